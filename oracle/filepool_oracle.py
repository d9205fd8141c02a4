"""Oracle of the CPU-side GPU-file pool (paper Section 3.1, "Scalable GPU File Pool") — TEST
INFRASTRUCTURE ONLY.

The paper's statement: all files exist from start-up and are free; persisting a new KV chunk
"only selects an empty GPU file and installs a CPU-side hash mapping"; creation and reclamation
stay off the critical path.  Policy details the paper leaves open, as read here: the empty
file with the lowest id is selected (chunks saved one after another become neighbours in the
store), a chunk that is already stored shares its file, and when no file is empty the least
recently used chunk that no in-flight batch pins is reclaimed.  Plain Python containers, no
code shared with the C++ pool.  Pins: tests/test_filepool_cpu.py."""
from __future__ import annotations

from typing import Dict, List, Optional, Tuple

OK, EINVAL, EAGAIN, ENOENT = 0, -1, -3, -7


class FilePoolOracle:
    def __init__(self, n_slots: int):
        self.free: List[int] = list(range(n_slots))      # kept sorted
        self.index: Dict[int, int] = {}                   # key -> slot
        self.key_of: Dict[int, int] = {}                  # slot -> key
        self.pins: Dict[int, int] = {}
        self.recency: List[int] = []                      # slots, least recent first
        self.evictions = 0

    def _touch(self, slot):
        self.recency.remove(slot)
        self.recency.append(slot)

    def insert(self, key) -> Tuple[int, Optional[int], bool]:
        if key in self.index:
            self._touch(self.index[key])
            return OK, self.index[key], True
        if self.free:
            slot = self.free.pop(0)
        else:
            victims = [s for s in self.recency if self.pins.get(s, 0) == 0]
            if not victims:
                return EAGAIN, None, False
            slot = victims[0]
            del self.index[self.key_of[slot]]
            self.recency.remove(slot)
            self.evictions += 1
        self.index[key] = slot
        self.key_of[slot] = key
        self.pins[slot] = 0
        self.recency.append(slot)
        return OK, slot, False

    def lookup(self, key):
        if key not in self.index:
            return ENOENT, None
        self._touch(self.index[key])
        return OK, self.index[key]

    def match_prefix(self, keys, pin=False):
        out = []
        for k in keys:
            if k not in self.index:
                break
            s = self.index[k]
            self._touch(s)
            if pin:
                self.pins[s] += 1
            out.append(s)
        return out

    def pin(self, slot, delta):
        if slot not in self.key_of or self.index.get(self.key_of[slot]) != slot:
            return EINVAL
        if self.pins[slot] + delta < 0:
            return EINVAL
        self.pins[slot] += delta
        return OK

    def remove(self, key):
        if key not in self.index:
            return ENOENT
        s = self.index[key]
        if self.pins[s]:
            return EAGAIN
        del self.index[key]
        del self.key_of[s]
        self.recency.remove(s)
        self.free.append(s)
        self.free.sort()
        return OK
