"""CPU-side GPU-file pool: a hand-worked sequence pins the policy, then the C-ABI pool is
compared call by call with the oracle on seeded random traffic."""
import time

import numpy as np
import pytest

from oracle.filepool_oracle import FilePoolOracle
from paper_2605_03375_b200 import tutti as T


def test_hand_worked_sequence():
    o, c = FilePoolOracle(4), T.FilePool(4)

    def ins(k):
        a = o.insert(k)
        b = c.tutti_filepool_insert(k, allow=(T.EAGAIN,))
        assert a[0] == b[0] and (a[0] != 0 or (a[1], a[2]) == (b[1], b[2]))
        return a
    # empty files are taken in ascending id: consecutive chunks become neighbours
    assert [ins(k)[1] for k in (100, 101, 102)] == [0, 1, 2]
    assert ins(101) == (0, 1, True)                       # already stored: shared, not duplicated
    assert c.tutti_filepool_lookup(555)[0] == T.ENOENT
    # prefix match stops at the first missing chunk
    assert list(c.tutti_filepool_match_prefix(np.array([100, 101, 999, 102], dtype=np.uint64))) == [0, 1]
    assert o.match_prefix([100, 101, 999, 102]) == [0, 1]
    assert ins(103)[1] == 3
    # pool full: the least recently used unpinned chunk goes; 102 (slot 2) is the oldest use
    assert ins(104) == (0, 2, False)
    assert c.tutti_filepool_lookup(102)[0] == T.ENOENT
    # pin everything: nothing can be reclaimed
    for s in range(4):
        assert c.tutti_filepool_pin(s, 1) == 0 and o.pin(s, 1) == 0
    assert ins(105)[0] == T.EAGAIN
    assert c.tutti_filepool_remove(100) == T.EAGAIN
    assert c.tutti_filepool_pin(0, -1) == 0 and o.pin(0, -1) == 0
    assert c.tutti_filepool_pin(0, -1, allow=(T.EINVAL,)) == T.EINVAL
    assert c.tutti_filepool_remove(100) == 0 and o.remove(100) == 0
    assert ins(106) == (0, 0, False)                      # the freed file is reused
    st = c.tutti_filepool_stats()
    assert (st["used"], st["free"], st["evictions"]) == (4, 0, 1) and o.evictions == 1
    c.close()


@pytest.mark.parametrize("seed", range(6))
def test_random_traffic_matches_oracle(seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(4, 40))
    o, c = FilePoolOracle(n), T.FilePool(n)
    pinned = []
    for step in range(4000):
        op = rng.random()
        key = int(rng.integers(0, 3 * n))
        if op < 0.45:
            a = o.insert(key)
            b = c.tutti_filepool_insert(key, allow=(T.EAGAIN,))
            assert a[0] == b[0]
            if a[0] == 0:
                assert (a[1], a[2]) == (b[1], b[2])
        elif op < 0.6:
            a, b = o.lookup(key), c.tutti_filepool_lookup(key)
            assert a[0] == b[0] and (a[0] != 0 or a[1] == b[1])
        elif op < 0.8:
            keys = rng.integers(0, 3 * n, size=int(rng.integers(0, 6))).astype(np.uint64)
            pin = bool(rng.random() < 0.4)
            a = o.match_prefix([int(k) for k in keys], pin)
            b = list(c.tutti_filepool_match_prefix(keys, pin))
            assert a == b
            if pin:
                pinned += a
        elif op < 0.9 and pinned:
            s = pinned.pop(int(rng.integers(0, len(pinned))))
            assert o.pin(s, -1) == c.tutti_filepool_pin(s, -1, allow=(T.EINVAL,))
        else:
            assert o.remove(key) == c.tutti_filepool_remove(key)
        if step % 500 == 0:
            st = c.tutti_filepool_stats()
            assert st["used"] == len(o.index) and st["free"] == len(o.free)
            assert st["evictions"] == o.evictions
    # every live slot holds exactly one key, no slot is both free and used
    assert len(set(o.index.values())) == len(o.index)
    assert not set(o.index.values()) & set(o.free)
    c.close()


def test_index_rate_is_far_from_the_io_path():
    """The index must sustain far more operations per second than a layer-wise transfer needs
    (config 2 touches 1,024 chunks per batch)."""
    n = 200_000
    c = T.FilePool(n)
    t0 = time.perf_counter()
    for k in range(20_000):
        c.tutti_filepool_insert(k)
    keys = np.arange(20_000, dtype=np.uint64)
    t1 = time.perf_counter()
    for _ in range(50):
        assert len(c.tutti_filepool_match_prefix(keys)) == 20_000
    t2 = time.perf_counter()
    lookups_per_s = 50 * 20_000 / (t2 - t1)
    assert lookups_per_s > 2e5                  # typically > 1e7; a loaded test box stays far above this
    assert 20_000 / (t1 - t0) > 5e3             # through ctypes, one call per insert
    c.close()
