"""Oracle of the slack-aware I/O scheduler (paper Section 3.3) — TEST INFRASTRUCTURE ONLY.

Plain Python restatement of the policy, in the paper's order:
  1. look the layer's slack window (duration, SM budget) up by (input length, prefix length);
  2. reads have priority: launch the largest number of queued read IOCBs whose profiled
     kernel time fits the window; if fewer fit than the layer about to run needs, launch the
     needed ones anyway ("immediately launches the required reads to avoid stalling");
  3. writes only after the reads, and only with window left; what does not fit stays queued;
  4. during decode only writes are flushed, best effort, against the decode window.
Reads are served in layer order, first come first served within a layer; writes oldest first.
Kernel times come from a profiled table (time of n IOCBs on s SMs), interpolated linearly.
Shares no code with the C++ scheduler.  Pins: tests/test_sched_cpu.py (hand-worked cases,
invariants)."""
from __future__ import annotations

import bisect
from typing import Dict, List, Tuple

import numpy as np

READ, WRITE = 0, 1
PREFILL, DECODE = 0, 1


class SchedOracle:
    def __init__(self, n_layers: int, token_step: int, max_input: int, max_prefix: int):
        self.n_layers, self.step = n_layers, token_step
        self.ni, self.nj = max_input // token_step + 1, max_prefix // token_step + 1
        self.slack: Dict[Tuple[int, int], Tuple[float, int]] = {}
        self.decode = (0.0, 0)
        self.io: List[Dict[int, List[Tuple[int, float]]]] = [{}, {}]
        self.reads: List[Tuple[int, int]] = []      # (layer, iocb)
        self.writes: List[Tuple[int, int]] = []

    # ---- offline profiles ------------------------------------------------------------
    def set_slack(self, l_input, l_prefix, us, sms):
        self.slack[(l_input // self.step, l_prefix // self.step)] = (float(np.float32(us)), sms)

    def set_decode_slack(self, us, sms):
        self.decode = (float(np.float32(us)), sms)

    def set_io_time(self, op, sms, n, us):
        pts = self.io[op].setdefault(sms, [])
        for k, (m, _) in enumerate(pts):
            if m == n:
                pts[k] = (n, np.float32(us))
                return
        bisect.insort(pts, (n, np.float32(us)))

    def _curve(self, op, sms):
        m = self.io[op]
        if not m:
            return None
        if sms in m:
            return m[sms]
        below = [k for k in sorted(m) if k != 0 and k <= sms]
        if below:
            return m[below[-1]]
        nonzero = [k for k in sorted(m) if k != 0]
        return m[nonzero[0]] if nonzero else m[sorted(m)[0]]

    def io_time(self, op, sms, n) -> np.float32:
        """float32 arithmetic throughout, as the tables hold float32."""
        f = np.float32
        pts = self._curve(op, sms)
        if n == 0 or not pts:
            return f(0)
        if len(pts) == 1 or n <= pts[0][0]:
            return f(f(pts[0][1] * f(n)) / f(pts[0][0]))
        for (n0, t0), (n1, t1) in zip(pts[:-1], pts[1:]):
            if n <= n1:
                frac = f(f(n - n0) / f(n1 - n0))
                return f(t0 + f(frac * f(t1 - t0)))
        (n0, t0), (n1, t1) = pts[-2], pts[-1]
        slope = f(f(t1 - t0) / f(n1 - n0))
        return f(t1 + f(slope * f(n - n1)))

    def _max_fit(self, op, sms, budget, limit):
        if self._curve(op, sms) is None:
            return 0
        n = 0
        while n < limit and self.io_time(op, sms, n + 1) <= np.float32(budget):
            n += 1
        return n

    # ---- queues ----------------------------------------------------------------------
    def enqueue(self, op, layer, first, n):
        for k in range(n):
            if op == READ:
                pos = len(self.reads)
                for i, (l, _) in enumerate(self.reads):
                    if l > layer:
                        pos = i
                        break
                self.reads.insert(pos, (layer, first + k))
            else:
                self.writes.append((layer, first + k))

    # ---- the decision ----------------------------------------------------------------
    def next(self, phase, layer, l_input, l_prefix):
        """Returns [(opcode, first_iocb, n_iocb, sm_count, layer_of_first)]."""
        if phase == PREFILL:
            i = min(l_input // self.step, self.ni - 1)
            j = min(l_prefix // self.step, self.nj - 1)
            us, sms = self.slack.get((i, j), (0.0, 0))
        else:
            us, sms = self.decode
        us = np.float32(us)
        picked: List[Tuple[int, int, int]] = []        # (op, layer, iocb)
        left = us
        if phase == PREFILL:
            required = sum(1 for (l, _) in self.reads if l <= layer)
            fit = self._max_fit(READ, sms, us, len(self.reads)) if us > 0 else 0
            take = max(fit, required)
            t = self.io_time(READ, sms, take)
            for _ in range(take):
                l, i = self.reads.pop(0)
                picked.append((READ, l, i))
            left = np.float32(0) if take > fit else np.float32(us - t)
        if left > 0 and self.writes:
            fit = self._max_fit(WRITE, sms, left, len(self.writes))
            for _ in range(fit):
                l, i = self.writes.pop(0)
                picked.append((WRITE, l, i))
        launches: List[List[int]] = []
        for op, l, i in picked:
            if launches and launches[-1][0] == op and launches[-1][1] + launches[-1][2] == i:
                launches[-1][2] += 1
            else:
                launches.append([op, i, 1, sms, l])
        return [tuple(x) for x in launches]
