"""Slack-aware I/O scheduler (host logic): hand-worked cases that pin the oracle to the
policy the paper states, invariants, and launch-by-launch parity of the C-ABI scheduler
with the oracle on seeded random scenarios."""
import numpy as np
import pytest

from oracle.sched_oracle import DECODE, PREFILL, READ, WRITE, SchedOracle
from paper_2605_03375_b200 import tutti as T


def both(n_layers=4, step=32, max_in=4096, max_pre=4096):
    return SchedOracle(n_layers, step, max_in, max_pre), T.Scheduler(n_layers, step, max_in, max_pre)


def apply(pair, name, *args):
    o, c = pair
    getattr(o, name)(*args)
    getattr(c, "tutti_sched_" + name)(*args)


def decide(pair, phase, layer, l_in, l_pre):
    o, c = pair
    a = o.next(phase, layer, l_in, l_pre)
    b = [x[:5] for x in c.tutti_sched_next(phase, layer, l_in, l_pre)]
    assert a == b
    return a


def test_hand_worked_policy():
    """100 us per read IOCB, 150 us per write IOCB on 16 SMs; windows of 350 us."""
    pair = both()
    for n in (1, 2, 4, 8):
        apply(pair, "set_io_time", READ, 16, n, 100.0 * n)
        apply(pair, "set_io_time", WRITE, 16, n, 150.0 * n)
    apply(pair, "set_slack", 1024, 512, 350.0, 16)
    apply(pair, "set_slack", 1024, 2048, 0.0, 0)             # high reuse: no window at all
    apply(pair, "set_decode_slack", 320.0, 16)
    # a request arrives: two read IOCBs per layer for 4 layers
    for layer in range(4):
        apply(pair, "enqueue", READ, layer, 10 + 2 * layer, 2)
    # before layer 0: 3 reads fit (300 <= 350 < 400); layer 0 needs 2 -> 3 launched, one merged run
    assert decide(pair, PREFILL, 0, 1024, 512) == [(READ, 10, 3, 16, 0)]
    # a write is queued; before layer 1: reads first (1 required + prefetch up to 3), then no
    # window is left for a 150 us write after 300 us of reads
    apply(pair, "enqueue", WRITE, 0, 50, 2)
    assert decide(pair, PREFILL, 1, 1024, 512) == [(READ, 13, 3, 16, 1)]
    # before layer 2: only 2 reads remain (200 us) -> 150 us left -> exactly one write fits
    assert decide(pair, PREFILL, 2, 1024, 512) == [(READ, 16, 2, 16, 3), (WRITE, 50, 1, 16, 0)]
    # before layer 3: nothing to read, 350 us -> two writes would fit, one is queued
    assert decide(pair, PREFILL, 3, 1024, 512) == [(WRITE, 51, 1, 16, 0)]
    assert pair[1].tutti_sched_pending() == (0, 0)
    # no window (window table says 0): required reads are launched anyway, writes are deferred
    apply(pair, "enqueue", READ, 0, 100, 2)
    apply(pair, "enqueue", READ, 1, 102, 2)
    apply(pair, "enqueue", WRITE, 0, 60, 3)
    assert decide(pair, PREFILL, 0, 1024, 2048) == [(READ, 100, 2, 0, 0)]
    assert pair[1].tutti_sched_pending() == (2, 3)
    # decode: writes only, best effort: 320 us holds two 150 us writes
    assert decide(pair, DECODE, 0, 0, 0) == [(WRITE, 60, 2, 16, 0)]
    assert decide(pair, DECODE, 0, 0, 0) == [(WRITE, 62, 1, 16, 0)]
    assert decide(pair, DECODE, 0, 0, 0) == []
    pair[1].close()


def test_interpolation_and_sm_fallback():
    pair = both()
    apply(pair, "set_io_time", READ, 8, 1, 120.0)
    apply(pair, "set_io_time", READ, 8, 4, 420.0)
    apply(pair, "set_io_time", READ, 32, 2, 80.0)
    o, c = pair
    for sms, n, want in [(8, 1, 120.0), (8, 2, 220.0), (8, 4, 420.0), (8, 6, 620.0),
                         (16, 3, 320.0),        # 16 SMs unprofiled -> the 8-SM curve
                         (32, 1, 40.0), (32, 5, 200.0),
                         (4, 1, 120.0),         # below every profiled count -> smallest
                         (8, 0, 0.0)]:
        assert abs(float(o.io_time(READ, sms, n)) - want) < 1e-3
        assert c.tutti_sched_io_time(READ, sms, n) == float(o.io_time(READ, sms, n))
    c.close()


@pytest.mark.parametrize("seed", range(12))
def test_random_scenarios_match_oracle_and_invariants(seed):
    rng = np.random.default_rng(seed)
    n_layers = int(rng.integers(2, 9))
    pair = both(n_layers=n_layers)
    o, c = pair
    sm_set = [8, 16, 32]
    for op in (READ, WRITE):
        for sms in sm_set:
            base = float(rng.uniform(20, 200)) * (1.5 if op == WRITE else 1.0) * 16 / sms
            t = 0.0
            for n in (1, 2, 4, 8, 16):
                t = base * n * float(rng.uniform(0.9, 1.1)) + 5.0
                apply(pair, "set_io_time", op, sms, n, t)
    for li in range(0, 4097, 512):
        for lp in range(0, 4097, 512):
            if rng.random() < 0.8:
                apply(pair, "set_slack", li, lp, float(rng.uniform(0, 1500)), int(rng.choice(sm_set)))
    apply(pair, "set_decode_slack", float(rng.uniform(100, 800)), 8)
    next_iocb = 0
    issued = []
    queued_r, queued_w = [], []
    for req in range(6):
        l_in, l_pre = int(rng.integers(0, 4097)), int(rng.integers(0, 4097))
        for layer in range(n_layers):
            k = int(rng.integers(0, 4))
            apply(pair, "enqueue", READ, layer, next_iocb, k)
            queued_r += [(layer, next_iocb + i) for i in range(k)]
            next_iocb += k
        for layer in range(n_layers):
            before_r = sorted(queued_r)
            out = decide(pair, PREFILL, layer, l_in, l_pre)
            us, sms = o.slack.get((min(l_in // 32, o.ni - 1), min(l_pre // 32, o.nj - 1)), (0.0, 0))
            reads = [i for (op, f, n, s, l) in out if op == READ for i in range(f, f + n)]
            writes = [i for (op, f, n, s, l) in out if op == WRITE for i in range(f, f + n)]
            # reads come before writes in the launch list
            ops = [op for (op, *_rest) in out]
            assert ops == sorted(ops)
            # every read the layer needs was launched (now or earlier)
            still = [x for x in queued_r if x[1] not in reads]
            assert all(l > layer for (l, _) in still)
            # reads are taken in (layer, arrival) order
            assert reads == [i for (_, i) in before_r[:len(reads)]]
            # the launched group fits the window unless it is exactly the required set
            required = sum(1 for (l, _) in before_r if l <= layer)
            if len(reads) > required:
                assert float(o.io_time(READ, sms, len(reads))) <= us + 1e-3
            if writes:
                assert float(o.io_time(READ, sms, len(reads))) + \
                    float(o.io_time(WRITE, sms, len(writes))) <= us + 1e-2
                assert writes == [i for (_, i) in queued_w[:len(writes)]]
            queued_r = still
            queued_w = queued_w[len(writes):]
            issued += reads + writes
            # the layer produces new KV to store
            k = int(rng.integers(0, 3))
            apply(pair, "enqueue", WRITE, layer, next_iocb, k)
            queued_w += [(layer, next_iocb + i) for i in range(k)]
            next_iocb += k
        assert not queued_r
    for _ in range(200):
        out = decide(pair, DECODE, 0, 0, 0)
        if not out:
            break
        assert all(op == WRITE for (op, *_r) in out)
        issued += [i for (op, f, n, s, l) in out for i in range(f, f + n)]
    assert c.tutti_sched_pending() == (0, 0) or float(o.io_time(WRITE, 8, 1)) > o.decode[0]
    assert len(issued) == len(set(issued))                  # every IOCB launched at most once
    c.close()


def test_small_output_array_loses_nothing():
    import ctypes as C
    s = T.Scheduler(2, 32, 1024, 1024)
    s.tutti_sched_set_io_time(READ, 8, 1, 10.0)
    s.tutti_sched_set_slack(0, 0, 1000.0, 8)
    for i in (3, 7, 11):                                    # three non-adjacent IOCBs
        s.tutti_sched_enqueue(READ, 0, i, 1)
    out = (T.Launch * 2)()
    n = C.c_uint32()
    rc = s.lib.tutti_sched_next(s.h, 0, 0, 0, 0, out, 2, C.byref(n))
    assert rc == T.EAGAIN and n.value == 3 and s.tutti_sched_pending() == (3, 0)
    got = s.tutti_sched_next(PREFILL, 0, 0, 0)
    assert [g[1] for g in got] == [3, 7, 11] and s.tutti_sched_pending() == (0, 0)
    assert s.tutti_sched_enqueue(READ, 5, 0, 1, allow=(T.EINVAL,)) == T.EINVAL
    s.close()
