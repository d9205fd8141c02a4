"""CPU-side checks of the C-ABI library: it loads without a GPU, exports every symbol the
header declares, its layout call agrees with the oracle's, and the host-side ring
accounting behaves (wrap-around, full ring, FIFO release)."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import oracle
from paper_2605_03375_b200 import tutti as T

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_loads_and_exports_header_symbols():
    lib = T.load()
    header = open(os.path.join(ROOT, "include", "tutti.h")).read()
    declared = set(re.findall(r"\b(tutti_[a-z_0-9]+)\s*\(", header))
    assert declared, "no declarations found"
    for name in sorted(declared):
        assert hasattr(lib, name), f"{name} declared in tutti.h but not exported"
    assert declared == set(T.EXPORTS)
    assert lib.tutti_version() > 0
    assert lib.tutti_strerror(T.EAGAIN).decode().startswith("try again")


GEOMS = [
    (1, 8, 128, 2, 16, 256, 1, 1, 8),
    (32, 8, 128, 2, 16, 256, 1, 1, 1280),
    (80, 8, 128, 2, 16, 1024, 1, 0, 320),
    (32, 8, 128, 2, 1, 256, 3, 1, 2113),
    (64, 8, 128, 2, 64, 64, 4, 0, 4096),
    (5, 1, 8, 2, 2, 4, 2, 0, 7),
]


@pytest.mark.parametrize("g", GEOMS)
def test_layout_matches_oracle(g):
    a = T.tutti_obj_layout(T.Geom(*g))
    b = oracle.obj_layout(oracle.geom(*g))
    for name, _ in T.Layout._fields_:
        assert getattr(a, name) == getattr(b, name), name


def test_layout_rejects_bad_geometry():
    lib = T.load()
    out = T.Layout()
    bad = [
        (0, 8, 128, 2, 16, 256, 1, 1, 8),       # zero layers
        (1, 8, 128, 2, 16, 250, 1, 1, 8),       # object not a multiple of the block
        (1, 8, 128, 2, 16, 256, 9, 1, 8),       # too many devices
        (1, 8, 128, 2, 16, 256, 1, 7, 8),       # unknown layout
        (1, 1, 3, 2, 16, 256, 1, 1, 8),         # token bytes not a multiple of 16
        (1, 8, 128, 2, 16, 256, 1, 1, 0),       # no slots
    ]
    for g in bad:
        assert lib.tutti_obj_layout(C.byref(T.Geom(*g)), C.byref(out)) == T.EINVAL
    assert lib.tutti_obj_layout(None, C.byref(out)) == T.EINVAL


class HostRing:
    def __init__(self, depth, cap):
        self.lib = T.load()
        self.h = self.lib.tutti_hostring_create(depth, cap)
        assert self.h

    def reserve(self, n, s):
        a, b = C.c_uint32(), C.c_uint32()
        rc = self.lib.tutti_hostring_reserve(self.h, n, s, C.byref(a), C.byref(b))
        return rc, a.value, b.value

    def release(self, i):
        return self.lib.tutti_hostring_release(self.h, i)

    def cancel_last(self, first):
        return self.lib.tutti_hostring_cancel_last(self.h, first)

    def live(self):
        a, b = C.c_uint32(), C.c_uint32()
        self.lib.tutti_hostring_live(self.h, C.byref(a), C.byref(b))
        return a.value, b.value

    def __del__(self):
        self.lib.tutti_hostring_destroy(self.h)


def test_hostring_reserve_release_wrap():
    r = HostRing(4, 100)
    assert T.load().tutti_hostring_create(3, 10) is None        # depth must be a power of two
    assert r.reserve(0, 1)[0] == T.EINVAL
    assert r.reserve(5, 1)[0] == T.EINVAL
    assert r.reserve(1, 101)[0] == T.EINVAL
    assert r.reserve(2, 40) == (0, 0, 0)
    assert r.reserve(1, 40) == (0, 2, 40)
    assert r.reserve(2, 1)[0] == T.EAGAIN                       # only one IOCB slot left
    assert r.reserve(1, 30)[0] == T.EAGAIN                      # 20 entries left at the end, 0 in front
    assert r.live() == (3, 80)
    assert r.release(7) == T.EINVAL                             # never reserved
    assert r.release(1) == 0                                    # out of order: nothing freed yet
    assert r.release(1) == T.EINVAL                             # twice
    assert r.live() == (3, 80)
    assert r.release(0) == 0                                    # first group complete -> freed
    assert r.live() == (1, 40)
    assert r.reserve(1, 30) == (0, 3, 0)                        # wraps to the front of the arena
    assert r.reserve(1, 15)[0] == T.EAGAIN                      # front gap is 40 - 30 = 10
    assert r.reserve(1, 10) == (0, 4, 30)
    assert r.release(2) == 0 and r.release(3) == 0 and r.release(4) == 0
    assert r.live() == (0, 0)
    assert r.reserve(4, 100) == (0, 5, 0)                       # empty ring starts at entry 0 again
    assert r.reserve(1, 0)[0] == T.EAGAIN
    for i in range(5, 9):
        assert r.release(i) == 0
    assert r.reserve(1, 0) == (0, 9, 0)


def test_hostring_many_cycles_never_overlap():
    rng = np.random.default_rng(3)
    depth, cap = 8, 1000
    r = HostRing(depth, cap)
    live = []                       # (first, n, base, cnt)
    expect_idx = 0
    for step in range(3000):
        if live and (rng.random() < 0.45 or len(live) > 6):
            k = int(rng.integers(0, len(live)))
            first, n, base, cnt, rel = live[k]
            i = int(rng.integers(0, n))
            if i not in rel:
                assert r.release(first + i) == 0
                rel.add(i)
            while live and len(live[0][4]) == live[0][1]:
                live.pop(0)
        else:
            n, s = int(rng.integers(1, 4)), int(rng.integers(0, 400))
            rc, first, base = r.reserve(n, s)
            if rc == 0:
                assert first == expect_idx
                expect_idx += n
                assert base + s <= cap
                for f2, n2, b2, c2, _ in live:
                    assert base + s <= b2 or b2 + c2 <= base or s == 0 or c2 == 0
                live.append((first, n, base, s, set()))
            else:
                assert rc == T.EAGAIN
        iocbs, ents = r.live()
        assert iocbs == sum(x[1] for x in live) <= depth
        assert ents == sum(x[3] for x in live)
    assert expect_idx > 500


def test_context_needs_a_gpu():
    import torch
    if torch.cuda.is_available():
        pytest.skip("GPU present")
    lib = T.load()
    h = C.c_void_p()
    g = T.Geom(*GEOMS[0])
    assert lib.tutti_ctx_create(C.byref(g), 0, C.byref(h)) == T.ECUDA
    assert lib.tutti_last_cuda_error().decode() != ""
    with pytest.raises(T.TuttiError):
        T.Context(g)


def test_struct_sizes_match_the_header():
    """The binding's ctypes structs and numpy record types have the sizes the library
    asserts at compile time."""
    assert C.sizeof(T.Geom) == 40 and C.sizeof(T.Layout) == 80 and C.sizeof(T.Batch) == 56
    assert C.sizeof(T.Cqe) == 16 and C.sizeof(T.IocbInfo) == 48 and C.sizeof(T.Launch) == 24
    assert T.SQE_DTYPE.itemsize == 32 and T.SGL_DTYPE.itemsize == 16
    assert oracle.SQE_DTYPE.itemsize == 32 and oracle.SGL_DTYPE.itemsize == 16


def test_hostring_cancel_last_restores_the_previous_state():
    r = HostRing(8, 100)
    assert r.reserve(2, 30) == (0, 0, 0)
    assert r.reserve(3, 50) == (0, 2, 30)
    assert r.cancel_last(0) == T.EINVAL                 # not the newest group
    assert r.cancel_last(2) == 0
    assert r.live() == (2, 30)
    assert r.reserve(1, 60) == (0, 2, 30)               # same index and arena position again
    assert r.cancel_last(2) == 0 and r.cancel_last(0) == 0
    assert r.live() == (0, 0)
    assert r.reserve(4, 100) == (0, 0, 0)
    assert r.release(1) == 0
    assert r.cancel_last(0) == T.EINVAL                 # already partly consumed


def test_null_handles_are_refused_without_a_gpu():
    """Entry points that take a context and a ring answer TUTTI_EINVAL for null handles before
    they touch the device: no GPU is needed to see that."""
    lib = T.load()
    n, ns, b, f, k = C.c_uint32(), C.c_uint32(), C.c_uint64(), C.c_uint32(), C.c_uint32()
    assert lib.tutti_stage_plan(None, None, None, 0, None, C.byref(n), C.byref(ns), C.byref(b)) == T.EINVAL
    assert lib.tutti_stage_copy_layer(None, None, 0, T.OP_READ, None, 0, None) == T.EINVAL
    assert lib.tutti_build_sqes_staged(None, None, None, 0, T.OP_READ, None, 0, None,
                                       C.byref(f), C.byref(k)) == T.EINVAL
    assert lib.tutti_build_sqes(None, None, None, 0, T.OP_READ, None, C.byref(f), C.byref(k)) == T.EINVAL
    assert lib.tutti_kv_restore_layer(None, None, 0, 1, 0, None) == T.EINVAL
    assert lib.tutti_kv_save_layer(None, None, 0, 1, 0, None) == T.EINVAL
