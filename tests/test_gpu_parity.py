"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the
same seeded inputs — descriptors element by element, pool and store bytes bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_03375_b200 import tutti as T
from paper_2605_03375_b200 import workload as wl
from tests.devcase import DeviceCase

pytestmark = pytest.mark.gpu

CASES = {
    "cfg1": dict(index=1),
    "cfg1-scattered-slots": dict(index=1, consecutive_slots=False, slot_mean_run=1.5,
                                 slot_space_factor=3.0),
    "cfg2-small": dict(index=2, scale=0.05, n_layers=4),
    "cfg2-file-major": dict(index=2, scale=0.03, n_layers=3, layout=wl.LAYOUT_FILE_MAJOR),
    "cfg2-2dev-interleaved": dict(index=2, scale=0.04, n_layers=2, n_devices=2,
                                  pool_interleaved=True),
    "cfg3-small": dict(index=3, scale=0.03, n_layers=2, store_kind="hbm"),
    "cfg4-small": dict(index=4, scale=0.04, n_layers=2),
    "cfg4-3dev-file-major": dict(index=4, scale=0.03, n_layers=2, n_devices=3,
                                 layout=wl.LAYOUT_FILE_MAJOR),
    "block-per-object": dict(index=2, scale=0.02, n_layers=2, obj_tokens=16, slot_mean_run=3.0),
    "big-blocks-64k": dict(index=2, scale=0.03, n_layers=2, block_tokens=32, obj_tokens=256),
    "odd-token-bytes": dict(index=4, scale=0.03, n_layers=2, n_kv_heads=3, head_dim=8,
                            block_tokens=4, obj_tokens=32),
    "fp8-kv": dict(index=2, scale=0.04, n_layers=2, elem_bytes=1),
    "padded-block-stride": dict(index=2, scale=0.04, n_layers=2, pool_pad_bytes=4096),
    "padded-stride-1-token-pages": dict(index=4, scale=0.03, n_layers=2, pool_pad_bytes=48,
                                        pool_interleaved=True),
    "hnd-pool": dict(index=2, scale=0.05, n_layers=2, pool_hnd=True),
    "hnd-pool-small-blocks": dict(index=4, scale=0.03, n_layers=2, pool_hnd=True, n_kv_heads=4,
                                  head_dim=64, block_tokens=2, obj_tokens=32),
    "hnd-pool-interleaved-2dev": dict(index=2, scale=0.04, n_layers=2, pool_hnd=True, n_devices=2,
                                      pool_interleaved=True, layout=wl.LAYOUT_FILE_MAJOR),
    # requests with a common prefix: the shared objects are read once (repeat entries)
    "shared-prefix-8-requests": dict(index=2, scale=0.25, n_layers=2, hit_tokens=[2048] * 8,
                                     shared_prefix_frac=0.75),
    "shared-prefix-1-token-pages": dict(index=4, scale=0.05, n_layers=2, shared_prefix_frac=1.0),
    "shared-prefix-hnd-2dev": dict(index=2, scale=0.05, n_layers=2, hit_tokens=[1024] * 3,
                                   shared_prefix_frac=0.5, pool_hnd=True, n_devices=2),
    "shared-prefix-one-block-objects": dict(index=2, scale=0.02, n_layers=2, obj_tokens=16,
                                            hit_tokens=[512, 512, 256], shared_prefix_frac=1.0),
    # more sharers than one stage's 32 lanes: the copy engines feed them in several rounds
    "shared-by-40-requests": dict(index=2, scale=0.02, n_layers=2, hit_tokens=[512] * 40,
                                  shared_prefix_frac=1.0),
}


def mk(name):
    c = dict(CASES[name])
    return wl.config(c.pop("index"), c.pop("scale", 1.0), **c)


def same_records(a, b):
    return a.dtype.itemsize == b.dtype.itemsize and a.tobytes() == b.tobytes()


@pytest.mark.parametrize("name", list(CASES))
@pytest.mark.parametrize("engine", [T.ENGINE_LDST, T.ENGINE_BULK])
def test_restore_and_save_match_oracle(name, engine):
    w = mk(name)
    dc = DeviceCase(w, capacity=2048)
    try:
        dc.ctx.tutti_set_option(T.OPT_COPY_ENGINE, engine)
        for layer in sorted({0, w.n_layers - 1}):
            # descriptors
            rc, first, n = dc.ring.tutti_build_sqes(dc.batch, layer, T.OP_READ)
            sq, sg, num, infos = dc.read_build(first, n)
            orc, osq, osg, onum = dc.oracle_descriptors(layer, oracle.OP_READ, 2048)
            assert orc == 0
            assert all(i.status == 0 and i.ready for i in infos)
            assert same_records(sq, osq) and same_records(sg, osg)
            assert list(num[:len(onum)]) == list(onum) and not num[len(onum):].any()
            # restore
            dc.ring.tutti_kv_restore_layer(first, n)
            cqes = dc.poll_all(first, n)
            assert sorted(c[0] for c in cqes) == list(range(first, first + n))
            assert all(c[1] == 0 for c in cqes)
            assert sum(c[2] for c in cqes) == int(osg["len"].astype(np.uint64).sum())
            got = dc.pool_dev[layer].cpu().numpy()
            want = dc.oracle_restore(layer)
            assert np.array_equal(got, want)
            # save the restored pool into a zeroed store
            for t in dc.store_dev:
                t.zero_()
            rc, first, n = dc.ring.tutti_build_sqes(dc.batch, layer, T.OP_WRITE)
            dc.ring.tutti_kv_save_layer(first, n)
            cqes = dc.poll_all(first, n)
            assert all(c[1] == 0 for c in cqes)
            st_want = [np.zeros_like(s) for s in dc.store_host]
            dc.oracle_save(layer, want, st_want)
            for t, s in zip(dc.store_dev, st_want):
                assert np.array_equal(t.cpu().numpy(), s)
            # round trip: what was saved equals the original store on the covered ranges
            for t, s0, s1 in zip(dc.store_dev, dc.store_host, st_want):
                cov = s1 != 0
                assert np.array_equal(t.cpu().numpy()[cov], s0[cov])
            for t, s in zip(dc.store_dev, dc.store_host):
                t.copy_(torch.from_numpy(s))
    finally:
        dc.close()


@pytest.mark.parametrize("engine", [T.ENGINE_LDST, T.ENGINE_BULK])
@pytest.mark.parametrize("sm_count", [0, 8, 32])
def test_small_iocbs_ring_wrap_and_capped_mode(engine, sm_count):
    """1-token pages with 4 contexts per IOCB and a ring of 64: many IOCBs per layer, the
    ring and the SGL arena wrap, completions arrive in any order."""
    w2 = wl.config(4, 0.04, n_layers=2, slot_mean_run=1.2, slot_space_factor=2.0)
    dc = DeviceCase(w2, depth=64, capacity=4, sgl_capacity=int(2.5 * 2 * len(w2.block_ids)))
    try:
        dc.ctx.tutti_set_option(T.OPT_COPY_ENGINE, engine)
        seen = []
        for it in range(14):
            layer = it % 2
            dc.pool_dev[layer].copy_(torch.from_numpy(dc.pool_host[layer]))
            rc, first, n = dc.ring.tutti_build_sqes(dc.batch, layer, T.OP_READ)
            assert n > 1
            sq, sg, num, infos = dc.read_build(first, n)
            orc, osq, osg, onum = dc.oracle_descriptors(layer, oracle.OP_READ, 4)
            assert same_records(sq, osq) and same_records(sg, osg)
            assert list(num[:len(onum)]) == list(onum)
            dc.ring.tutti_kv_restore_layer(first, n, sm_count)
            cqes = dc.poll_all(first, n)
            assert sorted(c[0] for c in cqes) == list(range(first, first + n))
            assert sum(c[2] for c in cqes) == int(osg["len"].astype(np.uint64).sum())
            assert np.array_equal(dc.pool_dev[layer].cpu().numpy(), dc.oracle_restore(layer))
            seen.append(first)
        assert seen[-1] >= 64          # the index counter ran past the ring depth
    finally:
        dc.close()


def test_host_prepared_descriptors():
    """CPU-prepared IOCBs (the paper's own split): oracle-built descriptors, uploaded and
    executed by the copy kernels, with entry lengths that differ."""
    w = mk("cfg2-small")
    dc = DeviceCase(w, depth=8, capacity=2048)
    try:
        for engine in (T.ENGINE_LDST, T.ENGINE_BULK):
            dc.ctx.tutti_set_option(T.OPT_COPY_ENGINE, engine)
            layer = 1
            dc.pool_dev[layer].copy_(torch.from_numpy(dc.pool_host[layer]))
            orc, osq, osg, onum = dc.oracle_descriptors(layer, oracle.OP_READ, 2048)
            rc, first = dc.ring.tutti_ring_reserve(1, len(osg))
            dc.ring.tutti_ring_fill_host(first, osq, osg)
            dc.ring.tutti_kv_restore_layer(first, 1)
            (idx, status, nbytes), = dc.poll_all(first, 1)
            assert (idx, status, nbytes) == (first, 0, int(osq["len"].sum()))
            assert np.array_equal(dc.pool_dev[layer].cpu().numpy(), dc.oracle_restore(layer))
        # split every entry in two unequal parts: same bytes, variable lengths
        sg2 = np.zeros(2 * len(osg), dtype=osg.dtype)
        sg2["addr"][0::2] = osg["addr"]
        sg2["len"][0::2] = 4096
        sg2["addr"][1::2] = osg["addr"] + 4096
        sg2["len"][1::2] = osg["len"] - 4096
        sg2["id"] = np.repeat(osg["id"], 2)
        sq2 = osq.copy()
        sq2["sgl_first"] *= 2
        sq2["sgl_count"] *= 2
        dc.pool_dev[layer].copy_(torch.from_numpy(dc.pool_host[layer]))
        rc, first = dc.ring.tutti_ring_reserve(1, len(sg2))
        dc.ring.tutti_ring_fill_host(first, sq2, sg2)
        dc.ring.tutti_kv_restore_layer(first, 1)
        (idx, status, nbytes), = dc.poll_all(first, 1)
        assert status == 0 and nbytes == int(osg["len"].astype(np.uint64).sum())
        assert np.array_equal(dc.pool_dev[layer].cpu().numpy(), dc.oracle_restore(layer))
    finally:
        dc.close()


def test_pinned_host_store_zero_copy():
    w = wl.config(3, 0.03, n_layers=2)
    assert w.store_kind == "host"
    dc = DeviceCase(w, host_store=True)
    try:
        layer = 1
        rc, first, n = dc.ring.tutti_build_sqes(dc.batch, layer, T.OP_READ)
        dc.ring.tutti_kv_restore_layer(first, n)
        cqes = dc.poll_all(first, n)
        assert all(c[1] == 0 for c in cqes)
        assert np.array_equal(dc.pool_dev[layer].cpu().numpy(), dc.oracle_restore(layer))
        # save back into the pinned store
        want = dc.oracle_restore(layer)
        for t in dc.store_dev:
            t.zero_()
        rc, first, n = dc.ring.tutti_build_sqes(dc.batch, layer, T.OP_WRITE)
        dc.ring.tutti_kv_save_layer(first, n)
        dc.poll_all(first, n)
        torch.cuda.synchronize()
        st_want = [np.zeros_like(s) for s in dc.store_host]
        dc.oracle_save(layer, want, st_want)
        for t, s in zip(dc.store_dev, st_want):
            assert np.array_equal(t.numpy(), s)
    finally:
        dc.close()


def test_plan_reuse_across_layers_and_launch_count():
    """With a plan epoch the batch is sorted once; every later layer costs one build launch
    and one copy launch, independent of the number of blocks."""
    w = mk("cfg2-small")
    dc = DeviceCase(w)
    try:
        dc.batch.plan_epoch = 7
        k0, h0 = dc.ring.tutti_ring_stats()
        for layer in range(w.n_layers):
            rc, first, n = dc.ring.tutti_build_sqes(dc.batch, layer, T.OP_READ)
            sq, sg, num, infos = dc.read_build(first, n)
            orc, osq, osg, onum = dc.oracle_descriptors(layer, oracle.OP_READ, 2048)
            assert same_records(sq, osq) and same_records(sg, osg)
            dc.ring.tutti_kv_restore_layer(first, n)
            dc.poll_all(first, n)
            assert np.array_equal(dc.pool_dev[layer].cpu().numpy(), dc.oracle_restore(layer))
        k1, h1 = dc.ring.tutti_ring_stats()
        assert k1 - k0 == 1 + 2 * w.n_layers           # one plan, then emit + copy per layer
        assert h1 - h0 == 3 * w.n_layers               # build, restore, poll: O(1) per layer
    finally:
        dc.close()


def test_empty_batch_and_zero_hits():
    w = wl.make_workload("z", seed=5, n_layers=1, hit_tokens=[0, 256, 0], block_tokens=16,
                         obj_tokens=256, n_pool_blocks=64)
    dc = DeviceCase(w)
    try:
        rc, first, n = dc.ring.tutti_build_sqes(dc.batch, 0, T.OP_READ)
        dc.ring.tutti_kv_restore_layer(first, n)
        cqes = dc.poll_all(first, n)
        assert sum(c[2] for c in cqes) == 256 * 2 * 2048
        assert np.array_equal(dc.pool_dev[0].cpu().numpy(), dc.oracle_restore(0))
        # a batch with no requests at all: one IOCB with no contexts, completes with 0 bytes
        empty = T.Batch(0, 0, 0, 0, None, None, None, None, None)
        rc, first, n = dc.ring.tutti_build_sqes(empty, 0, T.OP_READ)
        assert n == 1
        info, sq = dc.ring.tutti_ring_read_iocb(first)
        assert info.num_ioctx == 0 and info.total_entries == 0 and info.ready
        dc.ring.tutti_kv_restore_layer(first, n)
        assert dc.poll_all(first, n) == [(first, 0, 0)]
    finally:
        dc.close()


@pytest.mark.parametrize("capacity", [2048, 8])
def test_all_layers_built_in_one_launch(capacity):
    """tutti_build_sqes_layers: one launch prepares every layer; each layer's IOCBs hold
    exactly the descriptors of a single-layer build, and one copy launch executes them all."""
    w = mk("cfg2-small")
    n_items = 2 * len(w.obj_slot)
    per = max(1, -(-n_items // capacity))
    depth = 1
    while depth < 2 * per * w.n_layers:
        depth *= 2
    dc = DeviceCase(w, depth=depth, capacity=capacity, sgl_capacity=2 * len(w.block_ids) * (w.n_layers + 1))
    try:
        k0, _ = dc.ring.tutti_ring_stats()
        rc, first, per_layer = dc.ring.tutti_build_sqes_layers(dc.batch, 0, w.n_layers, T.OP_READ)
        assert per_layer == per
        k1, _ = dc.ring.tutti_ring_stats()
        assert k1 - k0 == 2                                   # plan + one emit for all layers
        for layer in range(w.n_layers):
            sq, sg, num, infos = dc.read_build(first + layer * per_layer, per_layer)
            orc, osq, osg, onum = dc.oracle_descriptors(layer, oracle.OP_READ, capacity)
            assert same_records(sq, osq) and same_records(sg, osg)
            assert list(num[:len(onum)]) == list(onum) and not num[len(onum):].any()
            assert all(i.layer == layer and i.status == 0 for i in infos)
        dc.ring.tutti_kv_restore_layer(first, per_layer * w.n_layers)
        cqes = dc.poll_all(first, per_layer * w.n_layers)
        assert all(c[1] == 0 for c in cqes)
        for layer in range(w.n_layers):
            assert np.array_equal(dc.pool_dev[layer].cpu().numpy(), dc.oracle_restore(layer))
        # a range that leaves the layer count is refused
        rc, *_ = dc.ring.tutti_build_sqes_layers(dc.batch, 2, w.n_layers, T.OP_READ, allow=(T.EINVAL,))
        assert rc == T.EINVAL
    finally:
        dc.close()


@pytest.mark.parametrize("hnd", [False, True])
def test_mixed_hbm_and_pinned_host_storage_devices(hnd):
    """Objects striped round-robin over two storage devices of different kinds: device 0 in
    HBM, device 1 in pinned host memory (read and written zero-copy)."""
    w = wl.config(2, 0.04, n_layers=2, n_devices=2, pool_hnd=hnd)
    dc = DeviceCase(w, host_devices=(1,))
    try:
        layer = 1
        rc, first, n = dc.ring.tutti_build_sqes(dc.batch, layer, T.OP_READ)
        sq, sg, num, infos = dc.read_build(first, n)
        assert set(sq["dev"].tolist()) == {0, 1}
        dc.ring.tutti_kv_restore_layer(first, n)
        assert all(c[1] == 0 for c in dc.poll_all(first, n))
        want = dc.oracle_restore(layer)
        assert np.array_equal(dc.pool_dev[layer].cpu().numpy(), want)
        for t in dc.store_dev:
            t.zero_()
        rc, first, n = dc.ring.tutti_build_sqes(dc.batch, layer, T.OP_WRITE)
        dc.ring.tutti_kv_save_layer(first, n, 8)
        assert all(c[1] == 0 for c in dc.poll_all(first, n))
        torch.cuda.synchronize()
        st = [np.zeros_like(s) for s in dc.store_host]
        dc.oracle_save(layer, want, st)
        for t, s in zip(dc.store_dev, st):
            assert np.array_equal(t.cpu().numpy(), s)
    finally:
        dc.close()


@pytest.mark.parametrize("engine", [T.ENGINE_LDST, T.ENGINE_BULK])
@pytest.mark.parametrize("sm_count", [0, 8])
@pytest.mark.parametrize("tokens", [1024, 4096 + 256 + 16])
def test_whole_pass_of_a_short_prefix_in_one_launch(engine, sm_count, tokens):
    """32 layers of a short prefix built by one launch and executed by one copy launch (both
    directions): many small IOCBs, over which the copy agents spread instead of queueing at
    the first one.  Completions are consumed with one tutti_ring_poll_range call."""
    w = wl.config(2, 1.0, n_layers=32, hit_tokens=[tokens])
    dc = DeviceCase(w, depth=64, capacity=2048, sgl_capacity=2 * len(w.block_ids) * 33)
    try:
        dc.ctx.tutti_set_option(T.OPT_COPY_ENGINE, engine)
        rc, first, per = dc.ring.tutti_build_sqes_layers(dc.batch, 0, 32, T.OP_READ)
        assert per == 1
        assert dc.ring.tutti_ring_poll_range(first, 32)[0] == T.EAGAIN      # nothing issued yet
        dc.ring.tutti_kv_restore_layer(first, 32, sm_count)
        rc, nbytes, err, done = dc.ring.tutti_ring_poll_range(first, 32, 5_000_000_000)
        assert (rc, err, done) == (T.OK, 0, 32)
        assert nbytes == 32 * tokens * 2 * int(dc.ctx.layout.token_bytes)
        assert dc.ring.tutti_ring_poll_range(first, 1)[0] == T.EINVAL       # released: no longer live
        want = {}
        for layer in (0, 1, 13, 31):
            want[layer] = dc.oracle_restore(layer)
            assert np.array_equal(dc.pool_dev[layer].cpu().numpy(), want[layer])
        for t in dc.store_dev:
            t.zero_()
        rc, first, per = dc.ring.tutti_build_sqes_layers(dc.batch, 0, 32, T.OP_WRITE)
        dc.ring.tutti_kv_save_layer(first, 32, sm_count)
        rc, nbytes, err, done = dc.ring.tutti_ring_poll_range(first, 32, 5_000_000_000)
        assert (rc, err, done) == (T.OK, 0, 32)
        torch.cuda.synchronize()
        st = [np.zeros_like(s) for s in dc.store_host]
        for layer in range(32):
            pool = want.get(layer)
            if pool is None:
                pool = dc.oracle_restore(layer)
            dc.oracle_save(layer, pool, st)
        for t, s in zip(dc.store_dev, st):
            assert np.array_equal(t.cpu().numpy(), s)
    finally:
        dc.close()


@pytest.mark.parametrize("engine", [T.ENGINE_LDST, T.ENGINE_BULK])
@pytest.mark.parametrize("sm_count", [0, 8])
@pytest.mark.parametrize("chunk", [0, 8192])
@pytest.mark.parametrize("name", ["shared-prefix-8-requests", "shared-by-40-requests"])
def test_shared_prefix_batch_grid_and_capped(engine, sm_count, chunk, name):
    """8 requests sharing 75 % of their prefix: the shared objects are named once in the
    descriptors and go to all eight requests' blocks, on all SMs and SM-capped, with stages
    that hold a whole block and with stages that hold a piece of one.  Claims of 1, 2 and 3
    chunks cut the groups of repeats at every possible place."""
    w = mk(name)
    dc = DeviceCase(w, capacity=16, depth=32)
    try:
        dc.ctx.tutti_set_option(T.OPT_COPY_ENGINE, engine)
        if chunk:
            dc.ctx.tutti_set_option(T.OPT_BULK_CHUNK_BYTES, chunk)
        layer = 1
        rc, first, n = dc.ring.tutti_build_sqes(dc.batch, layer, T.OP_READ)
        sq, sg, num, infos = dc.read_build(first, n)
        orc, osq, osg, onum = dc.oracle_descriptors(layer, oracle.OP_READ, 16)
        assert same_records(sq, osq) and same_records(sg, osg)
        n_dup = int(((sg["id"] & oracle.SGL_DUP) != 0).sum())
        assert n_dup > len(sg) // 2                                  # most entries are repeats
        assert int(sq["len"].sum()) < int(sg["len"].astype(np.uint64).sum()) // 2
        dc.ring.tutti_kv_restore_layer(first, n, sm_count)
        cqes = dc.poll_all(first, n)
        assert all(c[1] == 0 for c in cqes)
        assert sum(c[2] for c in cqes) == int(sg["len"].astype(np.uint64).sum())   # bytes landed
        want = dc.oracle_restore(layer)
        assert np.array_equal(dc.pool_dev[layer].cpu().numpy(), want)
        for claim in (1, 2, 3):
            dc.ctx.tutti_set_option(T.OPT_CLAIM_CHUNKS, claim)
            dc.pool_dev[layer].copy_(torch.from_numpy(dc.pool_host[layer]))
            rc, first, n = dc.ring.tutti_build_sqes(dc.batch, layer, T.OP_READ)
            dc.ring.tutti_kv_restore_layer(first, n, sm_count)
            rc, nbytes, err, done = dc.ring.tutti_ring_poll_range(first, n, 5_000_000_000)
            assert (rc, err, done) == (T.OK, 0, n)
            assert nbytes == int(sg["len"].astype(np.uint64).sum())
            assert np.array_equal(dc.pool_dev[layer].cpu().numpy(), want)
    finally:
        dc.close()


@pytest.mark.parametrize("name", ["cfg2-small", "shared-prefix-8-requests", "cfg4-small",
                                  "shared-prefix-1-token-pages", "hnd-pool"])
@pytest.mark.parametrize("per", [5, 64, 2048])
def test_iocbs_cut_by_bytes(name, per):
    """tutti_ring_set_iocb_bytes: IOCBs of equal work.  Contexts, entries and per-IOCB counts
    equal the oracle's, every IOCB moves at most its budget, and the bytes land as always —
    single-layer and multi-layer builds, both engines, capped and on all SMs."""
    w = mk(name)
    n_ent = 2 * len(w.block_ids)
    per_layer = max(1, -(-n_ent // per))
    depth = 1
    while depth < 2 * per_layer * w.n_layers:
        depth *= 2
    cap = 64 if per <= 64 else 2048
    dc = DeviceCase(w, depth=depth, capacity=cap, sgl_capacity=n_ent * (w.n_layers + 2))
    try:
        bb = int(dc.ctx.layout.block_bytes)
        assert dc.ring.tutti_ring_set_iocb_bytes(4096 * bb, allow=(T.EINVAL,)) == T.EINVAL
        assert dc.ring.tutti_ring_set_iocb_bytes(bb - 16, allow=(T.EINVAL,)) == T.EINVAL
        dc.ring.tutti_ring_set_iocb_bytes(per * bb)
        for engine, sm_count in ((T.ENGINE_BULK, 0), (T.ENGINE_LDST, 8)):
            dc.ctx.tutti_set_option(T.OPT_COPY_ENGINE, engine)
            for l in range(w.n_layers):
                dc.pool_dev[l].copy_(torch.from_numpy(dc.pool_host[l]))
            rc, first, n = dc.ring.tutti_build_sqes_layers(dc.batch, 0, w.n_layers, T.OP_READ)
            assert n == per_layer
            for layer in range(w.n_layers):
                sq, sg, num, infos = dc.read_build(first + layer * n, n)
                orc, osq, osg, onum = dc.oracle_descriptors(layer, oracle.OP_READ, cap, per)
                assert orc == 0
                assert same_records(sq, osq) and same_records(sg, osg)
                assert list(num[:len(onum)]) == list(onum) and not num[len(onum):].any()
                assert all(i.status == 0 and i.bytes <= per * bb + 64 * bb for i in infos)
                assert sum(i.bytes for i in infos) == int(osg["len"].astype(np.uint64).sum())
            # issue the IOCBs of every layer in two launches, out of order
            half = (n * w.n_layers) // 2
            if half:
                dc.ring.tutti_kv_restore_layer(first + half, n * w.n_layers - half, sm_count)
                dc.ring.tutti_kv_restore_layer(first, half, sm_count)
            else:
                dc.ring.tutti_kv_restore_layer(first, n * w.n_layers, sm_count)
            rc, nbytes, err, done = dc.ring.tutti_ring_poll_range(first, n * w.n_layers, 5_000_000_000)
            assert (rc, err, done) == (T.OK, 0, n * w.n_layers)
            for layer in range(w.n_layers):
                assert np.array_equal(dc.pool_dev[layer].cpu().numpy(), dc.oracle_restore(layer))
        # back to IOCBs of a fixed number of contexts
        dc.ring.tutti_ring_set_iocb_bytes(0)
        rc, first, n = dc.ring.tutti_build_sqes(dc.batch, 0, T.OP_READ)
        sq, sg, num, infos = dc.read_build(first, n)
        orc, osq, osg, onum = dc.oracle_descriptors(0, oracle.OP_READ, cap)
        assert same_records(sq, osq) and n == max(1, -(-2 * len(w.obj_slot) // cap))
        dc.ring.tutti_kv_restore_layer(first, n)
        dc.poll_all(first, n)
    finally:
        dc.close()


@pytest.mark.parametrize("name", ["cfg2-small", "shared-prefix-8-requests", "cfg4-small",
                                  "cfg2-2dev-interleaved", "hnd-pool"])
@pytest.mark.parametrize("host_store", [False, True])
@pytest.mark.parametrize("min_ctx", [0, "median"])
def test_staged_transfer_matches_oracle(name, host_store, min_ctx):
    """Staged restore and save: the copy engines move every context between the store and a
    staging buffer in HBM (one copy per context), the kernels scatter / gather between that
    buffer and the pool.  The pool after a staged restore and the store after a staged save
    are the oracle's, byte for byte; descriptors are those of an ordinary build."""
    w = mk(name)
    dc = DeviceCase(w, host_store=host_store)
    try:
        dc.batch.plan_epoch = 11
        layer = w.n_layers - 1
        orc, osq, osg, onum = dc.oracle_descriptors(layer, oracle.OP_READ, 2048)
        # "median": the contexts below the median length stay on the zero-copy path (their
        # entries keep pointing into the store), the others go through the staging buffer
        lens = osq["len"].astype(np.uint64)
        min_ctx = int(np.median(lens)) if min_ctx == "median" else 0
        rc, n_ctx, n_st, need = dc.ring.tutti_stage_plan(dc.batch, min_ctx)
        assert n_ctx == len(osq) and n_st == int((lens >= min_ctx).sum())
        assert need == int(lens[lens >= min_ctx].sum())
        stage = torch.zeros(need + 64, dtype=torch.uint8, device=dc.dev)
        # a stage that is too small is refused before anything is enqueued
        assert dc.ring.tutti_stage_copy_layer(layer, T.OP_READ, stage.data_ptr(), need - 16,
                                              allow=(T.EINVAL,)) == T.EINVAL
        # restore: copies in, then the scatter kernel
        dc.ring.tutti_stage_copy_layer(layer, T.OP_READ, stage.data_ptr(), need)
        rc, first, n = dc.ring.tutti_build_sqes_staged(dc.batch, layer, T.OP_READ, stage.data_ptr(), need)
        sq, sg, num, infos = dc.read_build(first, n)
        assert same_records(sq, osq) and same_records(sg, osg)
        dc.ring.tutti_kv_restore_layer(first, n)
        cqes = dc.poll_all(first, n)
        assert all(c[1] == 0 for c in cqes)
        assert sum(c[2] for c in cqes) == int(osg["len"].astype(np.uint64).sum())
        want = dc.oracle_restore(layer)
        assert np.array_equal(dc.pool_dev[layer].cpu().numpy(), want)
        # save: the gather kernel, then copies out, into a zeroed store
        for t in dc.store_dev:
            t.zero_()
        stage.zero_()
        rc, first, n = dc.ring.tutti_build_sqes_staged(dc.batch, layer, T.OP_WRITE, stage.data_ptr(), need)
        dc.ring.tutti_kv_save_layer(first, n)
        dc.ring.tutti_stage_copy_layer(layer, T.OP_WRITE, stage.data_ptr(), need)
        assert all(c[1] == 0 for c in dc.poll_all(first, n))
        torch.cuda.synchronize()
        st_want = [np.zeros_like(s) for s in dc.store_host]
        dc.oracle_save(layer, want, st_want)
        for t, s in zip(dc.store_dev, st_want):
            assert np.array_equal(t.cpu().numpy(), s)
        # another batch on the ring invalidates nothing silently: a build for a batch the stage
        # plan has not seen is refused
        other = T.Batch(dc.batch.n_req, dc.batch.n_obj, dc.batch.n_blk, 12, dc.batch.hit_tokens,
                        dc.batch.obj_start, dc.batch.obj_slot, dc.batch.blk_start, dc.batch.block_ids)
        rc, *_ = dc.ring.tutti_build_sqes_staged(other, layer, T.OP_READ, stage.data_ptr(), need,
                                                 allow=(T.EINVAL,))
        assert rc == T.EINVAL
    finally:
        dc.close()


@pytest.mark.parametrize("name", ["cfg2-small", "shared-prefix-8-requests", "cfg4-small"])
@pytest.mark.parametrize("sm_count", [0, 8])
def test_staged_transfer_with_cut_iocbs_on_a_wrapping_ring(name, sm_count):
    """Staged transfers composed with the rest: IOCBs cut by bytes (several per layer, a context
    split between two of them), a ring so small that it wraps and a build meets TUTTI_EAGAIN
    until the host has polled, capped and all-SM launches, every layer in turn, both directions.
    Descriptors are the oracle's for the cut build, bytes are the oracle's."""
    w = mk(name)
    n_ent = 2 * len(w.block_ids)
    per = max(3, n_ent // 5)                      # about 5 IOCBs per layer
    per_layer = -(-n_ent // per)
    depth = 1
    while depth < 2 * per_layer:
        depth *= 2                                # room for two builds, not for three
    dc = DeviceCase(w, depth=depth, capacity=2048, sgl_capacity=3 * n_ent, host_store=True)
    try:
        bb = int(dc.ctx.layout.block_bytes)
        dc.ring.tutti_ring_set_iocb_bytes(per * bb)
        dc.batch.plan_epoch = 5
        rc, n_ctx, n_st, need = dc.ring.tutti_stage_plan(dc.batch, 0)
        stage_in = torch.zeros(need, dtype=torch.uint8, device=dc.dev)
        stage_out = torch.zeros(need, dtype=torch.uint8, device=dc.dev)
        orig = [s.copy() for s in dc.store_host]
        outstanding = []
        saw_eagain = False
        for it in range(3 * w.n_layers):
            layer = it % w.n_layers
            dc.pool_dev[layer].copy_(torch.from_numpy(dc.pool_host[layer]))
            want = dc.oracle_restore(layer)
            for op, stage in ((T.OP_READ, stage_in), (T.OP_WRITE, stage_out)):
                if op == T.OP_READ:
                    dc.ring.tutti_stage_copy_layer(layer, T.OP_READ, stage.data_ptr(), need)
                rc, first, n = dc.ring.tutti_build_sqes_staged(dc.batch, layer, op, stage.data_ptr(),
                                                               need, allow=(T.EAGAIN,))
                if rc == T.EAGAIN:
                    saw_eagain = True
                    for f, k in outstanding:
                        rcp, nbytes, err, done = dc.ring.tutti_ring_poll_range(f, k, 5_000_000_000)
                        assert (rcp, err, done) == (T.OK, 0, k)
                    outstanding = []
                    rc, first, n = dc.ring.tutti_build_sqes_staged(dc.batch, layer, op,
                                                                   stage.data_ptr(), need)
                assert n == per_layer
                if it < w.n_layers:
                    sq, sg, num, infos = dc.read_build(first, n)
                    orc, osq, osg, onum = dc.oracle_descriptors(layer, op, 2048, per)
                    assert orc == 0 and same_records(sq, osq) and same_records(sg, osg)
                    assert list(num[:len(onum)]) == list(onum)
                if op == T.OP_READ:
                    dc.ring.tutti_kv_restore_layer(first, n, sm_count)
                else:
                    dc.ring.tutti_kv_save_layer(first, n, sm_count)
                    dc.ring.tutti_stage_copy_layer(layer, T.OP_WRITE, stage.data_ptr(), need)
                outstanding.append((first, n))
            torch.cuda.synchronize()
            assert np.array_equal(dc.pool_dev[layer].cpu().numpy(), want)
        for f, k in outstanding:
            rcp, nbytes, err, done = dc.ring.tutti_ring_poll_range(f, k, 5_000_000_000)
            assert (rcp, err, done) == (T.OK, 0, k)
        assert saw_eagain
        # restore then save leaves the store as it was
        torch.cuda.synchronize()
        for t, s in zip(dc.store_dev, orig):
            assert np.array_equal(t.cpu().numpy(), s)
    finally:
        dc.close()
