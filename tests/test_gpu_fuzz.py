"""Seeded random geometries and batches: every case checks descriptors, restore and save
against the oracle, with a random engine, SM cap and IOCB capacity, a third of them as staged
transfers.  Also two rings driven
concurrently on two streams."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_03375_b200 import tutti as T
from paper_2605_03375_b200 import workload as wl
from tests.devcase import DeviceCase

pytestmark = pytest.mark.gpu


def random_workload(seed):
    rng = np.random.default_rng(1000 + seed)
    heads = int(rng.choice([1, 2, 3, 4, 8]))
    dim = int(rng.choice([8, 16, 32, 64, 128]))
    elem = int(rng.choice([1, 2, 4]))
    while (heads * dim * elem) % 16:
        dim *= 2
    bt = int(rng.choice([1, 2, 4, 8, 16, 32]))
    obj_blocks = int(rng.choice([1, 2, 4, 16]))
    n_req = int(rng.integers(1, 7))
    hits = [int(rng.integers(0, 40)) * bt for _ in range(n_req)]
    if sum(hits) == 0:
        hits[0] = 3 * bt
    hnd = bool(rng.random() < 0.35) and (dim * elem) % 16 == 0   # the library's rule for HND
    return wl.make_workload(
        f"fuzz{seed}", seed=5000 + seed, n_layers=int(rng.integers(1, 4)), hit_tokens=hits,
        block_tokens=bt, obj_tokens=bt * obj_blocks, n_kv_heads=heads, head_dim=dim,
        elem_bytes=elem, n_devices=int(rng.choice([1, 1, 2, 3])),
        layout=int(rng.choice([wl.LAYOUT_FILE_MAJOR, wl.LAYOUT_LAYER_MAJOR])),
        slot_mean_run=float(rng.choice([1.0, 2.0, 6.0])), slot_space_factor=float(rng.choice([1.1, 2.0])),
        pool_round=64, pool_interleaved=bool(rng.random() < 0.4), pool_hnd=hnd,
        pool_pad_bytes=int(rng.choice([0, 0, 16, 256])),
        # a third of the cases: requests share leading objects (read once, repeat entries)
        shared_prefix_frac=float(np.random.default_rng(9000 + seed).choice([0.0, 0.0, 0.5, 1.0]))), rng


@pytest.mark.parametrize("seed", range(int(__import__("os").environ.get("TUTTI_FUZZ_CASES", "40"))))
def test_random_case(seed):
    w, rng = random_workload(seed)
    capacity = int(rng.choice([1, 3, 64, 2048]))
    n_items = 2 * len(w.obj_slot)
    depth = 1
    while depth < 2 * max(1, -(-n_items // capacity)):
        depth *= 2
    dc = DeviceCase(w, depth=depth, capacity=capacity)
    try:
        dc.ctx.tutti_set_option(T.OPT_COPY_ENGINE, int(rng.choice([0, 1, 2])))
        sm_count = int(rng.choice([0, 0, 3, 16]))
        layer = int(rng.integers(0, w.n_layers))
        flag = oracle.OP_HND if w.pool_hnd else 0
        # a third of the cases move the bytes staged (copy engine between store and a staging
        # buffer, kernels between that buffer and the pool), with every context staged or only
        # those of at least the median length
        srng = np.random.default_rng(7000 + seed)
        staged = srng.random() < 0.35
        stage = None
        if staged:
            orc, osq, osg, onum = dc.oracle_descriptors(layer, oracle.OP_READ, capacity)
            lens = osq["len"].astype(np.uint64)
            min_ctx = int(np.median(lens)) if (len(lens) and srng.random() < 0.5) else 0
            dc.batch.plan_epoch = 1 + seed
            rc, n_ctx, n_st, need = dc.ring.tutti_stage_plan(dc.batch, min_ctx)
            assert (n_ctx, n_st) == (len(lens), int((lens >= min_ctx).sum()))
            assert need == int(lens[lens >= min_ctx].sum())
            stage = torch.zeros(max(need, 16), dtype=torch.uint8, device=dc.dev)

        def build(op):
            if not staged:
                return dc.ring.tutti_build_sqes(dc.batch, layer, op)
            if op == T.OP_READ:
                dc.ring.tutti_stage_copy_layer(layer, op, stage.data_ptr(), stage.numel())
            return dc.ring.tutti_build_sqes_staged(dc.batch, layer, op, stage.data_ptr(), stage.numel())

        rc, first, n = build(T.OP_READ)
        sq, sg, num, infos = dc.read_build(first, n)
        orc, osq, osg, onum = dc.oracle_descriptors(layer, oracle.OP_READ, capacity)
        assert orc == 0 and all(i.status == 0 for i in infos)
        assert sq.tobytes() == osq.tobytes() and sg.tobytes() == osg.tobytes()
        assert np.all(osq["opcode"] == flag)
        assert list(num[:len(onum)]) == list(onum) and not num[len(onum):].any()
        dc.ring.tutti_kv_restore_layer(first, n, sm_count)
        cqes = dc.poll_all(first, n)
        assert all(c[1] == 0 for c in cqes)
        assert sum(c[2] for c in cqes) == int(osg["len"].astype(np.uint64).sum())
        want = dc.oracle_restore(layer)
        assert np.array_equal(dc.pool_dev[layer].cpu().numpy(), want)
        for t in dc.store_dev:
            t.zero_()
        rc, first, n = build(T.OP_WRITE)
        dc.ring.tutti_kv_save_layer(first, n, sm_count)
        if staged:
            dc.ring.tutti_stage_copy_layer(layer, T.OP_WRITE, stage.data_ptr(), stage.numel())
        assert all(c[1] == 0 for c in dc.poll_all(first, n))
        torch.cuda.synchronize()
        st_want = [np.zeros_like(s) for s in dc.store_host]
        dc.oracle_save(layer, want, st_want)
        for t, s in zip(dc.store_dev, st_want):
            assert np.array_equal(t.cpu().numpy(), s)
    finally:
        dc.close()


def test_two_rings_on_two_streams():
    """Two rings of one context, each on its own stream, restoring different layers at the
    same time: neither disturbs the other."""
    w = wl.config(2, 0.06, n_layers=4)
    dc = DeviceCase(w)
    ring2 = T.Ring(dc.ctx, 8, 2048, 4 * len(w.block_ids), 2 * len(w.obj_slot))
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    try:
        for rep in range(3):
            for l in range(w.n_layers):
                dc.pool_dev[l].copy_(torch.from_numpy(dc.pool_host[l]))
            torch.cuda.synchronize()
            issued = []
            for l in range(0, w.n_layers, 2):
                a = dc.ring.tutti_build_sqes(dc.batch, l, T.OP_READ, stream=s1)
                b = ring2.tutti_build_sqes(dc.batch, l + 1, T.OP_READ, stream=s2)
                dc.ring.tutti_kv_restore_layer(a[1], a[2], stream=s1)
                ring2.tutti_kv_restore_layer(b[1], b[2], 8, stream=s2)
                issued.append((a, b))
            for a, b in issued:
                for i in range(a[1], a[1] + a[2]):
                    rc, cqe = dc.ring.tutti_ring_poll(i, 5_000_000_000)
                    assert rc == T.OK and cqe.status == 0
                for i in range(b[1], b[1] + b[2]):
                    rc, cqe = ring2.tutti_ring_poll(i, 5_000_000_000)
                    assert rc == T.OK and cqe.status == 0
            torch.cuda.synchronize()
            for l in range(w.n_layers):
                assert np.array_equal(dc.pool_dev[l].cpu().numpy(), dc.oracle_restore(l))
    finally:
        torch.cuda.synchronize()
        ring2.close()
        dc.close()


@pytest.mark.parametrize("seed", range(6))
def test_random_op_sequences_on_a_small_ring(seed):
    """Random interleavings of build / restore / save / poll on a ring that is too small to
    hold everything: TUTTI_EAGAIN is answered by polling the oldest work, and at the end the
    pools and the store hold exactly what the oracle gets by applying the same operations in
    issue order."""
    rng = np.random.default_rng(77 + seed)
    w = wl.config(2, 0.03, n_layers=3, n_devices=int(rng.choice([1, 2])),
                  pool_interleaved=bool(seed & 1), slot_mean_run=2.0)
    n_blk, n_obj = len(w.block_ids), len(w.obj_slot)
    capacity = int(rng.choice([4, 16, 2048]))
    per_build = max(1, -(-2 * n_obj // capacity))
    depth = 1
    while depth < 2 * per_build:
        depth *= 2
    dc = DeviceCase(w, depth=depth, capacity=capacity, sgl_capacity=int(2 * n_blk * 2.5))
    try:
        dc.ctx.tutti_set_option(T.OPT_COPY_ENGINE, int(rng.choice([1, 2])))
        pools = {l: dc.pool_host[l].copy() for l in range(w.n_layers)}
        store = [s.copy() for s in dc.store_host]
        outstanding = []                     # (first, n) in issue order
        n_again = 0

        def poll_oldest():
            first, n = outstanding.pop(0)
            assert all(c[1] == 0 for c in dc.poll_all(first, n))

        for step in range(40):
            layer = int(rng.integers(0, w.n_layers))
            op = T.OP_READ if rng.random() < 0.6 else T.OP_WRITE
            if step % 7 == 3:                # scribble over a pool so that saves move new data
                noise = torch.randint(0, 255, (dc.pool_dev[layer].numel(),), dtype=torch.uint8,
                                      device=dc.dev)
                torch.cuda.synchronize()
                dc.pool_dev[layer].copy_(noise)
                pools[layer] = noise.cpu().numpy()
            while True:
                rc, first, n = dc.ring.tutti_build_sqes(dc.batch, layer, op, allow=(T.EAGAIN,))
                if rc == T.OK:
                    break
                n_again += 1
                assert outstanding, "ring full with nothing outstanding"
                poll_oldest()
            sm = int(rng.choice([0, 0, 4]))
            if op == T.OP_READ:
                dc.ring.tutti_kv_restore_layer(first, n, sm)
                assert oracle.restore_layer(dc.og, layer, dc.obatch, store, pools[layer], dc.k_off,
                                            dc.v_off, dc.stride, w.n_pool_blocks) == 0
            else:
                dc.ring.tutti_kv_save_layer(first, n, sm)
                assert oracle.save_layer(dc.og, layer, dc.obatch, store, pools[layer], dc.k_off,
                                         dc.v_off, dc.stride, w.n_pool_blocks) == 0
            outstanding.append((first, n))
            if rng.random() < 0.3 and outstanding:
                poll_oldest()
        while outstanding:
            poll_oldest()
        torch.cuda.synchronize()
        for l in range(w.n_layers):
            assert np.array_equal(dc.pool_dev[l].cpu().numpy(), pools[l])
        for t, s in zip(dc.store_dev, store):
            assert np.array_equal(t.cpu().numpy(), s)
        assert n_again > 0 or depth >= 80 * per_build
    finally:
        dc.close()


@pytest.mark.parametrize("seed", range(12))
def test_random_host_prepared_descriptors(seed):
    """CPU-prepared IOCBs with entries cut at random 16-byte boundaries (differing lengths),
    in both directions and on both engines."""
    rng = np.random.default_rng(300 + seed)
    w = wl.config(2, 0.03, n_layers=2, n_devices=int(rng.choice([1, 2])), slot_mean_run=2.0,
                  pool_interleaved=bool(seed & 1))
    dc = DeviceCase(w, depth=8, capacity=2048, sgl_capacity=64 * len(w.block_ids))
    try:
        dc.ctx.tutti_set_option(T.OPT_COPY_ENGINE, int(rng.choice([1, 2])))
        layer = int(rng.integers(0, 2))
        op = T.OP_READ if seed % 3 else T.OP_WRITE
        orc, osq, osg, onum = dc.oracle_descriptors(layer, op, 2048)
        # cut every entry into 1..4 pieces at random multiples of 16 bytes
        addr, ln, ident, counts = [], [], [], []
        for e in osg:
            total = int(e["len"])
            k = int(rng.integers(1, 5))
            cuts = sorted(set((rng.integers(1, total // 16, size=k - 1) * 16).tolist())) if k > 1 else []
            edges = [0] + cuts + [total]
            counts.append(len(edges) - 1)
            for a, b in zip(edges[:-1], edges[1:]):
                addr.append(int(e["addr"]) + a)
                ln.append(b - a)
                ident.append(int(e["id"]))
        sg2 = np.zeros(len(addr), dtype=osg.dtype)
        sg2["addr"], sg2["len"], sg2["id"] = addr, ln, ident
        cum = np.concatenate([[0], np.cumsum(counts)])
        sq2 = osq.copy()
        sq2["sgl_first"] = cum[osq["sgl_first"]]
        sq2["sgl_count"] = cum[osq["sgl_first"] + osq["sgl_count"]] - cum[osq["sgl_first"]]
        if op == T.OP_WRITE:
            noise = torch.randint(0, 255, (dc.pool_dev[layer].numel(),), dtype=torch.uint8, device=dc.dev)
            dc.pool_dev[layer].copy_(noise)
            for t in dc.store_dev:
                t.zero_()
        rc, first = dc.ring.tutti_ring_reserve(1, len(sg2))
        dc.ring.tutti_ring_fill_host(first, sq2, sg2)
        info, _ = dc.ring.tutti_ring_read_iocb(first)
        assert info.entry_len == 0 or len(set(ln)) == 1
        sm = int(rng.choice([0, 5]))
        (dc.ring.tutti_kv_restore_layer if op == T.OP_READ else dc.ring.tutti_kv_save_layer)(first, 1, sm)
        (idx, status, nbytes), = dc.poll_all(first, 1)
        assert status == 0 and nbytes == int(osg["len"].astype(np.uint64).sum())
        if op == T.OP_READ:
            assert np.array_equal(dc.pool_dev[layer].cpu().numpy(), dc.oracle_restore(layer))
        else:
            st = [np.zeros_like(s) for s in dc.store_host]
            dc.oracle_save(layer, dc.pool_dev[layer].cpu().numpy(), st)
            for t, s in zip(dc.store_dev, st):
                assert np.array_equal(t.cpu().numpy(), s)
    finally:
        dc.close()


@pytest.mark.parametrize("seed", range(10))
def test_random_multi_layer_builds_and_launches(seed):
    """Several layers built by one launch and executed by launches that cover random ranges
    of their IOCBs."""
    w, rng = random_workload(700 + seed)
    w = wl.make_workload("ml", seed=w.seed, n_layers=int(rng.integers(2, 6)),
                         hit_tokens=w.hit_tokens, block_tokens=w.block_tokens,
                         obj_tokens=w.obj_tokens, n_kv_heads=w.n_kv_heads, head_dim=w.head_dim,
                         elem_bytes=w.elem_bytes, n_devices=w.n_devices, layout=w.layout,
                         pool_round=64, pool_interleaved=w.pool_interleaved, pool_hnd=w.pool_hnd,
                         pool_pad_bytes=w.pool_pad_bytes, slot_mean_run=2.0)
    capacity = int(rng.choice([2, 16, 2048]))
    per = max(1, -(-2 * len(w.obj_slot) // capacity))
    depth = 1
    while depth < 2 * per * w.n_layers:
        depth *= 2
    dc = DeviceCase(w, depth=depth, capacity=capacity,
                    sgl_capacity=max(64, 2 * len(w.block_ids) * (w.n_layers + 1)))
    try:
        dc.ctx.tutti_set_option(T.OPT_COPY_ENGINE, int(rng.choice([0, 1, 2])))
        l0 = int(rng.integers(0, w.n_layers - 1))
        nl = int(rng.integers(1, w.n_layers - l0 + 1))
        rc, first, per_layer = dc.ring.tutti_build_sqes_layers(dc.batch, l0, nl, T.OP_READ)
        total = per_layer * nl
        # execute in random consecutive pieces
        at = 0
        while at < total:
            k = int(rng.integers(1, total - at + 1))
            dc.ring.tutti_kv_restore_layer(first + at, k, int(rng.choice([0, 0, 7])))
            at += k
        cqes = dc.poll_all(first, total)
        assert all(c[1] == 0 for c in cqes)
        for l in range(l0, l0 + nl):
            assert np.array_equal(dc.pool_dev[l].cpu().numpy(), dc.oracle_restore(l))
        for l in list(range(0, l0)) + list(range(l0 + nl, w.n_layers)):
            assert np.array_equal(dc.pool_dev[l].cpu().numpy(), dc.pool_host[l])   # untouched
    finally:
        dc.close()
