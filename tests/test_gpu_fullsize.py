"""Config 2 at full size, in the launch configuration the bench times: sampled tokens the
oracle locates one by one, whole layers compared byte for byte with the oracle's run on host
copies, untouched blocks, and the save direction."""
import argparse

import numpy as np
import pytest
import torch

import bench
import oracle
from tests.devcase import verify_replica_samples
from paper_2605_03375_b200 import tutti as T

pytestmark = pytest.mark.gpu


def _args(**kw):
    d = dict(config=2, scale=1.0, layers=0, engine=0, resident_layers=3, ioctx_per_iocb=2048,
             ctas_per_sm=0, bulk_warps=0, bulk_stages=0, claim=0, layers_per_launch=0)
    d.update(kw)
    return argparse.Namespace(**d)


@pytest.mark.parametrize("engine", [0, 1])
def test_config2_full_size(engine):
    rep = bench.Replica(_args(engine=engine), 0)
    try:
        w = rep.w
        assert (w.n_layers, w.n_req, len(w.block_ids)) == (32, 8, 16384)
        pools_before = [p.clone() for p in rep.pool]
        moved = rep.step(directions=(T.OP_READ,))
        assert moved == 32 * rep.payload_per_layer == 32 << 30
        torch.cuda.synchronize()
        assert verify_replica_samples(rep, 512)
        # whole layers against the oracle on host copies (layers 29..31 own the 3 pool buffers)
        og = oracle.geom(1, w.n_kv_heads, w.head_dim, w.elem_bytes, w.block_tokens, w.obj_tokens,
                         w.n_devices, w.layout, w.n_slots)
        ob = (w.hit_tokens, w.obj_start, w.obj_slot, w.blk_start, w.block_ids)
        lb = int(rep.lo.stride_layer)
        for l in (30, 31):
            store_l = [s[l * lb:(l + 1) * lb].cpu().numpy() for s in rep.store]
            want = pools_before[l % rep.R].cpu().numpy()
            assert oracle.restore_layer(og, 0, ob, store_l, want, 0, rep.v_off, rep.block_bytes,
                                        w.n_pool_blocks) == 0
            got = rep.pool[l % rep.R].cpu().numpy()
            assert np.array_equal(got, want)
            # blocks outside the block table kept their background bytes
            before = pools_before[l % rep.R].cpu().numpy()
            for b in w.occupied_blocks[::97]:
                for plane in (0, rep.v_off):
                    o = plane + int(b) * rep.block_bytes
                    assert np.array_equal(got[o:o + rep.block_bytes], before[o:o + rep.block_bytes])
        # save direction: zero one layer of the store, save, compare with the oracle's save
        l = 31
        orig = rep.store[0][l * lb:(l + 1) * lb].clone()
        rep.store[0][l * lb:(l + 1) * lb].zero_()
        rep.batch.plan_epoch = 0
        rc, first, n = rep.ring.tutti_build_sqes(rep.batch, l, T.OP_WRITE)
        rep.ring.tutti_kv_save_layer(first, n)
        for i in range(first, first + n):
            rc, cqe = rep.ring.tutti_ring_poll(i, 10_000_000_000)
            assert rc == T.OK and cqe.status == 0
        want_store = [np.zeros(lb, dtype=np.uint8)]
        assert oracle.save_layer(og, 0, ob, want_store, rep.pool[l % rep.R].cpu().numpy(), 0,
                                 rep.v_off, rep.block_bytes, w.n_pool_blocks) == 0
        got_store = rep.store[0][l * lb:(l + 1) * lb].cpu().numpy()
        assert np.array_equal(got_store, want_store[0])
        cov = want_store[0] != 0
        assert np.array_equal(got_store[cov], orig.cpu().numpy()[cov])     # round trip
    finally:
        rep.close()


def test_config2_full_size_every_layer_resident():
    """The bench's own residency: all 32 pool layers and the whole store in HBM, one build
    launch and one copy launch for the whole pass.  The oracle names, token by token, the
    store bytes and pool bytes that must be equal — sampled from every layer — and two
    early layers are compared whole."""
    rep = bench.Replica(_args(resident_layers=0), 0)
    try:
        w = rep.w
        if rep.R < w.n_layers:
            pytest.skip("not enough free HBM for 32 resident pool layers")
        assert rep.layers_per_launch == 32
        whole = (3, 17)
        before = {l: rep.pool[l].clone() for l in whole}
        assert rep.step(directions=(T.OP_READ,)) == 32 << 30
        torch.cuda.synchronize()
        assert verify_replica_samples(rep, 4096)           # layers drawn uniformly from all 32
        og = oracle.geom(1, w.n_kv_heads, w.head_dim, w.elem_bytes, w.block_tokens, w.obj_tokens,
                         w.n_devices, w.layout, w.n_slots)
        ob = (w.hit_tokens, w.obj_start, w.obj_slot, w.blk_start, w.block_ids)
        lb = int(rep.lo.stride_layer)
        for l in whole:
            store_l = [s[l * lb:(l + 1) * lb].cpu().numpy() for s in rep.store]
            want = before[l].cpu().numpy()
            assert oracle.restore_layer(og, 0, ob, store_l, want, 0, rep.v_off, rep.block_bytes,
                                        w.n_pool_blocks) == 0
            assert np.array_equal(rep.pool[l].cpu().numpy(), want)
        # and the save of the whole pass puts every sampled token back where the oracle says
        for s_ in rep.store:
            s_.zero_()
        assert rep.step(directions=(T.OP_WRITE,)) == 32 << 30
        torch.cuda.synchronize()
        assert verify_replica_samples(rep, 4096)
    finally:
        rep.close()


def test_one_object_per_block_at_full_batch_size():
    """The paper's own granularity (one object per paged block) on the config-2 batch: 32,768
    items — more than the shared-memory sort holds, so the plan sorts in ring scratch — and
    sixteen IOCBs per layer."""
    from paper_2605_03375_b200 import workload as wl
    from tests.devcase import DeviceCase
    w = wl.config(2, 1.0, n_layers=1, obj_tokens=16, slot_mean_run=1.3, slot_space_factor=2.0)
    assert len(w.obj_slot) == 16384
    dc = DeviceCase(w, depth=64, capacity=2048)
    try:
        layer = 0
        rc, first, n = dc.ring.tutti_build_sqes(dc.batch, layer, T.OP_READ)
        assert n == 16
        sq, sg, num, infos = dc.read_build(first, n)
        orc, osq, osg, onum = dc.oracle_descriptors(layer, oracle.OP_READ, 2048)
        assert orc == 0 and len(osq) > 2048
        assert sq.tobytes() == osq.tobytes() and sg.tobytes() == osg.tobytes()
        assert list(num[:len(onum)]) == list(onum) and not num[len(onum):].any()
        dc.ring.tutti_kv_restore_layer(first, n)
        cqes = dc.poll_all(first, n)
        assert sum(c[2] for c in cqes) == 1 << 30 and all(c[1] == 0 for c in cqes)
        assert np.array_equal(dc.pool_dev[layer].cpu().numpy(), dc.oracle_restore(layer))
    finally:
        dc.close()


def _whole_layer_check(rep, l, pool_before):
    """Layer l's pool buffer against the oracle's restore on host copies."""
    w = rep.w
    og = oracle.geom(1, w.n_kv_heads, w.head_dim, w.elem_bytes, w.block_tokens, w.obj_tokens,
                     w.n_devices, w.layout, w.n_slots)
    ob = (w.hit_tokens, w.obj_start, w.obj_slot, w.blk_start, w.block_ids)
    lb = int(rep.lo.stride_layer)
    store_l = [s[l * lb:(l + 1) * lb].cpu().numpy() for s in rep.store]
    want = pool_before.cpu().numpy()
    assert oracle.restore_layer(og, 0, ob, store_l, want, 0, rep.v_off, rep.block_bytes,
                                w.n_pool_blocks) == 0
    assert np.array_equal(rep.pool[l % rep.R].cpu().numpy(), want)


def test_config4_full_size_per_layer():
    """1-token pages, 64 requests with partial hits: a layer at full size (about 2 GiB in
    2 KiB fragments, >1 M SGL entries), 64 contexts per IOCB so that a layer spans dozens of
    IOCBs; sampled tokens and one whole layer."""
    rep = bench.Replica(_args(config=4, layers=2, resident_layers=2, ioctx_per_iocb=64), 0)
    try:
        w = rep.w
        assert w.n_req == 64 and w.block_tokens == 1 and len(w.block_ids) > 400_000
        before = rep.pool[1].clone()
        moved = rep.step(directions=(T.OP_READ,))
        assert moved == 2 * rep.payload_per_layer
        assert verify_replica_samples(rep, 512)
        _whole_layer_check(rep, 1, before)
    finally:
        rep.close()


def test_config3_full_size_per_layer_from_pinned_host():
    """Llama-3-70B-shaped batch (2 x 128K tokens, 1024-token objects) restored zero-copy from
    pinned host memory, then saved back to it."""
    rep = bench.Replica(_args(config=3, layers=2, resident_layers=2), 0, host_store=True)
    try:
        w = rep.w
        assert (w.n_req, w.obj_tokens, len(w.block_ids)) == (2, 1024, 16384)
        before = rep.pool[1].clone()
        rep.step(directions=(T.OP_READ,))
        assert verify_replica_samples(rep, 256)
        _whole_layer_check(rep, 1, before)
        orig = [s.clone() for s in rep.store]
        for s in rep.store:
            s.zero_()
        rep.step(directions=(T.OP_WRITE,))
        torch.cuda.synchronize()
        for s, o in zip(rep.store, orig):
            cov = s != 0
            assert torch.equal(s[cov], o[cov]) and int(cov.sum()) > 0.9 * 2 * rep.payload_per_layer
    finally:
        rep.close()


@pytest.mark.parametrize("sm_count", [8, 32])
def test_config5_capped_restore_beside_a_gemm(sm_count):
    """Config 2's restore as persistent CTAs inside a green-context SM partition while bf16
    GEMMs run in the other partition: the bytes are still exactly the oracle's."""
    rep = bench.Replica(_args(config=2, layers=2, resident_layers=2), 0)
    try:
        try:
            io_s, comp_s, got_io, got_comp = rep.ctx.tutti_sm_partition_create(sm_count)
        except T.TuttiError as e:
            pytest.skip(f"green contexts unavailable: {e}")
        assert got_io >= sm_count and got_io + got_comp <= 148
        io_stream = torch.cuda.ExternalStream(io_s, device=rep.dev)
        comp_stream = torch.cuda.ExternalStream(comp_s, device=rep.dev)
        a = torch.randn(4096, 4096, device=rep.dev, dtype=torch.bfloat16)
        c = torch.empty_like(a)
        with torch.cuda.stream(comp_stream):
            torch.matmul(a, a, out=c)
        torch.cuda.synchronize()
        ref = (a.float() @ a.float())
        before = rep.pool[1].clone()
        with torch.cuda.stream(comp_stream):
            for _ in range(60):
                torch.matmul(a, a, out=c)
        rep.stream = io_stream
        rep.two_streams = False
        moved = rep.step(sm_count=got_io, directions=(T.OP_READ,))
        torch.cuda.synchronize()
        assert moved == 2 * rep.payload_per_layer
        assert verify_replica_samples(rep, 256)
        _whole_layer_check(rep, 1, before)
        assert torch.allclose(c.float(), ref, rtol=2e-2, atol=2.0)       # the GEMM was not disturbed
        rep.ctx.tutti_sm_partition_destroy()
    finally:
        rep.close()


def test_config2_staged_duplex_pass_from_pinned_host():
    """The staged pass the bench's end-to-end leg times (copy engines between the pinned-host
    store and staging buffers in HBM, kernels between staging and pool, both directions at
    once): after it, every layer's pool is the oracle's restore, and the store, which every
    layer was saved back to, still holds its bytes."""
    rep = bench.Replica(_args(config=2, layers=3, resident_layers=3), 0, host_store=True)
    try:
        w = rep.w
        assert (w.n_req, len(w.block_ids)) == (8, 16384)
        before = [p.clone() for p in rep.pool]
        orig = [s.clone() for s in rep.store]
        moved = rep.step_staged(upload_tables=True)
        moved += rep.finish_staged()
        torch.cuda.synchronize()
        assert moved == 2 * w.n_layers * rep.payload_per_layer
        assert verify_replica_samples(rep, 256)
        for l in range(w.n_layers):
            _whole_layer_check(rep, l, before[l])
        for s, o in zip(rep.store, orig):
            assert torch.equal(s, o)
        # the save half on its own: into a zeroed store, the covered bytes come back
        for s in rep.store:
            s.zero_()
        need = rep.stage_bufs[2].numel()
        l = w.n_layers - 1
        rc, fw, nw = rep.ring.tutti_build_sqes_staged(rep.batch, l, T.OP_WRITE,
                                                      rep.stage_bufs[2].data_ptr(), need,
                                                      stream=rep.stream)
        rep.ring.tutti_kv_save_layer(fw, nw, 0, stream=rep.stream)
        rep.ring.tutti_stage_copy_layer(l, T.OP_WRITE, rep.stage_bufs[2].data_ptr(), need,
                                        stream=rep.stream)
        assert rep.poll_list([(fw, nw)]) == rep.payload_per_layer
        torch.cuda.synchronize()
        lb = int(rep.lo.stride_layer)
        for s, o in zip(rep.store, orig):
            cov = s != 0
            assert torch.equal(s[cov], o[cov])
            assert int(cov[l * lb:(l + 1) * lb].sum()) > 0.9 * rep.payload_per_layer
            assert int(cov.sum()) == int(cov[l * lb:(l + 1) * lb].sum())
    finally:
        rep.close()
