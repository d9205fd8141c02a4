"""Config 2 at full size, in the launch configuration the bench times: sampled tokens the
oracle locates one by one, whole layers compared byte for byte with the oracle's run on host
copies, untouched blocks, and the save direction."""
import argparse

import numpy as np
import pytest
import torch

import bench
import oracle
from paper_2605_03375_b200 import tutti as T

pytestmark = pytest.mark.gpu


def _args(**kw):
    d = dict(config=2, scale=1.0, layers=0, engine=0, resident_layers=3, ioctx_per_iocb=2048,
             ctas_per_sm=0, bulk_warps=0, bulk_stages=0, claim=0)
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
        assert rep.verify_samples(512)
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
