"""The allocation-free restore entry point against the ring-based one.

tutti_kv_restore_layer_noalloc serves callers that cannot allocate device memory (all of
HBM already belongs to the engine's pools, or allocator calls are forbidden where they
run), so it works out of a fixed scratch array inside the library.  Its result must be
the very bytes the ring path produces — twice in a row, because the second call finds the
scratch as the first one left it.  Collected last on purpose."""
import numpy as np
import pytest
import torch

from paper_2605_03375_b200 import tutti as T
from paper_2605_03375_b200 import workload as wl
from tests.devcase import DeviceCase

pytestmark = pytest.mark.gpu


def test_noalloc_restore_matches_ring_path_twice():
    w = wl.config(2, 0.05, n_layers=3)
    dc = DeviceCase(w)
    try:
        cqe = torch.zeros(2, dtype=torch.int64, device=dc.dev)
        for layer in (2, 0):                                    # two calls in a row
            # existing entry points
            dc.pool_dev[layer].copy_(torch.from_numpy(dc.pool_host[layer]))
            rc, first, n = dc.ring.tutti_build_sqes(dc.batch, layer, T.OP_READ)
            dc.ring.tutti_kv_restore_layer(first, n)
            ref_cqes = dc.poll_all(first, n)
            ref = dc.pool_dev[layer].clone()
            # the allocation-free entry point, same inputs, fresh pool
            dc.pool_dev[layer].copy_(torch.from_numpy(dc.pool_host[layer]))
            before = torch.cuda.memory_allocated(dc.dev)
            p = dc.pool_dev[layer].data_ptr()
            cqe.fill_(-1)
            T.tutti_kv_restore_layer_noalloc(
                dc.ctx.geom, 0, layer, dc.batch, p + dc.k_off, p + dc.v_off, dc.stride,
                w.n_pool_blocks, [t.data_ptr() for t in dc.store_dev],
                [t.numel() for t in dc.store_dev], cqe.data_ptr(), None)
            torch.cuda.synchronize()
            assert torch.cuda.memory_allocated(dc.dev) == before
            got = cqe.cpu().numpy().view(np.uint32)
            assert got[0] == 0 and got[1] == 0                  # iocb_idx 0, status OK
            assert int(cqe[1].item()) == sum(c[2] for c in ref_cqes)
            assert torch.equal(dc.pool_dev[layer], ref)         # bit-exact, as everywhere here
            assert np.array_equal(ref.cpu().numpy(), dc.oracle_restore(layer))
    finally:
        dc.close()


def test_noalloc_rejects_oversized_batch():
    w = wl.config(2, 0.05, n_layers=1)
    dc = DeviceCase(w)
    try:
        big = T.Batch(dc.batch.n_req, 2049, dc.batch.n_blk, 0, dc.batch.hit_tokens,
                      dc.batch.obj_start, dc.batch.obj_slot, dc.batch.blk_start,
                      dc.batch.block_ids)
        cqe = torch.zeros(2, dtype=torch.int64, device=dc.dev)
        p = dc.pool_dev[0].data_ptr()
        args = (p + dc.k_off, p + dc.v_off, dc.stride, w.n_pool_blocks,
                [t.data_ptr() for t in dc.store_dev], [t.numel() for t in dc.store_dev],
                cqe.data_ptr(), None)
        assert T.tutti_kv_restore_layer_noalloc(dc.ctx.geom, 0, 0, big, *args,
                                                allow=(T.EINVAL,)) == T.EINVAL
        big.n_obj = dc.batch.n_obj
        big.n_blk = 32769
        assert T.tutti_kv_restore_layer_noalloc(dc.ctx.geom, 0, 0, big, *args,
                                                allow=(T.EINVAL,)) == T.EINVAL
    finally:
        dc.close()
