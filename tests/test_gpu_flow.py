"""The pieces together, as a serving engine would use them: chunk keys go through the
CPU-side file pool, a finished request's KV is saved layer by layer, and a later request
that shares a prefix has it restored into other pool blocks — checked against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_03375_b200 import tutti as T
from paper_2605_03375_b200 import workload as wl
from tests import hostcase as hc

pytestmark = pytest.mark.gpu


def test_save_then_prefix_hit_restore():
    L, bt, ot, n_pool, n_slots = 3, 16, 256, 512, 64
    dev = torch.device("cuda", 0)
    geom = T.Geom(L, 8, 128, 2, bt, ot, 1, T.LAYOUT_LAYER_MAJOR, n_slots)
    ctx = T.Context(geom, 0)
    lo = ctx.layout
    og = oracle.geom(L, 8, 128, 2, bt, ot, 1, oracle.LAYER_MAJOR, n_slots)
    bb = int(lo.block_bytes)
    store = torch.zeros(int(lo.dev_bytes), dtype=torch.uint8, device=dev)
    ctx.tutti_store_register(0, store.data_ptr(), store.numel())
    pools = []
    for l in range(L):
        p = wl.fill_u16_torch(99, 0x200 + l, 0, n_pool * bb, dev).view(torch.uint8)
        pools.append(p)
        ctx.tutti_pool_register(l, p.data_ptr(), p.data_ptr() + n_pool * bb, bb, n_pool)
    ring = T.Ring(ctx, 16, 2048, 8192, 256)
    files = T.FilePool(n_slots)
    rng = np.random.default_rng(5)

    def batch_of(hit, slots, blocks):
        t = [torch.tensor(a, dtype=torch.int32, device=dev) for a in
             ([hit], [0, len(slots)], slots, [0, len(blocks)], blocks)]
        return T.make_batch(*t), ([hit], [0, len(slots)], slots, [0, len(blocks)], blocks)

    def run(batch, op):
        for l in range(L):
            rc, first, n = ring.tutti_build_sqes(batch, l, op)
            (ring.tutti_kv_restore_layer if op == T.OP_READ else ring.tutti_kv_save_layer)(first, n)
            for i in range(first, first + n):
                rc, cqe = ring.tutti_ring_poll(i, 5_000_000_000)
                assert rc == T.OK and cqe.status == 0

    # request A: 5 chunks (1280 tokens) living in random pool blocks; its KV is saved
    keys_a = [1000 + i for i in range(5)]
    blocks_a = rng.permutation(n_pool)[:5 * 16].tolist()
    slots_a = [files.tutti_filepool_insert(k)[1] for k in keys_a]
    assert slots_a == [0, 1, 2, 3, 4]
    ba, oa = batch_of(1280, slots_a, blocks_a)
    run(ba, T.OP_WRITE)
    # request B shares the first 3 chunks, then diverges; only the shared prefix is restored,
    # into different blocks
    keys_b = np.array(keys_a[:3] + [7777, 7778], dtype=np.uint64)
    hit_slots = files.tutti_filepool_match_prefix(keys_b, pin=True).tolist()
    assert hit_slots == [0, 1, 2]
    free_blocks = [b for b in rng.permutation(n_pool).tolist() if b not in blocks_a]
    blocks_b = free_blocks[:3 * 16]
    pools_before = [p.clone() for p in pools]
    bb_, ob = batch_of(3 * 256, hit_slots, blocks_b)
    run(bb_, T.OP_READ)
    torch.cuda.synchronize()
    store_host = [store.cpu().numpy()]
    for l in range(L):
        got = pools[l].cpu().numpy()
        want = pools_before[l].cpu().numpy()
        assert oracle.restore_layer(og, l, ob, store_host, want, 0, n_pool * bb, bb, n_pool) == 0
        assert np.array_equal(got, want)
        # the restored blocks hold request A's KV for the shared tokens, plane by plane
        for plane in (0, n_pool * bb):
            for j in range(3 * 16):
                a = plane + blocks_a[j] * bb
                b = plane + blocks_b[j] * bb
                assert np.array_equal(got[a:a + bb], got[b:b + bb])
    for s in hit_slots:
        files.tutti_filepool_pin(s, -1)
    ring.close()
    ctx.close()
    files.close()
