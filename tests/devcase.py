"""A workload placed on the GPU: store devices, pool layers and batch tables as torch
tensors registered with a library context, next to the host copies the oracle works on."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2605_03375_b200 import tutti as T
from tests import hostcase as hc


class DeviceCase:
    def __init__(self, w, layers=None, host_store=False, depth=8, capacity=2048,
                 sgl_capacity=None, max_items=None, device=0, host_devices=()):
        self.w = w
        self.og = oracle.geom_of(w)
        self.olo = oracle.obj_layout(self.og)
        self.layers = list(range(w.n_layers)) if layers is None else list(layers)
        self.dev = torch.device("cuda", device)
        self.ctx = T.Context(T.geom_of(w), device)
        self.hnd = bool(getattr(w, "pool_hnd", False))
        if self.hnd:
            self.ctx.tutti_set_option(T.OPT_POOL_LAYOUT, T.POOL_HND)
        lo = self.ctx.layout
        assert lo.dev_bytes == self.olo.dev_bytes
        # object store
        self.store_host = hc.make_store(w, self.olo, None if layers is None or
                                        w.layout != 1 else self.layers)
        self.store_dev = []
        for d, a in enumerate(self.store_host):
            if host_store or d in host_devices:
                t = torch.from_numpy(a.copy()).pin_memory()
                kind = T.STORE_HOST_PINNED
            else:
                t = torch.from_numpy(a).to(self.dev)
                kind = T.STORE_HBM
            self.store_dev.append(t)
            self.ctx.tutti_store_register(d, t.data_ptr(), t.numel(), kind)
        # pool layers
        self.pool_bytes, self.k_off, self.v_off, self.stride = hc.pool_geometry(w, self.olo)
        self.pool_host = {}
        self.pool_dev = {}
        for l in self.layers:
            p = hc.make_pool_layer(w, self.olo, l)
            self.pool_host[l] = p
            t = torch.from_numpy(p).to(self.dev)
            self.pool_dev[l] = t
            self.ctx.tutti_pool_register(l, t.data_ptr() + self.k_off, t.data_ptr() + self.v_off,
                                         self.stride, w.n_pool_blocks)
        # batch tables
        def up(a, dt):
            return torch.from_numpy(np.ascontiguousarray(a).astype(dt).view(np.int32)).to(self.dev)
        self.tensors = (up(w.hit_tokens, np.uint32), up(w.obj_start, np.uint32),
                        up(w.obj_slot, np.uint32), up(w.blk_start, np.uint32),
                        up(w.block_ids, np.int32))
        self.batch = T.make_batch(*self.tensors)
        n_blk = len(w.block_ids)
        n_obj = len(w.obj_slot)
        self.ring = T.Ring(self.ctx, depth, capacity,
                           sgl_capacity or max(2 * n_blk * 2, 64),
                           max_items or max(2 * n_obj, 2))
        self.obatch = hc.batch_of(w)

    def close(self):
        torch.cuda.synchronize()
        self.ring.close()
        self.ctx.close()

    # ---- oracle side -----------------------------------------------------
    def oracle_descriptors(self, layer, opcode, capacity, entries_per_iocb=0):
        base = self.pool_dev[layer].data_ptr()
        if self.hnd:
            opcode |= oracle.OP_HND
        return oracle.build_descriptors(self.og, layer, opcode, self.obatch, base + self.k_off,
                                        base + self.v_off, self.stride, capacity, entries_per_iocb)

    def oracle_restore(self, layer):
        pool = self.pool_host[layer].copy()
        rc = oracle.restore_layer(self.og, layer, self.obatch, self.store_host, pool, self.k_off,
                                  self.v_off, self.stride, self.w.n_pool_blocks, self.hnd)
        assert rc == 0
        return pool

    def oracle_save(self, layer, pool_host, store_host):
        rc = oracle.save_layer(self.og, layer, self.obatch, store_host, pool_host, self.k_off,
                               self.v_off, self.stride, self.w.n_pool_blocks, self.hnd)
        assert rc == 0

    # ---- CUDA side -------------------------------------------------------
    def read_build(self, first, n):
        """All contexts, SGL entries and per-IOCB counts of a build, in order."""
        sqes, sgl, num, infos = [], [], [], []
        for i in range(first, first + n):
            info, s = self.ring.tutti_ring_read_iocb(i)
            infos.append(info)
            num.append(info.num_ioctx)
            sqes.append(s)
            sgl.append(self.ring.tutti_ring_read_sgl(i, info.total_entries))
        return np.concatenate(sqes), np.concatenate(sgl), np.asarray(num, dtype=np.uint32), infos

    def poll_all(self, first, n, timeout_ns=5_000_000_000):
        out = []
        for i in range(first, first + n):
            rc, cqe = self.ring.tutti_ring_poll(i, timeout_ns)
            assert rc == T.OK, f"poll {i}: {rc}"
            out.append((cqe.iocb_idx, cqe.status, cqe.bytes))
        return out


def verify_replica_samples(rep, n_samples=256):
    """Sampled outputs at full size for a bench.Replica: for random (token, head) rows the oracle
    names the store bytes and the pool bytes that must be equal after a restore."""
    w = rep.w
    og = oracle.geom_of(w)
    ob = (w.hit_tokens, w.obj_start, w.obj_slot, w.blk_start, w.block_ids)
    rng = np.random.default_rng(4321)
    row = w.head_dim * w.elem_bytes
    for _ in range(n_samples):
        l = int(rng.integers(w.n_layers - rep.R, w.n_layers))    # layers whose pool buffer is still theirs
        r = int(rng.integers(0, w.n_req))
        t = int(rng.integers(0, int(w.hit_tokens[r])))
        kv = int(rng.integers(0, 2))
        hd = int(rng.integers(0, w.n_kv_heads))
        d, so, blk, bo = oracle.row_location(og, l, ob, r, t, kv, hd, w.pool_hnd)
        po = kv * rep.v_off + blk * rep.block_bytes + bo
        a = rep.store[d][so:so + row].to(rep.dev)
        b = rep.pool[l % rep.R][po:po + row]
        if not torch.equal(a, b):
            return False
    return True
