"""Host-side buffers for a workload: store devices and one pool layer as numpy
arrays, filled from the seeded generators.  Used by the oracle pins and by the
GPU parity tests (which upload the same bytes).  Sizes come from the oracle's
own layout function, so nothing here depends on the CUDA library."""
from __future__ import annotations

import numpy as np

import oracle
from paper_2605_03375_b200 import workload as wl

STREAM_STORE = 0x100      # + device index
STREAM_POOL = 0x200       # + layer index
CANARY = 0xA5


def pool_geometry(w, lo):
    """(pool_bytes, k_off, v_off, block_stride) of one pool layer."""
    bb = int(lo.block_bytes)
    n = w.n_pool_blocks
    pad = int(getattr(w, "pool_pad_bytes", 0))
    if w.pool_interleaved:
        return 2 * n * (bb + pad), 0, bb + pad, 2 * (bb + pad)
    return 2 * n * (bb + pad), 0, n * (bb + pad), bb + pad


def make_store(w, lo, layers=None):
    """One uint8 array per device.  With `layers` given only those layers' bytes are
    generated (LAYER_MAJOR keeps a layer contiguous); the rest stays zero."""
    out = []
    for d in range(w.n_devices):
        nbytes = int(lo.dev_bytes)
        if layers is None:
            a = wl.fill_u16_numpy(w.seed, STREAM_STORE + d, 0, nbytes // 2).view(np.uint8).copy()
        else:
            a = np.zeros(nbytes, dtype=np.uint8)
            assert w.layout == wl.LAYOUT_LAYER_MAJOR
            for l in layers:
                b0 = l * int(lo.stride_layer)
                nb = int(lo.stride_layer)
                a[b0:b0 + nb] = wl.fill_u16_numpy(w.seed, STREAM_STORE + d, b0 // 2,
                                                  nb // 2).view(np.uint8)
        out.append(a)
    return out


def make_pool_layer(w, lo, layer):
    """Pool layer: occupied blocks hold seeded background data, all other bytes a canary."""
    nbytes, k_off, v_off, stride = pool_geometry(w, lo)
    bb = int(lo.block_bytes)
    pool = np.full(nbytes, CANARY, dtype=np.uint8)
    bg = wl.fill_u16_numpy(w.seed, STREAM_POOL + layer, 0, nbytes // 2).view(np.uint8)
    for plane_off in (k_off, v_off):
        for b in w.occupied_blocks:
            o = plane_off + int(b) * stride
            pool[o:o + bb] = bg[o:o + bb]
    return pool


def batch_of(w):
    return (w.hit_tokens, w.obj_start, w.obj_slot, w.blk_start, w.block_ids)
