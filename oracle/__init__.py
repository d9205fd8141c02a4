"""ctypes front end of the CPU oracle (oracle/tutti_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the
bench's CPU-baseline leg.  Nothing here imports the CUDA package, and the CUDA
package never imports this.

All functions take plain numpy arrays.  A *store* is a list of uint8 arrays, one
per storage device; a *pool layer* is one uint8 array plus the byte offsets of
its K and V planes and the byte stride between consecutive blocks.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import List, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tutti_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

OK, EINVAL, ENOSPC = 0, -1, -2
FILE_MAJOR, LAYER_MAJOR = 0, 1
OP_READ, OP_WRITE = 0, 1
OP_HND = 0x100       # opcode flag: head-major pool blocks
SGL_DUP = 0x80000000  # SGL identifier flag: same object bytes as the entry before


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no GPU toolchain involved)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = f"{_LIB}.{os.getpid()}.tmp"       # several processes may build at once
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-Wall", "-Wextra", "-shared", "-fPIC",
                               "-pthread", _SRC, "-o", tmp])
        os.replace(tmp, _LIB)
    return _LIB


class Geom(C.Structure):
    _fields_ = [("n_layers", C.c_uint32), ("n_kv_heads", C.c_uint32), ("head_dim", C.c_uint32),
                ("elem_bytes", C.c_uint32), ("block_tokens", C.c_uint32),
                ("obj_tokens", C.c_uint32), ("n_devices", C.c_uint32), ("layout", C.c_uint32),
                ("n_slots", C.c_uint64)]


class Layout(C.Structure):
    _fields_ = [(n, C.c_uint64) for n in
                ("token_bytes", "block_bytes", "obj_kv_bytes", "obj_bytes", "blocks_per_obj",
                 "n_slots_local", "stride_kv", "stride_layer", "stride_slot", "dev_bytes")]


SQE_DTYPE = np.dtype([("src_off", "<u8"), ("len", "<u8"), ("sgl_first", "<u4"),
                      ("sgl_count", "<u4"), ("dev", "<u4"), ("opcode", "<u2"), ("layer", "<u2")])
SGL_DTYPE = np.dtype([("addr", "<u8"), ("len", "<u4"), ("id", "<u4")])
assert SQE_DTYPE.itemsize == 32 and SGL_DTYPE.itemsize == 16

_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
    return _lib


def geom(n_layers, n_kv_heads, head_dim, elem_bytes, block_tokens, obj_tokens, n_devices, layout,
         n_slots) -> Geom:
    return Geom(n_layers, n_kv_heads, head_dim, elem_bytes, block_tokens, obj_tokens, n_devices,
                layout, n_slots)


def geom_of(w) -> Geom:
    """Geometry of a workload description (any object with the same field names)."""
    return geom(w.n_layers, w.n_kv_heads, w.head_dim, w.elem_bytes, w.block_tokens, w.obj_tokens,
                w.n_devices, w.layout, w.n_slots)


def obj_layout(g: Geom) -> Layout:
    out = Layout()
    rc = lib().orc_obj_layout(C.byref(g), C.byref(out))
    if rc != OK:
        raise ValueError(f"orc_obj_layout: {rc}")
    return out


def _p(a: np.ndarray, ctype):
    return a.ctypes.data_as(C.POINTER(ctype))


def _batch(hit_tokens, obj_start, obj_slot, blk_start, block_ids):
    hit = np.ascontiguousarray(hit_tokens, dtype=np.uint32)
    os_ = np.ascontiguousarray(obj_start, dtype=np.uint32)
    osl = np.ascontiguousarray(obj_slot, dtype=np.uint32)
    bs = np.ascontiguousarray(blk_start, dtype=np.uint32)
    bi = np.ascontiguousarray(block_ids, dtype=np.int32)
    assert os_.shape[0] == hit.shape[0] + 1 and bs.shape[0] == hit.shape[0] + 1
    keep = (hit, os_, osl, bs, bi)
    args = (C.c_uint32(hit.shape[0]), _p(hit, C.c_uint32), _p(os_, C.c_uint32),
            _p(osl, C.c_uint32), _p(bs, C.c_uint32), _p(bi, C.c_int32))
    return keep, args


def _store_ptrs(store: Sequence[np.ndarray]):
    for s in store:
        assert s.dtype == np.uint8 and s.flags["C_CONTIGUOUS"]
    arr = (C.c_void_p * len(store))(*[s.ctypes.data for s in store])
    return arr


def _move(fn, g, layer, batch, store, pool, k_off, v_off, block_stride, n_pool_blocks, pool_hnd):
    keep, bargs = _batch(*batch)
    assert pool.dtype == np.uint8 and pool.flags["C_CONTIGUOUS"]
    sp = _store_ptrs(store)
    base = pool.ctypes.data
    rc = fn(C.byref(g), C.c_uint32(layer), *bargs, sp, C.c_void_p(base + k_off),
            C.c_void_p(base + v_off), C.c_uint64(block_stride), C.c_uint64(n_pool_blocks),
            C.c_int(1 if pool_hnd else 0))
    del keep
    return rc


def restore_layer(g: Geom, layer: int, batch, store: Sequence[np.ndarray], pool: np.ndarray,
                  k_off: int, v_off: int, block_stride: int, n_pool_blocks: int,
                  pool_hnd: bool = False) -> int:
    """store -> pool for every cached token; `batch` = (hit_tokens, obj_start,
    obj_slot, blk_start, block_ids).  Modifies `pool` in place.  pool_hnd: pool blocks are
    [head][token][dim] instead of [token][head][dim]."""
    return _move(lib().orc_restore_layer, g, layer, batch, store, pool, k_off, v_off,
                 block_stride, n_pool_blocks, pool_hnd)


def save_layer(g: Geom, layer: int, batch, store: Sequence[np.ndarray], pool: np.ndarray,
               k_off: int, v_off: int, block_stride: int, n_pool_blocks: int,
               pool_hnd: bool = False) -> int:
    """pool -> store for every cached token.  Modifies `store` in place."""
    return _move(lib().orc_save_layer, g, layer, batch, store, pool, k_off, v_off,
                 block_stride, n_pool_blocks, pool_hnd)


def move_layer_blocks_mt(g: Geom, layer: int, batch, store: Sequence[np.ndarray], pool: np.ndarray,
                         k_off: int, v_off: int, block_stride: int, n_pool_blocks: int,
                         to_pool: bool, n_threads: int, pool_hnd: bool = False) -> int:
    """The restore (to_pool) or save map, one memcpy per block and K/V half, with the batch's
    blocks dealt out over n_threads host threads.  Same result as restore_layer / save_layer."""
    keep, bargs = _batch(*batch)
    assert pool.dtype == np.uint8 and pool.flags["C_CONTIGUOUS"]
    sp = _store_ptrs(store)
    base = pool.ctypes.data
    rc = lib().orc_move_layer_blocks_mt(
        C.byref(g), C.c_uint32(layer), *bargs, sp, C.c_void_p(base + k_off),
        C.c_void_p(base + v_off), C.c_uint64(block_stride), C.c_uint64(n_pool_blocks),
        C.c_int(1 if pool_hnd else 0), C.c_int(1 if to_pool else 0), C.c_uint32(n_threads))
    del keep
    return rc


def token_location(g: Geom, layer: int, batch, r: int, t: int, kv: int
                   ) -> Tuple[int, int, int, int]:
    """(device, store byte offset, pool block id, byte offset inside the block)
    of token t of request r."""
    keep, bargs = _batch(*batch)
    dev = C.c_uint32()
    soff = C.c_uint64()
    blk = C.c_int64()
    roff = C.c_uint64()
    rc = lib().orc_token_location(C.byref(g), C.c_uint32(layer), *bargs[2:],
                                  C.c_uint32(r), C.c_uint64(t), C.c_uint32(kv), C.byref(dev),
                                  C.byref(soff), C.byref(blk), C.byref(roff))
    del keep
    if rc != OK:
        raise ValueError(f"orc_token_location: {rc}")
    return dev.value, soff.value, blk.value, roff.value


def row_location(g: Geom, layer: int, batch, r: int, t: int, kv: int, head: int,
                 pool_hnd: bool = False) -> Tuple[int, int, int, int]:
    """(device, store byte offset, pool block id, byte offset inside the block) of one head's
    row of token t of request r, for token-major or head-major pool blocks."""
    keep, bargs = _batch(*batch)
    dev = C.c_uint32()
    soff = C.c_uint64()
    blk = C.c_int64()
    boff = C.c_uint64()
    rc = lib().orc_row_location(C.byref(g), C.c_uint32(layer), *bargs[2:], C.c_uint32(r),
                                C.c_uint64(t), C.c_uint32(kv), C.c_uint32(head),
                                C.c_int(1 if pool_hnd else 0), C.byref(dev), C.byref(soff),
                                C.byref(blk), C.byref(boff))
    del keep
    if rc != OK:
        raise ValueError(f"orc_row_location: {rc}")
    return dev.value, soff.value, blk.value, boff.value


def build_descriptors(g: Geom, layer: int, opcode: int, batch, k_base_addr: int,
                      v_base_addr: int, block_stride: int, capacity: int,
                      entries_per_iocb: int = 0):
    """Returns (rc, sqes, sgl, num_ioctx) — structured arrays SQE_DTYPE / SGL_DTYPE and the
    per-IOCB context counts.  entries_per_iocb != 0: IOCBs are cut every that many
    scatter-gather entries (equal work) instead of every `capacity` contexts."""
    keep, bargs = _batch(*batch)
    hit, os_, osl, bs, bi = keep
    max_sgl = 2 * int(bi.shape[0]) + 1
    max_iocb = (2 * int(osl.shape[0]) + 1) // max(capacity, 1) + 2
    if entries_per_iocb:
        max_iocb = max_sgl // entries_per_iocb + 2
    max_sqe = 2 * int(osl.shape[0]) + 1 + max_iocb
    sqes = np.zeros(max_sqe, dtype=SQE_DTYPE)
    sgl = np.zeros(max_sgl, dtype=SGL_DTYPE)
    num = np.zeros(max_iocb, dtype=np.uint32)
    n_sqe, n_sgl, n_iocb = C.c_uint32(), C.c_uint32(), C.c_uint32()
    rc = lib().orc_build_budget(C.byref(g), C.c_uint32(layer), C.c_uint32(opcode), *bargs,
                         C.c_uint64(k_base_addr), C.c_uint64(v_base_addr),
                         C.c_uint64(block_stride), C.c_uint32(capacity),
                         C.c_uint32(entries_per_iocb),
                         C.c_void_p(sqes.ctypes.data), C.c_uint32(max_sqe),
                         C.c_void_p(sgl.ctypes.data), C.c_uint32(max_sgl), _p(num, C.c_uint32),
                         C.c_uint32(max_iocb), C.byref(n_sqe), C.byref(n_sgl), C.byref(n_iocb))
    if rc != OK:
        return rc, None, None, None
    return rc, sqes[:n_sqe.value].copy(), sgl[:n_sgl.value].copy(), num[:n_iocb.value].copy()


def exec_descriptors(sqes: np.ndarray, sgl: np.ndarray, store: Sequence[np.ndarray],
                     pool: np.ndarray, pool_base_addr: int, n_kv_heads: int = 0,
                     row_bytes: int = 0) -> int:
    """Perform the transfers the descriptors describe on host copies."""
    sqes = np.ascontiguousarray(sqes)
    sgl = np.ascontiguousarray(sgl)
    assert sqes.dtype == SQE_DTYPE and sgl.dtype == SGL_DTYPE
    sp = _store_ptrs(store)
    sb = np.asarray([s.nbytes for s in store], dtype=np.uint64)
    return lib().orc_exec(C.c_void_p(sqes.ctypes.data), C.c_uint32(sqes.shape[0]),
                          C.c_void_p(sgl.ctypes.data), C.c_uint32(sgl.shape[0]), sp,
                          _p(sb, C.c_uint64), C.c_uint32(len(store)),
                          C.c_void_p(pool.ctypes.data), C.c_uint64(pool_base_addr),
                          C.c_uint64(pool.nbytes), C.c_uint32(n_kv_heads), C.c_uint32(row_bytes))
