"""Thin ctypes binding over libtutti.so — the same names as include/tutti.h.

Argument marshalling only: every step of the path runs in the library's CUDA
kernels.  There is no CPU fallback: if the library cannot be loaded, importing
this module raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence, Tuple

import numpy as np

from . import _build

OK, EINVAL, ENOMEM, EAGAIN, ETIMEDOUT, EFAULT, ECUDA, ENOENT = 0, -1, -2, -3, -4, -5, -6, -7
LAYOUT_FILE_MAJOR, LAYOUT_LAYER_MAJOR = 0, 1
OP_READ, OP_WRITE = 0, 1
STORE_HBM, STORE_HOST_PINNED = 0, 1
OPT_COPY_ENGINE, OPT_WAIT_NS, OPT_CTAS_PER_SM, OPT_BULK_WARPS, OPT_BULK_STAGES, OPT_CLAIM_CHUNKS, \
    OPT_BULK_CHUNK_BYTES, OPT_POOL_LAYOUT, OPT_INJECT_BULK_TIMEOUT = 1, 2, 3, 4, 5, 6, 7, 8, 9
POOL_NHD, POOL_HND = 0, 1
OP_FLAG_HND = 0x100
ENGINE_AUTO, ENGINE_LDST, ENGINE_BULK = 0, 1, 2


class Geom(C.Structure):
    _fields_ = [("n_layers", C.c_uint32), ("n_kv_heads", C.c_uint32), ("head_dim", C.c_uint32),
                ("elem_bytes", C.c_uint32), ("block_tokens", C.c_uint32),
                ("obj_tokens", C.c_uint32), ("n_devices", C.c_uint32), ("layout", C.c_uint32),
                ("n_slots", C.c_uint64)]


class Layout(C.Structure):
    _fields_ = [(n, C.c_uint64) for n in
                ("token_bytes", "block_bytes", "obj_kv_bytes", "obj_bytes", "blocks_per_obj",
                 "n_slots_local", "stride_kv", "stride_layer", "stride_slot", "dev_bytes")]


class Batch(C.Structure):
    _fields_ = [("n_req", C.c_uint32), ("n_obj", C.c_uint32), ("n_blk", C.c_uint32),
                ("plan_epoch", C.c_uint32), ("hit_tokens", C.c_void_p), ("obj_start", C.c_void_p),
                ("obj_slot", C.c_void_p), ("blk_start", C.c_void_p), ("block_ids", C.c_void_p)]


class Cqe(C.Structure):
    _fields_ = [("iocb_idx", C.c_uint32), ("status", C.c_int32), ("bytes", C.c_uint64)]


class Launch(C.Structure):
    _fields_ = [("opcode", C.c_uint32), ("first_iocb", C.c_uint32), ("n_iocb", C.c_uint32),
                ("sm_count", C.c_uint32), ("layer", C.c_uint32), ("est_us", C.c_float)]


class IocbInfo(C.Structure):
    _fields_ = [("iocb_idx", C.c_uint32), ("ready", C.c_uint32), ("num_ioctx", C.c_uint32),
                ("opcode", C.c_uint32), ("layer", C.c_uint32), ("status", C.c_int32),
                ("sgl_base", C.c_uint32), ("entry_first", C.c_uint32),
                ("total_entries", C.c_uint32), ("entry_len", C.c_uint32), ("bytes", C.c_uint64)]


SQE_DTYPE = np.dtype([("src_off", "<u8"), ("len", "<u8"), ("sgl_first", "<u4"),
                      ("sgl_count", "<u4"), ("dev", "<u4"), ("opcode", "<u2"), ("layer", "<u2")])
SGL_DTYPE = np.dtype([("addr", "<u8"), ("len", "<u4"), ("id", "<u4")])

EXPORTS = [
    "tutti_obj_layout", "tutti_build_sqes", "tutti_kv_restore_layer", "tutti_kv_save_layer",
    "tutti_ring_poll", "tutti_ctx_create", "tutti_ctx_destroy", "tutti_pool_register",
    "tutti_store_register", "tutti_set_option", "tutti_ring_create", "tutti_ring_destroy",
    "tutti_ring_reserve", "tutti_ring_fill_host", "tutti_ring_read_iocb", "tutti_ring_read_sgl",
    "tutti_ring_stats", "tutti_sm_partition_create", "tutti_sm_partition_destroy",
    "tutti_hostring_create", "tutti_hostring_destroy", "tutti_hostring_reserve",
    "tutti_hostring_release", "tutti_hostring_live", "tutti_hostring_cancel_last", "tutti_strerror", "tutti_last_cuda_error",
    "tutti_version", "tutti_kv_restore_layer_noalloc",
    "tutti_sched_create", "tutti_sched_destroy", "tutti_sched_set_slack",
    "tutti_sched_set_decode_slack", "tutti_sched_set_io_time", "tutti_sched_io_time",
    "tutti_sched_enqueue", "tutti_sched_next", "tutti_sched_pending",
    "tutti_filepool_create", "tutti_filepool_destroy", "tutti_filepool_insert",
    "tutti_filepool_lookup", "tutti_filepool_match_prefix", "tutti_filepool_pin",
    "tutti_filepool_remove", "tutti_filepool_stats", "tutti_build_sqes_layers",
    "tutti_stream_wait_iocb", "tutti_ring_last_launch_sms", "tutti_ring_poll_range",
    "tutti_ring_set_iocb_bytes", "tutti_sched_profile",
    "tutti_stage_plan", "tutti_stage_copy_layer", "tutti_build_sqes_staged",
]

_lib: Optional[C.CDLL] = None


def load(path: Optional[str] = None) -> C.CDLL:
    """Load (building first if the sources are newer) the C-ABI library."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    if path is None:
        path = _build.LIB_PATH
        if not os.path.exists(path):
            _build.build_library()
    lib = C.CDLL(path)
    vp, u32, u64 = C.c_void_p, C.c_uint32, C.c_uint64
    P = C.POINTER
    sig = {
        "tutti_obj_layout": (C.c_int, [P(Geom), P(Layout)]),
        "tutti_build_sqes": (C.c_int, [vp, vp, P(Batch), u32, u32, vp, P(u32), P(u32)]),
        "tutti_build_sqes_layers": (C.c_int, [vp, vp, P(Batch), u32, u32, u32, vp, P(u32), P(u32)]),
        "tutti_kv_restore_layer": (C.c_int, [vp, vp, u32, u32, u32, vp]),
        "tutti_kv_save_layer": (C.c_int, [vp, vp, u32, u32, u32, vp]),
        "tutti_ring_poll": (C.c_int, [vp, u32, P(Cqe), u64]),
        "tutti_stream_wait_iocb": (C.c_int, [vp, u32, vp]),
        "tutti_ring_poll_range": (C.c_int, [vp, u32, u32, P(u64), P(C.c_int32), P(u32), u64]),
        "tutti_ctx_create": (C.c_int, [P(Geom), C.c_int, P(vp)]),
        "tutti_ctx_destroy": (C.c_int, [vp]),
        "tutti_pool_register": (C.c_int, [vp, u32, vp, vp, u64, u64]),
        "tutti_store_register": (C.c_int, [vp, u32, vp, u64, u32]),
        "tutti_set_option": (C.c_int, [vp, u32, u64]),
        "tutti_ring_create": (C.c_int, [vp, u32, u32, u32, u32, P(vp)]),
        "tutti_ring_destroy": (C.c_int, [vp]),
        "tutti_ring_reserve": (C.c_int, [vp, u32, u32, P(u32)]),
        "tutti_ring_fill_host": (C.c_int, [vp, vp, u32, vp, u32, vp, u32, u32, vp]),
        "tutti_ring_read_iocb": (C.c_int, [vp, u32, P(IocbInfo), vp, u32]),
        "tutti_ring_read_sgl": (C.c_int, [vp, u32, vp, u32, P(u32)]),
        "tutti_ring_stats": (C.c_int, [vp, P(u64), P(u64)]),
        "tutti_ring_set_iocb_bytes": (C.c_int, [vp, u64]),
        "tutti_stage_plan": (C.c_int, [vp, vp, P(Batch), u64, vp, P(u32), P(u32), P(u64)]),
        "tutti_stage_copy_layer": (C.c_int, [vp, vp, u32, u32, vp, u64, vp]),
        "tutti_build_sqes_staged": (C.c_int, [vp, vp, P(Batch), u32, u32, vp, u64, vp, P(u32), P(u32)]),
        "tutti_ring_last_launch_sms": (C.c_int, [vp, vp, u32, P(u32)]),
        "tutti_sm_partition_create": (C.c_int, [vp, u32, P(vp), P(vp), P(u32), P(u32)]),
        "tutti_sm_partition_destroy": (C.c_int, [vp]),
        "tutti_hostring_create": (vp, [u32, u32]),
        "tutti_hostring_destroy": (None, [vp]),
        "tutti_hostring_reserve": (C.c_int, [vp, u32, u32, P(u32), P(u32)]),
        "tutti_hostring_release": (C.c_int, [vp, u32]),
        "tutti_hostring_live": (C.c_int, [vp, P(u32), P(u32)]),
        "tutti_hostring_cancel_last": (C.c_int, [vp, u32]),
        "tutti_strerror": (C.c_char_p, [C.c_int]),
        "tutti_last_cuda_error": (C.c_char_p, []),
        "tutti_version": (u32, []),
        "tutti_sched_create": (C.c_int, [u32, u32, u32, u32, P(vp)]),
        "tutti_sched_destroy": (C.c_int, [vp]),
        "tutti_sched_set_slack": (C.c_int, [vp, u32, u32, C.c_float, u32]),
        "tutti_sched_set_decode_slack": (C.c_int, [vp, C.c_float, u32]),
        "tutti_sched_set_io_time": (C.c_int, [vp, u32, u32, u32, C.c_float]),
        "tutti_sched_io_time": (C.c_int, [vp, u32, u32, u32, P(C.c_float)]),
        "tutti_sched_enqueue": (C.c_int, [vp, u32, u32, u32, u32]),
        "tutti_sched_next": (C.c_int, [vp, u32, u32, u32, u32, P(Launch), u32, P(u32)]),
        "tutti_sched_pending": (C.c_int, [vp, P(u32), P(u32)]),
        "tutti_sched_profile": (C.c_int, [vp, vp, vp, P(Batch), u32, u32, P(u32), u32, u32, vp, P(u32)]),
        "tutti_filepool_create": (C.c_int, [u64, P(vp)]),
        "tutti_filepool_destroy": (C.c_int, [vp]),
        "tutti_filepool_insert": (C.c_int, [vp, u64, P(u32), P(C.c_int)]),
        "tutti_filepool_lookup": (C.c_int, [vp, u64, P(u32)]),
        "tutti_filepool_match_prefix": (C.c_int, [vp, vp, u32, vp, P(u32), C.c_int]),
        "tutti_filepool_pin": (C.c_int, [vp, u32, C.c_int]),
        "tutti_filepool_remove": (C.c_int, [vp, u64]),
        "tutti_filepool_stats": (C.c_int, [vp, P(u64), P(u64), P(u64), P(u64), P(u64)]),
        "tutti_kv_restore_layer_noalloc": (C.c_int, [P(Geom), C.c_int, u32, P(Batch), vp, vp, u64,
                                                     u64, P(vp), P(u64), vp, vp]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    if path == _build.LIB_PATH:
        _lib = lib
    return lib


class TuttiError(RuntimeError):
    def __init__(self, code: int, what: str):
        lib = load()
        msg = lib.tutti_strerror(code).decode()
        if code == ECUDA:
            msg += ": " + lib.tutti_last_cuda_error().decode()
        super().__init__(f"{what}: {msg} ({code})")
        self.code = code


def _check(code: int, what: str, allow: Sequence[int] = ()) -> int:
    if code != OK and code not in allow:
        raise TuttiError(code, what)
    return code


def geom_of(w) -> Geom:
    """Geometry struct of a workload description (any object with these fields)."""
    return Geom(w.n_layers, w.n_kv_heads, w.head_dim, w.elem_bytes, w.block_tokens, w.obj_tokens,
                w.n_devices, w.layout, w.n_slots)


def tutti_obj_layout(geom: Geom) -> Layout:
    out = Layout()
    _check(load().tutti_obj_layout(C.byref(geom), C.byref(out)), "tutti_obj_layout")
    return out


def _stream_ptr(stream) -> Optional[int]:
    if stream is None:
        return None
    if isinstance(stream, int):
        return stream
    return int(stream.cuda_stream)          # torch.cuda.Stream / ExternalStream


class Context:
    """tutti_ctx_t with its registrations."""

    def __init__(self, geom: Geom, device: int = 0):
        self.lib = load()
        self.geom = geom
        self.layout = tutti_obj_layout(geom)
        h = C.c_void_p()
        _check(self.lib.tutti_ctx_create(C.byref(geom), device, C.byref(h)), "tutti_ctx_create")
        self.h = h
        self.device = device

    def close(self):
        if self.h:
            self.lib.tutti_ctx_destroy(self.h)
            self.h = None

    def tutti_pool_register(self, layer: int, k_base: int, v_base: int, block_stride: int,
                            n_blocks: int):
        _check(self.lib.tutti_pool_register(self.h, layer, k_base, v_base, block_stride, n_blocks),
               "tutti_pool_register")

    def tutti_store_register(self, dev: int, base: int, nbytes: int, kind: int = STORE_HBM):
        _check(self.lib.tutti_store_register(self.h, dev, base, nbytes, kind),
               "tutti_store_register")

    def tutti_set_option(self, option: int, value: int):
        _check(self.lib.tutti_set_option(self.h, option, value), "tutti_set_option")

    def tutti_sm_partition_create(self, io_sms: int) -> Tuple[int, int, int, int]:
        """(io_stream, compute_stream, io_sms, compute_sms) — raw CUstream handles."""
        a, b = C.c_void_p(), C.c_void_p()
        n1, n2 = C.c_uint32(), C.c_uint32()
        _check(self.lib.tutti_sm_partition_create(self.h, io_sms, C.byref(a), C.byref(b),
                                                  C.byref(n1), C.byref(n2)),
               "tutti_sm_partition_create")
        return a.value, b.value, n1.value, n2.value

    def tutti_sm_partition_destroy(self):
        _check(self.lib.tutti_sm_partition_destroy(self.h), "tutti_sm_partition_destroy")


def make_batch(hit_tokens, obj_start, obj_slot, blk_start, block_ids, plan_epoch: int = 0) -> Batch:
    """Batch struct over device tensors (torch, already on the GPU; dtypes int32)."""
    n_req = int(hit_tokens.numel())
    b = Batch(n_req, int(obj_slot.numel()), int(block_ids.numel()), plan_epoch,
              hit_tokens.data_ptr(), obj_start.data_ptr(), obj_slot.data_ptr(),
              blk_start.data_ptr(), block_ids.data_ptr())
    b._keep = (hit_tokens, obj_start, obj_slot, blk_start, block_ids)
    return b


class Ring:
    """tutti_ring_t."""

    def __init__(self, ctx: Context, depth: int, ioctx_per_iocb: int, sgl_capacity: int,
                 max_items: int):
        self.ctx = ctx
        self.lib = ctx.lib
        h = C.c_void_p()
        _check(self.lib.tutti_ring_create(ctx.h, depth, ioctx_per_iocb, sgl_capacity, max_items,
                                          C.byref(h)), "tutti_ring_create")
        self.h = h
        self.ioctx_per_iocb = ioctx_per_iocb

    def close(self):
        if self.h:
            self.lib.tutti_ring_destroy(self.h)
            self.h = None

    def tutti_build_sqes(self, batch: Batch, layer: int, opcode: int, stream=None,
                         allow: Sequence[int] = ()) -> Tuple[int, int, int]:
        first, n = C.c_uint32(), C.c_uint32()
        rc = self.lib.tutti_build_sqes(self.ctx.h, self.h, C.byref(batch), layer, opcode,
                                       _stream_ptr(stream), C.byref(first), C.byref(n))
        _check(rc, "tutti_build_sqes", allow)
        return rc, first.value, n.value

    def tutti_build_sqes_layers(self, batch: Batch, first_layer: int, n_layers: int, opcode: int,
                                stream=None, allow: Sequence[int] = ()) -> Tuple[int, int, int]:
        """(rc, first_iocb, iocbs_per_layer): one launch builds n_layers consecutive layers."""
        first, per = C.c_uint32(), C.c_uint32()
        rc = self.lib.tutti_build_sqes_layers(self.ctx.h, self.h, C.byref(batch), first_layer,
                                              n_layers, opcode, _stream_ptr(stream),
                                              C.byref(first), C.byref(per))
        _check(rc, "tutti_build_sqes_layers", allow)
        return rc, first.value, per.value

    def tutti_kv_restore_layer(self, first_iocb: int, n_iocb: int, sm_count: int = 0, stream=None,
                               allow: Sequence[int] = ()) -> int:
        return _check(self.lib.tutti_kv_restore_layer(self.ctx.h, self.h, first_iocb, n_iocb,
                                                      sm_count, _stream_ptr(stream)),
                      "tutti_kv_restore_layer", allow)

    def tutti_kv_save_layer(self, first_iocb: int, n_iocb: int, sm_count: int = 0, stream=None,
                            allow: Sequence[int] = ()) -> int:
        return _check(self.lib.tutti_kv_save_layer(self.ctx.h, self.h, first_iocb, n_iocb,
                                                   sm_count, _stream_ptr(stream)),
                      "tutti_kv_save_layer", allow)

    def tutti_ring_poll(self, iocb_idx: int, timeout_ns: int = 0) -> Tuple[int, Cqe]:
        cqe = Cqe()
        rc = self.lib.tutti_ring_poll(self.h, iocb_idx, C.byref(cqe), timeout_ns)
        _check(rc, "tutti_ring_poll", (EAGAIN, EINVAL))
        return rc, cqe

    def tutti_ring_poll_range(self, first_iocb: int, n_iocb: int, timeout_ns: int = 0
                              ) -> Tuple[int, int, int, int]:
        """(rc, bytes_total, first_error, n_done) for the IOCBs [first_iocb, first_iocb + n_iocb)."""
        b, e, n = C.c_uint64(), C.c_int32(), C.c_uint32()
        rc = self.lib.tutti_ring_poll_range(self.h, first_iocb, n_iocb, C.byref(b), C.byref(e),
                                            C.byref(n), timeout_ns)
        _check(rc, "tutti_ring_poll_range", (EAGAIN, EINVAL))
        return rc, b.value, e.value, n.value

    def tutti_stream_wait_iocb(self, iocb_idx: int, stream, allow: Sequence[int] = ()) -> int:
        """Work enqueued on `stream` after this call starts once the IOCB has completed."""
        return _check(self.lib.tutti_stream_wait_iocb(self.h, iocb_idx, _stream_ptr(stream)),
                      "tutti_stream_wait_iocb", allow)

    def tutti_ring_reserve(self, n_iocb: int, n_sgl: int, allow: Sequence[int] = ()):
        first = C.c_uint32()
        rc = _check(self.lib.tutti_ring_reserve(self.h, n_iocb, n_sgl, C.byref(first)),
                    "tutti_ring_reserve", allow)
        return rc, first.value

    def tutti_ring_fill_host(self, iocb_idx: int, sqes: np.ndarray, sgl: np.ndarray,
                             sgl_offset: int = 0, stream=None, allow: Sequence[int] = ()) -> int:
        sqes = np.ascontiguousarray(sqes)
        sgl = np.ascontiguousarray(sgl)
        assert sqes.dtype.itemsize == 32 and sgl.dtype.itemsize == 16
        return _check(self.lib.tutti_ring_fill_host(self.ctx.h, self.h, iocb_idx,
                                                    sqes.ctypes.data, len(sqes), sgl.ctypes.data,
                                                    len(sgl), sgl_offset, _stream_ptr(stream)),
                      "tutti_ring_fill_host", allow)

    def tutti_ring_read_iocb(self, iocb_idx: int) -> Tuple[IocbInfo, np.ndarray]:
        info = IocbInfo()
        sqes = np.zeros(self.ioctx_per_iocb, dtype=SQE_DTYPE)
        _check(self.lib.tutti_ring_read_iocb(self.h, iocb_idx, C.byref(info), sqes.ctypes.data,
                                             len(sqes)), "tutti_ring_read_iocb")
        return info, sqes[:info.num_ioctx].copy()

    def tutti_ring_read_sgl(self, iocb_idx: int, max_entries: int) -> np.ndarray:
        sgl = np.zeros(max(max_entries, 1), dtype=SGL_DTYPE)
        n = C.c_uint32()
        _check(self.lib.tutti_ring_read_sgl(self.h, iocb_idx, sgl.ctypes.data, max_entries,
                                            C.byref(n)), "tutti_ring_read_sgl")
        return sgl[:min(n.value, max_entries)].copy()

    def tutti_stage_plan(self, batch: Batch, min_ctx_bytes: int = 0, stream=None,
                         allow: Sequence[int] = ()):
        """(rc, n_ctx, n_staged, bytes_per_layer): the batch's contexts are fetched to the host,
        once; contexts below min_ctx_bytes stay on the zero-copy path."""
        n, ns, b = C.c_uint32(), C.c_uint32(), C.c_uint64()
        rc = _check(self.lib.tutti_stage_plan(self.ctx.h, self.h, C.byref(batch), min_ctx_bytes,
                                              _stream_ptr(stream), C.byref(n), C.byref(ns),
                                              C.byref(b)),
                    "tutti_stage_plan", allow)
        return rc, n.value, ns.value, b.value

    def tutti_stage_copy_layer(self, layer: int, opcode: int, stage: int, stage_bytes: int,
                               stream=None, allow: Sequence[int] = ()) -> int:
        """Copy-engine leg of a staged transfer: store -> stage (READ) or stage -> store (WRITE)."""
        return _check(self.lib.tutti_stage_copy_layer(self.ctx.h, self.h, layer, opcode, stage,
                                                      stage_bytes, _stream_ptr(stream)),
                      "tutti_stage_copy_layer", allow)

    def tutti_build_sqes_staged(self, batch: Batch, layer: int, opcode: int, stage: int,
                                stage_bytes: int, stream=None, allow: Sequence[int] = ()):
        first, n = C.c_uint32(), C.c_uint32()
        rc = _check(self.lib.tutti_build_sqes_staged(self.ctx.h, self.h, C.byref(batch), layer,
                                                     opcode, stage, stage_bytes,
                                                     _stream_ptr(stream), C.byref(first), C.byref(n)),
                    "tutti_build_sqes_staged", allow)
        return rc, first.value, n.value

    def tutti_ring_set_iocb_bytes(self, nbytes: int, allow: Sequence[int] = ()) -> int:
        """IOCBs of (nearly) equal work: cut by bytes instead of by context count (0 = off)."""
        return _check(self.lib.tutti_ring_set_iocb_bytes(self.h, nbytes),
                      "tutti_ring_set_iocb_bytes", allow)

    def tutti_ring_last_launch_sms(self) -> np.ndarray:
        """SM id of every CTA of the most recent copy launch (synchronises)."""
        out = np.zeros(4096, dtype=np.uint32)
        n = C.c_uint32()
        _check(self.lib.tutti_ring_last_launch_sms(self.h, out.ctypes.data, len(out), C.byref(n)),
               "tutti_ring_last_launch_sms")
        return out[:min(n.value, len(out))].copy()

    def tutti_ring_stats(self) -> Tuple[int, int]:
        a, b = C.c_uint64(), C.c_uint64()
        _check(self.lib.tutti_ring_stats(self.h, C.byref(a), C.byref(b)), "tutti_ring_stats")
        return a.value, b.value


def tutti_kv_restore_layer_noalloc(geom: Geom, device: int, layer: int, batch: Batch, k_base: int,
                                   v_base: int, block_stride: int, n_blocks: int,
                                   store_base: Sequence[int], store_bytes: Sequence[int],
                                   cqe_out: int, stream=None, allow: Sequence[int] = ()) -> int:
    """Build + restore one layer using only the library's fixed device scratch: for callers
    that may not allocate (no context, no ring).  `cqe_out` is the address of 16 bytes of
    device or pinned host memory that receive {iocb_idx, status, bytes}."""
    n = len(store_base)
    bases = (C.c_void_p * n)(*store_base)
    sizes = (C.c_uint64 * n)(*store_bytes)
    return _check(load().tutti_kv_restore_layer_noalloc(C.byref(geom), device, layer,
                                                        C.byref(batch), k_base, v_base,
                                                        block_stride, n_blocks, bases, sizes,
                                                        cqe_out, _stream_ptr(stream)),
                  "tutti_kv_restore_layer_noalloc", allow)


PHASE_PREFILL, PHASE_DECODE = 0, 1


class Scheduler:
    """tutti_sched_t: the slack-aware I/O scheduler (host logic only)."""

    def __init__(self, n_layers: int, token_step: int, max_input_tokens: int,
                 max_prefix_tokens: int):
        self.lib = load()
        h = C.c_void_p()
        _check(self.lib.tutti_sched_create(n_layers, token_step, max_input_tokens,
                                           max_prefix_tokens, C.byref(h)), "tutti_sched_create")
        self.h = h

    def close(self):
        if self.h:
            self.lib.tutti_sched_destroy(self.h)
            self.h = None

    def tutti_sched_set_slack(self, l_input, l_prefix, slack_us, sm_budget):
        _check(self.lib.tutti_sched_set_slack(self.h, l_input, l_prefix, slack_us, sm_budget),
               "tutti_sched_set_slack")

    def tutti_sched_set_decode_slack(self, slack_us, sm_budget):
        _check(self.lib.tutti_sched_set_decode_slack(self.h, slack_us, sm_budget),
               "tutti_sched_set_decode_slack")

    def tutti_sched_set_io_time(self, opcode, sm_count, n_iocb, us):
        _check(self.lib.tutti_sched_set_io_time(self.h, opcode, sm_count, n_iocb, us),
               "tutti_sched_set_io_time")

    def tutti_sched_io_time(self, opcode, sm_count, n_iocb) -> float:
        us = C.c_float()
        _check(self.lib.tutti_sched_io_time(self.h, opcode, sm_count, n_iocb, C.byref(us)),
               "tutti_sched_io_time")
        return us.value

    def tutti_sched_profile(self, ring: "Ring", batch: Batch, layer: int, opcode: int,
                            sm_counts: Sequence[int], reps: int = 3, stream=None) -> int:
        """Time the I/O kernels against the IOCB count on every SM count and fill the table;
        returns the number of table entries written."""
        arr = (C.c_uint32 * len(sm_counts))(*sm_counts)
        n = C.c_uint32()
        _check(self.lib.tutti_sched_profile(ring.ctx.h, ring.h, self.h, C.byref(batch), layer,
                                            opcode, arr, len(sm_counts), reps,
                                            _stream_ptr(stream), C.byref(n)),
               "tutti_sched_profile")
        return n.value

    def tutti_sched_enqueue(self, opcode, layer, first_iocb, n_iocb, allow: Sequence[int] = ()):
        return _check(self.lib.tutti_sched_enqueue(self.h, opcode, layer, first_iocb, n_iocb),
                      "tutti_sched_enqueue", allow)

    def tutti_sched_next(self, phase, layer, l_input, l_prefix, max_out: int = 64):
        """[(opcode, first_iocb, n_iocb, sm_count, layer, est_us)] to launch now."""
        out = (Launch * max_out)()
        n = C.c_uint32()
        rc = self.lib.tutti_sched_next(self.h, phase, layer, l_input, l_prefix, out, max_out,
                                       C.byref(n))
        if rc == EAGAIN:
            return self.tutti_sched_next(phase, layer, l_input, l_prefix, n.value)
        _check(rc, "tutti_sched_next")
        return [(o.opcode, o.first_iocb, o.n_iocb, o.sm_count, o.layer, o.est_us)
                for o in out[:n.value]]

    def tutti_sched_pending(self) -> Tuple[int, int]:
        a, b = C.c_uint32(), C.c_uint32()
        _check(self.lib.tutti_sched_pending(self.h, C.byref(a), C.byref(b)), "tutti_sched_pending")
        return a.value, b.value


class FilePool:
    """tutti_filepool_t: CPU-side chunk-key -> object-slot index with a pre-allocated slot pool."""

    def __init__(self, n_slots: int):
        self.lib = load()
        h = C.c_void_p()
        _check(self.lib.tutti_filepool_create(n_slots, C.byref(h)), "tutti_filepool_create")
        self.h = h

    def close(self):
        if self.h:
            self.lib.tutti_filepool_destroy(self.h)
            self.h = None

    def tutti_filepool_insert(self, key: int, allow: Sequence[int] = ()):
        slot, was = C.c_uint32(), C.c_int()
        rc = _check(self.lib.tutti_filepool_insert(self.h, key, C.byref(slot), C.byref(was)),
                    "tutti_filepool_insert", allow)
        return rc, slot.value, bool(was.value)

    def tutti_filepool_lookup(self, key: int):
        slot = C.c_uint32()
        rc = _check(self.lib.tutti_filepool_lookup(self.h, key, C.byref(slot)),
                    "tutti_filepool_lookup", (ENOENT,))
        return rc, slot.value

    def tutti_filepool_match_prefix(self, keys: np.ndarray, pin: bool = False) -> np.ndarray:
        keys = np.ascontiguousarray(keys, dtype=np.uint64)
        slots = np.zeros(max(len(keys), 1), dtype=np.uint32)
        n = C.c_uint32()
        _check(self.lib.tutti_filepool_match_prefix(self.h, keys.ctypes.data, len(keys),
                                                    slots.ctypes.data, C.byref(n), int(pin)),
               "tutti_filepool_match_prefix")
        return slots[:n.value].copy()

    def tutti_filepool_pin(self, slot: int, delta: int, allow: Sequence[int] = ()):
        return _check(self.lib.tutti_filepool_pin(self.h, slot, delta), "tutti_filepool_pin", allow)

    def tutti_filepool_remove(self, key: int):
        return _check(self.lib.tutti_filepool_remove(self.h, key), "tutti_filepool_remove",
                      (ENOENT, EAGAIN))

    def tutti_filepool_stats(self):
        v = [C.c_uint64() for _ in range(5)]
        _check(self.lib.tutti_filepool_stats(self.h, *[C.byref(x) for x in v]),
               "tutti_filepool_stats")
        return dict(zip(("used", "free", "hits", "misses", "evictions"), (x.value for x in v)))
