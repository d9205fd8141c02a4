"""Seeded synthetic inputs for the KV restore/save path.

This module only *draws inputs*: KV bytes, block tables, object maps, pool
occupancy.  It holds none of the method's arithmetic (no object-store offsets,
no descriptor logic), so the CPU oracle and the CUDA path can both be fed from
it without sharing any of the code under test.

Inputs are shaped like the long-context serving workloads of the paper's
evaluation (prefixes of thousands to >100K tokens, paged KV pools with 16-token
blocks or 1-token pages, Section 4 "Workloads"); no dataset item is reproduced.

KV bytes are bf16 ~N(0,1) from a counter-based generator, so that any range of
any buffer can be produced on the host (numpy) or on the device (torch integer
ops) with identical bits: element 4w+k of a stream is
``TABLE[(mix64(w + start) >> 16k) & 0xFFFF]`` where ``TABLE`` holds the bf16
values of the standard normal quantiles (k + 1/2) / 65536.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Optional

import numpy as np

LAYOUT_FILE_MAJOR = 0
LAYOUT_LAYER_MAJOR = 1

BASE_SEED = 20260503

_M64 = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15
_C1 = 0xBF58476D1CE4E5B9
_C2 = 0x94D049BB133111EB


def _mix64_int(z: int) -> int:
    z &= _M64
    z ^= z >> 30
    z = (z * _C1) & _M64
    z ^= z >> 27
    z = (z * _C2) & _M64
    z ^= z >> 31
    return z


def stream_start(seed: int, stream: int) -> int:
    """64-bit starting counter of stream `stream` under `seed`."""
    return _mix64_int(_mix64_int(seed) ^ ((stream * _GOLDEN) & _M64))


_TABLE: Optional[np.ndarray] = None


def normal_table_bf16() -> np.ndarray:
    """uint16[65536]: bf16 bit patterns of the N(0,1) quantiles (k+0.5)/65536."""
    global _TABLE
    if _TABLE is None:
        from scipy.special import ndtri

        q = (np.arange(65536, dtype=np.float64) + 0.5) / 65536.0
        f = ndtri(q).astype(np.float32)
        bits = f.view(np.uint32).astype(np.uint64)
        rnd = ((bits >> np.uint64(16)) & np.uint64(1)) + np.uint64(0x7FFF)
        _TABLE = ((bits + rnd) >> np.uint64(16)).astype(np.uint16)
    return _TABLE


def fill_u16_numpy(seed: int, stream: int, first_elem: int, n_elem: int) -> np.ndarray:
    """bf16 bit patterns of elements [first_elem, first_elem+n_elem) of a stream."""
    if n_elem == 0:
        return np.zeros(0, dtype=np.uint16)
    w0 = first_elem // 4
    w1 = (first_elem + n_elem + 3) // 4
    start = stream_start(seed, stream)
    with np.errstate(over="ignore"):
        z = np.arange(w0, w1, dtype=np.uint64) + np.uint64(start)
        z ^= z >> np.uint64(30)
        z *= np.uint64(_C1)
        z ^= z >> np.uint64(27)
        z *= np.uint64(_C2)
        z ^= z >> np.uint64(31)
    shifts = np.array([0, 16, 32, 48], dtype=np.uint64)
    idx = ((z[:, None] >> shifts[None, :]) & np.uint64(0xFFFF)).astype(np.int64).reshape(-1)
    out = normal_table_bf16()[idx]
    lo = first_elem - 4 * w0
    return out[lo:lo + n_elem]


def _s64(x: int) -> int:
    x &= _M64
    return x - (1 << 64) if x >= (1 << 63) else x


def fill_u16_torch(seed: int, stream: int, first_elem: int, n_elem: int, device,
                   out=None, chunk_words: int = 1 << 24):
    """Same bits as fill_u16_numpy, produced with torch integer ops on `device`.

    Returns an int16 tensor (bf16 bit patterns); if `out` (int16/bf16 viewable,
    n_elem elements) is given it is filled in place.  first_elem and n_elem must
    be multiples of 4.
    """
    import torch

    assert first_elem % 4 == 0 and n_elem % 4 == 0
    table = torch.from_numpy(normal_table_bf16().view(np.int16).copy()).to(device)
    if out is None:
        out = torch.empty(n_elem, dtype=torch.int16, device=device)
    out16 = out.view(torch.int16).reshape(-1)
    assert out16.numel() == n_elem
    start = _s64(stream_start(seed, stream))
    w0 = first_elem // 4
    n_words = n_elem // 4
    shifts = torch.tensor([0, 16, 32, 48], dtype=torch.int64, device=device)
    done = 0
    while done < n_words:
        n = min(chunk_words, n_words - done)
        z = torch.arange(w0 + done, w0 + done + n, dtype=torch.int64, device=device)
        z += start
        z ^= (z >> 30) & ((1 << 34) - 1)
        z *= _s64(_C1)
        z ^= (z >> 27) & ((1 << 37) - 1)
        z *= _s64(_C2)
        z ^= (z >> 31) & ((1 << 33) - 1)
        idx = (z[:, None] >> shifts[None, :]) & 0xFFFF
        out16[4 * done:4 * (done + n)] = table[idx.reshape(-1)]
        done += n
    return out


# ----------------------------------------------------------------------------
# Workload descriptions (geometry + block tables + object maps)
# ----------------------------------------------------------------------------

@dataclasses.dataclass
class Workload:
    """One batch of prefix hits against a paged KV pool and an object store.

    Arrays follow the CSR convention: request r owns objects
    obj_slot[obj_start[r]:obj_start[r+1]] (logical chunk order) and blocks
    block_ids[blk_start[r]:blk_start[r+1]] (logical block order).
    """
    name: str
    seed: int
    n_layers: int
    n_kv_heads: int
    head_dim: int
    elem_bytes: int
    block_tokens: int
    obj_tokens: int
    n_devices: int
    layout: int
    n_slots: int
    n_pool_blocks: int
    pool_interleaved: bool
    store_kind: str                 # "hbm" | "host"
    hit_tokens: np.ndarray          # uint32[n_req]
    obj_start: np.ndarray           # uint32[n_req+1]
    obj_slot: np.ndarray            # uint32[n_obj]
    blk_start: np.ndarray           # uint32[n_req+1]
    block_ids: np.ndarray           # int32[n_blk]
    occupied_blocks: np.ndarray     # int32[]: pool blocks holding background data
    pool_hnd: bool = False          # pool blocks are [head][token][dim] (else [token][head][dim])
    pool_pad_bytes: int = 0         # unused bytes after every block (block stride > block bytes)

    @property
    def n_req(self) -> int:
        return int(self.hit_tokens.shape[0])

    @property
    def total_tokens(self) -> int:
        return int(self.hit_tokens.astype(np.int64).sum())


def _geometric_runs(rng: np.random.Generator, n_slots: int, mean_run: float) -> list:
    """Cut [0, n_slots) into consecutive runs with geometric lengths, shuffled."""
    runs = []
    s = 0
    p = 1.0 / mean_run
    while s < n_slots:
        ln = int(rng.geometric(p))
        ln = min(ln, n_slots - s)
        runs.append((s, ln))
        s += ln
    order = rng.permutation(len(runs))
    return [runs[i] for i in order]


def _assign_slots(rng, objs_per_req, n_slots, mean_run):
    """Objects of each request take slots in seeded runs of consecutive ids
    (prefixes grow turn by turn, so neighbours in a prefix are often neighbours
    in the store)."""
    runs = _geometric_runs(rng, n_slots, mean_run)
    out = []
    ri = 0
    for need in objs_per_req:
        slots = []
        while len(slots) < need:
            if ri >= len(runs):
                raise ValueError("slot space too small for the batch")
            s, ln = runs[ri]
            take = min(ln, need - len(slots))
            slots.extend(range(s, s + take))
            if take < ln:
                runs[ri] = (s + take, ln - take)
            else:
                ri += 1
        out.append(np.asarray(slots, dtype=np.uint32))
    return out


def _pool_with_free_list(rng, needed_blocks: int, occupancy: float, round_to: int):
    """Pool in which `occupancy` of the blocks already hold other requests'
    data; the rest form a seeded random free list that requests pop in order."""
    n_pool = int(math.ceil(needed_blocks / (1.0 - occupancy)))
    n_pool = ((n_pool + round_to - 1) // round_to) * round_to
    perm = rng.permutation(n_pool).astype(np.int32)
    n_occ = min(int(round(n_pool * occupancy)), n_pool - needed_blocks)
    occupied = np.sort(perm[:n_occ])
    free_list = perm[n_occ:]
    return n_pool, occupied, free_list


def _csr(lengths) -> np.ndarray:
    out = np.zeros(len(lengths) + 1, dtype=np.uint32)
    out[1:] = np.cumsum(np.asarray(lengths, dtype=np.int64))
    return out


def make_workload(name: str, *, seed: int, n_layers: int, hit_tokens, block_tokens: int,
                  obj_tokens: int, n_kv_heads: int = 8, head_dim: int = 128,
                  elem_bytes: int = 2, n_devices: int = 1,
                  layout: int = LAYOUT_LAYER_MAJOR, slot_mean_run: float = 8.0,
                  slot_space_factor: float = 1.25, occupancy: float = 0.6,
                  pool_round: int = 1024, pool_interleaved: bool = False,
                  store_kind: str = "hbm", n_pool_blocks: Optional[int] = None,
                  consecutive_slots: bool = False, pool_hnd: bool = False,
                  pool_pad_bytes: int = 0, shared_prefix_frac: float = 0.0) -> Workload:
    rng = np.random.default_rng(seed)
    hit = np.asarray(hit_tokens, dtype=np.uint32)
    assert np.all(hit % block_tokens == 0)
    blks = (hit // block_tokens).astype(np.int64)
    objs = ((hit.astype(np.int64) + obj_tokens - 1) // obj_tokens)
    needed = int(blks.sum())
    if n_pool_blocks is None:
        n_pool, occupied, free_list = _pool_with_free_list(rng, needed, occupancy, pool_round)
    else:
        n_pool = n_pool_blocks
        perm = rng.permutation(n_pool).astype(np.int32)
        free_list = perm[:needed]
        occupied = np.sort(perm[needed:needed + int(occupancy * (n_pool - needed))])
    block_ids = free_list[:needed].astype(np.int32).copy()
    n_obj = int(objs.sum())
    if consecutive_slots:
        n_slots = max(n_obj, 1)
        per_req = []
        s = 0
        for k in objs:
            per_req.append(np.arange(s, s + int(k), dtype=np.uint32))
            s += int(k)
    else:
        n_slots = max(int(math.ceil(n_obj * slot_space_factor)), 1)
        n_slots = ((n_slots + n_devices - 1) // n_devices) * n_devices
        per_req = _assign_slots(rng, [int(k) for k in objs], n_slots, slot_mean_run)
    if shared_prefix_frac > 0.0 and len(per_req) > 1:
        # requests with a common prefix: the leading objects of every request are the very
        # objects of request 0 (stored once, shared by all), the rest stays private
        n_share = int(min(len(p) for p in per_req) * shared_prefix_frac)
        for p in per_req[1:]:
            p[:n_share] = per_req[0][:n_share]
    obj_slot = np.concatenate(per_req) if per_req else np.zeros(0, dtype=np.uint32)
    return Workload(name=name, seed=seed, n_layers=n_layers, n_kv_heads=n_kv_heads,
                    head_dim=head_dim, elem_bytes=elem_bytes, block_tokens=block_tokens,
                    obj_tokens=obj_tokens, n_devices=n_devices, layout=layout,
                    n_slots=n_slots, n_pool_blocks=n_pool, pool_interleaved=pool_interleaved,
                    store_kind=store_kind, hit_tokens=hit, obj_start=_csr(objs),
                    obj_slot=obj_slot.astype(np.uint32), blk_start=_csr(blks),
                    block_ids=block_ids, occupied_blocks=occupied.astype(np.int32),
                    pool_hnd=pool_hnd, pool_pad_bytes=pool_pad_bytes)


def config(index: int, scale: float = 1.0, **overrides) -> Workload:
    """The five benchmark configurations.  `scale` < 1 shrinks request count /
    prefix length (for CPU-sized parity cases); scale = 1 is the full size.

    1: tiny restore; 2: Llama-3-8B-shaped, HBM object store; 3: Llama-3-70B-shaped,
    pinned-host object store; 4: 1-token pages with partial prefix hits;
    5: config 2 again (run SM-capped beside a GEMM).
    """
    seed = BASE_SEED + index
    rng = np.random.default_rng(seed ^ 0x5EED)
    if index == 1:
        kw = dict(n_layers=1, hit_tokens=[2048], block_tokens=16, obj_tokens=256,
                  n_pool_blocks=1024, consecutive_slots=True)
    elif index in (2, 5):
        n_req = max(1, int(round(8 * min(1.0, scale * 4))))
        toks = max(256, int(32768 * scale) // 256 * 256)
        kw = dict(n_layers=32, hit_tokens=[toks] * n_req, block_tokens=16, obj_tokens=256,
                  slot_mean_run=8.0)
    elif index == 3:
        toks = max(1024, int(131072 * scale) // 1024 * 1024)
        kw = dict(n_layers=80, hit_tokens=[toks] * 2, block_tokens=16, obj_tokens=1024,
                  slot_mean_run=8.0, store_kind="host")
    elif index == 4:
        n_req = max(2, int(round(64 * min(1.0, scale * 4))))
        lo, hi = 512, 16384
        hi = max(lo + 1, int(hi * scale)) if scale < 1.0 else hi
        lo = min(lo, max(1, hi // 8))
        hits = rng.integers(lo, hi + 1, size=n_req)
        kw = dict(n_layers=32, hit_tokens=hits, block_tokens=1, obj_tokens=256,
                  slot_mean_run=4.0)
    else:
        raise ValueError("config index must be 1..5")
    kw.update(overrides)
    bt = kw["block_tokens"]
    kw["hit_tokens"] = [max(bt, int(h) // bt * bt) for h in kw["hit_tokens"]]
    return make_workload(f"cfg{index}", seed=seed, **kw)
