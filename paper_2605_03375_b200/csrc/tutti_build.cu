// Descriptor build on the GPU (paper Section 3.1 "block lookup and P2P table
// lookup to generate a batch of lightweight GPU I/O contexts", Section 3.2 IOCB /
// IOCTX format).  Two kernels:
//
//   plan_kernel   one CTA.  Items (object, K|V) -> keys (device, offset) -> sort ->
//                 adjacency flags -> prefix sums -> contexts for layer 0.  The
//                 result does not depend on the layer (a layer only adds a constant
//                 to every offset), so it is kept in the ring and reused while the
//                 caller's plan_epoch says the batch is unchanged.
//   emit_kernel   wide.  Per layer: contexts rebased to the layer and packed into
//                 IOCBs, one 16-byte SGL entry per pool block (block-table lookup),
//                 the object-side address of every entry, then a release-publish of
//                 the IOCB headers by the last CTA to finish.
//
// The paper prepares these descriptors on the CPU; here GPU threads do it so that
// no CPU thread touches per-block work.
#include "tutti_internal.h"

namespace tutti {

namespace {

constexpr int PLAN_THREADS = 1024;
constexpr uint32_t SMEM_SORT_ITEMS = 8192;   // (8 + 4) bytes each = 96 KiB
constexpr unsigned long long KEY_NONE = ~0ull;

__device__ __forceinline__ uint32_t find_request(const uint32_t *obj_start, uint32_t n_req,
                                                 uint32_t o) {
    // largest r with obj_start[r] <= o  (rows may be empty)
    uint32_t lo = 0, hi = n_req;           // invariant: obj_start[lo] <= o < obj_start[hi]
    while (hi - lo > 1) {
        uint32_t mid = (lo + hi) >> 1;
        if (__ldg(obj_start + mid) <= o) lo = mid; else hi = mid;
    }
    return lo;
}

// tokens of chunk c of a request that are part of the hit
__device__ __forceinline__ uint32_t valid_tokens(uint32_t hit, uint32_t c, uint32_t obj_tokens) {
    unsigned long long start = (unsigned long long)c * obj_tokens;
    if (start >= hit) return 0;
    unsigned long long left = hit - start;
    return left < obj_tokens ? (uint32_t)left : obj_tokens;
}

__device__ __forceinline__ void note_error(int32_t *where, int32_t code) {
    atomicCAS(where, 0, code);
}

__device__ __forceinline__ bool pair_less(unsigned long long ka, uint32_t ia, unsigned long long kb,
                                          uint32_t ib) {
    return ka < kb || (ka == kb && ia < ib);
}

// In-place bitonic sort of (key, idx) pairs, ascending by (key, idx); n is a power
// of two.  idx values are unique, so the order is total and equals a stable sort by key.
__device__ void bitonic_sort(unsigned long long *key, uint32_t *idx, uint32_t n) {
    for (uint32_t k = 2; k <= n; k <<= 1) {
        for (uint32_t j = k >> 1; j > 0; j >>= 1) {
            for (uint32_t t = threadIdx.x; t < (n >> 1); t += blockDim.x) {
                // t-th compare-exchange of this stage: partner indices differ in bit j
                uint32_t i = ((t & ~(j - 1)) << 1) | (t & (j - 1));
                uint32_t p = i | j;
                bool up = (i & k) == 0;
                unsigned long long ka = key[i], kb = key[p];
                uint32_t ia = idx[i], ib = idx[p];
                bool swap = up ? pair_less(kb, ib, ka, ia) : pair_less(ka, ia, kb, ib);
                if (swap) {
                    key[i] = kb; key[p] = ka;
                    idx[i] = ib; idx[p] = ia;
                }
            }
            __syncthreads();
        }
    }
}

// Sort key of item q = 2 * object + kv, or KEY_NONE when the object holds no hit token (or q
// is padding).  Items are ordered by (device, offset, length): the key is
// (device << 56) | (offset at layer 0 in blocks + blocks of the item - 1).  Offsets of items are
// multiples of an object half (blocks_per_obj blocks) and an item has 1..blocks_per_obj blocks,
// so the sum orders by offset first, then by length, and equal keys mean exactly the same
// bytes (a stored chunk hit by several requests).  A slot out of range is reported.
__device__ unsigned long long item_key(const GeomDev &g, const BatchDev &b, uint32_t q,
                                       int32_t &err) {
    if (q >= 2u * b.n_obj || b.n_req == 0) return KEY_NONE;
    const uint32_t o = q >> 1, kv = q & 1;
    const uint32_t r = find_request(b.obj_start, b.n_req, o);
    if (o < b.obj_start[r] || o >= b.obj_start[r + 1]) return KEY_NONE;
    const uint32_t c = o - b.obj_start[r];
    const uint32_t n_blk = valid_tokens(b.hit_tokens[r], c, g.obj_tokens) / g.block_tokens;
    if (n_blk == 0) return KEY_NONE;
    const unsigned long long slot = b.obj_slot[o];
    if (slot >= g.n_slots) {
        err = TUTTI_EFAULT;
        return KEY_NONE;
    }
    const unsigned long long dev = slot % g.n_devices;
    const unsigned long long off = (slot / g.n_devices) * g.stride_slot +
                                   (unsigned long long)kv * g.stride_kv;
    return (dev << 56) | (off / g.block_bytes + (n_blk - 1));
}

// ---- batches too large for one CTA's shared memory: the same bitonic network, run as a
// ---- few launches.  Stages whose partners lie inside one aligned tile of SORT_TILE
// ---- elements run in shared memory, one CTA per tile; the others are one global
// ---- compare-exchange pass each.
constexpr uint32_t SORT_TILE = 8192;

__global__ void __launch_bounds__(256)
plan_keys_kernel(RingDev ring, GeomDev g, BatchDev b, uint32_t np) {
    // plan_counts[1].status is zero on entry: the plan kernel that consumed it last cleared it
    const uint32_t q = blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= np) return;
    int32_t st = 0;
    ring.plan_key[q] = item_key(g, b, q, st);
    ring.plan_idx[q] = q;
    if (st) atomicCAS(&ring.plan_counts[1].status, 0, st);
}

__device__ __forceinline__ void cmp_exchange(unsigned long long *key, uint32_t *idx, uint32_t i,
                                             uint32_t p, bool up) {
    unsigned long long ka = key[i], kb = key[p];
    uint32_t ia = idx[i], ib = idx[p];
    bool swap = up ? pair_less(kb, ib, ka, ia) : pair_less(ka, ia, kb, ib);
    if (swap) {
        key[i] = kb; key[p] = ka;
        idx[i] = ib; idx[p] = ia;
    }
}

// For k = k_first, 2*k_first, ..., k_last: the stages j = min(k/2, SORT_TILE/2) ... 1.
__global__ void __launch_bounds__(PLAN_THREADS, 1)
bitonic_tile_kernel(unsigned long long *gkey, uint32_t *gidx, uint32_t k_first, uint32_t k_last) {
    extern __shared__ __align__(16) unsigned char dyn_smem[];
    unsigned long long *key = reinterpret_cast<unsigned long long *>(dyn_smem);
    uint32_t *idx = reinterpret_cast<uint32_t *>(dyn_smem + (size_t)SORT_TILE * 8);
    const uint32_t base = blockIdx.x * SORT_TILE;
    for (uint32_t i = threadIdx.x; i < SORT_TILE; i += blockDim.x) {
        key[i] = gkey[base + i];
        idx[i] = gidx[base + i];
    }
    __syncthreads();
    for (uint32_t k = k_first; k <= k_last && k != 0; k <<= 1) {
        uint32_t j0 = k >> 1;
        if (j0 > SORT_TILE / 2) j0 = SORT_TILE / 2;
        for (uint32_t j = j0; j > 0; j >>= 1) {
            for (uint32_t t = threadIdx.x; t < SORT_TILE / 2; t += blockDim.x) {
                uint32_t i = ((t & ~(j - 1)) << 1) | (t & (j - 1));
                cmp_exchange(key, idx, i, i | j, ((base + i) & k) == 0);
            }
            __syncthreads();
        }
    }
    for (uint32_t i = threadIdx.x; i < SORT_TILE; i += blockDim.x) {
        gkey[base + i] = key[i];
        gidx[base + i] = idx[i];
    }
}

// One stage (k, j) with j >= SORT_TILE: partners sit in different tiles.
__global__ void __launch_bounds__(256)
bitonic_global_kernel(unsigned long long *key, uint32_t *idx, uint32_t np, uint32_t k, uint32_t j) {
    const uint32_t t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= np / 2) return;
    const uint32_t i = ((t & ~(j - 1)) << 1) | (t & (j - 1));
    cmp_exchange(key, idx, i, i | j, (i & k) == 0);
}

struct ScanVals {
    uint32_t a;   // sum: blocks
    uint32_t b;   // sum of a 0/1 flag: context heads
    uint32_t m;   // running maximum: index of the latest group start
};

// Inclusive scan of (a, b, m) across the CTA for one element per thread, plus carry.  `a`
// (block counts) and `m` go through shuffles; `b` is a 0/1 flag (context head), so its
// warp-level prefix is a ballot and a population count.
__device__ ScanVals block_scan_incl(ScanVals v, ScanVals *warp_tot, ScanVals &carry) {
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        uint32_t ua = __shfl_up_sync(0xffffffffu, v.a, d);
        uint32_t um = __shfl_up_sync(0xffffffffu, v.m, d);
        if (lane >= (uint32_t)d) { v.a += ua; v.m = max(v.m, um); }
    }
    const uint32_t heads = __ballot_sync(0xffffffffu, v.b != 0);
    v.b = __popc(heads & (0xffffffffu >> (31 - lane)));
    const uint32_t n_warps = blockDim.x >> 5;
    if (lane == 31) warp_tot[warp] = v;
    __syncthreads();
    if (warp == 0) {
        ScanVals w = lane < n_warps ? warp_tot[lane] : ScanVals{0, 0, 0};
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            uint32_t ua = __shfl_up_sync(0xffffffffu, w.a, d);
            uint32_t ub = __shfl_up_sync(0xffffffffu, w.b, d);
            uint32_t um = __shfl_up_sync(0xffffffffu, w.m, d);
            if (lane >= (uint32_t)d) { w.a += ua; w.b += ub; w.m = max(w.m, um); }
        }
        if (lane < n_warps) warp_tot[lane] = w;
    }
    __syncthreads();
    ScanVals off = carry;
    if (warp > 0) {
        off.a += warp_tot[warp - 1].a;
        off.b += warp_tot[warp - 1].b;
        off.m = max(off.m, warp_tot[warp - 1].m);
    }
    v.a += off.a; v.b += off.b; v.m = max(v.m, off.m);
    ScanVals tot = warp_tot[n_warps - 1];
    __syncthreads();
    if (threadIdx.x == 0) { carry.a += tot.a; carry.b += tot.b; carry.m = max(carry.m, tot.m); }
    __syncthreads();
    return v;
}

__global__ void __launch_bounds__(PLAN_THREADS, 1)
plan_kernel(RingDev ring, GeomDev g, BatchDev b, uint32_t np, int use_smem, int presorted) {
    extern __shared__ __align__(16) unsigned char dyn_smem[];
    __shared__ ScanVals warp_tot[32];
    __shared__ ScanVals carry;
    __shared__ int32_t s_status;
    __shared__ uint32_t s_nact;

    // the emit kernel launched behind this one may become resident now (it waits for this
    // kernel's completion before it reads the plan)
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    unsigned long long *key = use_smem ? reinterpret_cast<unsigned long long *>(dyn_smem)
                                       : ring.plan_key;
    uint32_t *idx = use_smem ? reinterpret_cast<uint32_t *>(dyn_smem + (size_t)np * 8)
                             : ring.plan_idx;
    if (threadIdx.x == 0) { s_status = 0; s_nact = 0; carry.a = 0; carry.b = 0; carry.m = 0; }
    __syncthreads();

    // per-request preconditions
    for (uint32_t r = threadIdx.x; r < b.n_req; r += blockDim.x) {
        uint32_t hit = b.hit_tokens[r];
        uint32_t n_o = b.obj_start[r + 1] - b.obj_start[r];
        uint32_t n_b = b.blk_start[r + 1] - b.blk_start[r];
        bool bad = (hit % g.block_tokens) != 0 ||
                   b.obj_start[r + 1] < b.obj_start[r] || b.blk_start[r + 1] < b.blk_start[r] ||
                   b.obj_start[r + 1] > b.n_obj || b.blk_start[r + 1] > b.n_blk ||
                   (unsigned long long)n_o * g.obj_tokens < hit ||
                   (unsigned long long)n_b * g.block_tokens < hit;
        if (bad) note_error(&s_status, TUTTI_EINVAL);
    }

    // step 1: items and their keys (device, offset at layer 0)
    if (!presorted) {
        for (uint32_t q = threadIdx.x; q < np; q += blockDim.x) {
            int32_t st = 0;
            key[q] = item_key(g, b, q, st);
            idx[q] = q;
            if (st) note_error(&s_status, st);
        }
    } else if (threadIdx.x == 0) {
        if (ring.plan_counts[1].status != 0) s_status = ring.plan_counts[1].status;
        ring.plan_counts[1].status = 0;            // found while the keys were computed; consumed
    }
    __syncthreads();

    // step 2: order by (device, offset), ties by item id = (request, chunk, K before V)
    if (!presorted) bitonic_sort(key, idx, np);

    // active items are the prefix before the first KEY_NONE
    for (uint32_t i = threadIdx.x; i < np; i += blockDim.x)
        if (key[i] != KEY_NONE && (i + 1 == np || key[i + 1] == KEY_NONE)) s_nact = i + 1;
    __syncthreads();
    const uint32_t n_act = s_status ? 0 : s_nact;

    const unsigned long long OFF_MASK = (1ull << 56) - 1;
    // blocks per item (kept in plan_sqe_of until the scans have run), byte offset, item id
    for (uint32_t i = threadIdx.x; i < n_act; i += blockDim.x) {
        uint32_t q = idx[i], o = q >> 1;
        uint32_t r = find_request(b.obj_start, b.n_req, o);
        uint32_t valid = valid_tokens(b.hit_tokens[r], o - b.obj_start[r], g.obj_tokens);
        const uint32_t n_blk = valid / g.block_tokens;
        const unsigned long long k = key[i];
        ring.plan_sqe_of[i] = n_blk;
        ring.plan_item[i] = q;
        ring.plan_off[i] = (k & ~OFF_MASK) | (((k & OFF_MASK) - (n_blk - 1)) * g.block_bytes);
    }
    __syncthreads();

    // steps 3-4: flags.  An item repeats its predecessor when the keys are equal (the same
    // bytes, hit by another request): such a group is one source.  A group starts a new
    // context unless it begins exactly where the previous group's bytes end on the same
    // device.  Packed with the block count: bit 31 context head, bit 30 repeat.
    for (uint32_t i = threadIdx.x; i < n_act; i += blockDim.x) {
        uint32_t head = 1, rep = 0;
        if (i > 0) {
            const unsigned long long k = key[i], kp = key[i - 1];
            rep = (k == kp);
            // end of the previous item = end of its group (all members name the same bytes)
            const unsigned long long end_prev = (kp & OFF_MASK) + 1;          // in blocks
            const unsigned long long start = (k & OFF_MASK) - (ring.plan_sqe_of[i] - 1);
            head = !rep && (((kp >> 56) != (k >> 56)) || (end_prev != start));
        }
        ring.plan_cumblk[i] = (head << 31) | (rep << 30) | ring.plan_sqe_of[i];
    }
    __syncthreads();

    // step 5: prefix sums of (blocks, context heads) and the running group start; every
    // thread touches only its own item
    for (uint32_t base = 0; base < n_act; base += blockDim.x) {
        uint32_t i = base + threadIdx.x;
        ScanVals v{0, 0, 0};
        uint32_t nblk = 0, head = 0, rep = 0;
        if (i < n_act) {
            uint32_t packed = ring.plan_cumblk[i];
            nblk = packed & 0x3fffffffu;
            head = packed >> 31;
            rep = (packed >> 30) & 1u;
            v.a = nblk; v.b = head; v.m = rep ? 0u : i;
        }
        ScanVals s = block_scan_incl(v, warp_tot, carry);
        if (i < n_act) {
            uint32_t excl = s.a - nblk;
            uint32_t sq = s.b - 1;
            ring.plan_cumblk[i] = excl;
            ring.plan_sqe_of[i] = sq;
            ring.plan_grp[i] = s.m;                  // index of the first item of this group
            if (head) {
                const unsigned long long po = ring.plan_off[i];
                tutti_sqe_t e;
                e.src_off = po & OFF_MASK;
                e.len = 0;
                e.sgl_first = excl;
                e.sgl_count = 0;
                e.dev = (uint32_t)(po >> 56);
                e.opcode = 0;
                e.layer = 0;
                ring.plan_sqe[sq] = e;
            }
        }
    }
    __syncthreads();
    const uint32_t n_entries = carry.a, n_sqe = carry.b;
    if (threadIdx.x == 0) ring.plan_cumblk[n_act] = n_entries;
    __syncthreads();

    // group sizes (written at every group's first item) and the end of every context: its
    // entries cover all members of its groups, its length names the bytes once
    for (uint32_t i = threadIdx.x; i < n_act; i += blockDim.x) {
        const bool group_ends = (i + 1 == n_act) || (ring.plan_grp[i + 1] == i + 1);
        if (group_ends) ring.plan_k[ring.plan_grp[i]] = i + 1 - ring.plan_grp[i];
        uint32_t sq = ring.plan_sqe_of[i];
        bool last = (i + 1 == n_act) || (ring.plan_sqe_of[i + 1] != sq);
        if (last) {
            const uint32_t n_blk = ring.plan_cumblk[i + 1] - ring.plan_cumblk[i];
            const unsigned long long end = (ring.plan_off[i] & OFF_MASK) +
                                           (unsigned long long)n_blk * g.block_bytes;
            ring.plan_sqe[sq].sgl_count = ring.plan_cumblk[i + 1] - ring.plan_sqe[sq].sgl_first;
            ring.plan_sqe[sq].len = end - ring.plan_sqe[sq].src_off;
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        PlanCounts pc;
        pc.n_items = n_act;
        pc.n_sqe = n_sqe;
        pc.n_entries = n_entries;
        pc.status = s_status;
        *ring.plan_counts = pc;
    }
}

constexpr int EMIT_THREADS = 256;

struct EmitParams {
    uint32_t layer, opcode;
    uint64_t k_base, v_base, block_stride, n_pool_blocks;
    uint64_t store_base[TUTTI_MAX_DEVICES];
    uint64_t store_bytes[TUTTI_MAX_DEVICES];
    uint32_t first_iocb, n_iocb, sgl_base, sgl_reserved;
    uint32_t entries_per_iocb;   // 0: IOCBs of `capacity` contexts; else IOCBs cut by entries
    uint64_t stage_base;         // != 0: the object side of every entry is this staging buffer,
    uint64_t stage_bytes;        //       which holds the contexts' bytes packed in context order
    const PoolLayerDev *pools;   // per-layer pool table for launches that cover several layers
};

// IOCBs of equal work: boundary k of a build is scatter-gather entry k * entries_per_iocb moved
// back to the first entry of its source block (a repeat is never separated from the bytes it
// repeats).  A cut: the boundary's entry index, the context that holds it and the object-side
// offset (layer 0) its source block starts at.
struct Cut {
    uint32_t entry;
    uint32_t sq;
    unsigned long long src;
};

__device__ Cut cut_at(const RingDev &ring, const GeomDev &g, uint32_t n_items, uint32_t n_entries,
                      unsigned long long y) {
    Cut c{n_entries, 0xffffffffu, 0};
    if (y >= n_entries) return c;
    // the item whose share of the entries, [cumblk[i], cumblk[i + 1]), holds y
    uint32_t lo = 0, hi = n_items;
    while (hi - lo > 1) {
        const uint32_t mid = (lo + hi) >> 1;
        if (ring.plan_cumblk[mid] <= y) lo = mid; else hi = mid;
    }
    // its group lists block j of the source k_copies times in a row
    const uint32_t gs = ring.plan_grp[lo];
    const uint32_t first = ring.plan_cumblk[gs], k_copies = ring.plan_k[gs];
    const uint32_t j = ((uint32_t)y - first) / k_copies;
    c.entry = first + j * k_copies;
    c.sq = ring.plan_sqe_of[gs];
    c.src = (ring.plan_off[gs] & ((1ull << 56) - 1)) + (unsigned long long)j * g.block_bytes;
    return c;
}

// blockIdx.y selects the layer of a multi-layer launch: layer p.layer + y, whose IOCBs and
// arena range follow those of the layer before it.
__global__ void __launch_bounds__(EMIT_THREADS)
emit_kernel(RingDev ring, GeomDev g, BatchDev b, EmitParams p) {
    // Everything earlier in the stream (the plan kernel, or whatever ran before this build)
    // has completed once this returns; only then may the copy kernel launched behind this one
    // become resident, where its agents wait for the READY words written at the end.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (p.pools) {
        const PoolLayerDev pl = p.pools[p.layer + blockIdx.y];
        p.k_base = pl.k_base;
        p.v_base = pl.v_base;
        p.block_stride = pl.block_stride;
        p.n_pool_blocks = pl.n_blocks;
    }
    p.layer += blockIdx.y;
    p.first_iocb += blockIdx.y * p.n_iocb;
    p.sgl_base += blockIdx.y * p.sgl_reserved;
    const PlanCounts pc = *ring.plan_counts;
    IocbHdr *hdr0 = &ring.hdrs[p.first_iocb & (ring.depth - 1)];
    int32_t status = pc.status;
    if (status == 0 && pc.n_entries > p.sgl_reserved) status = TUTTI_EINVAL;
    const uint32_t n_sqe = status ? 0 : pc.n_sqe;
    const uint32_t n_items = status ? 0 : pc.n_items;
    const uint32_t n_entries = status ? 0 : pc.n_entries;
    const unsigned long long layer_off = (unsigned long long)p.layer * g.stride_layer;

    // IOCB headers (step 7 of the path): CTA 0
    const uint32_t per = p.entries_per_iocb;
    if (blockIdx.x == 0) {
        for (uint32_t k = threadIdx.x; k < p.n_iocb; k += blockDim.x) {
            uint32_t idx = p.first_iocb + k;
            IocbHdr *h = &ring.hdrs[idx & (ring.depth - 1)];
            uint32_t e0, e1, n_ctx;
            if (per == 0) {
                unsigned long long s0 = (unsigned long long)k * ring.capacity;
                unsigned long long s1 = s0 + ring.capacity;
                e0 = s0 < n_sqe ? ring.plan_sqe[s0].sgl_first : n_entries;
                e1 = s1 < n_sqe ? ring.plan_sqe[s1].sgl_first : n_entries;
                n_ctx = s0 < n_sqe ? (uint32_t)((s1 < n_sqe ? s1 : n_sqe) - s0) : 0;
            } else {
                const Cut a = cut_at(ring, g, n_items, n_entries, (unsigned long long)k * per);
                const Cut b = cut_at(ring, g, n_items, n_entries, (unsigned long long)(k + 1) * per);
                e0 = a.entry;
                e1 = b.entry;
                n_ctx = 0;
                if (e1 > e0) {
                    // contexts with entries in [e0, e1): from the one holding e0 to the one
                    // holding e1 - 1
                    const uint32_t last = (b.sq == 0xffffffffu) ? n_sqe - 1
                                          : (e1 > ring.plan_sqe[b.sq].sgl_first ? b.sq : b.sq - 1);
                    n_ctx = last - a.sq + 1;
                }
            }
            h->num_ioctx = n_ctx;
            h->opcode = p.opcode;
            h->layer = p.layer;
            h->status = (n_ctx > ring.capacity && status == 0) ? TUTTI_EINVAL : status;
            h->sgl_base = p.sgl_base;
            h->entry_first = e0;
            h->total_entries = (n_ctx > ring.capacity) ? 0 : e1 - e0;
            h->entry_len = (uint32_t)g.block_bytes;
            h->claim_cursor = 0;
            h->done_bytes = 0;
            h->bytes = (n_ctx > ring.capacity) ? 0 : (unsigned long long)(e1 - e0) * g.block_bytes;
        }
    }

    // contexts, rebased to this layer and packed into IOCBs
    const uint32_t gtid = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t gthreads = gridDim.x * blockDim.x;
    if (per == 0) {
        for (uint32_t k = gtid; k < n_sqe; k += gthreads) {
            tutti_sqe_t e = ring.plan_sqe[k];
            e.src_off += layer_off;
            e.opcode = (uint16_t)p.opcode;
            e.layer = (uint16_t)p.layer;
            uint32_t slot = (p.first_iocb + k / ring.capacity) & (ring.depth - 1);
            ring.sqes[(size_t)slot * ring.capacity + k % ring.capacity] = e;
        }
    } else {
        // one IOCB per CTA at a time; a context that crosses a boundary is cut there
        for (uint32_t k = blockIdx.x; k < p.n_iocb; k += gridDim.x) {
            const Cut a = cut_at(ring, g, n_items, n_entries, (unsigned long long)k * per);
            const Cut b = cut_at(ring, g, n_items, n_entries, (unsigned long long)(k + 1) * per);
            if (b.entry <= a.entry) continue;
            const uint32_t last = (b.sq == 0xffffffffu) ? n_sqe - 1
                                  : (b.entry > ring.plan_sqe[b.sq].sgl_first ? b.sq : b.sq - 1);
            const uint32_t n_ctx = last - a.sq + 1;
            if (n_ctx > ring.capacity) continue;                 // reported in the header
            const uint32_t slot = (p.first_iocb + k) & (ring.depth - 1);
            for (uint32_t q = threadIdx.x; q < n_ctx; q += blockDim.x) {
                const tutti_sqe_t whole = ring.plan_sqe[a.sq + q];
                const uint32_t w_end = whole.sgl_first + whole.sgl_count;
                tutti_sqe_t e = whole;
                const unsigned long long src0 = whole.sgl_first >= a.entry ? whole.src_off : a.src;
                const unsigned long long src1 = w_end <= b.entry ? whole.src_off + whole.len : b.src;
                e.src_off = src0 + layer_off;
                e.len = src1 - src0;
                e.sgl_first = max(whole.sgl_first, a.entry);
                e.sgl_count = min(w_end, b.entry) - e.sgl_first;
                e.opcode = (uint16_t)p.opcode;
                e.layer = (uint16_t)p.layer;
                ring.sqes[(size_t)slot * ring.capacity + q] = e;
            }
        }
    }

    // SGL entries: a group of G lanes per item, lanes over the item's blocks.  G is the
    // power of two that covers an object's blocks (32 for big objects, 1 when every object
    // is a single block), so small objects do not leave most of a warp idle.
    const uint32_t lane = threadIdx.x & 31;
    uint32_t G = 1;
    while (G < 32 && G < g.blocks_per_obj) G <<= 1;
    const uint32_t per_warp = 32 / G;                   // items handled side by side
    const uint32_t sub = lane / G, sl = lane % G, leader = sub * G;
    const uint32_t gwarp = gtid >> 5, nwarps = gthreads >> 5;
    for (uint32_t i0 = gwarp * per_warp; i0 < n_items; i0 += nwarps * per_warp) {
        const uint32_t i = i0 + sub;
        const bool live = i < n_items;
        // leader: the item, its place in its group (copy c of k), the group's first entry,
        // its row in the block table and the object-side address of its first byte
        uint32_t q = 0, n_blk = 0, g_first = 0, k_copies = 1, c_copy = 0;
        unsigned long long meta0 = 0, meta1 = 0;
        if (live && sl == 0) {
            q = ring.plan_item[i];
            n_blk = ring.plan_cumblk[i + 1] - ring.plan_cumblk[i];
            const uint32_t gs = ring.plan_grp[i];
            g_first = ring.plan_cumblk[gs];
            k_copies = ring.plan_k[gs];
            c_copy = i - gs;
            const uint32_t o = q >> 1;
            uint32_t r = find_request(b.obj_start, b.n_req, o);
            uint32_t c = o - b.obj_start[r];
            meta0 = (unsigned long long)b.blk_start[r] + (unsigned long long)c * g.blocks_per_obj;
            const unsigned long long po = ring.plan_off[i];
            const uint32_t dev = (uint32_t)(po >> 56);
            const unsigned long long off = (po & ((1ull << 56) - 1)) + layer_off;
            const unsigned long long end = off + (unsigned long long)n_blk * g.block_bytes;
            if (end > p.store_bytes[dev]) {
                note_error(&hdr0->emit_status, TUTTI_EFAULT);
                meta1 = 0;
                n_blk = 0;                             // nothing is emitted for this item
            } else if (p.stage_base == 0 ||
                       ring.plan_stage[ring.plan_sqe_of[gs]] == STAGE_NONE) {
                meta1 = p.store_base[dev] + off;       // this context's bytes stay in the store
            } else {
                // staged transfer: the item's bytes sit in the staging buffer at its context's
                // place plus its distance from the context's first byte
                const uint32_t sq = ring.plan_sqe_of[gs];
                const unsigned long long at =
                    (unsigned long long)ring.plan_stage[sq] * g.block_bytes +
                    ((po & ((1ull << 56) - 1)) - ring.plan_sqe[sq].src_off);
                if (at + (unsigned long long)n_blk * g.block_bytes > p.stage_bytes) {
                    note_error(&hdr0->emit_status, TUTTI_EFAULT);
                    meta1 = 0;
                    n_blk = 0;
                } else {
                    meta1 = p.stage_base + at;
                }
            }
        }
        // the group leader read the item; its lanes get it by shuffle
        q = __shfl_sync(0xffffffffu, q, leader);
        n_blk = __shfl_sync(0xffffffffu, n_blk, leader);
        g_first = __shfl_sync(0xffffffffu, g_first, leader);
        k_copies = __shfl_sync(0xffffffffu, k_copies, leader);
        c_copy = __shfl_sync(0xffffffffu, c_copy, leader);
        const unsigned long long row0 = __shfl_sync(0xffffffffu, meta0, leader);
        const unsigned long long obj0 = __shfl_sync(0xffffffffu, meta1, leader);
        if (!live) continue;
        const unsigned long long pool_base = (q & 1) ? p.v_base : p.k_base;
        for (uint32_t j = sl; j < n_blk; j += G) {
            unsigned long long bi = row0 + j;
            tutti_sgl_t ent;
            ent.len = (uint32_t)g.block_bytes;
            if (bi >= b.n_blk) {
                note_error(&hdr0->emit_status, TUTTI_EFAULT);
                continue;
            }
            int32_t id = b.block_ids[bi];
            if (id < 0 || (unsigned long long)id >= p.n_pool_blocks) {
                note_error(&hdr0->emit_status, TUTTI_EFAULT);
                continue;
            }
            // block j of the source: one entry per member of the group, side by side; all
            // but the first are flagged as taking the bytes of the entry before them
            ent.addr = pool_base + (unsigned long long)id * p.block_stride;
            ent.id = (uint32_t)id | (c_copy ? TUTTI_SGL_FLAG_DUP : 0u);
            size_t at = (size_t)p.sgl_base + g_first + (size_t)j * k_copies + c_copy;
            ring.sgl[at] = ent;
            ring.obj_ptr[at] = obj0 + (unsigned long long)j * g.block_bytes;
        }
    }

    // publish: the last CTA to finish makes every IOCB of the build visible
    __syncthreads();
    __shared__ uint32_t s_last;
    if (threadIdx.x == 0) {
        __threadfence();
        uint32_t prev = atomicAdd(&hdr0->emit_done, 1u);
        s_last = (prev == gridDim.x - 1);
        __threadfence();
    }
    __syncthreads();
    if (!s_last) return;
    int32_t est = *((volatile int32_t *)&hdr0->emit_status);
    for (uint32_t k = threadIdx.x; k < p.n_iocb; k += blockDim.x) {
        uint32_t idx = p.first_iocb + k;
        IocbHdr *h = &ring.hdrs[idx & (ring.depth - 1)];
        if (est != 0) {
            h->status = est;
            h->total_entries = 0;
            h->bytes = 0;
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        hdr0->emit_done = 0;
        hdr0->emit_status = 0;
    }
    __threadfence();
    __syncthreads();
    for (uint32_t k = threadIdx.x; k < p.n_iocb; k += blockDim.x) {
        uint32_t idx = p.first_iocb + k;
        IocbHdr *h = &ring.hdrs[idx & (ring.depth - 1)];
        // release: descriptors before the state word
        asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(&h->state),
                     "r"(state_word(idx, PHASE_READY)) : "memory");
    }
}

uint32_t next_pow2(uint32_t v) {
    uint32_t p = 32;
    while (p < v) p <<= 1;
    return p;
}

}  // namespace

// The attribute is per device: set whenever a context is created, with its device current.
cudaError_t build_kernels_setup() {
    cudaError_t e = cudaFuncSetAttribute(plan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)(SMEM_SORT_ITEMS * 12));
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(bitonic_tile_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)(SORT_TILE * 12));
}

cudaError_t launch_plan(const RingDev &ring, const GeomDev &geom, const BatchDev &batch,
                        cudaStream_t stream, uint32_t *launches) {
    uint32_t np = next_pow2(2u * batch.n_obj);
    uint32_t n = 0;
    if (np <= SMEM_SORT_ITEMS) {
        // small batches get a small CTA: the kernel is a chain of block-wide barriers
        uint32_t threads = 64;
        while (threads < PLAN_THREADS && threads < np / 2) threads <<= 1;
        plan_kernel<<<1, threads, (size_t)np * 12, stream>>>(ring, geom, batch, np, 1, 0);
        n = 1;
    } else {
        // keys, then the sorting network as a handful of launches, then flags and scans
        plan_keys_kernel<<<(np + 255) / 256, 256, 0, stream>>>(ring, geom, batch, np);
        const uint32_t tiles = np / SORT_TILE;
        bitonic_tile_kernel<<<tiles, PLAN_THREADS, SORT_TILE * 12, stream>>>(ring.plan_key, ring.plan_idx,
                                                                           2, SORT_TILE);
        n = 2;
        for (uint32_t k = 2 * SORT_TILE; k <= np; k <<= 1) {
            for (uint32_t j = k >> 1; j >= SORT_TILE; j >>= 1) {
                bitonic_global_kernel<<<(np / 2 + 255) / 256, 256, 0, stream>>>(ring.plan_key, ring.plan_idx,
                                                                            np, k, j);
                ++n;
            }
            bitonic_tile_kernel<<<tiles, PLAN_THREADS, SORT_TILE * 12, stream>>>(ring.plan_key,
                                                                               ring.plan_idx, k, k);
            ++n;
        }
        plan_kernel<<<1, PLAN_THREADS, 0, stream>>>(ring, geom, batch, np, 0, 1);
        ++n;
    }
    if (launches) *launches = n;
    return cudaGetLastError();
}

cudaError_t launch_emit(const RingDev &ring, const GeomDev &geom, const BatchDev &batch,
                        uint32_t layer, uint32_t n_layers, uint32_t opcode, const PoolLayer &pool,
                        const PoolLayerDev *pools, const uint64_t *store_base,
                        const uint64_t *store_bytes, uint32_t first_iocb, uint32_t n_iocb,
                        uint32_t sgl_base, uint32_t sgl_reserved, uint32_t entries_per_iocb,
                        uint64_t stage_base, uint64_t stage_bytes, int device_sms,
                        cudaStream_t stream) {
    EmitParams p;
    p.entries_per_iocb = entries_per_iocb;
    p.stage_base = stage_base;
    p.stage_bytes = stage_bytes;
    p.layer = layer;
    p.opcode = opcode;
    p.k_base = pool.k_base;
    p.v_base = pool.v_base;
    p.block_stride = pool.block_stride;
    p.n_pool_blocks = pool.n_blocks;
    p.pools = pools;
    for (int d = 0; d < TUTTI_MAX_DEVICES; ++d) {
        p.store_base[d] = store_base[d];
        p.store_bytes[d] = store_bytes[d];
    }
    p.first_iocb = first_iocb;       // of the first layer; n_iocb and sgl_reserved are per layer
    p.n_iocb = n_iocb;
    p.sgl_base = sgl_base;
    p.sgl_reserved = sgl_reserved;
    uint32_t items = 2u * batch.n_obj;
    uint32_t G = 1;
    while (G < 32 && G < geom.blocks_per_obj) G <<= 1;
    const uint32_t per_cta = 8 * (32 / G);             // 8 warps, 32/G items side by side
    uint32_t ctas = (items + per_cta - 1) / per_cta;
    uint32_t cap = (uint32_t)device_sms * 2u;
    if (n_layers > 1) cap = cap / (n_layers < 8 ? n_layers : 8) + 1;   // the layers share the SMs
    if (ctas > cap) ctas = cap;
    if (ctas == 0) ctas = 1;
    return launch_dependent(emit_kernel, dim3(ctas, n_layers), dim3(EMIT_THREADS), 0, stream, ring,
                            geom, batch, p);
}

}  // namespace tutti
