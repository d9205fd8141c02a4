// Paged scatter / gather between contiguous KV objects and the block-table-indexed
// KV pool (layer-wise Retrieve / Store of paper Section 3.1 and 3.4), executed from
// the IOCBs of the submission ring (Section 3.2 step 3, issue_io), with completion
// entries written to the CQ by the kernel itself.
//
// Two engines over the same descriptors:
//   ldst   256-thread CTAs; every lane moves 16 bytes per instruction, eight
//          independent loads in flight per lane before the first store; a warp owns a
//          4 KiB sub-range of a tile, its lanes 0..7 fetch the SGL entries of that
//          sub-range once and broadcast them with shuffles.
//   bulk   persistent CTAs whose warps each run a ring of shared-memory stages:
//          cp.async.bulk global->shared (mbarrier completion) then shared->global,
//          so a handful of threads keep >100 KiB in flight per SM.  This is the
//          engine of the SM-capped mode.  Head-major pool blocks are transposed on the
//          way through the stage by tiled tensor copies (cp.async.bulk.tensor, one box
//          of [block_tokens][row] per head).
// Both claim work in chunks with one atomicAdd per claim on the IOCB's cursor and
// account completion in bytes; the agent that lands the last byte writes the CQE.
//
// Every wait is bounded: a timed-out wait records TUTTI_ETIMEDOUT in the IOCB
// status and the kernel still terminates normally.
#include "tutti_internal.h"

namespace tutti {

namespace {

constexpr uint32_t CHUNK_BYTES = 32768;       // work unit of both engines
constexpr int LDST_THREADS = 256;             // one copy group of the ldst engine
constexpr int LDST_MAX_GROUPS = 4;            // groups per CTA in a capped launch
constexpr int LDST_PAD_SMEM = 120 * 1024;     // more than half an SM's shared memory
constexpr uint32_t MBAR_TRY_LIMIT = 1u << 22;

struct CopyParams {
    RingDev ring;
    uint32_t first_iocb, n_iocb, opcode;
    unsigned long long wait_ns;
    uint32_t claim_chunks;
    uint32_t stages;        // bulk engine: stages per warp
    uint32_t chunk_bytes;   // bulk engine: bytes per stage (a power of two, 4..32 KiB)
    uint32_t inject_timeout; // bulk engine: report the first wait of every stage as run out
    uint32_t *smid_log;     // [grid] SM every CTA of the launch ran on (inspection)
    PermGeom perm;          // head-major pool blocks
};

// Offset inside a head-major pool block of the byte that sits at `off` in the
// token-major object: off = (t * heads + h) * row + x  ->  (h * tokens + t) * row + x.
__device__ __forceinline__ uint32_t hnd_offset(uint32_t off, const PermGeom &g) {
    const uint32_t t = off / g.token_bytes, y = off - t * g.token_bytes;
    const uint32_t hh = y / g.row_bytes, x = y - hh * g.row_bytes;
    return (hh * g.block_tokens + t) * g.row_bytes + x;
}

__device__ __forceinline__ unsigned long long globaltimer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ uint32_t smid() {
    uint32_t v;
    asm volatile("mov.u32 %0, %%smid;" : "=r"(v));
    return v;
}

__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t *p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Completion entry into pinned host memory: entry, system fence, then its sequence word.
__device__ void post_cqe(const RingDev &ring, uint32_t iocb_idx, int32_t status,
                         unsigned long long bytes) {
    uint32_t pos = atomicAdd(ring.cq_reserve, 1u);
    CqSlot *slot = &ring.cq[pos & (ring.depth - 1)];
    volatile tutti_cqe_t *c = &slot->cqe;
    c->iocb_idx = iocb_idx;
    c->status = status;
    c->bytes = bytes;
    __threadfence_system();
    *((volatile uint32_t *)&slot->seq) = pos + 1;
    __threadfence_system();
}

enum { IOCB_RUN = 0, IOCB_SKIP = 1 };

// One agent (thread) waits until the IOCB is published.  Returns IOCB_RUN when it is
// ready, IOCB_SKIP when it is already complete or when the wait ran out (in which
// case exactly one agent posts a TUTTI_ETIMEDOUT completion).
__device__ int wait_iocb_ready(const RingDev &ring, IocbHdr *h, uint32_t idx,
                               unsigned long long wait_ns) {
    const uint32_t ready = state_word(idx, PHASE_READY), done = state_word(idx, PHASE_DONE);
    const unsigned long long t0 = globaltimer_ns();
    for (uint32_t it = 0;; ++it) {
        uint32_t s = ld_acquire_u32(&h->state);
        if (s == ready) return IOCB_RUN;
        if (s == done) return IOCB_SKIP;
        if (globaltimer_ns() - t0 > wait_ns || it > (1u << 24)) {
            if (atomicCAS(&h->state, s, done) == s) {
                __threadfence();
                post_cqe(ring, idx, TUTTI_ETIMEDOUT, 0);
                return IOCB_SKIP;
            }
        }
        __nanosleep(64);
    }
}

// An IOCB with nothing to move (empty, or carrying a build error): one agent wins the
// READY -> DONE transition and posts the completion.
__device__ void complete_empty(const RingDev &ring, IocbHdr *h, uint32_t idx) {
    if (atomicCAS(&h->state, state_word(idx, PHASE_READY), state_word(idx, PHASE_DONE)) ==
        state_word(idx, PHASE_READY))
        post_cqe(ring, idx, h->status, 0);
}

constexpr int BULK_MAX_STAGES = 8;

// Geometry of the chunks of one IOCB with uniform entry length.
struct ChunkGeom {
    uint32_t elen;       // entry length
    uint32_t per_chunk;  // entries per chunk when elen <= chunk bytes (1..32), else 0
    uint32_t pieces;     // pieces per entry when elen > chunk bytes, else 0
    uint32_t n_chunks;
    uint32_t total;
};

__device__ __forceinline__ ChunkGeom chunk_geom(uint32_t total, uint32_t elen, uint32_t CB) {
    ChunkGeom g;
    g.elen = elen;
    g.total = total;
    if (elen <= CB) {
        uint32_t pc = CB / elen;
        g.per_chunk = pc > 32 ? 32 : pc;
        g.pieces = 0;
        g.n_chunks = (total + g.per_chunk - 1) / g.per_chunk;
    } else {
        g.per_chunk = 0;
        g.pieces = (elen + CB - 1) / CB;
        g.n_chunks = total * g.pieces;
    }
    return g;
}


// Number of claim units (what claim_cursor counts) of a published IOCB under this launch's
// engine: tiles / chunks for uniform entries, entries for the per-entry paths.  0xffffffff for
// an IOCB the engine will refuse (it must be opened, not skipped).  `bulk_chunk` is the bulk
// engine's stage size, 0 for the ldst engine; `tm_valid` says whether head-major blocks can be
// staged.  The copy loops use the very same function, so a look-ahead that skips IOCBs whose
// cursor has passed this count can never skip unclaimed work.
__device__ __forceinline__ uint32_t claim_units(const IocbHdr *h, const PermGeom &perm,
                                                uint32_t bulk_chunk, bool tm_valid) {
    const uint32_t total = h->total_entries, elen = h->entry_len;
    const bool hnd = (h->opcode & TUTTI_OP_FLAG_HND) != 0;
    if (hnd && (elen == 0 || elen != perm.block_tokens * perm.token_bytes)) return 0xffffffffu;
    if (bulk_chunk) {
        const bool hnd_staged = hnd && elen <= bulk_chunk && tm_valid && perm.n_heads <= 32;
        if (elen == 0 || (hnd && !hnd_staged)) return total;      // per-entry vector path
        if (hnd_staged) return total;                              // one block per stage
        return chunk_geom(total, elen, bulk_chunk).n_chunks;
    }
    if (elen != 0 && (elen & 511u) == 0)
        return (uint32_t)(((unsigned long long)total * elen + CHUNK_BYTES - 1) / CHUNK_BYTES);
    return total;
}

// Warp-collective look-ahead over the IOCBs [bi, n_iocb) of a launch: 32 headers are read at
// a time, and the leading ones that need no copying — already complete, or published with
// nothing to move (the unused tail of a build's reservation, or a build error) — are
// skipped without a round trip each; so are IOCBs whose work has all been claimed already
// (many small IOCBs in one launch: an agent does not open what others are finishing).  The
// `designated` warp (one per launch) completes the published-but-empty ones, one lane per
// IOCB.  Returns the first IOCB that is either not published yet or has unclaimed work
// (n_iocb if none).
__device__ uint32_t skip_idle_iocbs(const RingDev &ring, uint32_t first_iocb, uint32_t bi,
                                    uint32_t n_iocb, bool designated, const PermGeom &perm,
                                    uint32_t bulk_chunk, bool tm_valid, bool *ready_out = nullptr) {
    const uint32_t lane = threadIdx.x & 31;
    bool ready_seen = false;
    while (bi < n_iocb) {
        const uint32_t k = bi + lane;
        bool idle = false, empty_ready = false, ready = false;
        IocbHdr *h = nullptr;
        uint32_t idx = first_iocb + k;
        if (k < n_iocb) {
            h = &ring.hdrs[idx & (ring.depth - 1)];
            const uint32_t st = ld_acquire_u32(&h->state);
            if (st == state_word(idx, PHASE_DONE)) {
                idle = true;
            } else if (st == state_word(idx, PHASE_READY)) {
                ready = true;
                empty_ready = (h->total_entries == 0 || h->status != 0);
                // every unit already claimed by other agents: nothing left to take here
                idle = empty_ready ||
                       *((volatile uint32_t *)&h->claim_cursor) >= claim_units(h, perm, bulk_chunk, tm_valid);
            }
        }
        const uint32_t mask = __ballot_sync(0xffffffffu, idle);
        const uint32_t lead = (mask == 0xffffffffu) ? 32u : (uint32_t)(__ffs(~mask) - 1);
        if (designated && empty_ready && lane < lead) complete_empty(ring, h, idx);
        bi += lead;
        if (lead < 32u) {
            // the IOCB the walk stops at was seen published (acquire): no second look needed
            ready_seen = __shfl_sync(0xffffffffu, ready, lead);
            __syncwarp();       // the other lanes read that header after this lane's acquire
            break;
        }
    }
    if (ready_out) *ready_out = ready_seen && bi < n_iocb;
    return bi < n_iocb ? bi : n_iocb;
}

// Account `bytes` landed; the agent that completes the IOCB posts the CQE.
__device__ void account_done(const RingDev &ring, IocbHdr *h, uint32_t idx,
                             unsigned long long bytes) {
    if (bytes == 0) return;
    __threadfence();
    unsigned long long before = atomicAdd(&h->done_bytes, bytes);
    if (before + bytes == h->bytes) {
        __threadfence();
        int32_t st = *((volatile int32_t *)&h->status);
        *((volatile uint32_t *)&h->state) = state_word(idx, PHASE_DONE);
        post_cqe(ring, idx, st, h->bytes);
    }
}

__device__ __forceinline__ uint4 ld_stream(const void *p) {
    uint4 v;
    asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ void st_stream(void *p, const uint4 &v) {
    asm volatile("st.global.L1::no_allocate.v4.u32 [%0], {%1,%2,%3,%4};"
                 ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// ---------------------------------------------------------------------------
// ldst engine
// ---------------------------------------------------------------------------
// A CTA is one or more independent copy groups of LDST_THREADS threads, each with its
// own named barrier.  On all SMs the launch is many one-group CTAs; a capped launch is
// exactly sm_count CTAs of several groups (one CTA per SM, kept alone on its SM by a
// shared-memory pad), so the cap holds on any stream.
__device__ __forceinline__ void group_sync(uint32_t grp) {
    asm volatile("bar.sync %0, %1;" ::"r"(grp + 1), "n"(LDST_THREADS) : "memory");
}

template <int TO_POOL>
__global__ void __launch_bounds__(LDST_THREADS * LDST_MAX_GROUPS, 1)
copy_ldst_kernel(CopyParams p) {
    __shared__ uint32_t s_claim_g[LDST_MAX_GROUPS];
    __shared__ int s_mode_g[LDST_MAX_GROUPS];
    __shared__ uint32_t s_bi_g[LDST_MAX_GROUPS];
    const uint32_t grp = threadIdx.x / LDST_THREADS, tid = threadIdx.x % LDST_THREADS;
    const uint32_t lane = tid & 31, warp = tid >> 5;
    uint32_t &s_claim = s_claim_g[grp];
    int &s_mode = s_mode_g[grp];
    uint32_t &s_bi = s_bi_g[grp];
    if (threadIdx.x == 0 && p.smid_log) p.smid_log[blockIdx.x] = smid();
    for (uint32_t bi = 0; bi < p.n_iocb; ++bi) {
        // warp 0 looks ahead past IOCBs that need no copying
        if (warp == 0) {
            uint32_t nb = skip_idle_iocbs(p.ring, p.first_iocb, bi, p.n_iocb, blockIdx.x == 0 && grp == 0,
                                          p.perm, 0, false);
            if (lane == 0) s_bi = nb;
        }
        group_sync(grp);
        bi = s_bi;
        if (bi >= p.n_iocb) break;
        const uint32_t idx = p.first_iocb + bi;
        IocbHdr *h = &p.ring.hdrs[idx & (p.ring.depth - 1)];
        if (tid == 0) s_mode = wait_iocb_ready(p.ring, h, idx, p.wait_ns);
        group_sync(grp);
        const int mode = s_mode;
        group_sync(grp);
        if (mode == IOCB_SKIP) continue;
        const uint32_t total = h->total_entries;
        if (total == 0 || h->status != 0) {
            if (tid == 0) complete_empty(p.ring, h, idx);
            continue;
        }
        const uint32_t elen = h->entry_len;
        const size_t e_base = (size_t)h->sgl_base + h->entry_first;
        const tutti_sgl_t *sgl = p.ring.sgl + e_base;
        const uint64_t *obj = p.ring.obj_ptr + e_base;
        const bool hnd = (h->opcode & TUTTI_OP_FLAG_HND) != 0;
        if (hnd && (elen == 0 || elen != p.perm.block_tokens * p.perm.token_bytes)) {
            // a head-major entry must be exactly one block
            if (tid == 0) {
                atomicCAS(&h->status, 0, TUTTI_EINVAL);
                __threadfence();
                if (atomicCAS(&h->state, state_word(idx, PHASE_READY), state_word(idx, PHASE_DONE)) ==
                    state_word(idx, PHASE_READY))
                    post_cqe(p.ring, idx, TUTTI_EINVAL, 0);
            }
            continue;
        }

        if (elen != 0 && (elen & 511u) == 0) {
            // uniform entries, every 512-byte warp row lies inside one entry
            const unsigned long long total_bytes = (unsigned long long)total * elen;
            const uint32_t n_tiles = claim_units(h, p.perm, 0, false);
            const bool pow2 = (elen & (elen - 1)) == 0;
            const uint32_t shift = 31 - __clz(elen);
            for (;;) {
                if (tid == 0) s_claim = atomicAdd(&h->claim_cursor, p.claim_chunks);
                group_sync(grp);
                const uint32_t t0 = s_claim;
                if (t0 >= n_tiles) { group_sync(grp); break; }
                const uint32_t t1 = min(t0 + p.claim_chunks, n_tiles);
                for (uint32_t t = t0; t < t1; ++t) {
                    // this warp's 4 KiB sub-range of the tile: 8 rows of 512 bytes
                    const unsigned long long p0 = (unsigned long long)t * CHUNK_BYTES + warp * 4096u;
                    if (p0 >= total_bytes) continue;
                    const uint32_t e0 = pow2 ? (uint32_t)(p0 >> shift) : (uint32_t)(p0 / elen);
                    const uint32_t off0 = (uint32_t)(p0 - (unsigned long long)e0 * elen);
                    if (off0 + 4096u <= elen) {
                        // the whole sub-range lies in one entry (blocks of 4 KiB and more):
                        // lane 0 reads the entry once, every lane gets it by shuffle
                        unsigned long long a_pool = 0, a_obj = 0;
                        if (lane == 0) { a_pool = sgl[e0].addr; a_obj = obj[e0]; }
                        a_pool = __shfl_sync(0xffffffffu, a_pool, 0);
                        a_obj = __shfl_sync(0xffffffffu, a_obj, 0);
                        const uint32_t o_obj = off0 + lane * 16u;
                        uint4 v[8];
                        if (!hnd) {
                            const char *src = reinterpret_cast<const char *>(TO_POOL ? a_obj : a_pool) + o_obj;
                            char *dst = reinterpret_cast<char *>(TO_POOL ? a_pool : a_obj) + o_obj;
#pragma unroll
                            for (int k = 0; k < 8; ++k) v[k] = ld_stream(src + k * 512);
#pragma unroll
                            for (int k = 0; k < 8; ++k) st_stream(dst + k * 512, v[k]);
                            // restore of an object shared by several requests: the following
                            // entries of this claim that repeat these bytes (one entry per
                            // tile, so every warp of the group sees the same flags) are stored
                            // from the registers just loaded, and their tiles are skipped
                            while (TO_POOL && elen == CHUNK_BYTES && t + 1 < t1) {
                                unsigned long long a_next = 0;
                                uint32_t id_next = 0;
                                if (lane == 0) {
                                    const tutti_sgl_t ent = sgl[t + 1];
                                    a_next = ent.addr;
                                    id_next = ent.id;
                                }
                                id_next = __shfl_sync(0xffffffffu, id_next, 0);
                                if (!(id_next & TUTTI_SGL_FLAG_DUP)) break;
                                a_next = __shfl_sync(0xffffffffu, a_next, 0);
                                char *dst2 = reinterpret_cast<char *>(a_next) + o_obj;
#pragma unroll
                                for (int k = 0; k < 8; ++k) st_stream(dst2 + k * 512, v[k]);
                                ++t;
                            }
                        } else {
                            // head-major pool block: every 16-byte vector keeps its place in the
                            // object and goes to the transposed row of the block
#pragma unroll
                            for (int k = 0; k < 8; ++k) {
                                const uint32_t oo = o_obj + k * 512u;
                                const uint32_t op = hnd_offset(oo, p.perm);
                                v[k] = ld_stream(reinterpret_cast<const void *>(
                                    TO_POOL ? a_obj + oo : a_pool + op));
                            }
#pragma unroll
                            for (int k = 0; k < 8; ++k) {
                                const uint32_t oo = o_obj + k * 512u;
                                const uint32_t op = hnd_offset(oo, p.perm);
                                st_stream(reinterpret_cast<void *>(TO_POOL ? a_pool + op : a_obj + oo), v[k]);
                            }
                        }
                        continue;
                    }
                    // small entries (512 B .. 2 KiB, e.g. 1-token pages): lanes 0..7 fetch the
                    // entries this sub-range touches, once; rows pick theirs by shuffle
                    unsigned long long my_pool = 0, my_obj = 0;
                    if (lane < 8 && e0 + lane < total) {
                        my_pool = sgl[e0 + lane].addr;
                        my_obj = obj[e0 + lane];
                    }
#pragma unroll 1
                    for (int half = 0; half < 2; ++half) {
                        uint4 v[4];
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const unsigned long long pk = p0 + (unsigned long long)(half * 4 + k) * 512u;
                            const bool ok = pk < total_bytes;
                            const uint32_t e = ok ? (pow2 ? (uint32_t)(pk >> shift) : (uint32_t)(pk / elen)) : e0;
                            const uint32_t off = (uint32_t)(pk - (unsigned long long)e * elen) + lane * 16u;
                            const unsigned long long a = __shfl_sync(0xffffffffu, TO_POOL ? my_obj : my_pool, e - e0);
                            const uint32_t o2 = (hnd && !TO_POOL) ? hnd_offset(off, p.perm) : off;
                            if (ok) v[k] = ld_stream(reinterpret_cast<const void *>(a + o2));
                        }
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const unsigned long long pk = p0 + (unsigned long long)(half * 4 + k) * 512u;
                            const bool ok = pk < total_bytes;
                            const uint32_t e = ok ? (pow2 ? (uint32_t)(pk >> shift) : (uint32_t)(pk / elen)) : e0;
                            const uint32_t off = (uint32_t)(pk - (unsigned long long)e * elen) + lane * 16u;
                            const unsigned long long a = __shfl_sync(0xffffffffu, TO_POOL ? my_pool : my_obj, e - e0);
                            const uint32_t o2 = (hnd && TO_POOL) ? hnd_offset(off, p.perm) : off;
                            if (ok) st_stream(reinterpret_cast<void *>(a + o2), v[k]);
                        }
                    }
                }
                group_sync(grp);
                if (tid == 0) {
                    unsigned long long b0 = (unsigned long long)t0 * CHUNK_BYTES;
                    unsigned long long b1 = min((unsigned long long)t1 * CHUNK_BYTES, total_bytes);
                    account_done(p.ring, h, idx, b1 - b0);
                }
            }
        } else {
            // general entries (lengths may differ): one warp per entry
            const uint32_t per_claim = 64;
            for (;;) {
                if (tid == 0) s_claim = atomicAdd(&h->claim_cursor, per_claim);
                group_sync(grp);
                const uint32_t c0 = s_claim;
                if (c0 >= total) { group_sync(grp); break; }
                const uint32_t c1 = min(c0 + per_claim, total);
                unsigned long long moved = 0;
                for (uint32_t e = c0 + warp; e < c1; e += LDST_THREADS / 32) {
                    unsigned long long a_pool = 0, a_obj = 0;
                    uint32_t len = 0;
                    if (lane == 0) { a_pool = sgl[e].addr; len = sgl[e].len; a_obj = obj[e]; }
                    a_pool = __shfl_sync(0xffffffffu, a_pool, 0);
                    a_obj = __shfl_sync(0xffffffffu, a_obj, 0);
                    len = __shfl_sync(0xffffffffu, len, 0);
                    for (uint32_t o = lane * 16u; o < len; o += 512u) {
                        const uint32_t op = hnd ? hnd_offset(o, p.perm) : o;
                        const unsigned long long src = TO_POOL ? a_obj + o : a_pool + op;
                        const unsigned long long dst = TO_POOL ? a_pool + op : a_obj + o;
                        st_stream(reinterpret_cast<void *>(dst),
                                  ld_stream(reinterpret_cast<const void *>(src)));
                    }
                    moved += len;
                }
                __syncwarp();
                if (lane == 0) account_done(p.ring, h, idx, moved);
                group_sync(grp);
            }
        }
    }
}

// ---------------------------------------------------------------------------
// bulk-async engine
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait for a phase of an mbarrier; false when it gave up.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity) {
    for (uint32_t it = 0; it < MBAR_TRY_LIMIT; ++it)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst_smem, unsigned long long src, uint32_t bytes,
                                         uint32_t bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(dst_smem), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void bulk_s2g(unsigned long long dst, uint32_t src_smem, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                 ::"l"(dst), "r"(src_smem), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_commit() {
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
__device__ __forceinline__ void bulk_wait_read_1() {
    asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
}
__device__ __forceinline__ void bulk_wait_all() {
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// Tiled tensor copies: one head of one block, [block_tokens][row] in shared memory, against the
// store region seen as [token row][head][row].  Coordinates: word 0 of the row (always 16-byte
// aligned), head, token row.
__device__ __forceinline__ void tensor_g2s(uint32_t dst_smem, const CUtensorMap *map, uint32_t head,
                                           uint32_t row, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst_smem), "l"(reinterpret_cast<unsigned long long>(map)), "r"(0), "r"(head), "r"(row),
          "r"(bar) : "memory");
}
__device__ __forceinline__ void tensor_s2g(const CUtensorMap *map, uint32_t head, uint32_t row,
                                           uint32_t src_smem) {
    asm volatile(
        "cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%1, %2, %3}], [%4];"
        ::"l"(reinterpret_cast<unsigned long long>(map)), "r"(0), "r"(head), "r"(row), "r"(src_smem)
        : "memory");
}

// Each warp of the CTA is an independent agent with its own ring of stages, fed by a
// stream of chunks that runs across the IOCBs of the launch without draining in between.
// Shared memory: [warps][stages][chunk bytes] data, [warps][stages] mbarriers, then per
// stage the store descriptor of every lane (address, bytes, offset in the stage) and
// the chunk's byte count and IOCB.
template <int TO_POOL>
__global__ void __launch_bounds__(256, 1)
copy_bulk_kernel(CopyParams p, const __grid_constant__ StoreTensorMaps tm) {
    extern __shared__ __align__(128) unsigned char smem[];
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t n_warps = blockDim.x >> 5;
    if (threadIdx.x == 0 && p.smid_log) p.smid_log[blockIdx.x] = smid();
    const uint32_t S = p.stages;
    const uint32_t CB = p.chunk_bytes;
    unsigned char *data = smem + (size_t)warp * S * CB;
    unsigned long long *bars = reinterpret_cast<unsigned long long *>(
        smem + (size_t)n_warps * S * CB) + warp * S;
    unsigned char *meta = smem + (size_t)n_warps * S * (CB + 8);
    const size_t lanes_all = (size_t)n_warps * S * 32;
    unsigned long long *st_addr_of = reinterpret_cast<unsigned long long *>(meta) + (size_t)warp * S * 32;
    uint32_t *st_bytes_of = reinterpret_cast<uint32_t *>(meta + lanes_all * 8) + (size_t)warp * S * 32;
    uint32_t *st_off_of = reinterpret_cast<uint32_t *>(meta + lanes_all * 12) + (size_t)warp * S * 32;
    uint32_t *chunk_bytes_of = reinterpret_cast<uint32_t *>(meta + lanes_all * 16) + warp * S;
    uint32_t *chunk_iocb_of = reinterpret_cast<uint32_t *>(meta + lanes_all * 16 +
                                                           (size_t)n_warps * S * 4) + warp * S;

    if (lane == 0)
        for (uint32_t s = 0; s < S; ++s) mbar_init(smem_u32(&bars[s]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async();
    __syncwarp();

    uint32_t phase_bits = 0;   // parity of every stage's mbarrier (bit s)
    uint32_t head = 0, tail = 0;            // stages issued / drained (monotonic)
    bool failed = false;

    // ---- source side of the stream: the IOCB chunks are being claimed from
    uint32_t f_bi = 0;                      // next IOCB of the launch to open
    uint32_t f_start = 0, f_limit = p.n_iocb;   // starting point and end of the current sweep
    uint32_t claim = p.claim_chunks;            // chunks per work claim of this agent
    bool f_wrapped = false;
    IocbHdr *f_h = nullptr;
    ChunkGeom cg{0, 0, 0, 0, 0};
    const tutti_sgl_t *sgl = nullptr;
    const uint64_t *obj = nullptr;
    bool f_open = false;
    uint32_t f_cur_bi = 0;
    bool f_hnd = false;                     // head-major blocks, transposed through the stage
    uint32_t pending_claim = 0, cur = 0, cur_end = 0;
    // the next chunk, fetched ahead: one bulk load and one bulk store per lane
    bool have_next = false;
    uint32_t n_bi = 0, ld_bytes = 0, st_bytes = 0, st_off = 0;
    bool n_hnd = false;
    unsigned long long ld_addr = 0, st_addr = 0;

    // ---- sink side: bytes stored for the IOCB being accounted
    uint32_t acct_bi = 0;
    unsigned long long moved = 0;

    auto hdr_of = [&](uint32_t bi) -> IocbHdr * {
        return &p.ring.hdrs[(p.first_iocb + bi) & (p.ring.depth - 1)];
    };
    // all stores of this agent so far have landed: account what belongs to acct_bi
    auto flush_account = [&]() {
        if (moved == 0) return;
        bulk_wait_all();
        __syncwarp();
        if (lane == 0) account_done(p.ring, hdr_of(acct_bi), p.first_iocb + acct_bi, moved);
        __syncwarp();
        moved = 0;
    };

    // Entries of differing lengths (host-prepared IOCBs only): plain vector copies, one
    // entry per warp at a time, outside the staged pipeline.
    auto copy_varlen = [&](IocbHdr *h, uint32_t idx, uint32_t total, bool hnd) {
        for (;;) {
            uint32_t c0 = 0;
            if (lane == 0) c0 = atomicAdd(&h->claim_cursor, 8u);
            c0 = __shfl_sync(0xffffffffu, c0, 0);
            if (c0 >= total) break;
            const uint32_t c1 = min(c0 + 8u, total);
            unsigned long long mv = 0;
            for (uint32_t e = c0; e < c1; ++e) {
                unsigned long long a_pool = 0, a_obj = 0;
                uint32_t len = 0;
                if (lane == 0) { a_pool = sgl[e].addr; len = sgl[e].len; a_obj = obj[e]; }
                a_pool = __shfl_sync(0xffffffffu, a_pool, 0);
                a_obj = __shfl_sync(0xffffffffu, a_obj, 0);
                len = __shfl_sync(0xffffffffu, len, 0);
                for (uint32_t o = lane * 16u; o < len; o += 512u) {
                    const uint32_t op = hnd ? hnd_offset(o, p.perm) : o;
                    const unsigned long long src = TO_POOL ? a_obj + o : a_pool + op;
                    const unsigned long long dst = TO_POOL ? a_pool + op : a_obj + o;
                    st_stream(reinterpret_cast<void *>(dst), ld_stream(reinterpret_cast<const void *>(src)));
                }
                mv += len;
            }
            __syncwarp();
            if (lane == 0) account_done(p.ring, h, idx, mv);
        }
    };

    // Open the next IOCB that has staged work; false when the launch has none left.
    auto open_next_iocb = [&]() -> bool {
        for (;;) {
            if (f_bi >= f_limit) {
                // end of the launch's IOCBs: an agent that did not start at the first one goes
                // round once, over the IOCBs before its starting point
                if (f_wrapped || f_start == 0) break;
                f_wrapped = true;
                f_bi = 0;
                f_limit = f_start;
                continue;
            }
            bool seen_ready = false;
            f_bi = skip_idle_iocbs(p.ring, p.first_iocb, f_bi, f_limit,
                                   blockIdx.x == 0 && warp == 0, p.perm, CB, tm.valid != 0,
                                   &seen_ready);
            if (f_bi >= f_limit) continue;
            const uint32_t bi = f_bi++;
            const uint32_t idx = p.first_iocb + bi;
            IocbHdr *h = hdr_of(bi);
            if (!seen_ready) {
                int mode = 0;
                if (lane == 0) mode = wait_iocb_ready(p.ring, h, idx, p.wait_ns);
                mode = __shfl_sync(0xffffffffu, mode, 0);
                if (mode == IOCB_SKIP) continue;
            }
            const uint32_t total = h->total_entries;
            if (total == 0 || h->status != 0) {
                if (lane == 0) complete_empty(p.ring, h, idx);
                continue;
            }
            const size_t e_base = (size_t)h->sgl_base + h->entry_first;
            sgl = p.ring.sgl + e_base;
            obj = p.ring.obj_ptr + e_base;
            const bool hnd = (h->opcode & TUTTI_OP_FLAG_HND) != 0;
            if (hnd && h->entry_len != p.perm.block_tokens * p.perm.token_bytes) {
                if (lane == 0) {
                    atomicCAS(&h->status, 0, TUTTI_EINVAL);
                    __threadfence();
                    if (atomicCAS(&h->state, state_word(idx, PHASE_READY), state_word(idx, PHASE_DONE)) ==
                        state_word(idx, PHASE_READY))
                        post_cqe(p.ring, idx, TUTTI_EINVAL, 0);
                }
                continue;
            }
            // entries of differing lengths go through the per-entry vector path; so do
            // head-major blocks that do not fit one stage
            const bool hnd_staged = hnd && h->entry_len <= CB && tm.valid && p.perm.n_heads <= 32;
            if (h->entry_len == 0 || (hnd && !hnd_staged)) { copy_varlen(h, idx, total, hnd); continue; }
            f_h = h;
            f_cur_bi = bi;
            f_hnd = hnd_staged;
            cg = chunk_geom(total, h->entry_len, CB);
            if (f_hnd) cg.per_chunk = 1;                            // one block per stage
            cg.n_chunks = claim_units(h, p.perm, CB, tm.valid != 0);
            cur = cur_end = 0;
            if (lane == 0) pending_claim = atomicAdd(&h->claim_cursor, claim);
            return true;
        }
        return false;
    };

    // A launch of many small IOCBs (a whole pass of a short prefix): opening an IOCB costs a
    // few dependent round trips, so an agent should not have to open many for its share of the
    // work, and the agents should not all queue up at the first one.  With the first IOCB's
    // size as the estimate of all of them, a claim grows to about half an agent's share of the
    // launch (the option's value stays when one IOCB alone feeds every agent several times), and
    // agent a starts at the IOCB that this claim size assigns to it, walking on cyclically.
    // Half a share is too coarse a grain once the share is large (IOCBs of tens of MiB: the
    // last claims would decide when the launch ends): beyond MID_CLAIM units the claim stops
    // there and the agents are dealt out evenly over the IOCBs instead, so that each still
    // opens about one IOCB and takes its share from it in several claims.
    constexpr uint32_t MID_CLAIM = 8;
    if (p.n_iocb > 1) {
        uint32_t start = 0, cl = claim;
        if (lane == 0) {
            // (the kernel may have become resident while the build is still writing: the
            // first IOCB's publication is awaited like any other, bounded)
            IocbHdr *h0 = hdr_of(0);
            if (wait_iocb_ready(p.ring, h0, p.first_iocb, p.wait_ns) == IOCB_RUN &&
                h0->total_entries != 0 && h0->status == 0) {
                const uint32_t u = claim_units(h0, p.perm, CB, tm.valid != 0);
                const uint32_t n_agents = gridDim.x * n_warps;
                if (u != 0xffffffffu && u / claim < 8u * n_agents) {
                    const unsigned long long share =
                        ((unsigned long long)u * p.n_iocb + n_agents - 1) / n_agents;
                    const unsigned long long half = (share + 1) / 2;
                    if (half > cl) cl = (uint32_t)(half < u ? half : u);
                    const uint32_t agent = warp * gridDim.x + blockIdx.x;
                    if (cl > MID_CLAIM && cl > claim) {
                        cl = max(MID_CLAIM, claim);
                        start = min((uint32_t)((unsigned long long)agent * p.n_iocb / n_agents),
                                    p.n_iocb - 1);
                    } else {
                        const uint32_t per = u / cl + (u % cl != 0);   // agents one IOCB feeds
                        start = min(agent / per, p.n_iocb - 1);
                    }
                }
            }
        }
        f_start = f_bi = __shfl_sync(0xffffffffu, start, 0);
        claim = __shfl_sync(0xffffffffu, cl, 0);
    }

    // Work claims are taken one ahead of need (the atomic's latency hides behind the
    // copies of the current claim), and the addresses of the next chunk are fetched as
    // soon as the current chunk's loads are issued.
    auto fetch_next = [&]() {
        have_next = false;
        for (;;) {
            if (!f_open) {
                if (!open_next_iocb()) return;
                f_open = true;
            }
            if (cur == cur_end) {
                uint32_t c0 = __shfl_sync(0xffffffffu, pending_claim, 0);
                if (c0 >= cg.n_chunks) { f_open = false; continue; }
                cur = c0;
                cur_end = min(c0 + claim, cg.n_chunks);
                if (lane == 0) pending_claim = atomicAdd(&f_h->claim_cursor, claim);
            }
            break;
        }
        const uint32_t c = cur++;
        have_next = true;
        n_bi = f_cur_bi;
        n_hnd = f_hnd;
        ld_bytes = 0; st_bytes = 0; st_off = 0; ld_addr = 0; st_addr = 0;
        if (cg.per_chunk == 1) {
            // one entry per stage (a whole block; also every head-major block).  On a restore
            // the entries right after it that repeat its bytes (the same stored chunk going to
            // other requests' blocks) share the stage: one load, one store per destination.
            const uint32_t n_in = min(32u, cur_end - c);         // entries of this claim from c on
            unsigned long long a_obj = 0, a_pool = 0;
            uint32_t id_flags = 0;
            if (lane < n_in) {
                const tutti_sgl_t ent = sgl[c + lane];
                a_pool = ent.addr;
                id_flags = ent.id;
            }
            if (lane == 0) a_obj = obj[c];
            a_obj = __shfl_sync(0xffffffffu, a_obj, 0);
            const bool rep = TO_POOL && lane > 0 && lane < n_in && (id_flags & TUTTI_SGL_FLAG_DUP);
            const uint32_t reps = __ballot_sync(0xffffffffu, rep) | 1u;
            const uint32_t m = (reps == 0xffffffffu) ? 32u : (uint32_t)(__ffs(~reps) - 1);
            cur += m - 1;                                         // the repeats are consumed too
            if (f_hnd) {
                // object side as (device, token row) for the tensor map; the rows are spread
                // over the lanes, so every lane carries the packed source
                uint32_t dv = 0;
                for (uint32_t d = 1; d < tm.n_devices; ++d)
                    if (a_obj >= tm.base[d] && a_obj < tm.base[d] + tm.bytes[d]) dv = d;
                const unsigned long long rowi = (a_obj - tm.base[dv]) / p.perm.token_bytes;
                const unsigned long long packed = (rowi << 8) | dv;
                const unsigned long long pool0 = __shfl_sync(0xffffffffu, a_pool, 0);
                if (TO_POOL) {
                    ld_addr = packed;
                    ld_bytes = (lane == 0) ? cg.elen : 0;
                    st_addr = a_pool;
                    st_bytes = (lane < m) ? cg.elen : 0;
                } else {
                    ld_addr = pool0;
                    ld_bytes = (lane == 0) ? cg.elen : 0;
                    st_addr = packed;
                    st_bytes = (lane == 0) ? cg.elen : 0;
                }
            } else if (TO_POOL) {
                ld_addr = a_obj;
                ld_bytes = (lane == 0) ? cg.elen : 0;
                st_addr = a_pool;
                st_bytes = (lane < m) ? cg.elen : 0;
            } else {
                ld_addr = a_pool;
                ld_bytes = (lane == 0) ? cg.elen : 0;
                st_addr = a_obj;
                st_bytes = (lane == 0) ? cg.elen : 0;
            }
        } else if (cg.per_chunk) {
            const uint32_t e0 = c * cg.per_chunk;
            const uint32_t n_e = min(cg.per_chunk, cg.total - e0);
            unsigned long long a_obj = 0, a_pool = 0;
            uint32_t id_flags = 0;
            if (lane < n_e) {
                const tutti_sgl_t ent = sgl[e0 + lane];
                a_obj = obj[e0 + lane];
                a_pool = ent.addr;
                id_flags = ent.id;
            }
            // restore: an entry that repeats the bytes of the entry before it brings nothing
            // into the stage and is stored from its predecessor's place (the first entry of a
            // chunk always loads: its predecessor sits in another chunk)
            const bool rep = TO_POOL && lane > 0 && lane < n_e && (id_flags & TUTTI_SGL_FLAG_DUP);
            const uint32_t live = (n_e >= 32u) ? 0xffffffffu : ((1u << n_e) - 1u);
            const uint32_t uniq = live & ~__ballot_sync(0xffffffffu, rep);
            const uint32_t upto = 0xffffffffu >> (31 - lane);     // lanes 0..lane
            const uint32_t slot = (lane < n_e) ? (uint32_t)__popc(uniq & upto) - 1u : 0u;
            // the object side is contiguous in runs: one bulk copy per run
            unsigned long long prev = __shfl_up_sync(0xffffffffu, a_obj, 1);
            bool is_head = ((uniq >> lane) & 1u) && (lane == 0 || a_obj != prev + cg.elen);
            uint32_t heads = __ballot_sync(0xffffffffu, is_head);
            uint32_t run_bytes = 0;
            if (is_head) {
                uint32_t above = lane < 31 ? heads >> (lane + 1) : 0u;
                uint32_t next = above ? lane + __ffs(above) : n_e;
                const uint32_t below_next = (next >= 32u) ? 0xffffffffu : ((1u << next) - 1u);
                run_bytes = (uint32_t)__popc(uniq & below_next & ~(upto >> 1)) * cg.elen;
            }
            const uint32_t one = lane < n_e ? cg.elen : 0;
            st_off = slot * cg.elen;
            if (TO_POOL) { ld_addr = a_obj; ld_bytes = run_bytes; st_addr = a_pool; st_bytes = one; }
            else         { ld_addr = a_pool; ld_bytes = one; st_addr = a_obj; st_bytes = run_bytes; }
        } else {
            // entries longer than a stage are moved in pieces.  Chunks are numbered piece-major
            // inside blocks of 32 entries (piece 0 of entries 0..31, then piece 1 of them, ...),
            // so that consecutive chunks are the same piece of consecutive entries: on a
            // restore, entries that repeat their predecessor's bytes share the stage here too.
            // (A save has no repeats to fold and keeps entry-major order, which writes the
            // object side sequentially.)
            const uint32_t PB = TO_POOL ? 32u : 1u;               // entries per block
            const uint32_t span = PB * cg.pieces;
            const uint32_t blk = c / span, rem = c - blk * span;
            const uint32_t e_base = blk * PB;
            const uint32_t n_b = min(PB, cg.total - e_base);      // entries of this block
            const uint32_t piece = rem / n_b, ei = rem - piece * n_b;
            const uint32_t e = e_base + ei;
            const uint32_t off = piece * CB;
            const uint32_t bytes = min(CB, cg.elen - off);
            const uint32_t n_in = min(min(32u, cur_end - c), n_b - ei);
            unsigned long long a_obj = 0, a_pool = 0;
            uint32_t id_flags = 0;
            if (lane < n_in) {
                const tutti_sgl_t ent = sgl[e + lane];
                a_pool = ent.addr + off;
                id_flags = ent.id;
            }
            if (lane == 0) a_obj = obj[e] + off;
            const bool rep = TO_POOL && lane > 0 && lane < n_in && (id_flags & TUTTI_SGL_FLAG_DUP);
            const uint32_t reps = __ballot_sync(0xffffffffu, rep) | 1u;
            const uint32_t m = (reps == 0xffffffffu) ? 32u : (uint32_t)(__ffs(~reps) - 1);
            cur += m - 1;
            if (TO_POOL) {
                ld_addr = a_obj;
                ld_bytes = (lane == 0) ? bytes : 0;
                st_addr = a_pool;
                st_bytes = (lane < m) ? bytes : 0;
            } else if (lane == 0) {
                ld_addr = a_pool;
                st_addr = a_obj;
                ld_bytes = bytes; st_bytes = bytes;
            }
        }
    };
    fetch_next();

    for (;;) {
        // ---- issue loads while a stage is free (one stage of slack is kept for the
        //      store that may still be reading shared memory)
        while (!failed && have_next && head - tail < S - 1) {
            const uint32_t s = head % S;
            // the store that last used this stage must have finished reading it:
            // at most one newer store group may still be pending
            bulk_wait_read_1();
            __syncwarp();
            const uint32_t bar = smem_u32(&bars[s]);
            const uint32_t sbase = smem_u32(data + (size_t)s * CB);
            const uint32_t total_bytes = __reduce_add_sync(0xffffffffu, ld_bytes);
            const uint32_t landed_bytes = __reduce_add_sync(0xffffffffu, st_bytes);
            if (lane == 0) mbar_expect_tx(bar, total_bytes);
            __syncwarp();
            if (n_hnd && TO_POOL) {
                // token-major object -> head-major stage: one tiled tensor copy per head
                // (box = [block_tokens][row]), heads dealt out over the lanes
                if (lane < p.perm.n_heads)
                    tensor_g2s(sbase + lane * p.perm.block_tokens * p.perm.row_bytes,
                               &tm.map[ld_addr & 0xff], lane, (uint32_t)(ld_addr >> 8), bar);
            } else if (ld_bytes) {
                bulk_g2s(sbase + st_off, ld_addr, ld_bytes, bar);
            }
            st_addr_of[s * 32 + lane] = st_addr;
            st_bytes_of[s * 32 + lane] = st_bytes;
            st_off_of[s * 32 + lane] = st_off;
            if (lane == 0) {
                chunk_bytes_of[s] = landed_bytes;       // completion is counted in bytes landed
                chunk_iocb_of[s] = n_bi | (n_hnd ? 0x80000000u : 0u);
            }
            __syncwarp();
            ++head;
            fetch_next();
        }
        if (head == tail) {
            if (!failed || !have_next) break;
            // A wait ran out and every stage has been drained.  The chunks this agent has
            // claimed, and whatever the launch still offers, are accounted without being
            // copied (their IOCBs carry TUTTI_ETIMEDOUT): every IOCB still reaches its byte
            // count, so its completion entry is posted and nothing waits for it for ever.
            do {
                if (n_bi != acct_bi) {
                    flush_account();
                    acct_bi = n_bi;
                }
                if (lane == 0) atomicCAS(&hdr_of(n_bi)->status, 0, TUTTI_ETIMEDOUT);
                moved += __reduce_add_sync(0xffffffffu, st_bytes);
                fetch_next();
            } while (have_next);
            break;
        }

        // ---- drain the oldest stage: wait for its bytes, store them
        const uint32_t s = tail % S;
        const uint32_t bar = smem_u32(&bars[s]);
        const uint32_t sbase = smem_u32(data + (size_t)s * CB);
        const uint32_t s_tag = chunk_iocb_of[s];
        const uint32_t s_bi = s_tag & 0x7fffffffu;
        const bool s_hnd = (s_tag >> 31) != 0;
        if (s_bi != acct_bi) {
            // first chunk of a later IOCB: close the books of the previous one.  Only the
            // stores are waited for; the loads already in flight keep streaming.
            flush_account();
            acct_bi = s_bi;
        }
        bool arrived = !p.inject_timeout && mbar_wait_bounded(bar, (phase_bits >> s) & 1u);
        arrived = __all_sync(0xffffffffu, arrived);
        if (!arrived) {
            failed = true;
            if (lane == 0) atomicCAS(&hdr_of(s_bi)->status, 0, TUTTI_ETIMEDOUT);
            // the stage is given up, but its copy may still be on its way: one more bounded
            // wait, so that nothing lands in this CTA's shared memory after it has left
            (void)mbar_wait_bounded(bar, (phase_bits >> s) & 1u);
            __syncwarp();
        }
        phase_bits ^= (1u << s);
        const unsigned long long dst = st_addr_of[s * 32 + lane];
        const uint32_t nbytes = st_bytes_of[s * 32 + lane];
        const uint32_t off = st_off_of[s * 32 + lane];
        if (s_hnd && !TO_POOL) {
            // head-major stage -> token-major object, one tiled tensor copy per head
            if (arrived && lane < p.perm.n_heads)
                tensor_s2g(&tm.map[dst & 0xff], lane, (uint32_t)(dst >> 8),
                           sbase + lane * p.perm.block_tokens * p.perm.row_bytes);
        } else if (arrived && nbytes) {
            bulk_s2g(dst, sbase + off, nbytes);
        }
        bulk_commit();
        moved += chunk_bytes_of[s];
        ++tail;
    }
    flush_account();
}

}  // namespace

cudaError_t copy_kernels_setup() {
    cudaError_t e;
    const int max_smem = 227 * 1024;
    e = cudaFuncSetAttribute(copy_bulk_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(copy_bulk_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem);
    if (e != cudaSuccess) return e;
    // the ldst engine uses dynamic shared memory only as a pad that keeps a capped CTA alone
    // on its SM
    e = cudaFuncSetAttribute(copy_ldst_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, LDST_PAD_SMEM);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(copy_ldst_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, LDST_PAD_SMEM);
    if (e != cudaSuccess) return e;
    return build_kernels_setup();
}

cudaError_t launch_copy(const RingDev &ring, uint32_t first_iocb, uint32_t n_iocb, uint32_t opcode,
                        uint32_t sm_count, int device_sms, const CopyOptions &opt, bool host_store,
                        bool pool_hnd, const PermGeom &perm, const StoreTensorMaps *maps,
                        uint32_t *smid_log, cudaStream_t stream, uint32_t *launches,
                        uint32_t *grid_out) {
    static const StoreTensorMaps no_maps = {};
    const StoreTensorMaps &tm = maps ? *maps : no_maps;
    CopyParams p;
    p.ring = ring;
    p.first_iocb = first_iocb;
    p.n_iocb = n_iocb;
    p.opcode = opcode;
    p.wait_ns = opt.wait_ns;
    p.inject_timeout = opt.inject_timeout;
    p.smid_log = smid_log;
    uint32_t grid = 0;
    cudaError_t err = cudaSuccess;
    // measured: small claims balance best when every SM takes part, larger ones amortise the
    // claim's round trip when few SMs carry everything
    // (a capped launch on a pinned-host store is bound by the link, not by balance: long claims
    // keep a shared block and the entries repeating it in one agent's hands, so it crosses the
    // link once)
    p.claim_chunks = opt.claim_chunks ? opt.claim_chunks : (sm_count ? (host_store ? 16 : 4) : 2);
    uint32_t engine = opt.engine;
    // measured: bulk-async wins on HBM, also for head-major blocks when tensor maps exist
    if (engine == 0) engine = (host_store || (pool_hnd && !(maps && maps->valid))) ? 1 : 2;
    p.perm = perm;
    const uint32_t sms = sm_count ? sm_count : (uint32_t)device_sms;
    if (engine == 2) {
        // measured on B200: all SMs -> 2 warps x 3 stages x 32 KiB; a capped launch gets
        // closest to the per-SM ceiling (~49 GB/s each way) with 4 warps x 3 stages x 16 KiB
        const bool capped_hbm = sm_count != 0;
        uint32_t warps = opt.bulk_warps ? opt.bulk_warps : (capped_hbm ? 4 : 2);
        uint32_t stages = opt.bulk_stages ? opt.bulk_stages : 3;
        if (warps > 8) warps = 8;
        if (stages < 2) stages = 2;
        if (stages > BULK_MAX_STAGES) stages = BULK_MAX_STAGES;
        uint32_t cb = opt.bulk_chunk ? opt.bulk_chunk : (capped_hbm ? 16384u : CHUNK_BYTES);
        const size_t per_stage = cb + 8 + 32 * 16 + 8;
        while ((size_t)warps * stages * per_stage > 224u * 1024u) {
            if (stages > 2) --stages; else --warps;
        }
        p.stages = stages;
        p.chunk_bytes = cb;
        size_t smem = (size_t)warps * stages * per_stage;
        // a capped launch keeps one CTA per SM: pad shared memory so no second CTA fits
        if (sm_count && smem < 120u * 1024u) smem = 120u * 1024u;
        grid = sms;
        if (opcode == TUTTI_OP_READ)
            err = launch_dependent(copy_bulk_kernel<1>, dim3(sms), dim3(warps * 32), smem, stream, p, tm);
        else
            err = launch_dependent(copy_bulk_kernel<0>, dim3(sms), dim3(warps * 32), smem, stream, p, tm);
    } else {
        p.stages = 0;
        p.chunk_bytes = CHUNK_BYTES;
        uint32_t per_sm = opt.ctas_per_sm ? opt.ctas_per_sm : 4;
        if (per_sm > LDST_MAX_GROUPS) per_sm = LDST_MAX_GROUPS;
        // all SMs: per_sm one-group CTAs per SM.  Capped: exactly sm_count CTAs of per_sm
        // groups each, one per SM (the pad leaves no room for a second CTA).
        const uint32_t threads = sm_count ? per_sm * LDST_THREADS : LDST_THREADS;
        const size_t smem = sm_count ? LDST_PAD_SMEM : 0;
        grid = sm_count ? sm_count : sms * per_sm;
        if (opcode == TUTTI_OP_READ)
            err = launch_dependent(copy_ldst_kernel<1>, dim3(grid), dim3(threads), smem, stream, p);
        else
            err = launch_dependent(copy_ldst_kernel<0>, dim3(grid), dim3(threads), smem, stream, p);
    }
    if (launches) *launches = 1;
    if (grid_out) *grid_out = grid;
    return err;
}

}  // namespace tutti
