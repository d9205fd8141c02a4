// Internal definitions shared by the host side of the library and its kernels.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/tutti.h"
#include "host_ring.h"

namespace tutti {

// IOCB header in HBM (paper Section 3.2: an SQ entry is an IOCB holding up to
// ioctx_per_iocb I/O contexts plus num_ioctx).  64 bytes, one per ring slot.
// `state` carries the IOCB index so that a stale value from the slot's previous
// use is never mistaken for the current one.
struct __align__(64) IocbHdr {
    uint32_t state;          // state_word(idx, phase)
    uint32_t num_ioctx;
    uint32_t opcode;
    uint32_t layer;
    int32_t status;          // first error found while building or copying (0 = none)
    uint32_t sgl_base;       // arena index of the build's first SGL entry
    uint32_t entry_first;    // first entry of this IOCB, relative to sgl_base
    uint32_t total_entries;
    uint32_t entry_len;      // common length of all entries, 0 = lengths differ
    uint32_t claim_cursor;   // next unclaimed chunk
    unsigned long long done_bytes;  // bytes that have landed
    unsigned long long bytes;       // bytes this IOCB moves
    uint32_t emit_done;      // build: CTAs finished (first IOCB of a build only)
    int32_t emit_status;     // build: first error seen by any CTA
};
static_assert(sizeof(IocbHdr) == 64, "IocbHdr must be 64 bytes");

enum : uint32_t { PHASE_FREE = 0, PHASE_READY = 1, PHASE_DONE = 2 };
__host__ __device__ inline uint32_t state_word(uint32_t iocb_idx, uint32_t phase) {
    return (iocb_idx << 2) | phase;
}

// Completion queue slot in pinned host memory: the entry, then a sequence word
// written last (value = position in the CQ + 1).
struct __align__(32) CqSlot {
    tutti_cqe_t cqe;
    uint32_t seq;
    uint32_t pad[3];
};
static_assert(sizeof(CqSlot) == 32, "CqSlot must be 32 bytes");

// Batch-level plan (independent of the layer): items in (device, offset) order.
struct PlanCounts {
    uint32_t n_items;    // active items (objects x {K,V} with at least one hit token)
    uint32_t n_sqe;
    uint32_t n_entries;
    int32_t status;
};

struct PoolLayer {
    uint64_t k_base, v_base, block_stride, n_blocks;
    bool registered;
};

// Device-resident copy of a registered pool layer (table indexed by layer).
struct PoolLayerDev {
    uint64_t k_base, v_base, block_stride, n_blocks;
};

struct StoreDev {
    uint64_t base, bytes;
    uint32_t kind;
    bool registered;
    bool tmap_ok;      // a tensor map of the region exists
};

// Device-side view of a ring, passed by value to kernels.
// plan_stage[] of a context that is not staged (its entries keep pointing into the store)
constexpr uint32_t STAGE_NONE = 0xffffffffu;

struct RingDev {
    IocbHdr *hdrs;            // [depth]
    tutti_sqe_t *sqes;        // [depth * capacity]
    tutti_sgl_t *sgl;         // [sgl_capacity]   pool side of every entry
    uint64_t *obj_ptr;        // [sgl_capacity]   object-store side of every entry
    CqSlot *cq;               // [depth]          device alias of pinned host memory
    uint32_t *cq_reserve;     // CQ position counter (HBM)
    uint32_t depth;           // power of two
    uint32_t capacity;        // contexts per IOCB
    // plan scratch
    uint32_t *plan_item;      // [max_items]  item id (2*object + kv) in sorted order
    uint32_t *plan_cumblk;    // [max_items+1] exclusive prefix of blocks per item
    uint32_t *plan_sqe_of;    // [max_items]  context index of each item
    uint64_t *plan_off;       // [max_items]  (device << 56) | byte offset of the item at layer 0
    uint32_t *plan_grp;       // [max_items]  index of the first item of the item's group (items
                              //              that name exactly the same bytes form a group)
    uint32_t *plan_k;         // [max_items]  at a group's first item: members of the group
    uint32_t *plan_stage;     // [max_items]  per context: its place in a staging buffer, in blocks, or
                              //              STAGE_NONE; written by the host (tutti_stage_plan)
    tutti_sqe_t *plan_sqe;    // [max_items]  contexts for layer 0, opcode unset
    unsigned long long *plan_key;  // [pow2(max_items)] sort keys when they do not fit in shared memory
    uint32_t *plan_idx;       // [pow2(max_items)] sort payload, same
    PlanCounts *plan_counts;  // [2]: [0] the plan's result, [1].status scratch of the key pass
    uint32_t max_items;
};

struct GeomDev {
    uint32_t block_tokens, obj_tokens, blocks_per_obj, n_devices;
    uint64_t token_bytes, block_bytes, stride_kv, stride_layer, stride_slot, n_slots;
    uint64_t dev_bytes;
};

struct BatchDev {
    uint32_t n_req, n_obj, n_blk;
    const uint32_t *hit_tokens, *obj_start, *obj_slot, *blk_start;
    const int32_t *block_ids;
};

// What a head-major pool block needs to be addressed: tokens per block, heads, bytes of
// one head's row of a token, bytes of a whole token.
struct PermGeom {
    uint32_t block_tokens, n_heads, row_bytes, token_bytes;
};

// Tensor maps of the storage devices for head-major pool blocks: every device region seen as
// a 3-D array [token row][head][row of head_dim elements], box = one head of one block.
struct alignas(64) StoreTensorMaps {
    CUtensorMap map[TUTTI_MAX_DEVICES];
    uint64_t base[TUTTI_MAX_DEVICES];
    uint64_t bytes[TUTTI_MAX_DEVICES];
    uint32_t n_devices;
    uint32_t valid;         // 1 when the maps may be used
};

struct CopyOptions {
    uint32_t engine;        // 0 auto, 1 ld/st, 2 bulk
    uint64_t wait_ns;
    uint32_t ctas_per_sm;
    uint32_t bulk_warps, bulk_stages;
    uint32_t claim_chunks;
    uint32_t bulk_chunk;    // bytes per stage of the bulk engine (0 = 32 KiB)
    uint32_t inject_timeout; // test hook: the bulk engine's stage waits report "ran out"
};

// Programmatic dependent launch: a kernel launched with this attribute may become resident
// while the kernel before it in the stream is still running.  Used for the emit kernel
// (behind the plan kernel) and the copy kernels (behind the emit kernel): the dependent's
// launch latency and start-up overlap the tail of its predecessor.  Correctness never rests
// on it: the emit kernel executes griddepcontrol.wait before it touches anything (so everything
// earlier in the stream has completed by then, for it and for whatever is launched behind
// it), and the copy agents wait, bounded, on each IOCB's READY word with acquire semantics.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                    cudaStream_t stream, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}

// kernels (tutti_build.cu / tutti_copy.cu)
cudaError_t launch_plan(const RingDev &ring, const GeomDev &geom, const BatchDev &batch,
                        cudaStream_t stream, uint32_t *launches);
cudaError_t launch_emit(const RingDev &ring, const GeomDev &geom, const BatchDev &batch,
                        uint32_t layer, uint32_t n_layers, uint32_t opcode, const PoolLayer &pool,
                        const PoolLayerDev *pools, const uint64_t *store_base,
                        const uint64_t *store_bytes, uint32_t first_iocb, uint32_t n_iocb,
                        uint32_t sgl_base, uint32_t sgl_reserved, uint32_t entries_per_iocb,
                        uint64_t stage_base, uint64_t stage_bytes, int device_sms,
                        cudaStream_t stream);
cudaError_t launch_copy(const RingDev &ring, uint32_t first_iocb, uint32_t n_iocb, uint32_t opcode,
                        uint32_t sm_count, int device_sms, const CopyOptions &opt, bool host_store,
                        bool pool_hnd, const PermGeom &perm, const StoreTensorMaps *maps,
                        uint32_t *smid_log, cudaStream_t stream, uint32_t *launches,
                        uint32_t *grid_out);
// Per-device kernel attributes (dynamic shared memory opt-ins) of every kernel of the
// library; called with the device current whenever a context is created on it.
cudaError_t copy_kernels_setup();
cudaError_t build_kernels_setup();

}  // namespace tutti
