// tutti_kv_restore_layer_noalloc: one layer's build + restore for callers that are
// not allowed to allocate device memory — code running inside a serving engine's
// memory-pool-managed region, inside a CUDA-graph-style "no allocator calls" section,
// or in a process whose whole HBM budget was handed out at start-up.  Such callers
// cannot create a ring (tutti_ring_create allocates), so this entry point keeps the
// ring-side scratch — IOCB header, contexts, SGL entries, object-side addresses and
// the plan arrays — in one file-scope device array that every GPU loading the
// library holds until the process exits.
#include <mutex>
#include <string>

#include "tutti_internal.h"

using namespace tutti;

extern "C" void tutti_set_cuda_error_(const char *msg);

namespace {

constexpr uint32_t NA_MAX_ITEMS = 4096;       // objects x {K,V} per call
constexpr uint32_t NA_MAX_ENTRIES = 65536;    // pool blocks x {K,V} per call
constexpr uint32_t NA_POW2_ITEMS = 4096;

// layout of the scratch array (all offsets multiples of 256)
constexpr size_t OFF_HDR = 0;                                              // IocbHdr
constexpr size_t OFF_CQ = 256;                                             // CqSlot
constexpr size_t OFF_CQ_RESERVE = 512;                                     // uint32_t
constexpr size_t OFF_COUNTS = 768;                                         // PlanCounts
constexpr size_t CLEAR_BYTES = 1024;                                       // what a call zeroes
constexpr size_t OFF_SQES = 1024;
constexpr size_t OFF_PLAN_SQE = OFF_SQES + sizeof(tutti_sqe_t) * NA_MAX_ITEMS;
constexpr size_t OFF_PLAN_ITEM = OFF_PLAN_SQE + sizeof(tutti_sqe_t) * NA_MAX_ITEMS;
constexpr size_t OFF_PLAN_CUM = OFF_PLAN_ITEM + 4 * NA_MAX_ITEMS;
constexpr size_t OFF_PLAN_SQE_OF = OFF_PLAN_CUM + 4 * (NA_MAX_ITEMS + 64);
constexpr size_t OFF_PLAN_OFF = OFF_PLAN_SQE_OF + 4 * NA_MAX_ITEMS;
constexpr size_t OFF_PLAN_GRP = OFF_PLAN_OFF + 8 * NA_MAX_ITEMS;
constexpr size_t OFF_PLAN_K = OFF_PLAN_GRP + 4 * NA_MAX_ITEMS;
constexpr size_t OFF_PLAN_KEY = OFF_PLAN_K + 4 * NA_MAX_ITEMS;
constexpr size_t OFF_PLAN_IDX = OFF_PLAN_KEY + 8 * NA_POW2_ITEMS;
constexpr size_t OFF_SGL = OFF_PLAN_IDX + 4 * NA_POW2_ITEMS;
constexpr size_t OFF_OBJ = OFF_SGL + sizeof(tutti_sgl_t) * NA_MAX_ENTRIES;
constexpr size_t SCRATCH_BYTES = OFF_OBJ + 8 * (size_t)NA_MAX_ENTRIES;    // about 2 MiB
static_assert(OFF_SQES % 256 == 0 && OFF_SGL % 256 == 0 && OFF_OBJ % 256 == 0, "alignment");

// The scratch itself.  In host code this name is only a stand-in for the symbol: its
// device address comes from cudaGetSymbolAddress below, never from `&` or decay.
static __device__ __align__(256) unsigned char g_noalloc_scratch[SCRATCH_BYTES];

constexpr int MAX_GPUS = 64;
std::mutex g_mu;
unsigned char *g_scratch_addr[MAX_GPUS] = {nullptr};
int g_sms[MAX_GPUS] = {0};

int fail(cudaError_t e, const char *what) {
    std::string m = std::string(what) + ": " + cudaGetErrorName(e) + " (" + cudaGetErrorString(e) + ")";
    tutti_set_cuda_error_(m.c_str());
    return TUTTI_ECUDA;
}

// Header, counters and completion slot start from zero; the slot's status starts as
// "timed out", so a launch that never posts its completion is not read as a success.
__global__ void noalloc_reset_kernel(unsigned char *base) {
    uint32_t *w = reinterpret_cast<uint32_t *>(base);
    for (uint32_t i = threadIdx.x; i < CLEAR_BYTES / 4; i += blockDim.x) w[i] = 0;
    __syncthreads();
    if (threadIdx.x == 0) reinterpret_cast<CqSlot *>(base + OFF_CQ)->cqe.status = TUTTI_ETIMEDOUT;
}

// Once per device, with that device current: resolve the scratch address.
int setup_device(int device, unsigned char **out, int *sms) {
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_addr[device]) {
        unsigned char *ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress((void **)&ptr, g_noalloc_scratch);
        if (e != cudaSuccess || !ptr) return fail(e != cudaSuccess ? e : cudaErrorInvalidSymbol, "cudaGetSymbolAddress");
        int n = 0;
        e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, device);
        if (e != cudaSuccess) return fail(e, "cudaDeviceGetAttribute");
        e = copy_kernels_setup();
        if (e != cudaSuccess) return fail(e, "kernel attributes");
        g_sms[device] = n;
        g_scratch_addr[device] = ptr;
    }
    *out = g_scratch_addr[device];
    *sms = g_sms[device];
    return TUTTI_OK;
}

}  // namespace

extern "C" int tutti_kv_restore_layer_noalloc(const tutti_geom_t *geom, int device, uint32_t layer,
                                              const tutti_batch_t *batch, void *k_base,
                                              void *v_base, uint64_t block_stride,
                                              uint64_t n_blocks, void *const *store_base,
                                              const uint64_t *store_bytes, tutti_cqe_t *cqe_out,
                                              void *stream) {
    if (!geom || !batch || !k_base || !v_base || !store_base || !store_bytes || !cqe_out)
        return TUTTI_EINVAL;
    tutti_layout_t lo;
    int rc = tutti_obj_layout(geom, &lo);
    if (rc) return rc;
    if (device < 0 || device >= MAX_GPUS || layer >= geom->n_layers) return TUTTI_EINVAL;
    if ((((uint64_t)k_base | (uint64_t)v_base | block_stride) & 15) || block_stride < lo.block_bytes ||
        n_blocks == 0 || n_blocks > 0x7fffffffull)
        return TUTTI_EINVAL;
    // the fixed scratch bounds the batch: reject anything larger, clearly
    if (2ull * batch->n_obj > NA_MAX_ITEMS || 2ull * batch->n_blk > NA_MAX_ENTRIES)
        return TUTTI_EINVAL;
    if (batch->n_req && (!batch->hit_tokens || !batch->obj_start || !batch->blk_start))
        return TUTTI_EINVAL;
    if ((batch->n_obj && !batch->obj_slot) || (batch->n_blk && !batch->block_ids)) return TUTTI_EINVAL;
    uint64_t sbase[TUTTI_MAX_DEVICES] = {0}, sbytes[TUTTI_MAX_DEVICES] = {0};
    for (uint32_t d = 0; d < geom->n_devices; ++d) {
        if (!store_base[d] || ((uint64_t)store_base[d] & 15) || store_bytes[d] < lo.dev_bytes)
            return TUTTI_EINVAL;
        sbase[d] = (uint64_t)store_base[d];
        sbytes[d] = store_bytes[d];
    }
    int prev = -1;
    cudaError_t e0 = cudaGetDevice(&prev);
    if (e0 != cudaSuccess) return fail(e0, "cudaGetDevice");
    if (prev != device && (e0 = cudaSetDevice(device)) != cudaSuccess) return fail(e0, "cudaSetDevice");
    unsigned char *base = nullptr;
    int sms = 0;
    rc = setup_device(device, &base, &sms);
    cudaStream_t st = (cudaStream_t)stream;
    if (rc == TUTTI_OK) {
        RingDev r;
        r.hdrs = reinterpret_cast<IocbHdr *>(base + OFF_HDR);
        r.sqes = reinterpret_cast<tutti_sqe_t *>(base + OFF_SQES);
        r.sgl = reinterpret_cast<tutti_sgl_t *>(base + OFF_SGL);
        r.obj_ptr = reinterpret_cast<uint64_t *>(base + OFF_OBJ);
        r.cq = reinterpret_cast<CqSlot *>(base + OFF_CQ);
        r.cq_reserve = reinterpret_cast<uint32_t *>(base + OFF_CQ_RESERVE);
        r.depth = 1;
        r.capacity = NA_MAX_ITEMS;
        r.plan_item = reinterpret_cast<uint32_t *>(base + OFF_PLAN_ITEM);
        r.plan_cumblk = reinterpret_cast<uint32_t *>(base + OFF_PLAN_CUM);
        r.plan_sqe_of = reinterpret_cast<uint32_t *>(base + OFF_PLAN_SQE_OF);
        r.plan_sqe = reinterpret_cast<tutti_sqe_t *>(base + OFF_PLAN_SQE);
        r.plan_off = reinterpret_cast<uint64_t *>(base + OFF_PLAN_OFF);
        r.plan_grp = reinterpret_cast<uint32_t *>(base + OFF_PLAN_GRP);
        r.plan_k = reinterpret_cast<uint32_t *>(base + OFF_PLAN_K);
        r.plan_stage = nullptr;                   // staged transfers are not offered here
        r.plan_key = reinterpret_cast<unsigned long long *>(base + OFF_PLAN_KEY);
        r.plan_idx = reinterpret_cast<uint32_t *>(base + OFF_PLAN_IDX);
        r.plan_counts = reinterpret_cast<PlanCounts *>(base + OFF_COUNTS);
        r.max_items = NA_MAX_ITEMS;
        GeomDev g;
        g.block_tokens = geom->block_tokens;
        g.obj_tokens = geom->obj_tokens;
        g.blocks_per_obj = (uint32_t)lo.blocks_per_obj;
        g.n_devices = geom->n_devices;
        g.token_bytes = lo.token_bytes;
        g.block_bytes = lo.block_bytes;
        g.stride_kv = lo.stride_kv;
        g.stride_layer = lo.stride_layer;
        g.stride_slot = lo.stride_slot;
        g.n_slots = geom->n_slots;
        g.dev_bytes = lo.dev_bytes;
        BatchDev b{batch->n_req, batch->n_obj, batch->n_blk, batch->hit_tokens, batch->obj_start,
                   batch->obj_slot, batch->blk_start, batch->block_ids};
        PoolLayer pool{(uint64_t)k_base, (uint64_t)v_base, block_stride, n_blocks, true};
        CopyOptions opt{2, 2000000ull, 4, 0, 0, 0, 0, 0};
        uint32_t launches = 0;
        // header, completion slot and counters must start at zero: the array still holds
        // whatever the previous call left there
        noalloc_reset_kernel<<<1, 256, 0, st>>>(base);
        cudaError_t e = cudaGetLastError();
        if (e == cudaSuccess) e = launch_plan(r, g, b, st, nullptr);
        if (e == cudaSuccess)
            e = launch_emit(r, g, b, layer, 1, TUTTI_OP_READ, pool, nullptr, sbase, sbytes, 0, 1, 0,
                            NA_MAX_ENTRIES, 0, 0, 0, sms, st);
        if (e == cudaSuccess)
            e = launch_copy(r, 0, 1, TUTTI_OP_READ, 0, sms, opt, false, false,
                            PermGeom{geom->block_tokens, geom->n_kv_heads,
                                     geom->head_dim * geom->elem_bytes, (uint32_t)lo.token_bytes},
                            nullptr, nullptr, st, &launches, nullptr);
        if (e == cudaSuccess)
            e = cudaMemcpyAsync(cqe_out, base + OFF_CQ, sizeof(tutti_cqe_t), cudaMemcpyDefault, st);
        if (e != cudaSuccess) rc = fail(e, "tutti_kv_restore_layer_noalloc");
    }
    if (prev != device) cudaSetDevice(prev);
    return rc;
}
