// Host side of the C ABI declared in include/tutti.h: contexts, registration
// tables, the ring and its completion queue.  All device work is in
// tutti_build.cu / tutti_copy.cu; nothing here falls back to the CPU.
#include <chrono>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <thread>
#include <vector>

#include "tutti_internal.h"

using namespace tutti;

// the wire formats the header promises
static_assert(sizeof(tutti_sqe_t) == 32, "I/O context is 32 bytes");
static_assert(sizeof(tutti_sgl_t) == 16, "SGL entry is 16 bytes (address 8, length 4, id 4)");
static_assert(sizeof(tutti_cqe_t) == 16, "completion entry is 16 bytes");
static_assert(sizeof(tutti_geom_t) == 40 && sizeof(tutti_layout_t) == 80 && sizeof(tutti_batch_t) == 56,
              "geometry / layout / batch structs have no hidden padding");

namespace {

thread_local std::string g_last_cuda_error;

int cuda_fail(cudaError_t e, const char *what) {
    g_last_cuda_error = std::string(what) + ": " + cudaGetErrorName(e) + " (" +
                        cudaGetErrorString(e) + ")";
    return TUTTI_ECUDA;
}

#define CK(call)                                           \
    do {                                                   \
        cudaError_t e__ = (call);                          \
        if (e__ != cudaSuccess) return cuda_fail(e__, #call); \
    } while (0)

bool is_pow2(uint32_t v) { return v && !(v & (v - 1)); }

uint32_t pow2_at_least(uint32_t v) {
    uint32_t p = 32;
    while (p < v) p <<= 1;
    return p;
}

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
        target = dev;
    }
    ~DeviceGuard() {
        if (ok && prev >= 0 && prev != target) cudaSetDevice(prev);
    }
    int target = -1;
};

}  // namespace

struct tutti_ctx {
    tutti_geom_t geom;
    tutti_layout_t layout;
    int device;
    int device_sms;
    std::vector<PoolLayer> pool;
    StoreDev store[TUTTI_MAX_DEVICES];
    CopyOptions opt;
    GeomDev gdev;
    void *partition = nullptr;   // SM partition state (tutti_partition.cu)
    bool pool_hnd = false;       // pool blocks are [head][token][dim]
    StoreTensorMaps maps;        // for the transposing bulk copies
    PoolLayerDev *d_pools = nullptr;   // device copy of the pool table (multi-layer builds)
};

struct tutti_ring {
    tutti_ctx *ctx;
    RingDev dev;
    HostRing *host;
    CqSlot *cq_host;            // host view of the CQ
    uint32_t cq_head = 0;       // next CQ position to consume
    std::vector<tutti_cqe_t> completed;   // per slot
    std::vector<uint8_t> have_cqe;        // per slot
    std::vector<uint8_t> opcode_of;       // per slot, opcode of the reservation (0xff = unknown)
    std::vector<uint8_t> issued;          // per slot: a copy launch that executes it was enqueued
    std::vector<uint64_t> fill_optr;      // tutti_ring_fill_host scratch (sized at create)
    std::vector<uint8_t> fill_seen;
    uint32_t entries_per_iocb = 0;        // IOCBs cut by entries (0: by context count)
    std::vector<uint8_t> staged;          // per slot: 0 the object side of the IOCB is the store,
                                          // 1 a staging buffer, 2 either, context by context
    // staged transfers: the batch's contexts (layer 0) on the host, and where each sits in a
    // staging buffer packed in context order
    std::vector<tutti_sqe_t> stage_ctx;
    std::vector<uint64_t> stage_off;
    uint64_t stage_layer_bytes = 0;
    bool stage_valid = false;
    bool stage_all = true;                // every context of the stage plan goes through staging
    tutti_batch_t stage_batch{};
    uint32_t *smid_log = nullptr;         // device: SM of every CTA of the last copy launch
    uint32_t smid_cap = 0, last_grid = 0;
    uint32_t sgl_capacity;
    // plan cache key
    bool plan_valid = false;
    tutti_batch_t plan_batch{};
    uint64_t kernel_launches = 0, host_calls = 0;
    std::vector<void *> allocs;
};

extern "C" {

// accessors for tutti_partition.cu
void **tutti_ctx_partition_slot_(tutti_ctx_t *ctx) { return &ctx->partition; }
int tutti_ctx_device_(tutti_ctx_t *ctx) { return ctx->device; }
void tutti_set_cuda_error_(const char *msg) { g_last_cuda_error = msg; }

uint32_t tutti_version(void) { return 0x000100; }

const char *tutti_last_cuda_error(void) { return g_last_cuda_error.c_str(); }

const char *tutti_strerror(int code) {
    switch (code) {
        case TUTTI_OK: return "ok";
        case TUTTI_EINVAL: return "invalid argument";
        case TUTTI_ENOMEM: return "out of memory";
        case TUTTI_EAGAIN: return "try again (ring full or not complete)";
        case TUTTI_ETIMEDOUT: return "device-side wait timed out";
        case TUTTI_EFAULT: return "block id or slot out of range";
        case TUTTI_ECUDA: return "CUDA error";
        case TUTTI_ENOENT: return "no such key";
        default: return "unknown";
    }
}

int tutti_obj_layout(const tutti_geom_t *g, tutti_layout_t *o) {
    if (!g || !o) return TUTTI_EINVAL;
    if (!g->n_layers || !g->n_kv_heads || !g->head_dim || !g->elem_bytes || !g->block_tokens ||
        !g->obj_tokens || !g->n_devices || !g->n_slots)
        return TUTTI_EINVAL;
    if (g->n_devices > TUTTI_MAX_DEVICES || g->n_layers > 65535) return TUTTI_EINVAL;
    if (g->layout != TUTTI_LAYOUT_FILE_MAJOR && g->layout != TUTTI_LAYOUT_LAYER_MAJOR)
        return TUTTI_EINVAL;
    if (g->obj_tokens % g->block_tokens) return TUTTI_EINVAL;
    uint64_t tb = (uint64_t)g->n_kv_heads * g->head_dim * g->elem_bytes;
    if (tb % 16) return TUTTI_EINVAL;
    uint64_t bb = tb * g->block_tokens;
    if (bb > 0xffffffffull) return TUTTI_EINVAL;      // an SGL entry's length is 32 bits
    o->token_bytes = tb;
    o->block_bytes = bb;
    o->obj_kv_bytes = tb * g->obj_tokens;
    o->obj_bytes = 2 * o->obj_kv_bytes;
    o->blocks_per_obj = g->obj_tokens / g->block_tokens;
    o->n_slots_local = (g->n_slots + g->n_devices - 1) / g->n_devices;
    o->stride_kv = o->obj_kv_bytes;
    if (g->layout == TUTTI_LAYOUT_FILE_MAJOR) {
        o->stride_layer = o->obj_bytes;
        o->stride_slot = o->obj_bytes * g->n_layers;
    } else {
        o->stride_slot = o->obj_bytes;
        o->stride_layer = o->obj_bytes * o->n_slots_local;
    }
    o->dev_bytes = o->obj_bytes * g->n_layers * o->n_slots_local;
    if (o->dev_bytes >= (1ull << 56)) return TUTTI_EINVAL;
    return TUTTI_OK;
}

int tutti_ctx_create(const tutti_geom_t *geom, int device, tutti_ctx_t **out) {
    if (!geom || !out) return TUTTI_EINVAL;
    tutti_layout_t lo;
    int rc = tutti_obj_layout(geom, &lo);
    if (rc) return rc;
    int n_dev = 0;
    CK(cudaGetDeviceCount(&n_dev));
    if (device < 0 || device >= n_dev) return TUTTI_EINVAL;
    DeviceGuard guard(device);
    if (!guard.ok) return cuda_fail(cudaErrorInvalidDevice, "cudaSetDevice");
    cudaDeviceProp prop;
    CK(cudaGetDeviceProperties(&prop, device));
    if (prop.major < 10) {
        g_last_cuda_error = "this library is built for sm_100a only";
        return TUTTI_ECUDA;
    }
    CK(copy_kernels_setup());
    tutti_ctx *c = new (std::nothrow) tutti_ctx();
    if (!c) return TUTTI_ENOMEM;
    c->geom = *geom;
    c->layout = lo;
    c->device = device;
    c->device_sms = prop.multiProcessorCount;
    c->pool.assign(geom->n_layers, PoolLayer{0, 0, 0, 0, false});
    for (auto &s : c->store) s = StoreDev{0, 0, 0, false, false};
    memset(&c->maps, 0, sizeof(c->maps));
    c->opt = CopyOptions{0, 2000000ull, 4, 0, 0, 0, 0, 0};   // 0 = chosen per launch
    c->gdev.block_tokens = geom->block_tokens;
    c->gdev.obj_tokens = geom->obj_tokens;
    c->gdev.blocks_per_obj = (uint32_t)lo.blocks_per_obj;
    c->gdev.n_devices = geom->n_devices;
    c->gdev.token_bytes = lo.token_bytes;
    c->gdev.block_bytes = lo.block_bytes;
    c->gdev.stride_kv = lo.stride_kv;
    c->gdev.stride_layer = lo.stride_layer;
    c->gdev.stride_slot = lo.stride_slot;
    c->gdev.n_slots = geom->n_slots;
    c->gdev.dev_bytes = lo.dev_bytes;
    cudaError_t e = cudaMalloc((void **)&c->d_pools, sizeof(PoolLayerDev) * geom->n_layers);
    if (e == cudaSuccess) e = cudaMemset(c->d_pools, 0, sizeof(PoolLayerDev) * geom->n_layers);
    if (e != cudaSuccess) {
        delete c;
        cuda_fail(e, "cudaMalloc(pool table)");
        return TUTTI_ENOMEM;
    }
    *out = c;
    return TUTTI_OK;
}

int tutti_ctx_destroy(tutti_ctx_t *ctx) {
    if (!ctx) return TUTTI_EINVAL;
    tutti_sm_partition_destroy(ctx);
    {
        DeviceGuard guard(ctx->device);
        if (ctx->d_pools) cudaFree(ctx->d_pools);
    }
    delete ctx;
    return TUTTI_OK;
}

int tutti_pool_register(tutti_ctx_t *ctx, uint32_t layer, void *k_base, void *v_base,
                        uint64_t block_stride, uint64_t n_blocks) {
    if (!ctx || layer >= ctx->geom.n_layers || !k_base || !v_base || !n_blocks) return TUTTI_EINVAL;
    uint64_t k = (uint64_t)k_base, v = (uint64_t)v_base;
    if ((k | v | block_stride) & 15) return TUTTI_EINVAL;
    if (block_stride < ctx->layout.block_bytes || n_blocks > 0x7fffffffull) return TUTTI_EINVAL;
    ctx->pool[layer] = PoolLayer{k, v, block_stride, n_blocks, true};
    PoolLayerDev pl{k, v, block_stride, n_blocks};
    DeviceGuard guard(ctx->device);
    CK(cudaMemcpy(ctx->d_pools + layer, &pl, sizeof(pl), cudaMemcpyHostToDevice));
    return TUTTI_OK;
}

int tutti_store_register(tutti_ctx_t *ctx, uint32_t dev, void *base, uint64_t bytes, uint32_t kind) {
    if (!ctx || dev >= ctx->geom.n_devices || !base) return TUTTI_EINVAL;
    if (((uint64_t)base & 15) || bytes < ctx->layout.dev_bytes) return TUTTI_EINVAL;
    if (kind != TUTTI_STORE_HBM && kind != TUTTI_STORE_HOST_PINNED) return TUTTI_EINVAL;
    ctx->store[dev] = StoreDev{(uint64_t)base, bytes, kind, true};
    // Tensor map of the region as [token row][head][row bytes / 4] 32-bit words, box = one
    // head of one block.  Only used for head-major pool blocks; if the driver refuses it
    // (or the shape is out of a tensor map's range) those fall back to vector copies.
    ctx->maps.base[dev] = (uint64_t)base;
    ctx->maps.bytes[dev] = bytes;
    ctx->maps.n_devices = ctx->geom.n_devices;
    const uint64_t row_bytes = (uint64_t)ctx->geom.head_dim * ctx->geom.elem_bytes;
    const uint64_t n_rows = ctx->layout.dev_bytes / ctx->layout.token_bytes;
    bool ok = kind == TUTTI_STORE_HBM && (row_bytes % 16) == 0 && row_bytes / 4 <= 256 &&
              ctx->geom.block_tokens <= 256 && n_rows < (1ull << 32) &&
              ctx->layout.token_bytes % 16 == 0 &&
              (ctx->geom.block_tokens * row_bytes) % 128 == 0;   // a head's slab in the stage
    if (ok) {
        typedef CUresult (*encode_fn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                      const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                      const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                      CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
        void *fp = nullptr;
        cudaDriverEntryPointQueryResult q;
        ok = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fp, cudaEnableDefault, &q) == cudaSuccess &&
             fp && q == cudaDriverEntryPointSuccess;
        if (ok) {
            cuuint64_t dims[3] = {row_bytes / 4, ctx->geom.n_kv_heads, n_rows};
            cuuint64_t strides[2] = {row_bytes, ctx->layout.token_bytes};      // bytes, dims 1 and 2
            cuuint32_t box[3] = {(cuuint32_t)(row_bytes / 4), 1, ctx->geom.block_tokens};
            cuuint32_t estr[3] = {1, 1, 1};
            CUresult r = ((encode_fn)fp)(&ctx->maps.map[dev], CU_TENSOR_MAP_DATA_TYPE_UINT32, 3, base, dims,
                                         strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                         CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            ok = r == CUDA_SUCCESS;
        }
    }
    bool all = ok;
    ctx->store[dev].tmap_ok = ok;
    for (uint32_t d = 0; d < ctx->geom.n_devices; ++d) all = all && ctx->store[d].registered && ctx->store[d].tmap_ok;
    ctx->maps.valid = all ? 1u : 0u;
    return TUTTI_OK;
}

int tutti_set_option(tutti_ctx_t *ctx, uint32_t option, uint64_t value) {
    if (!ctx) return TUTTI_EINVAL;
    switch (option) {
        case TUTTI_OPT_COPY_ENGINE:
            if (value > 2) return TUTTI_EINVAL;
            ctx->opt.engine = (uint32_t)value;
            return TUTTI_OK;
        case TUTTI_OPT_WAIT_NS:
            if (value > 2000000000ull) return TUTTI_EINVAL;    // waits stay short by design
            ctx->opt.wait_ns = value;
            return TUTTI_OK;
        case TUTTI_OPT_CTAS_PER_SM:
            if (value < 1 || value > 8) return TUTTI_EINVAL;
            ctx->opt.ctas_per_sm = (uint32_t)value;
            return TUTTI_OK;
        case TUTTI_OPT_BULK_WARPS:
            if (value < 1 || value > 8) return TUTTI_EINVAL;
            ctx->opt.bulk_warps = (uint32_t)value;
            return TUTTI_OK;
        case TUTTI_OPT_BULK_STAGES:
            if (value < 2 || value > 8) return TUTTI_EINVAL;
            ctx->opt.bulk_stages = (uint32_t)value;
            return TUTTI_OK;
        case TUTTI_OPT_CLAIM_CHUNKS:
            if (value < 1 || value > 1024) return TUTTI_EINVAL;
            ctx->opt.claim_chunks = (uint32_t)value;
            return TUTTI_OK;
        case TUTTI_OPT_POOL_LAYOUT:
            if (value > TUTTI_POOL_HND) return TUTTI_EINVAL;
            // the transposing copies move 16-byte vectors that must stay inside one head's row
            if (value == TUTTI_POOL_HND && ((uint64_t)ctx->geom.head_dim * ctx->geom.elem_bytes) % 16)
                return TUTTI_EINVAL;
            ctx->pool_hnd = value == TUTTI_POOL_HND;
            return TUTTI_OK;
        case TUTTI_OPT_BULK_CHUNK_BYTES:
            if (value < 4096 || value > 32768 || (value & (value - 1))) return TUTTI_EINVAL;
            ctx->opt.bulk_chunk = (uint32_t)value;
            return TUTTI_OK;
        case TUTTI_OPT_INJECT_BULK_TIMEOUT:
            if (value > 1) return TUTTI_EINVAL;
            ctx->opt.inject_timeout = (uint32_t)value;
            return TUTTI_OK;
        default:
            return TUTTI_EINVAL;
    }
}

// ---------------------------------------------------------------------------
// ring
// ---------------------------------------------------------------------------

static int ring_alloc(tutti_ring *r, void **p, size_t bytes, bool zero) {
    cudaError_t e = cudaMalloc(p, bytes ? bytes : 16);
    if (e != cudaSuccess) { cuda_fail(e, "cudaMalloc"); return TUTTI_ENOMEM; }
    r->allocs.push_back(*p);
    if (zero) {
        e = cudaMemset(*p, 0, bytes ? bytes : 16);
        if (e != cudaSuccess) return cuda_fail(e, "cudaMemset");
    }
    return TUTTI_OK;
}

int tutti_ring_create(tutti_ctx_t *ctx, uint32_t depth, uint32_t ioctx_per_iocb,
                      uint32_t sgl_capacity, uint32_t max_items, tutti_ring_t **out) {
    if (!ctx || !out || !is_pow2(depth) || depth > (1u << 16) || !ioctx_per_iocb ||
        ioctx_per_iocb > (1u << 16) || !sgl_capacity || !max_items || max_items > (1u << 24))
        return TUTTI_EINVAL;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return cuda_fail(cudaErrorInvalidDevice, "cudaSetDevice");
    tutti_ring *r = new (std::nothrow) tutti_ring();
    if (!r) return TUTTI_ENOMEM;
    r->ctx = ctx;
    r->sgl_capacity = sgl_capacity;
    r->host = new (std::nothrow) HostRing(depth, sgl_capacity);
    r->completed.resize(depth);
    r->have_cqe.assign(depth, 0);
    r->opcode_of.assign(depth, 0xff);
    r->issued.assign(depth, 0);
    r->staged.assign(depth, 0);
    r->fill_optr.resize(sgl_capacity < (1u << 16) ? sgl_capacity : (1u << 16));
    r->fill_seen.resize(r->fill_optr.size());
    r->smid_cap = (uint32_t)ctx->device_sms * 8u;
    RingDev &d = r->dev;
    memset(&d, 0, sizeof(d));
    d.depth = depth;
    d.capacity = ioctx_per_iocb;
    d.max_items = max_items;
    const uint32_t np = pow2_at_least(max_items);
    int rc = TUTTI_OK;
    auto A = [&](void **p, size_t bytes, bool zero) { if (rc == TUTTI_OK) rc = ring_alloc(r, p, bytes, zero); };
    A((void **)&d.hdrs, sizeof(IocbHdr) * depth, true);
    A((void **)&d.sqes, sizeof(tutti_sqe_t) * (size_t)depth * ioctx_per_iocb, false);
    A((void **)&d.sgl, sizeof(tutti_sgl_t) * (size_t)sgl_capacity, false);
    A((void **)&d.obj_ptr, sizeof(uint64_t) * (size_t)sgl_capacity, false);
    A((void **)&d.cq_reserve, 16, true);
    A((void **)&d.plan_item, sizeof(uint32_t) * (size_t)max_items, false);
    A((void **)&d.plan_cumblk, sizeof(uint32_t) * ((size_t)max_items + 1), false);
    A((void **)&d.plan_sqe_of, sizeof(uint32_t) * (size_t)max_items, false);
    A((void **)&d.plan_off, sizeof(uint64_t) * (size_t)max_items, false);
    A((void **)&d.plan_grp, sizeof(uint32_t) * (size_t)max_items, false);
    A((void **)&d.plan_k, sizeof(uint32_t) * (size_t)max_items, false);
    A((void **)&d.plan_stage, sizeof(uint32_t) * (size_t)max_items, false);
    A((void **)&d.plan_sqe, sizeof(tutti_sqe_t) * (size_t)max_items, false);
    A((void **)&d.plan_key, sizeof(unsigned long long) * (size_t)np, false);
    A((void **)&d.plan_idx, sizeof(uint32_t) * (size_t)np, false);
    A((void **)&d.plan_counts, 2 * sizeof(PlanCounts), true);
    A((void **)&r->smid_log, sizeof(uint32_t) * r->smid_cap, true);
    if (rc == TUTTI_OK) {
        // headers start out "done" for an index that is never issued first
        cudaError_t e = cudaHostAlloc((void **)&r->cq_host, sizeof(CqSlot) * depth,
                                      cudaHostAllocMapped | cudaHostAllocPortable);
        if (e != cudaSuccess) { cuda_fail(e, "cudaHostAlloc"); rc = TUTTI_ENOMEM; }
    }
    if (rc == TUTTI_OK) {
        memset(r->cq_host, 0, sizeof(CqSlot) * depth);
        cudaError_t e = cudaHostGetDevicePointer((void **)&d.cq, r->cq_host, 0);
        if (e != cudaSuccess) rc = cuda_fail(e, "cudaHostGetDevicePointer");
    }
    if (rc != TUTTI_OK) {
        tutti_ring_destroy(r);
        return rc;
    }
    *out = r;
    return TUTTI_OK;
}

int tutti_ring_destroy(tutti_ring_t *r) {
    if (!r) return TUTTI_EINVAL;
    DeviceGuard guard(r->ctx->device);
    cudaDeviceSynchronize();
    for (void *p : r->allocs) cudaFree(p);
    if (r->cq_host) cudaFreeHost(r->cq_host);
    delete r->host;
    delete r;
    return TUTTI_OK;
}

int tutti_ring_set_iocb_bytes(tutti_ring_t *r, uint64_t bytes) {
    if (!r) return TUTTI_EINVAL;
    if (bytes == 0) { r->entries_per_iocb = 0; return TUTTI_OK; }
    const uint64_t per = bytes / r->ctx->layout.block_bytes;
    // every context of an IOCB holds at least one entry, so `per` contexts always fit
    if (per == 0 || per > r->dev.capacity) return TUTTI_EINVAL;
    r->entries_per_iocb = (uint32_t)per;
    return TUTTI_OK;
}

int tutti_ring_stats(tutti_ring_t *r, uint64_t *kernel_launches, uint64_t *host_calls) {
    if (!r) return TUTTI_EINVAL;
    if (kernel_launches) *kernel_launches = r->kernel_launches;
    if (host_calls) *host_calls = r->host_calls;
    return TUTTI_OK;
}

static bool same_plan(const tutti_batch_t &a, const tutti_batch_t &b) {
    return a.plan_epoch != 0 && a.plan_epoch == b.plan_epoch && a.n_req == b.n_req &&
           a.n_obj == b.n_obj && a.n_blk == b.n_blk && a.hit_tokens == b.hit_tokens &&
           a.obj_start == b.obj_start && a.obj_slot == b.obj_slot && a.blk_start == b.blk_start &&
           a.block_ids == b.block_ids;
}

static int build_layers(tutti_ctx_t *ctx, tutti_ring_t *r, const tutti_batch_t *batch, uint32_t layer,
                        uint32_t n_layers, uint32_t opcode, void *stream, uint32_t *first_iocb,
                        uint32_t *iocbs_per_layer, uint64_t stage_base = 0, uint64_t stage_bytes = 0) {
    if (!ctx || !r || r->ctx != ctx || !batch || !first_iocb || !iocbs_per_layer) return TUTTI_EINVAL;
    r->host_calls++;
    if (n_layers == 0 || layer >= ctx->geom.n_layers || n_layers > ctx->geom.n_layers - layer ||
        (opcode != TUTTI_OP_READ && opcode != TUTTI_OP_WRITE))
        return TUTTI_EINVAL;
    for (uint32_t l = layer; l < layer + n_layers; ++l)
        if (!ctx->pool[l].registered) return TUTTI_EINVAL;
    for (uint32_t d = 0; d < ctx->geom.n_devices; ++d)
        if (!ctx->store[d].registered) return TUTTI_EINVAL;
    if (batch->n_req && (!batch->hit_tokens || !batch->obj_start || !batch->blk_start))
        return TUTTI_EINVAL;
    if ((batch->n_obj && !batch->obj_slot) || (batch->n_blk && !batch->block_ids)) return TUTTI_EINVAL;
    if (batch->n_obj > r->dev.max_items / 2 || batch->n_blk > 0x7fffffffu / 2) return TUTTI_EINVAL;
    const uint32_t items = 2u * batch->n_obj;
    const uint32_t need_sgl = 2u * batch->n_blk;
    uint32_t need_iocb = r->entries_per_iocb
                             ? (need_sgl + r->entries_per_iocb - 1) / r->entries_per_iocb
                             : (items + r->dev.capacity - 1) / r->dev.capacity;
    if (need_iocb == 0) need_iocb = 1;
    if ((uint64_t)need_sgl * n_layers > r->sgl_capacity) return TUTTI_EINVAL;
    if ((uint64_t)need_iocb * n_layers > r->dev.depth) return TUTTI_EINVAL;
    uint32_t first = 0, sgl_base = 0;
    int rc = r->host->reserve(need_iocb * n_layers, need_sgl * n_layers, &first, &sgl_base);
    if (rc == -3) return TUTTI_EAGAIN;
    if (rc) return TUTTI_EINVAL;
    for (uint32_t k = 0; k < need_iocb * n_layers; ++k) {
        uint32_t slot = (first + k) & (r->dev.depth - 1);
        r->have_cqe[slot] = 0;
        r->opcode_of[slot] = (uint8_t)opcode;
        r->issued[slot] = 0;
        r->staged[slot] = stage_base == 0 ? 0 : (r->stage_all ? 1 : 2);
    }
    DeviceGuard guard(ctx->device);
    cudaStream_t st = (cudaStream_t)stream;
    BatchDev b{batch->n_req, batch->n_obj, batch->n_blk, batch->hit_tokens, batch->obj_start,
               batch->obj_slot, batch->blk_start, batch->block_ids};
    // a launch that fails must not leave its reservation behind
#define CK_OR_CANCEL(call)                                         \
    do {                                                           \
        cudaError_t e__ = (call);                                  \
        if (e__ != cudaSuccess) {                                  \
            r->host->cancel_last(first);                           \
            r->plan_valid = false;                                 \
            return cuda_fail(e__, #call);                          \
        }                                                          \
    } while (0)
    if (!(r->plan_valid && same_plan(r->plan_batch, *batch))) {
        uint32_t plan_launches = 0;
        CK_OR_CANCEL(launch_plan(r->dev, ctx->gdev, b, st, &plan_launches));
        r->kernel_launches += plan_launches;
        r->plan_batch = *batch;
        r->plan_valid = batch->plan_epoch != 0;
    }
    uint64_t sbase[TUTTI_MAX_DEVICES] = {0}, sbytes[TUTTI_MAX_DEVICES] = {0};
    for (uint32_t d = 0; d < ctx->geom.n_devices; ++d) {
        sbase[d] = ctx->store[d].base;
        sbytes[d] = ctx->store[d].bytes;
    }
    const uint32_t op_flags = opcode | (ctx->pool_hnd ? TUTTI_OP_FLAG_HND : 0u);
    CK_OR_CANCEL(launch_emit(r->dev, ctx->gdev, b, layer, n_layers, op_flags, ctx->pool[layer],
                             n_layers > 1 ? ctx->d_pools : nullptr, sbase, sbytes, first, need_iocb,
                             sgl_base, need_sgl, r->entries_per_iocb, stage_base, stage_bytes,
                             ctx->device_sms, st));
#undef CK_OR_CANCEL
    r->kernel_launches++;
    *first_iocb = first;
    *iocbs_per_layer = need_iocb;
    return TUTTI_OK;
}

int tutti_build_sqes(tutti_ctx_t *ctx, tutti_ring_t *r, const tutti_batch_t *batch, uint32_t layer,
                     uint32_t opcode, void *stream, uint32_t *first_iocb, uint32_t *n_iocb) {
    return build_layers(ctx, r, batch, layer, 1, opcode, stream, first_iocb, n_iocb);
}

int tutti_build_sqes_layers(tutti_ctx_t *ctx, tutti_ring_t *r, const tutti_batch_t *batch,
                            uint32_t first_layer, uint32_t n_layers, uint32_t opcode, void *stream,
                            uint32_t *first_iocb, uint32_t *iocbs_per_layer) {
    return build_layers(ctx, r, batch, first_layer, n_layers, opcode, stream, first_iocb,
                        iocbs_per_layer);
}

static int issue(tutti_ctx_t *ctx, tutti_ring_t *r, uint32_t first, uint32_t n, uint32_t sm_count,
                 void *stream, uint32_t opcode) {
    if (!ctx || !r || r->ctx != ctx || n == 0 || n > r->dev.depth) return TUTTI_EINVAL;
    r->host_calls++;
    if (sm_count > (uint32_t)ctx->device_sms) return TUTTI_EINVAL;
    bool host_store = false;
    for (uint32_t d = 0; d < ctx->geom.n_devices; ++d)
        host_store |= ctx->store[d].kind == TUTTI_STORE_HOST_PINNED;
    bool all_staged = true, any_staged = false;
    for (uint32_t k = 0; k < n; ++k) {
        uint32_t idx = first + k;
        if (!r->host->is_live(idx)) return TUTTI_EINVAL;
        uint8_t op = r->opcode_of[idx & (r->dev.depth - 1)];
        if (op != 0xff && op != opcode) return TUTTI_EINVAL;
        const uint8_t sg = r->staged[idx & (r->dev.depth - 1)];
        all_staged = all_staged && sg == 1;
        any_staged = any_staged || sg != 0;
    }
    if (all_staged) host_store = false;      // the object side of these IOCBs is a buffer in HBM
    // head-major blocks are transposed with tensor maps of the store regions, which a staging
    // buffer is not part of: a launch with staged IOCBs takes the vector path, which follows any
    // address; staged and unstaged IOCBs do not share a launch there
    if (ctx->pool_hnd && any_staged) {
        for (uint32_t k = 0; k < n; ++k)
            if (r->staged[(first + k) & (r->dev.depth - 1)] == 0) return TUTTI_EINVAL;
    }
    const StoreTensorMaps *maps = (ctx->pool_hnd && any_staged) ? nullptr : &ctx->maps;
    DeviceGuard guard(ctx->device);
    uint32_t launches = 0;
    PermGeom pg{ctx->geom.block_tokens, ctx->geom.n_kv_heads,
                ctx->geom.head_dim * ctx->geom.elem_bytes, (uint32_t)ctx->layout.token_bytes};
    uint32_t grid = 0;
    CK(launch_copy(r->dev, first, n, opcode, sm_count, ctx->device_sms, ctx->opt, host_store,
                   ctx->pool_hnd, pg, maps, r->smid_log, (cudaStream_t)stream, &launches, &grid));
    r->kernel_launches += launches;
    r->last_grid = grid < r->smid_cap ? grid : r->smid_cap;
    for (uint32_t k = 0; k < n; ++k) r->issued[(first + k) & (r->dev.depth - 1)] = 1;
    return TUTTI_OK;
}

int tutti_kv_restore_layer(tutti_ctx_t *ctx, tutti_ring_t *ring, uint32_t first_iocb,
                           uint32_t n_iocb, uint32_t sm_count, void *stream) {
    return issue(ctx, ring, first_iocb, n_iocb, sm_count, stream, TUTTI_OP_READ);
}

int tutti_kv_save_layer(tutti_ctx_t *ctx, tutti_ring_t *ring, uint32_t first_iocb, uint32_t n_iocb,
                        uint32_t sm_count, void *stream) {
    return issue(ctx, ring, first_iocb, n_iocb, sm_count, stream, TUTTI_OP_WRITE);
}

// Consume whatever the device has appended to the CQ since the last call.
static void drain_cq(tutti_ring *r) {
    const uint32_t depth = r->dev.depth;
    for (;;) {
        CqSlot *slot = &r->cq_host[r->cq_head & (depth - 1)];
        uint32_t seq = __atomic_load_n(&slot->seq, __ATOMIC_ACQUIRE);
        if (seq != r->cq_head + 1) break;
        tutti_cqe_t c;
        c.iocb_idx = *(volatile uint32_t *)&slot->cqe.iocb_idx;
        c.status = *(volatile int32_t *)&slot->cqe.status;
        c.bytes = *(volatile uint64_t *)&slot->cqe.bytes;
        if (r->host->is_live(c.iocb_idx)) {
            uint32_t s = c.iocb_idx & (depth - 1);
            r->completed[s] = c;
            r->have_cqe[s] = 1;
        }
        r->cq_head++;
    }
}

// `waited_ns`: how long the caller has been waiting already (a range poll waits for its IOCBs
// one after the other; the busy phase is counted over the whole call, not per IOCB)
static int poll_one(tutti_ring_t *r, uint32_t iocb_idx, tutti_cqe_t *out, uint64_t timeout_ns,
                    uint64_t waited_ns) {
    if (!r || !out) return TUTTI_EINVAL;
    r->host_calls++;
    if (!r->host->is_live(iocb_idx)) return TUTTI_EINVAL;
    const uint32_t slot = iocb_idx & (r->dev.depth - 1);
    auto t0 = std::chrono::steady_clock::now();
    for (;;) {
        if (!r->have_cqe[slot]) drain_cq(r);
        if (r->have_cqe[slot]) {
            *out = r->completed[slot];
            r->host->release(iocb_idx);       // a repeated poll of a live index is harmless
            return TUTTI_OK;
        }
        if (timeout_ns == 0) return TUTTI_EAGAIN;
        auto dt = std::chrono::duration_cast<std::chrono::nanoseconds>(
                      std::chrono::steady_clock::now() - t0).count();
        if ((uint64_t)dt >= timeout_ns) return TUTTI_EAGAIN;
        // a busy phase for completions that are less than a millisecond away (a sleep, however
        // short, returns some 50 us late: more than a short pass takes), then the core is given
        // back between looks at the queue, for about 1/128 of the time waited so far
        if ((uint64_t)dt + waited_ns < 1000000) {
#if defined(__x86_64__) || defined(__i386__)
            __builtin_ia32_pause();
#else
            std::this_thread::yield();
#endif
        } else {
            long long nap_us = (long long)(((uint64_t)dt + waited_ns) / 128000);
            if (nap_us < 5) nap_us = 5;
            if (nap_us > 100) nap_us = 100;
            std::this_thread::sleep_for(std::chrono::microseconds(nap_us));
        }
    }
}

int tutti_ring_poll(tutti_ring_t *r, uint32_t iocb_idx, tutti_cqe_t *out, uint64_t timeout_ns) {
    return poll_one(r, iocb_idx, out, timeout_ns, 0);
}

int tutti_ring_poll_range(tutti_ring_t *r, uint32_t first_iocb, uint32_t n_iocb, uint64_t *bytes_total,
                          int32_t *first_error, uint32_t *n_done, uint64_t timeout_ns) {
    if (!r || n_iocb == 0 || n_iocb > r->dev.depth) return TUTTI_EINVAL;
    uint64_t bytes = 0;
    int32_t err = 0;
    uint32_t done = 0;
    int rc = TUTTI_OK;
    auto t0 = std::chrono::steady_clock::now();
    for (; done < n_iocb; ++done) {
        uint64_t left = 0, waited = 0;
        if (timeout_ns) {
            auto dt = std::chrono::duration_cast<std::chrono::nanoseconds>(
                          std::chrono::steady_clock::now() - t0).count();
            waited = (uint64_t)dt;
            left = waited < timeout_ns ? timeout_ns - waited : 1;
        }
        tutti_cqe_t c;
        rc = poll_one(r, first_iocb + done, &c, left, waited);
        if (rc != TUTTI_OK) break;
        bytes += c.bytes;
        if (c.status != 0 && err == 0) err = c.status;
    }
    if (bytes_total) *bytes_total = bytes;
    if (first_error) *first_error = err;
    if (n_done) *n_done = done;
    return rc;
}

int tutti_stage_plan(tutti_ctx_t *ctx, tutti_ring_t *r, const tutti_batch_t *batch,
                     uint64_t min_ctx_bytes, void *stream, uint32_t *n_ctx, uint32_t *n_staged,
                     uint64_t *bytes_per_layer) {
    if (!ctx || !r || r->ctx != ctx || !batch || batch->plan_epoch == 0) return TUTTI_EINVAL;
    r->host_calls++;
    if (batch->n_req && (!batch->hit_tokens || !batch->obj_start || !batch->blk_start))
        return TUTTI_EINVAL;
    if ((batch->n_obj && !batch->obj_slot) || (batch->n_blk && !batch->block_ids)) return TUTTI_EINVAL;
    if (batch->n_obj > r->dev.max_items / 2) return TUTTI_EINVAL;
    DeviceGuard guard(ctx->device);
    cudaStream_t st = (cudaStream_t)stream;
    r->stage_valid = false;
    if (!(r->plan_valid && same_plan(r->plan_batch, *batch))) {
        BatchDev b{batch->n_req, batch->n_obj, batch->n_blk, batch->hit_tokens, batch->obj_start,
                   batch->obj_slot, batch->blk_start, batch->block_ids};
        uint32_t plan_launches = 0;
        CK(launch_plan(r->dev, ctx->gdev, b, st, &plan_launches));
        r->kernel_launches += plan_launches;
        r->plan_batch = *batch;
        r->plan_valid = true;
    }
    // once per batch: the plan's contexts come to the host (they do not depend on the layer)
    CK(cudaStreamSynchronize(st));
    PlanCounts pc;
    CK(cudaMemcpy(&pc, r->dev.plan_counts, sizeof(pc), cudaMemcpyDeviceToHost));
    if (pc.status != 0) return pc.status;
    r->stage_ctx.resize(pc.n_sqe);
    r->stage_off.resize(pc.n_sqe);
    if (pc.n_sqe)
        CK(cudaMemcpy(r->stage_ctx.data(), r->dev.plan_sqe, sizeof(tutti_sqe_t) * pc.n_sqe,
                      cudaMemcpyDeviceToHost));
    // a context of at least min_ctx_bytes goes through the staging buffer, packed behind the
    // staged contexts before it; a smaller one stays with the kernels (a copy engine pays a
    // fixed start-up per copy)
    uint64_t at = 0;
    uint32_t staged = 0;
    const uint64_t bb = ctx->layout.block_bytes;
    std::vector<uint32_t> place(pc.n_sqe);
    for (uint32_t k = 0; k < pc.n_sqe; ++k) {
        if (r->stage_ctx[k].len >= min_ctx_bytes) {
            if (at / bb >= STAGE_NONE) return TUTTI_EINVAL;
            r->stage_off[k] = at;
            place[k] = (uint32_t)(at / bb);
            at += r->stage_ctx[k].len;
            ++staged;
        } else {
            r->stage_off[k] = UINT64_MAX;
            place[k] = STAGE_NONE;
        }
    }
    if (pc.n_sqe)
        CK(cudaMemcpy(r->dev.plan_stage, place.data(), sizeof(uint32_t) * pc.n_sqe,
                      cudaMemcpyHostToDevice));
    r->stage_layer_bytes = at;
    r->stage_all = (staged == pc.n_sqe);
    r->stage_batch = *batch;
    r->stage_valid = true;
    if (n_ctx) *n_ctx = pc.n_sqe;
    if (n_staged) *n_staged = staged;
    if (bytes_per_layer) *bytes_per_layer = at;
    return TUTTI_OK;
}

int tutti_stage_copy_layer(tutti_ctx_t *ctx, tutti_ring_t *r, uint32_t layer, uint32_t opcode,
                           void *stage, uint64_t stage_bytes, void *stream) {
    if (!ctx || !r || r->ctx != ctx || !stage || layer >= ctx->geom.n_layers ||
        (opcode != TUTTI_OP_READ && opcode != TUTTI_OP_WRITE))
        return TUTTI_EINVAL;
    r->host_calls++;
    if (!r->stage_valid) return TUTTI_EINVAL;
    if (stage_bytes < r->stage_layer_bytes || ((uint64_t)stage & 15)) return TUTTI_EINVAL;
    DeviceGuard guard(ctx->device);
    cudaStream_t st = (cudaStream_t)stream;
    const uint64_t layer_off = (uint64_t)layer * ctx->layout.stride_layer;
    for (size_t k = 0; k < r->stage_ctx.size(); ++k) {
        const tutti_sqe_t &c = r->stage_ctx[k];
        if (r->stage_off[k] == UINT64_MAX) continue;          // not staged: the kernels move it
        if (c.dev >= ctx->geom.n_devices || !ctx->store[c.dev].registered) return TUTTI_EINVAL;
        if (c.src_off + layer_off + c.len > ctx->store[c.dev].bytes) return TUTTI_EFAULT;
        char *in_store = reinterpret_cast<char *>(ctx->store[c.dev].base + c.src_off + layer_off);
        char *in_stage = reinterpret_cast<char *>(stage) + r->stage_off[k];
        if (opcode == TUTTI_OP_READ)
            CK(cudaMemcpyAsync(in_stage, in_store, c.len, cudaMemcpyDefault, st));
        else
            CK(cudaMemcpyAsync(in_store, in_stage, c.len, cudaMemcpyDefault, st));
    }
    return TUTTI_OK;
}

int tutti_build_sqes_staged(tutti_ctx_t *ctx, tutti_ring_t *r, const tutti_batch_t *batch,
                            uint32_t layer, uint32_t opcode, void *stage, uint64_t stage_bytes,
                            void *stream, uint32_t *first_iocb, uint32_t *n_iocb) {
    if (!stage || ((uint64_t)stage & 15) || !r || !batch) return TUTTI_EINVAL;
    if (!r->stage_valid || !same_plan(r->stage_batch, *batch)) return TUTTI_EINVAL;
    if (stage_bytes < r->stage_layer_bytes) return TUTTI_EINVAL;
    return build_layers(ctx, r, batch, layer, 1, opcode, stream, first_iocb, n_iocb, (uint64_t)stage,
                        stage_bytes);
}

int tutti_sched_profile(tutti_ctx_t *ctx, tutti_ring_t *r, tutti_sched_t *sched,
                        const tutti_batch_t *batch, uint32_t layer, uint32_t opcode,
                        const uint32_t *sm_counts, uint32_t n_sm, uint32_t reps, void *stream,
                        uint32_t *n_points) {
    if (!ctx || !r || r->ctx != ctx || !sched || !batch || !sm_counts || n_sm == 0 || reps == 0 ||
        (opcode != TUTTI_OP_READ && opcode != TUTTI_OP_WRITE))
        return TUTTI_EINVAL;
    DeviceGuard guard(ctx->device);
    cudaStream_t st = (cudaStream_t)stream;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    CK(cudaEventCreate(&e0));
    cudaError_t ce = cudaEventCreate(&e1);
    if (ce != cudaSuccess) { cudaEventDestroy(e0); return cuda_fail(ce, "cudaEventCreate"); }
    uint32_t points = 0;
    int rc = TUTTI_OK;
    // one build to learn how many IOCBs of a layer carry work (the rest of a reservation is empty)
    uint32_t first = 0, n = 0, used = 0;
    rc = tutti_build_sqes(ctx, r, batch, layer, opcode, stream, &first, &n);
    if (rc == TUTTI_OK) {
        for (uint32_t k = 0; k < n && rc == TUTTI_OK; ++k) {
            tutti_iocb_info_t info;
            rc = tutti_ring_read_iocb(r, first + k, &info, nullptr, 0);
            if (rc == TUTTI_OK && info.status != 0) rc = info.status;
            if (rc == TUTTI_OK && info.total_entries) used = k + 1;
        }
        int rc2 = issue(ctx, r, first, n, 0, stream, opcode);
        if (rc == TUTTI_OK) rc = rc2;
        if (rc2 == TUTTI_OK) tutti_ring_poll_range(r, first, n, nullptr, nullptr, nullptr, 5000000000ull);
    }
    for (uint32_t si = 0; si < n_sm && rc == TUTTI_OK && used; ++si) {
        const uint32_t sms = sm_counts[si];
        for (uint32_t cnt = 1; rc == TUTTI_OK; cnt = (cnt * 2 < used || cnt == used) ? cnt * 2 : used) {
            if (cnt > used) break;
            float best = 0.f;
            for (uint32_t rep = 0; rep < reps && rc == TUTTI_OK; ++rep) {
                rc = tutti_build_sqes(ctx, r, batch, layer, opcode, stream, &first, &n);
                if (rc != TUTTI_OK) break;
                // the launch under test, alone on the stream, between two events
                ce = cudaStreamSynchronize(st);
                if (ce == cudaSuccess) ce = cudaEventRecord(e0, st);
                if (ce != cudaSuccess) { rc = cuda_fail(ce, "cudaEventRecord"); break; }
                rc = issue(ctx, r, first, cnt, sms, stream, opcode);
                if (rc != TUTTI_OK) break;
                ce = cudaEventRecord(e1, st);
                // the rest of the build runs too, so that every reserved IOCB completes
                if (cnt < n) rc = issue(ctx, r, first + cnt, n - cnt, sms, stream, opcode);
                if (ce == cudaSuccess) ce = cudaEventSynchronize(e1);
                float ms = 0.f;
                if (ce == cudaSuccess) ce = cudaEventElapsedTime(&ms, e0, e1);
                if (ce != cudaSuccess) { rc = cuda_fail(ce, "cudaEventElapsedTime"); break; }
                int32_t err = 0;
                int prc = tutti_ring_poll_range(r, first, n, nullptr, &err, nullptr, 5000000000ull);
                if (rc == TUTTI_OK && prc != TUTTI_OK) rc = prc;
                if (rc == TUTTI_OK && err != 0) rc = err;
                if (rep == 0 || ms < best) best = ms;
            }
            if (rc == TUTTI_OK) {
                rc = tutti_sched_set_io_time(sched, opcode, sms, cnt, best * 1e3f);
                ++points;
            }
            if (cnt == used) break;
        }
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (n_points) *n_points = points;
    return rc;
}

int tutti_stream_wait_iocb(tutti_ring_t *r, uint32_t iocb_idx, void *stream) {
    if (!r || !r->host->is_live(iocb_idx)) return TUTTI_EINVAL;
    r->host_calls++;
    // Only an IOCB whose copy launch is already enqueued may be waited for: that launch
    // terminates by itself (all its waits are bounded) and leaves the state word at DONE,
    // so the stream wait cannot outlive it.  Nothing is enqueued for any other index.
    if (!r->issued[iocb_idx & (r->dev.depth - 1)]) return TUTTI_EAGAIN;
    typedef CUresult (*wait_fn)(CUstream, CUdeviceptr, cuuint32_t, unsigned int);
    static wait_fn fn = nullptr;
    if (!fn) {
        void *fp = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuStreamWaitValue32", &fp, cudaEnableDefault, &q) != cudaSuccess ||
            !fp || q != cudaDriverEntryPointSuccess) {
            g_last_cuda_error = "cuStreamWaitValue32 is not available";
            return TUTTI_ECUDA;
        }
        fn = (wait_fn)fp;
    }
    DeviceGuard guard(r->ctx->device);
    const uint32_t slot = iocb_idx & (r->dev.depth - 1);
    CUdeviceptr addr = (CUdeviceptr)(uintptr_t)&r->dev.hdrs[slot].state;
    // ">=" in the cyclic sense the driver defines: also satisfied when the slot has moved on
    // to a later IOCB by the time the stream reaches the wait
    CUresult res = fn((CUstream)stream, addr, state_word(iocb_idx, PHASE_DONE), CU_STREAM_WAIT_VALUE_GEQ);
    if (res != CUDA_SUCCESS) {
        g_last_cuda_error = "cuStreamWaitValue32: CUresult " + std::to_string((int)res);
        return TUTTI_ECUDA;
    }
    return TUTTI_OK;
}

int tutti_ring_reserve(tutti_ring_t *r, uint32_t n_iocb, uint32_t n_sgl, uint32_t *first_iocb) {
    if (!r || !first_iocb) return TUTTI_EINVAL;
    r->host_calls++;
    uint32_t first = 0, base = 0;
    int rc = r->host->reserve(n_iocb, n_sgl, &first, &base);
    if (rc == -3) return TUTTI_EAGAIN;
    if (rc) return TUTTI_EINVAL;
    for (uint32_t k = 0; k < n_iocb; ++k) {
        uint32_t slot = (first + k) & (r->dev.depth - 1);
        r->have_cqe[slot] = 0;
        r->opcode_of[slot] = 0xff;
        r->issued[slot] = 0;
        r->staged[slot] = 0;
    }
    *first_iocb = first;
    return TUTTI_OK;
}

int tutti_ring_fill_host(tutti_ctx_t *ctx, tutti_ring_t *r, uint32_t iocb_idx,
                         const tutti_sqe_t *sqes, uint32_t n_sqe, const tutti_sgl_t *sgl,
                         uint32_t n_sgl, uint32_t sgl_offset, void *stream) {
    if (!ctx || !r || r->ctx != ctx) return TUTTI_EINVAL;
    if ((n_sqe && !sqes) || (n_sgl && !sgl) || n_sqe > r->dev.capacity) return TUTTI_EINVAL;
    const Group *g = r->host->group_of(iocb_idx);
    if (!g) return TUTTI_EINVAL;
    if ((uint64_t)sgl_offset + n_sgl > g->sgl_count) return TUTTI_EINVAL;
    // walk the contexts as a device would: object-side address of every entry
    if (n_sgl > r->fill_optr.size()) {        // grows once for an unusually long IOCB, then stays
        r->fill_optr.resize(n_sgl);
        r->fill_seen.resize(n_sgl);
    }
    uint64_t *optr = r->fill_optr.data();
    uint8_t *seen = r->fill_seen.data();
    memset(seen, 0, n_sgl);
    uint64_t total = 0;
    uint32_t common = n_sgl ? sgl[0].len : 0;
    uint32_t opcode = n_sqe ? sqes[0].opcode : TUTTI_OP_READ;
    for (uint32_t k = 0; k < n_sqe; ++k) {
        const tutti_sqe_t &s = sqes[k];
        if (s.dev >= ctx->geom.n_devices || !ctx->store[s.dev].registered) return TUTTI_EINVAL;
        if (s.opcode != opcode || (uint64_t)s.sgl_first + s.sgl_count > n_sgl) return TUTTI_EINVAL;
        if ((s.opcode & 0xff) > TUTTI_OP_WRITE || (s.opcode & ~(0xffu | TUTTI_OP_FLAG_HND)))
            return TUTTI_EINVAL;
        if ((s.opcode & TUTTI_OP_FLAG_HND) && ((uint64_t)ctx->geom.head_dim * ctx->geom.elem_bytes) % 16)
            return TUTTI_EINVAL;
        uint64_t cursor = s.src_off;
        for (uint32_t e = s.sgl_first; e < s.sgl_first + s.sgl_count; ++e) {
            if (seen[e] || (sgl[e].len & 15) || (sgl[e].addr & 15) || sgl[e].len == 0) return TUTTI_EINVAL;
            seen[e] = 1;
            if (sgl[e].id & TUTTI_SGL_FLAG_DUP) {
                // the object bytes of the entry before: same address, the walk stays put
                if (e == s.sgl_first || sgl[e].len != sgl[e - 1].len) return TUTTI_EINVAL;
                optr[e] = optr[e - 1];
            } else {
                if (cursor + sgl[e].len > ctx->store[s.dev].bytes) return TUTTI_EFAULT;
                optr[e] = ctx->store[s.dev].base + cursor;
                if (optr[e] & 15) return TUTTI_EINVAL;
                cursor += sgl[e].len;
            }
            total += sgl[e].len;
            if (sgl[e].len != common) common = 0;
        }
        if (cursor - s.src_off != s.len) return TUTTI_EINVAL;
    }
    for (uint32_t e = 0; e < n_sgl; ++e)
        if (!seen[e]) return TUTTI_EINVAL;
    DeviceGuard guard(ctx->device);
    cudaStream_t st = (cudaStream_t)stream;
    const uint32_t slot = iocb_idx & (r->dev.depth - 1);
    const size_t at = (size_t)g->sgl_begin + sgl_offset;
    if (n_sqe)
        CK(cudaMemcpyAsync(r->dev.sqes + (size_t)slot * r->dev.capacity, sqes,
                           sizeof(tutti_sqe_t) * n_sqe, cudaMemcpyHostToDevice, st));
    if (n_sgl) {
        CK(cudaMemcpyAsync(r->dev.sgl + at, sgl, sizeof(tutti_sgl_t) * n_sgl, cudaMemcpyHostToDevice, st));
        CK(cudaMemcpyAsync(r->dev.obj_ptr + at, optr, sizeof(uint64_t) * n_sgl,
                           cudaMemcpyHostToDevice, st));
    }
    IocbHdr h;
    memset(&h, 0, sizeof(h));
    h.state = state_word(iocb_idx, PHASE_READY);
    h.num_ioctx = n_sqe;
    h.opcode = opcode;
    h.layer = n_sqe ? sqes[0].layer : 0;
    h.sgl_base = g->sgl_begin;
    h.entry_first = sgl_offset;
    h.total_entries = n_sgl;
    h.entry_len = common;
    h.bytes = total;
    // stream order publishes the header after the descriptors it refers to
    CK(cudaMemcpyAsync(&r->dev.hdrs[slot], &h, sizeof(h), cudaMemcpyHostToDevice, st));
    r->opcode_of[slot] = (uint8_t)(opcode & 0xff);
    return TUTTI_OK;
}

int tutti_ring_read_iocb(tutti_ring_t *r, uint32_t iocb_idx, tutti_iocb_info_t *info,
                         tutti_sqe_t *sqes, uint32_t max_sqes) {
    if (!r || !info || !r->host->is_live(iocb_idx)) return TUTTI_EINVAL;
    DeviceGuard guard(r->ctx->device);
    CK(cudaDeviceSynchronize());
    const uint32_t slot = iocb_idx & (r->dev.depth - 1);
    IocbHdr h;
    CK(cudaMemcpy(&h, &r->dev.hdrs[slot], sizeof(h), cudaMemcpyDeviceToHost));
    info->iocb_idx = iocb_idx;
    info->ready = h.state == state_word(iocb_idx, PHASE_READY) ||
                  h.state == state_word(iocb_idx, PHASE_DONE);
    info->num_ioctx = h.num_ioctx;
    info->opcode = h.opcode;
    info->layer = h.layer;
    info->status = h.status;
    info->sgl_base = h.sgl_base;
    info->entry_first = h.entry_first;
    info->total_entries = h.total_entries;
    info->entry_len = h.entry_len;
    info->bytes = h.bytes;
    uint32_t n = h.num_ioctx < max_sqes ? h.num_ioctx : max_sqes;
    if (sqes && n && info->ready)
        CK(cudaMemcpy(sqes, r->dev.sqes + (size_t)slot * r->dev.capacity, sizeof(tutti_sqe_t) * n,
                      cudaMemcpyDeviceToHost));
    return TUTTI_OK;
}

int tutti_ring_read_sgl(tutti_ring_t *r, uint32_t iocb_idx, tutti_sgl_t *sgl, uint32_t max_entries,
                        uint32_t *n_entries) {
    if (!r || !n_entries || !r->host->is_live(iocb_idx)) return TUTTI_EINVAL;
    DeviceGuard guard(r->ctx->device);
    CK(cudaDeviceSynchronize());
    const uint32_t slot = iocb_idx & (r->dev.depth - 1);
    IocbHdr h;
    CK(cudaMemcpy(&h, &r->dev.hdrs[slot], sizeof(h), cudaMemcpyDeviceToHost));
    *n_entries = h.total_entries;
    uint32_t n = h.total_entries < max_entries ? h.total_entries : max_entries;
    if (sgl && n)
        CK(cudaMemcpy(sgl, r->dev.sgl + (size_t)h.sgl_base + h.entry_first, sizeof(tutti_sgl_t) * n,
                      cudaMemcpyDeviceToHost));
    return TUTTI_OK;
}

int tutti_ring_last_launch_sms(tutti_ring_t *r, uint32_t *smids, uint32_t max_ctas, uint32_t *n_ctas) {
    if (!r || !n_ctas || (max_ctas && !smids)) return TUTTI_EINVAL;
    DeviceGuard guard(r->ctx->device);
    CK(cudaDeviceSynchronize());
    *n_ctas = r->last_grid;
    uint32_t n = r->last_grid < max_ctas ? r->last_grid : max_ctas;
    if (n) CK(cudaMemcpy(smids, r->smid_log, sizeof(uint32_t) * n, cudaMemcpyDeviceToHost));
    return TUTTI_OK;
}

// ---------------------------------------------------------------------------
// host-side accounting on its own
// ---------------------------------------------------------------------------
struct tutti_hostring {
    HostRing ring;
    tutti_hostring(uint32_t d, uint32_t s) : ring(d, s) {}
};

tutti_hostring_t *tutti_hostring_create(uint32_t depth, uint32_t sgl_capacity) {
    if (!is_pow2(depth) || !sgl_capacity) return nullptr;
    return new (std::nothrow) tutti_hostring(depth, sgl_capacity);
}
void tutti_hostring_destroy(tutti_hostring_t *h) { delete h; }
int tutti_hostring_reserve(tutti_hostring_t *h, uint32_t n_iocb, uint32_t n_sgl, uint32_t *first_iocb,
                           uint32_t *sgl_base) {
    if (!h || !first_iocb || !sgl_base) return TUTTI_EINVAL;
    int rc = h->ring.reserve(n_iocb, n_sgl, first_iocb, sgl_base);
    return rc == -3 ? TUTTI_EAGAIN : (rc ? TUTTI_EINVAL : TUTTI_OK);
}
int tutti_hostring_release(tutti_hostring_t *h, uint32_t iocb_idx) {
    if (!h) return TUTTI_EINVAL;
    return h->ring.release(iocb_idx) ? TUTTI_EINVAL : TUTTI_OK;
}
int tutti_hostring_cancel_last(tutti_hostring_t *h, uint32_t first_iocb) {
    if (!h) return TUTTI_EINVAL;
    return h->ring.cancel_last(first_iocb) ? TUTTI_EINVAL : TUTTI_OK;
}
int tutti_hostring_live(const tutti_hostring_t *h, uint32_t *iocbs, uint32_t *sgl_entries) {
    if (!h) return TUTTI_EINVAL;
    if (iocbs) *iocbs = h->ring.live_iocbs();
    if (sgl_entries) *sgl_entries = h->ring.live_sgl();
    return TUTTI_OK;
}

}  // extern "C"
