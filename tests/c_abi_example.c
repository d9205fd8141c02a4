/*
 * The C ABI used from plain C, with no Python and no torch: one layer of a small batch is
 * restored from an HBM object store into a paged pool and saved back.  Build and run:
 *
 *   nvcc tests/c_abi_example.c -Iinclude -Lpaper_2605_03375_b200 -ltutti \
 *        -Xlinker -rpath -Xlinker $PWD/paper_2605_03375_b200 -o c_abi_example && ./c_abi_example
 *
 * Prints "OK ..." and exits 0 when every restored block holds the object bytes the block
 * table says it should, and the save reproduces the store.
 */
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "tutti.h"

#define CHECK(x)                                                                   \
    do {                                                                           \
        int rc__ = (x);                                                            \
        if (rc__ != 0) {                                                           \
            fprintf(stderr, "%s -> %d (%s) %s\n", #x, rc__, tutti_strerror(rc__), \
                    tutti_last_cuda_error());                                      \
            return 1;                                                              \
        }                                                                          \
    } while (0)
#define CU(x)                                                              \
    do {                                                                   \
        cudaError_t e__ = (x);                                             \
        if (e__ != cudaSuccess) {                                          \
            fprintf(stderr, "%s -> %s\n", #x, cudaGetErrorString(e__));    \
            return 1;                                                      \
        }                                                                  \
    } while (0)

int main(void)
{
    /* 2 layers, 8 KV heads x 128 x 2 bytes, 16-token blocks, 256-token objects */
    tutti_geom_t geom = {2, 8, 128, 2, 16, 256, 1, TUTTI_LAYOUT_LAYER_MAJOR, 8};
    tutti_layout_t lo;
    CHECK(tutti_obj_layout(&geom, &lo));
    const uint32_t n_pool = 256, n_tok = 1024 + 32, layer = 1;  /* last object is partial */
    const uint32_t n_blk = n_tok / 16, n_obj = (n_tok + 255) / 256;

    /* host-side inputs: store bytes, block table (a fixed permutation), object slots */
    uint8_t *h_store = (uint8_t *)malloc(lo.dev_bytes);
    for (uint64_t i = 0; i < lo.dev_bytes; ++i) h_store[i] = (uint8_t)((i * 2654435761u) >> 13);
    int32_t block_ids[128];
    for (uint32_t j = 0; j < n_blk; ++j) block_ids[j] = (int32_t)((j * 37u + 11u) % n_pool);
    uint32_t hit[1] = {n_tok}, obj_start[2] = {0, n_obj}, blk_start[2] = {0, n_blk};
    uint32_t obj_slot[8] = {5, 6, 7, 2, 0, 0, 0, 0};

    uint8_t *d_store, *d_pool;
    void *d_hit, *d_os, *d_slot, *d_bs, *d_ids;
    const size_t pool_bytes = 2ull * n_pool * lo.block_bytes;
    CU(cudaMalloc((void **)&d_store, lo.dev_bytes));
    CU(cudaMalloc((void **)&d_pool, pool_bytes));
    CU(cudaMemcpy(d_store, h_store, lo.dev_bytes, cudaMemcpyHostToDevice));
    CU(cudaMemset(d_pool, 0xA5, pool_bytes));
    CU(cudaMalloc(&d_hit, sizeof hit));
    CU(cudaMalloc(&d_os, sizeof obj_start));
    CU(cudaMalloc(&d_slot, sizeof obj_slot));
    CU(cudaMalloc(&d_bs, sizeof blk_start));
    CU(cudaMalloc(&d_ids, sizeof block_ids));
    CU(cudaMemcpy(d_hit, hit, sizeof hit, cudaMemcpyHostToDevice));
    CU(cudaMemcpy(d_os, obj_start, sizeof obj_start, cudaMemcpyHostToDevice));
    CU(cudaMemcpy(d_slot, obj_slot, sizeof obj_slot, cudaMemcpyHostToDevice));
    CU(cudaMemcpy(d_bs, blk_start, sizeof blk_start, cudaMemcpyHostToDevice));
    CU(cudaMemcpy(d_ids, block_ids, sizeof block_ids, cudaMemcpyHostToDevice));

    tutti_ctx_t *ctx;
    tutti_ring_t *ring;
    CHECK(tutti_ctx_create(&geom, 0, &ctx));
    CHECK(tutti_store_register(ctx, 0, d_store, lo.dev_bytes, TUTTI_STORE_HBM));
    for (uint32_t l = 0; l < geom.n_layers; ++l)   /* both layers share the pool memory here */
        CHECK(tutti_pool_register(ctx, l, d_pool, d_pool + n_pool * lo.block_bytes, lo.block_bytes, n_pool));
    CHECK(tutti_ring_create(ctx, 8, TUTTI_DEFAULT_IOCTX_PER_IOCB, 4096, 64, &ring));

    tutti_batch_t batch = {1, n_obj, n_blk, 0, (const uint32_t *)d_hit, (const uint32_t *)d_os,
                           (const uint32_t *)d_slot, (const uint32_t *)d_bs, (const int32_t *)d_ids};
    cudaStream_t stream;
    CU(cudaStreamCreate(&stream));
    uint32_t first, n;
    tutti_cqe_t cqe;
    CHECK(tutti_build_sqes(ctx, ring, &batch, layer, TUTTI_OP_READ, stream, &first, &n));
    CHECK(tutti_kv_restore_layer(ctx, ring, first, n, 0, stream));
    uint64_t moved = 0;
    for (uint32_t i = first; i < first + n; ++i) {
        CHECK(tutti_ring_poll(ring, i, &cqe, 5000000000ull));
        if (cqe.status != 0) { fprintf(stderr, "IOCB %u status %d\n", i, cqe.status); return 1; }
        moved += cqe.bytes;
    }
    if (moved != 2ull * n_tok * lo.token_bytes) { fprintf(stderr, "moved %llu\n", (unsigned long long)moved); return 1; }

    /* check: token t of the request sits in block block_ids[t/16], row t%16, and came from
     * object slot obj_slot[t/256], token t%256 of its K (then V) half */
    uint8_t *h_pool = (uint8_t *)malloc(pool_bytes);
    CU(cudaMemcpy(h_pool, d_pool, pool_bytes, cudaMemcpyDeviceToHost));
    uint64_t bad = 0, touched = 0;
    for (uint32_t kv = 0; kv < 2; ++kv)
        for (uint32_t t = 0; t < n_tok; ++t) {
            uint64_t src = obj_slot[t / 256] * lo.stride_slot + layer * lo.stride_layer +
                           kv * lo.stride_kv + (uint64_t)(t % 256) * lo.token_bytes;
            uint64_t dst = (uint64_t)kv * n_pool * lo.block_bytes +
                           (uint64_t)block_ids[t / 16] * lo.block_bytes + (t % 16) * lo.token_bytes;
            bad += memcmp(h_pool + dst, h_store + src, lo.token_bytes) != 0;
            touched += lo.token_bytes;
        }
    uint64_t canary = 0;
    for (size_t i = 0; i < pool_bytes; ++i) canary += h_pool[i] == 0xA5;
    if (bad || canary < pool_bytes - touched) { fprintf(stderr, "restore mismatch: %llu tokens\n", (unsigned long long)bad); return 1; }

    /* save back into a cleared store; the covered ranges must come back identical */
    CU(cudaMemset(d_store, 0, lo.dev_bytes));
    CHECK(tutti_build_sqes(ctx, ring, &batch, layer, TUTTI_OP_WRITE, stream, &first, &n));
    CHECK(tutti_kv_save_layer(ctx, ring, first, n, 0, stream));
    int32_t first_error = 0;
    uint32_t n_done = 0;
    CHECK(tutti_ring_poll_range(ring, first, n, &moved, &first_error, &n_done, 5000000000ull));
    if (first_error != 0 || n_done != n) { fprintf(stderr, "save status %d\n", first_error); return 1; }
    uint8_t *h_back = (uint8_t *)malloc(lo.dev_bytes);
    CU(cudaMemcpy(h_back, d_store, lo.dev_bytes, cudaMemcpyDeviceToHost));
    for (uint32_t kv = 0; kv < 2; ++kv)
        for (uint32_t t = 0; t < n_tok; ++t) {
            uint64_t src = obj_slot[t / 256] * lo.stride_slot + layer * lo.stride_layer +
                           kv * lo.stride_kv + (uint64_t)(t % 256) * lo.token_bytes;
            bad += memcmp(h_back + src, h_store + src, lo.token_bytes) != 0;
        }
    if (bad) { fprintf(stderr, "save mismatch: %llu tokens\n", (unsigned long long)bad); return 1; }

    /* the same restore as a staged transfer: the contexts are copied as they are into a staging
     * buffer (here device to device; the copy engines' job when the store is pinned host
     * memory), the kernel scatters from there into the pool */
    CU(cudaMemcpy(d_store, h_store, lo.dev_bytes, cudaMemcpyHostToDevice));
    CU(cudaMemset(d_pool, 0xA5, pool_bytes));
    batch.plan_epoch = 1;
    uint32_t n_ctx = 0, n_staged = 0;
    uint64_t stage_bytes = 0;
    CHECK(tutti_stage_plan(ctx, ring, &batch, 0, stream, &n_ctx, &n_staged, &stage_bytes));
    if (n_ctx == 0 || n_staged != n_ctx || stage_bytes != 2ull * n_tok * lo.token_bytes) {
        fprintf(stderr, "stage plan: %u contexts, %u staged, %llu bytes\n", n_ctx, n_staged,
                (unsigned long long)stage_bytes);
        return 1;
    }
    uint8_t *d_stage;
    CU(cudaMalloc((void **)&d_stage, stage_bytes));
    CHECK(tutti_stage_copy_layer(ctx, ring, layer, TUTTI_OP_READ, d_stage, stage_bytes, stream));
    CHECK(tutti_build_sqes_staged(ctx, ring, &batch, layer, TUTTI_OP_READ, d_stage, stage_bytes, stream,
                                  &first, &n));
    CHECK(tutti_kv_restore_layer(ctx, ring, first, n, 0, stream));
    CHECK(tutti_ring_poll_range(ring, first, n, &moved, &first_error, &n_done, 5000000000ull));
    if (first_error != 0 || n_done != n || moved != stage_bytes) { fprintf(stderr, "staged restore status %d\n", first_error); return 1; }
    uint8_t *h_pool2 = (uint8_t *)malloc(pool_bytes);
    CU(cudaMemcpy(h_pool2, d_pool, pool_bytes, cudaMemcpyDeviceToHost));
    if (memcmp(h_pool2, h_pool, pool_bytes) != 0) { fprintf(stderr, "staged restore differs from the direct one\n"); return 1; }

    uint64_t launches, calls;
    tutti_ring_stats(ring, &launches, &calls);
    printf("OK restored and saved %llu bytes; %llu kernel launches, %llu host calls\n",
           (unsigned long long)moved, (unsigned long long)launches, (unsigned long long)calls);
    tutti_ring_destroy(ring);
    tutti_ctx_destroy(ctx);
    return 0;
}
