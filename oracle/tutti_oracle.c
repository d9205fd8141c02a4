/*
 * CPU oracle for the per-layer KV restore / save path and its descriptor build.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, obviously-correct
 * statement of what the path computes.  It shares no code, header, table or
 * helper with the CUDA library and must never be called from the product path;
 * only the tests, the smoke check and the bench's CPU-baseline leg use it.
 *
 * What it states (paper sections in brackets):
 *   orc_obj_layout     object id -> (device, byte offset): a "GPU file" holds
 *                      2 x L objects, one key and one value object per layer;
 *                      files are spread round-robin over the storage devices
 *                      [Section 3.1, "Scalable GPU File Pool"].
 *   orc_restore_layer  layer-wise Retrieve: for every cached token of every
 *   orc_save_layer     request, the token's K and V bytes move between the
 *                      contiguous object and the paged block the block table
 *                      names; layer-wise Store is the same map reversed
 *                      [Section 2.1 paged KV blocks; Section 3.1 layer-wise
 *                      batched Store/Retrieve; Section 3.4 retrieve_layer /
 *                      store_layer].
 *   orc_build          the batch of I/O contexts for one layer: (file offset,
 *                      length, scatter-gather list) per contiguous run, 16-byte
 *                      SGL entries (address 8 B, length 4 B, identifier 4 B),
 *                      packed into IOCBs of a fixed number of contexts
 *                      [Section 3.1 "P2P Memory Mapping Table"; Section 3.2].
 *   orc_exec           what executing such descriptors means (the transfer a
 *                      device would perform for each context).
 *   orc_move_layer_blocks_mt
 *                      the same restore / save map taken one paged block at a time
 *                      (a block's K or V bytes are one run on both sides, so one
 *                      memcpy of block_bytes per block and half) with the blocks of
 *                      the batch dealt out over host threads.  It exists to time the
 *                      host's cores as a baseline; it is pinned byte for byte to
 *                      orc_restore_layer / orc_save_layer.
 *
 * The paper gives no sorting/coalescing rule (only the motivation that small
 * scattered requests waste bandwidth, Section 2.3/2.4); the rule used here is
 * the reading recorded in the design notes: order by (device, offset, length), stable
 * on (request, chunk, K-before-V); items that name exactly the same bytes (a stored
 * chunk shared by several requests of the batch, Section 3.1 "Scalable GPU File
 * Pool") form one source that is read once: its scatter-gather entries list, block
 * by block, every request's destination, the second and later ones flagged as
 * repeats; distinct sources that are exactly byte-adjacent on one device merge into
 * one context.
 *
 * Parity pins (tests/test_oracle_*.py): brute force on tiny pools against an
 * independent Python byte loop, array-shaped (numpy advanced indexing)
 * restatement, round-trip identity, untouched-byte checks, descriptor
 * prefix-sum / coverage invariants, exec(build) == restore, and the counts the
 * paper prints.  No function here is "parity unpinned".
 */
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_OK 0
#define ORC_EINVAL (-1)
#define ORC_ENOSPC (-2)

#define ORC_FILE_MAJOR 0
#define ORC_LAYER_MAJOR 1

#define ORC_OP_READ 0  /* object store -> paged pool (restore) */
#define ORC_OP_WRITE 1 /* paged pool -> object store (save)    */
#define ORC_OP_HND 0x100 /* flag: pool blocks are [head][token][dim] instead of [token][head][dim] */
/* Flag in the identifier of a scatter-gather entry: this entry takes (READ) the same object
 * bytes as the entry before it, i.e. one stored chunk goes to several requests' blocks. */
#define ORC_SGL_DUP 0x80000000u

typedef struct {
    uint32_t n_layers, n_kv_heads, head_dim, elem_bytes;
    uint32_t block_tokens, obj_tokens, n_devices, layout;
    uint64_t n_slots;
} orc_geom;

typedef struct {
    uint64_t token_bytes;   /* one token's K (or V) of one layer            */
    uint64_t block_bytes;   /* one paged block's K (or V) of one layer      */
    uint64_t obj_kv_bytes;  /* K half (= V half) of one object              */
    uint64_t obj_bytes;     /* K half followed by V half                    */
    uint64_t blocks_per_obj;
    uint64_t n_slots_local; /* object slots per device                      */
    uint64_t stride_kv, stride_layer, stride_slot;
    uint64_t dev_bytes;     /* bytes of store needed on each device         */
} orc_layout;

typedef struct {
    uint64_t src_off; /* object-side byte offset on device `dev`           */
    uint64_t len;
    uint32_t sgl_first, sgl_count;
    uint32_t dev;
    uint16_t opcode, layer;
} orc_sqe;

typedef struct {
    uint64_t addr; /* pool-side address */
    uint32_t len;
    uint32_t id;   /* pool block id     */
} orc_sgl;

/* Section 3.1: object = K half then V half of obj_tokens tokens of one layer. */
int orc_obj_layout(const orc_geom *g, orc_layout *o)
{
    if (!g || !o) return ORC_EINVAL;
    if (g->n_layers == 0 || g->n_kv_heads == 0 || g->head_dim == 0 || g->elem_bytes == 0 ||
        g->block_tokens == 0 || g->obj_tokens == 0 || g->n_devices == 0)
        return ORC_EINVAL;
    if (g->obj_tokens % g->block_tokens != 0) return ORC_EINVAL;
    if (g->layout != ORC_FILE_MAJOR && g->layout != ORC_LAYER_MAJOR) return ORC_EINVAL;
    o->token_bytes = (uint64_t)g->n_kv_heads * g->head_dim * g->elem_bytes;
    o->block_bytes = o->token_bytes * g->block_tokens;
    o->obj_kv_bytes = o->token_bytes * g->obj_tokens;
    o->obj_bytes = 2 * o->obj_kv_bytes;
    o->blocks_per_obj = g->obj_tokens / g->block_tokens;
    o->n_slots_local = (g->n_slots + g->n_devices - 1) / g->n_devices;
    o->stride_kv = o->obj_kv_bytes;
    if (g->layout == ORC_FILE_MAJOR) {
        /* a file = all layers of one chunk, files one after another */
        o->stride_layer = o->obj_bytes;
        o->stride_slot = (uint64_t)g->n_layers * o->obj_bytes;
    } else {
        /* all objects of a layer together, layers one after another */
        o->stride_slot = o->obj_bytes;
        o->stride_layer = o->n_slots_local * o->obj_bytes;
    }
    o->dev_bytes = o->n_slots_local * g->n_layers * o->obj_bytes;
    return ORC_OK;
}

/* Device and byte offset of the K (kv=0) or V (kv=1) half of object `slot`. */
static void object_location(const orc_geom *g, const orc_layout *lo, uint64_t slot,
                            uint32_t layer, uint32_t kv, uint32_t *dev, uint64_t *off)
{
    *dev = (uint32_t)(slot % g->n_devices); /* round-robin over devices */
    *off = (slot / g->n_devices) * lo->stride_slot + (uint64_t)layer * lo->stride_layer +
           (uint64_t)kv * lo->stride_kv;
}

static int check_batch(const orc_geom *g, uint32_t layer, uint32_t n_req,
                       const uint32_t *hit_tokens, const uint32_t *obj_start,
                       const uint32_t *blk_start)
{
    if (layer >= g->n_layers) return ORC_EINVAL;
    for (uint32_t r = 0; r < n_req; ++r) {
        uint64_t hit = hit_tokens[r];
        if (hit % g->block_tokens != 0) return ORC_EINVAL;
        uint64_t need_obj = (hit + g->obj_tokens - 1) / g->obj_tokens;
        uint64_t need_blk = hit / g->block_tokens;
        if ((uint64_t)obj_start[r + 1] - obj_start[r] < need_obj) return ORC_EINVAL;
        if ((uint64_t)blk_start[r + 1] - blk_start[r] < need_blk) return ORC_EINVAL;
    }
    return ORC_OK;
}

/*
 * Location of token t of request r: where it sits in the object store and in
 * which pool block / token row.  This is the whole map; restore and save only
 * differ in the direction of the copy.
 */
static int token_location(const orc_geom *g, const orc_layout *lo, uint32_t layer,
                          const uint32_t *obj_start, const uint32_t *obj_slot,
                          const uint32_t *blk_start, const int32_t *block_ids, uint32_t r,
                          uint64_t t, uint32_t kv, uint32_t *dev, uint64_t *store_off,
                          int64_t *block, uint64_t *row_off)
{
    uint64_t slot = obj_slot[obj_start[r] + t / g->obj_tokens];
    uint64_t off;
    if (slot >= g->n_slots) return ORC_EINVAL;
    object_location(g, lo, slot, layer, kv, dev, &off);
    *store_off = off + (t % g->obj_tokens) * lo->token_bytes;
    *block = block_ids[blk_start[r] + t / g->block_tokens];
    *row_off = (t % g->block_tokens) * lo->token_bytes;
    return ORC_OK;
}

int orc_token_location(const orc_geom *g, uint32_t layer, const uint32_t *obj_start,
                       const uint32_t *obj_slot, const uint32_t *blk_start,
                       const int32_t *block_ids, uint32_t r, uint64_t t, uint32_t kv,
                       uint32_t *dev, uint64_t *store_off, int64_t *block, uint64_t *row_off)
{
    orc_layout lo;
    int rc = orc_obj_layout(g, &lo);
    if (rc) return rc;
    return token_location(g, &lo, layer, obj_start, obj_slot, blk_start, block_ids, r, t, kv,
                          dev, store_off, block, row_off);
}

/* One head's row of one token: where it sits in the store and inside its pool block,
 * for either element order of the block. */
int orc_row_location(const orc_geom *g, uint32_t layer, const uint32_t *obj_start,
                     const uint32_t *obj_slot, const uint32_t *blk_start,
                     const int32_t *block_ids, uint32_t r, uint64_t t, uint32_t kv, uint32_t head,
                     int pool_hnd, uint32_t *dev, uint64_t *store_off, int64_t *block,
                     uint64_t *off_in_block)
{
    orc_layout lo;
    uint64_t tok_off;
    int rc = orc_obj_layout(g, &lo);
    if (rc) return rc;
    if (head >= g->n_kv_heads) return ORC_EINVAL;
    rc = token_location(g, &lo, layer, obj_start, obj_slot, blk_start, block_ids, r, t, kv, dev,
                        store_off, block, &tok_off);
    if (rc) return rc;
    uint64_t row = (uint64_t)g->head_dim * g->elem_bytes;
    *store_off += head * row;
    if (pool_hnd)
        *off_in_block = ((uint64_t)head * g->block_tokens + t % g->block_tokens) * row;
    else
        *off_in_block = tok_off + head * row;
    return ORC_OK;
}

static int move_layer(const orc_geom *g, uint32_t layer, uint32_t n_req,
                      const uint32_t *hit_tokens, const uint32_t *obj_start,
                      const uint32_t *obj_slot, const uint32_t *blk_start,
                      const int32_t *block_ids, uint8_t *const *store, uint8_t *pool_k,
                      uint8_t *pool_v, uint64_t block_stride, uint64_t n_pool_blocks, int to_pool,
                      int pool_hnd)
{
    orc_layout lo;
    int rc = orc_obj_layout(g, &lo);
    if (rc) return rc;
    rc = check_batch(g, layer, n_req, hit_tokens, obj_start, blk_start);
    if (rc) return rc;
    for (uint32_t r = 0; r < n_req; ++r) {
        for (uint64_t t = 0; t < hit_tokens[r]; ++t) {
            for (uint32_t kv = 0; kv < 2; ++kv) {
                uint32_t dev;
                uint64_t soff, roff;
                int64_t blk;
                rc = token_location(g, &lo, layer, obj_start, obj_slot, blk_start, block_ids, r,
                                    t, kv, &dev, &soff, &blk, &roff);
                if (rc) return rc;
                if (blk < 0 || (uint64_t)blk >= n_pool_blocks) return ORC_EINVAL;
                uint8_t *in_store = store[dev] + soff;
                if (!pool_hnd) {
                    /* block = [token][head][dim]: the token's bytes are one run */
                    uint8_t *in_pool = (kv ? pool_v : pool_k) + (uint64_t)blk * block_stride + roff;
                    if (to_pool)
                        memcpy(in_pool, in_store, lo.token_bytes);
                    else
                        memcpy(in_store, in_pool, lo.token_bytes);
                } else {
                    /* block = [head][token][dim]: one row of head_dim elements per head */
                    uint64_t row = (uint64_t)g->head_dim * g->elem_bytes;
                    uint64_t tok = t % g->block_tokens;
                    for (uint32_t hd = 0; hd < g->n_kv_heads; ++hd) {
                        uint8_t *in_pool = (kv ? pool_v : pool_k) + (uint64_t)blk * block_stride +
                                           ((uint64_t)hd * g->block_tokens + tok) * row;
                        if (to_pool)
                            memcpy(in_pool, in_store + hd * row, row);
                        else
                            memcpy(in_store + hd * row, in_pool, row);
                    }
                }
            }
        }
    }
    return ORC_OK;
}

/* Layer-wise Retrieve (Section 3.1 / 3.4): object store -> paged pool. */
int orc_restore_layer(const orc_geom *g, uint32_t layer, uint32_t n_req,
                      const uint32_t *hit_tokens, const uint32_t *obj_start,
                      const uint32_t *obj_slot, const uint32_t *blk_start,
                      const int32_t *block_ids, uint8_t *const *store, uint8_t *pool_k,
                      uint8_t *pool_v, uint64_t block_stride, uint64_t n_pool_blocks, int pool_hnd)
{
    return move_layer(g, layer, n_req, hit_tokens, obj_start, obj_slot, blk_start, block_ids,
                      store, pool_k, pool_v, block_stride, n_pool_blocks, 1, pool_hnd);
}

/* Layer-wise Store (Section 3.1 / 3.4): paged pool -> object store. */
int orc_save_layer(const orc_geom *g, uint32_t layer, uint32_t n_req,
                   const uint32_t *hit_tokens, const uint32_t *obj_start,
                   const uint32_t *obj_slot, const uint32_t *blk_start,
                   const int32_t *block_ids, uint8_t *const *store, uint8_t *pool_k,
                   uint8_t *pool_v, uint64_t block_stride, uint64_t n_pool_blocks, int pool_hnd)
{
    return move_layer(g, layer, n_req, hit_tokens, obj_start, obj_slot, blk_start, block_ids,
                      store, pool_k, pool_v, block_stride, n_pool_blocks, 0, pool_hnd);
}

/* ------------------------------------------------------------------------- */
/* Descriptor build, step by step (sequential).                               */
/* ------------------------------------------------------------------------- */

typedef struct {
    uint32_t dev;
    uint64_t src_off;
    uint64_t len;
    uint32_t n_blk;
    uint32_t r, c, kv;
    uint32_t seq; /* position in (r, c, kv) generation order */
} item_t;

static int item_cmp(const void *pa, const void *pb)
{
    const item_t *a = (const item_t *)pa, *b = (const item_t *)pb;
    if (a->dev != b->dev) return a->dev < b->dev ? -1 : 1;
    if (a->src_off != b->src_off) return a->src_off < b->src_off ? -1 : 1;
    /* items that start at the same byte: the shorter (a prefix ending inside the object)
     * first, so that items naming exactly the same bytes end up next to each other */
    if (a->len != b->len) return a->len < b->len ? -1 : 1;
    /* equal keys keep generation order: this makes qsort behave as a stable sort */
    if (a->seq != b->seq) return a->seq < b->seq ? -1 : 1;
    return 0;
}

/*
 * Step 5, second form: IOCBs of (nearly) equal work instead of equal context count, so that
 * "n IOCBs" is a unit of transfer time as it is with the paper's uniform IOCBs (Section 3.2:
 * an IOCB is a batch of 2048 equal I/O contexts; Section 3.3 profiles kernel time against the
 * IOCB count).  IOCB k takes the scatter-gather entries from boundary k to boundary k + 1,
 * where boundary k is entry k * entries_per_iocb moved back to the first entry of its source
 * block (a repeat is never separated from the bytes it repeats); a context that crosses a
 * boundary is cut there into two contexts.  The contexts are rewritten in place.
 */
static int pack_by_entries(orc_sqe *sqes, uint32_t ns, uint32_t max_sqe, const orc_sgl *sgl,
                           uint32_t ne, uint32_t capacity, uint32_t per, uint32_t *num_ioctx,
                           uint32_t max_iocb, uint32_t *n_sqe, uint32_t *n_sgl, uint32_t *n_iocb)
{
    uint32_t nb = (ne + per - 1) / per;
    if (nb == 0) nb = 1;
    if (nb > max_iocb) return ORC_ENOSPC;
    orc_sqe *whole = (orc_sqe *)malloc((ns ? ns : 1) * sizeof(orc_sqe));
    if (!whole) return ORC_ENOSPC;
    memcpy(whole, sqes, ns * sizeof(orc_sqe));
    uint32_t out = 0, s = 0;
    for (uint32_t k = 0; k < nb; ++k) {
        uint64_t y0 = (uint64_t)k * per, y1 = (uint64_t)(k + 1) * per;
        uint32_t lo = y0 < ne ? (uint32_t)y0 : ne, hi = y1 < ne ? (uint32_t)y1 : ne;
        while (lo < ne && lo > 0 && (sgl[lo].id & ORC_SGL_DUP)) --lo;
        while (hi < ne && hi > 0 && (sgl[hi].id & ORC_SGL_DUP)) --hi;
        uint32_t count = 0;
        /* the contexts that have entries in [lo, hi) */
        while (s < ns && whole[s].sgl_first + whole[s].sgl_count <= lo) ++s;
        for (uint32_t t = s; t < ns && whole[t].sgl_first < hi; ++t) {
            uint32_t a = whole[t].sgl_first > lo ? whole[t].sgl_first : lo;
            uint32_t b = whole[t].sgl_first + whole[t].sgl_count < hi
                             ? whole[t].sgl_first + whole[t].sgl_count : hi;
            if (a >= b) continue;
            if (out >= max_sqe) { free(whole); return ORC_ENOSPC; }
            orc_sqe *p = &sqes[out++];
            *p = whole[t];
            /* object bytes named before entry a, and by the entries [a, b) */
            uint64_t before = 0, named = 0;
            for (uint32_t e = whole[t].sgl_first; e < a; ++e)
                if (!(sgl[e].id & ORC_SGL_DUP)) before += sgl[e].len;
            for (uint32_t e = a; e < b; ++e)
                if (!(sgl[e].id & ORC_SGL_DUP)) named += sgl[e].len;
            p->src_off = whole[t].src_off + before;
            p->len = named;
            p->sgl_first = a;
            p->sgl_count = b - a;
            ++count;
        }
        if (count > capacity) { free(whole); return ORC_EINVAL; }
        num_ioctx[k] = count;
    }
    free(whole);
    *n_sqe = out;
    *n_sgl = ne;
    *n_iocb = nb;
    return ORC_OK;
}

/*
 * Build one layer's descriptors.
 *   sqes[max_sqe], sgl[max_sgl], num_ioctx[max_iocb] are outputs; *n_sqe, *n_sgl,
 *   *n_iocb the counts produced.  SQE k belongs to IOCB k / capacity at position
 *   k % capacity.  n_iocb = ceil(n_sqe / capacity), at least 1 (an empty batch
 *   yields one IOCB with num_ioctx = 0).  With entries_per_iocb != 0 the IOCBs are cut by
 *   scatter-gather entries instead (see pack_by_entries): n_iocb = ceil(n_sgl /
 *   entries_per_iocb), IOCB b holds num_ioctx[b] consecutive contexts of the output.
 */
int orc_build_budget(const orc_geom *g, uint32_t layer, uint32_t opcode, uint32_t n_req,
                     const uint32_t *hit_tokens, const uint32_t *obj_start,
                     const uint32_t *obj_slot, const uint32_t *blk_start,
                     const int32_t *block_ids, uint64_t k_base_addr, uint64_t v_base_addr,
                     uint64_t block_stride, uint32_t capacity, uint32_t entries_per_iocb,
                     orc_sqe *sqes, uint32_t max_sqe, orc_sgl *sgl, uint32_t max_sgl,
                     uint32_t *num_ioctx, uint32_t max_iocb, uint32_t *n_sqe, uint32_t *n_sgl,
                     uint32_t *n_iocb)
{
    orc_layout lo;
    int rc = orc_obj_layout(g, &lo);
    if (rc) return rc;
    rc = check_batch(g, layer, n_req, hit_tokens, obj_start, blk_start);
    if (rc) return rc;
    if (capacity == 0 || ((opcode & 0xff) != ORC_OP_READ && (opcode & 0xff) != ORC_OP_WRITE))
        return ORC_EINVAL;

    /* step 1: items, one per hit object and per K / V half */
    uint64_t n_items = 0;
    for (uint32_t r = 0; r < n_req; ++r)
        n_items += 2 * (((uint64_t)hit_tokens[r] + g->obj_tokens - 1) / g->obj_tokens);
    item_t *items = (item_t *)malloc((n_items ? n_items : 1) * sizeof(item_t));
    if (!items) return ORC_ENOSPC;
    uint32_t q = 0;
    for (uint32_t r = 0; r < n_req; ++r) {
        uint64_t hit = hit_tokens[r];
        uint64_t n_chunks = (hit + g->obj_tokens - 1) / g->obj_tokens;
        for (uint64_t c = 0; c < n_chunks; ++c) {
            uint64_t valid = hit - c * g->obj_tokens;
            if (valid > g->obj_tokens) valid = g->obj_tokens;
            uint64_t slot = obj_slot[obj_start[r] + c];
            if (slot >= g->n_slots) { free(items); return ORC_EINVAL; }
            for (uint32_t kv = 0; kv < 2; ++kv) {
                item_t *it = &items[q];
                object_location(g, &lo, slot, layer, kv, &it->dev, &it->src_off);
                it->len = valid * lo.token_bytes;
                it->n_blk = (uint32_t)(valid / g->block_tokens);
                it->r = r; it->c = (uint32_t)c; it->kv = kv; it->seq = q;
                ++q;
            }
        }
    }

    /* step 2: order by (device, offset, length), stable */
    qsort(items, n_items, sizeof(item_t), item_cmp);

    /* step 3 + 4: sweep over the distinct sources.  A group = an item and the items right
     * after it that name exactly the same bytes (same device, offset and length).  A group
     * opens a new context unless it starts where the previous group's bytes end; its SGL
     * entries go block by block, and for each block one entry per member of the group, in
     * sorted order, all but the first flagged as repeats of the bytes just named. */
    uint32_t ns = 0, ne = 0;
    const item_t *prev = NULL; /* first item of the previous group */
    for (uint64_t i = 0; i < n_items;) {
        const item_t *it = &items[i];
        uint64_t k = 1;
        while (i + k < n_items && items[i + k].dev == it->dev &&
               items[i + k].src_off == it->src_off && items[i + k].len == it->len)
            ++k;
        int fresh = !prev || prev->dev != it->dev || prev->src_off + prev->len != it->src_off;
        if (fresh) {
            if (ns >= max_sqe) { free(items); return ORC_ENOSPC; }
            orc_sqe *s = &sqes[ns++];
            s->src_off = it->src_off;
            s->len = 0;
            s->sgl_first = ne;
            s->sgl_count = 0;
            s->dev = it->dev;
            s->opcode = (uint16_t)opcode;
            s->layer = (uint16_t)layer;
        }
        orc_sqe *s = &sqes[ns - 1];
        s->len += it->len;                       /* the bytes are named once */
        s->sgl_count += (uint32_t)(k * it->n_blk);
        for (uint32_t j = 0; j < it->n_blk; ++j) {
            for (uint64_t c = 0; c < k; ++c) {
                const item_t *m = &items[i + c];
                if (ne >= max_sgl) { free(items); return ORC_ENOSPC; }
                int32_t id = block_ids[blk_start[m->r] + (uint64_t)m->c * lo.blocks_per_obj + j];
                if (id < 0) { free(items); return ORC_EINVAL; }
                sgl[ne].addr = (m->kv ? v_base_addr : k_base_addr) + (uint64_t)id * block_stride;
                sgl[ne].len = (uint32_t)lo.block_bytes;
                sgl[ne].id = (uint32_t)id | (c ? ORC_SGL_DUP : 0u);
                ++ne;
            }
        }
        prev = it;
        i += k;
    }
    free(items);

    if (entries_per_iocb != 0)
        return pack_by_entries(sqes, ns, max_sqe, sgl, ne, capacity, entries_per_iocb, num_ioctx,
                               max_iocb, n_sqe, n_sgl, n_iocb);

    /* step 5: pack into IOCBs of `capacity` contexts */
    uint32_t nb = (ns + capacity - 1) / capacity;
    if (nb == 0) nb = 1;
    if (nb > max_iocb) return ORC_ENOSPC;
    for (uint32_t b = 0; b < nb; ++b) {
        uint32_t left = ns - (ns < b * capacity ? ns : b * capacity);
        num_ioctx[b] = left < capacity ? left : capacity;
    }
    *n_sqe = ns;
    *n_sgl = ne;
    *n_iocb = nb;
    return ORC_OK;
}

int orc_build(const orc_geom *g, uint32_t layer, uint32_t opcode, uint32_t n_req,
              const uint32_t *hit_tokens, const uint32_t *obj_start, const uint32_t *obj_slot,
              const uint32_t *blk_start, const int32_t *block_ids, uint64_t k_base_addr,
              uint64_t v_base_addr, uint64_t block_stride, uint32_t capacity, orc_sqe *sqes,
              uint32_t max_sqe, orc_sgl *sgl, uint32_t max_sgl, uint32_t *num_ioctx,
              uint32_t max_iocb, uint32_t *n_sqe, uint32_t *n_sgl, uint32_t *n_iocb)
{
    return orc_build_budget(g, layer, opcode, n_req, hit_tokens, obj_start, obj_slot, blk_start,
                            block_ids, k_base_addr, v_base_addr, block_stride, capacity, 0, sqes,
                            max_sqe, sgl, max_sgl, num_ioctx, max_iocb, n_sqe, n_sgl, n_iocb);
}

/*
 * Execute descriptors: for each context, walk its SGL entries with a cursor
 * on the object side.  READ moves object bytes to the entry's address, WRITE
 * the other way.  An entry flagged as a repeat uses the object bytes of the entry
 * before it and does not advance the cursor.  Pool addresses are translated to the host copy of the pool
 * by  host = pool_host + (addr - pool_base_addr).
 */
int orc_exec(const orc_sqe *sqes, uint32_t n_sqe, const orc_sgl *sgl, uint32_t n_sgl,
             uint8_t *const *store, const uint64_t *store_bytes, uint32_t n_devices,
             uint8_t *pool_host, uint64_t pool_base_addr, uint64_t pool_bytes,
             uint32_t n_kv_heads, uint32_t row_bytes)
{
    for (uint32_t k = 0; k < n_sqe; ++k) {
        const orc_sqe *s = &sqes[k];
        if (s->dev >= n_devices) return ORC_EINVAL;
        if ((uint64_t)s->sgl_first + s->sgl_count > n_sgl) return ORC_EINVAL;
        int to_pool = (s->opcode & 0xff) == ORC_OP_READ;
        uint64_t cursor = s->src_off, at = s->src_off;
        for (uint32_t e = s->sgl_first; e < s->sgl_first + s->sgl_count; ++e) {
            if (sgl[e].addr < pool_base_addr) return ORC_EINVAL;
            uint64_t poff = sgl[e].addr - pool_base_addr;
            if (poff + sgl[e].len > pool_bytes) return ORC_EINVAL;
            if (sgl[e].id & ORC_SGL_DUP) {
                /* the bytes of the entry before: the cursor stays where it is */
                if (e == s->sgl_first || sgl[e].len != sgl[e - 1].len) return ORC_EINVAL;
            } else {
                at = cursor;
                cursor += sgl[e].len;
            }
            if (at + sgl[e].len > store_bytes[s->dev]) return ORC_EINVAL;
            uint8_t *obj = store[s->dev] + at, *blk = pool_host + poff;
            if (!(s->opcode & ORC_OP_HND)) {
                if (to_pool) memcpy(blk, obj, sgl[e].len); else memcpy(obj, blk, sgl[e].len);
            } else {
                /* the entry is one block: object side [token][head][row], pool side
                 * [head][token][row] */
                uint64_t tok_bytes = (uint64_t)n_kv_heads * row_bytes;
                if (tok_bytes == 0 || sgl[e].len % tok_bytes) return ORC_EINVAL;
                uint64_t n_tok = sgl[e].len / tok_bytes;
                for (uint64_t t = 0; t < n_tok; ++t)
                    for (uint32_t hd = 0; hd < n_kv_heads; ++hd) {
                        uint8_t *o = obj + t * tok_bytes + (uint64_t)hd * row_bytes;
                        uint8_t *q = blk + ((uint64_t)hd * n_tok + t) * row_bytes;
                        if (to_pool) memcpy(q, o, row_bytes); else memcpy(o, q, row_bytes);
                    }
            }
        }
        if (cursor - s->src_off != s->len) return ORC_EINVAL;
    }
    return ORC_OK;
}

/* ------------------------------------------------------------------------- */
/* The restore / save map at block granularity, on several host threads.      */
/* ------------------------------------------------------------------------- */

typedef struct {
    const orc_geom *g;
    const orc_layout *lo;
    uint32_t layer, n_req;
    const uint32_t *hit_tokens, *obj_start, *obj_slot, *blk_start;
    const int32_t *block_ids;
    uint8_t *const *store;
    uint8_t *pool_k, *pool_v;
    uint64_t block_stride, n_pool_blocks;
    int to_pool, pool_hnd;
    uint64_t first, last; /* this thread's share of the batch's blocks, [first, last) */
    int rc, threaded;
} mt_job;

static void *mt_worker(void *arg)
{
    mt_job *j = (mt_job *)arg;
    const orc_geom *g = j->g;
    const orc_layout *lo = j->lo;
    uint64_t seen = 0; /* blocks of the requests before r */
    j->rc = ORC_OK;
    for (uint32_t r = 0; r < j->n_req; ++r) {
        uint64_t nb = j->hit_tokens[r] / g->block_tokens;
        uint64_t b0 = j->first > seen ? j->first - seen : 0;
        uint64_t b1 = j->last < seen + nb ? (j->last > seen ? j->last - seen : 0) : nb;
        for (uint64_t b = b0; b < b1; ++b) {
            uint64_t t = b * g->block_tokens; /* first token of the block */
            for (uint32_t kv = 0; kv < 2; ++kv) {
                uint32_t dev;
                uint64_t soff, roff;
                int64_t blk;
                int rc = token_location(g, lo, j->layer, j->obj_start, j->obj_slot, j->blk_start,
                                        j->block_ids, r, t, kv, &dev, &soff, &blk, &roff);
                if (rc) { j->rc = rc; return NULL; }
                if (blk < 0 || (uint64_t)blk >= j->n_pool_blocks) { j->rc = ORC_EINVAL; return NULL; }
                uint8_t *in_store = j->store[dev] + soff;
                uint8_t *in_pool = (kv ? j->pool_v : j->pool_k) + (uint64_t)blk * j->block_stride;
                if (!j->pool_hnd) {
                    if (j->to_pool) memcpy(in_pool, in_store, lo->block_bytes);
                    else memcpy(in_store, in_pool, lo->block_bytes);
                } else {
                    uint64_t row = (uint64_t)g->head_dim * g->elem_bytes;
                    for (uint32_t tok = 0; tok < g->block_tokens; ++tok)
                        for (uint32_t hd = 0; hd < g->n_kv_heads; ++hd) {
                            uint8_t *o = in_store + tok * lo->token_bytes + hd * row;
                            uint8_t *q = in_pool + ((uint64_t)hd * g->block_tokens + tok) * row;
                            if (j->to_pool) memcpy(q, o, row); else memcpy(o, q, row);
                        }
                }
            }
        }
        seen += nb;
    }
    return NULL;
}

/* to_pool != 0: restore, else save.  n_threads >= 1; returns the oracle's codes. */
int orc_move_layer_blocks_mt(const orc_geom *g, uint32_t layer, uint32_t n_req,
                             const uint32_t *hit_tokens, const uint32_t *obj_start,
                             const uint32_t *obj_slot, const uint32_t *blk_start,
                             const int32_t *block_ids, uint8_t *const *store, uint8_t *pool_k,
                             uint8_t *pool_v, uint64_t block_stride, uint64_t n_pool_blocks,
                             int pool_hnd, int to_pool, uint32_t n_threads)
{
    orc_layout lo;
    int rc = orc_obj_layout(g, &lo);
    if (rc) return rc;
    rc = check_batch(g, layer, n_req, hit_tokens, obj_start, blk_start);
    if (rc) return rc;
    if (n_threads == 0 || n_threads > 1024) return ORC_EINVAL;
    uint64_t total = 0;
    for (uint32_t r = 0; r < n_req; ++r) total += hit_tokens[r] / g->block_tokens;
    mt_job *jobs = (mt_job *)calloc(n_threads, sizeof(mt_job));
    pthread_t *tids = (pthread_t *)calloc(n_threads, sizeof(pthread_t));
    if (!jobs || !tids) { free(jobs); free(tids); return ORC_ENOSPC; }
    for (uint32_t k = 0; k < n_threads; ++k) {
        mt_job *j = &jobs[k];
        j->g = g; j->lo = &lo; j->layer = layer; j->n_req = n_req;
        j->hit_tokens = hit_tokens; j->obj_start = obj_start; j->obj_slot = obj_slot;
        j->blk_start = blk_start; j->block_ids = block_ids; j->store = store;
        j->pool_k = pool_k; j->pool_v = pool_v; j->block_stride = block_stride;
        j->n_pool_blocks = n_pool_blocks; j->to_pool = to_pool; j->pool_hnd = pool_hnd;
        j->first = total * k / n_threads;
        j->last = total * (k + 1) / n_threads;
        j->threaded = 0;
        /* the calling thread takes the last share (and any share no thread could be made for) */
        if (k + 1 < n_threads && pthread_create(&tids[k], NULL, mt_worker, j) == 0)
            j->threaded = 1;
        else
            mt_worker(j);
    }
    for (uint32_t k = 0; k < n_threads; ++k)
        if (jobs[k].threaded) pthread_join(tids[k], NULL);
    for (uint32_t k = 0; k < n_threads; ++k)
        if (jobs[k].rc) rc = jobs[k].rc;
    free(jobs);
    free(tids);
    return rc;
}
