/*
 * tutti.h — C ABI of the B200 (sm_100a) KV-cache object-store hot path.
 *
 * The library moves prefix KV cache, one layer at a time, between contiguous
 * per-layer KV objects (the storage tier; here an object store in HBM or in
 * pinned host memory read zero-copy) and a fragmented, block-table-indexed paged
 * KV pool in HBM, and builds the I/O submission descriptors for that transfer on
 * the GPU, into a GPU-resident submission/completion ring.  The host does O(1)
 * work per layer and no per-block work (paper Section 3.1, last paragraph).
 *
 * Conventions
 *   - Every call returns TUTTI_OK (0) or a negative TUTTI_E* code.  Device-side
 *     problems never trap: they arrive as `status` of the completion entry.
 *   - "device pointer" = address valid in kernels on the context's GPU (HBM, or
 *     the device alias of pinned mapped host memory).  "host pointer" = ordinary
 *     host memory.  Streams are passed as `void*` holding a CUstream/cudaStream_t
 *     (NULL = the legacy default stream).
 *   - Nothing on the per-layer path (build / restore / save / poll) allocates
 *     memory or synchronises the host with the device (Section 3.2, "Zero-Copy
 *     Ring Buffers": no runtime allocation, copying or CPU-GPU synchronisation).
 *   - One ring is driven by one host thread at a time (no internal locking).
 */
#ifndef TUTTI_H_
#define TUTTI_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define TUTTI_OK 0
#define TUTTI_EINVAL (-1)    /* bad argument or broken precondition                      */
#define TUTTI_ENOMEM (-2)    /* allocation failed at create time                         */
#define TUTTI_EAGAIN (-3)    /* ring / SGL arena full, or completion not there yet       */
#define TUTTI_ETIMEDOUT (-4) /* a bounded device-side wait ran out                       */
#define TUTTI_EFAULT (-5)    /* a block id or object slot points outside its region      */
#define TUTTI_ECUDA (-6)     /* a CUDA call failed; see tutti_last_cuda_error()          */
#define TUTTI_ENOENT (-7)    /* key not in the file pool                                 */

#define TUTTI_LAYOUT_FILE_MAJOR 0  /* a file = all layers of one chunk; files back to back */
#define TUTTI_LAYOUT_LAYER_MAJOR 1 /* all objects of a layer together; layers back to back */

#define TUTTI_OP_READ 0  /* object store -> paged pool  (restore / Retrieve) */
#define TUTTI_OP_WRITE 1 /* paged pool  -> object store (save / Store)       */
/* Opcode flag carried by contexts and IOCBs built while the pool layout is head-major:
 * a pool block is [head][token][dim] instead of [token][head][dim] (Section 2.1 gives
 * the paged layout as [Block, h, d]; objects always stay token-major), so the copy
 * transposes rows of head_dim elements inside every block. */
#define TUTTI_OP_FLAG_HND 0x100

#define TUTTI_STORE_HBM 0
#define TUTTI_STORE_HOST_PINNED 1

#define TUTTI_MAX_DEVICES 8
#define TUTTI_DEFAULT_IOCTX_PER_IOCB 2048 /* Section 3.2: one IOCB holds 2048 I/O contexts */

/* Options for tutti_set_option(). */
#define TUTTI_OPT_COPY_ENGINE 1 /* 0 auto, 1 vector load/store kernel, 2 bulk-async (TMA) kernel */
#define TUTTI_OPT_WAIT_NS 2     /* budget of the device-side wait for an IOCB to become ready
                                   (default 2 ms, at most 2 s).  An IOCB whose build has not been
                                   published within it completes with TUTTI_ETIMEDOUT and moves
                                   nothing; this is retryable: poll it, build the layer again and
                                   issue the new IOCBs                                            */
#define TUTTI_OPT_CTAS_PER_SM 3 /* resident CTAs per SM of the load/store kernel (grid mode)     */
#define TUTTI_OPT_BULK_WARPS 4  /* copy warps per CTA of the bulk-async kernel                   */
#define TUTTI_OPT_BULK_STAGES 5 /* shared-memory stages per copy warp of the bulk-async kernel   */
#define TUTTI_OPT_CLAIM_CHUNKS 6 /* chunks taken per work claim                                   */
#define TUTTI_OPT_POOL_LAYOUT 8  /* TUTTI_POOL_NHD (default) or TUTTI_POOL_HND: element order inside a
                                   pool block; applies to builds made after it is set.  HND needs
                                   head_dim * elem_bytes to be a multiple of 16 (TUTTI_EINVAL)  */
#define TUTTI_POOL_NHD 0
#define TUTTI_POOL_HND 1
#define TUTTI_OPT_BULK_CHUNK_BYTES 7 /* bytes per shared-memory stage of the bulk-async kernel: a
                                        power of two, 4096..32768                                 */
#define TUTTI_OPT_INJECT_BULK_TIMEOUT 9 /* 1: the bulk-async kernel reports every wait for a stage's
                                           bytes as run out (host-side fault injection for the
                                           error path: the IOCBs complete with TUTTI_ETIMEDOUT and
                                           move nothing; no GPU fault is involved)                */

/*
 * Geometry of the KV cache and of the object store (Section 3.1, "Scalable GPU
 * File Pool").  An object holds obj_tokens tokens of one layer: its K half then
 * its V half, each [obj_tokens][n_kv_heads][head_dim] elements; the paper's
 * one-object-per-block case is obj_tokens == block_tokens.  Object slot s lives
 * on storage device s mod n_devices (round-robin placement).
 */
typedef struct tutti_geom {
    uint32_t n_layers;
    uint32_t n_kv_heads;
    uint32_t head_dim;
    uint32_t elem_bytes;
    uint32_t block_tokens; /* tokens per paged KV block                      */
    uint32_t obj_tokens;   /* tokens per object; a multiple of block_tokens  */
    uint32_t n_devices;    /* storage devices, 1..TUTTI_MAX_DEVICES          */
    uint32_t layout;       /* TUTTI_LAYOUT_*                                 */
    uint64_t n_slots;      /* object slots in the store, over all devices    */
} tutti_geom_t;

/* Derived sizes and strides.  Byte offset of the K (kv=0) / V (kv=1) half of slot s,
 * layer l, on device s mod n_devices:
 *     (s / n_devices) * stride_slot + l * stride_layer + kv * stride_kv          */
typedef struct tutti_layout {
    uint64_t token_bytes;   /* K (or V) of one token of one layer              */
    uint64_t block_bytes;   /* K (or V) of one paged block of one layer        */
    uint64_t obj_kv_bytes;  /* one half of an object                           */
    uint64_t obj_bytes;     /* K half + V half                                 */
    uint64_t blocks_per_obj;
    uint64_t n_slots_local; /* slots per device = ceil(n_slots / n_devices)    */
    uint64_t stride_kv;
    uint64_t stride_layer;
    uint64_t stride_slot;
    uint64_t dev_bytes;     /* bytes each device's store region must provide   */
} tutti_layout_t;

/*
 * One batch of prefix hits.  All five arrays are DEVICE pointers owned by the
 * caller; they must stay valid and unchanged until every IOCB built from them has
 * been polled.  CSR form: request r owns objects obj_slot[obj_start[r] ..
 * obj_start[r+1]) in chunk order and pool blocks block_ids[blk_start[r] ..
 * blk_start[r+1]) in logical block order.  hit_tokens[r] must be a multiple of
 * block_tokens; row r must list at least ceil(hit/obj_tokens) objects and
 * hit/block_tokens blocks (extra entries are never read).
 * The scalar fields are host-known sizes: n_obj = obj_start[n_req], n_blk =
 * blk_start[n_req].
 * plan_epoch: 0 = the sorted/coalesced plan is recomputed on every build.  A
 * non-zero value promises that a batch with the same epoch, pointers and sizes has
 * the same contents, so the plan of the previous build on the ring is reused (it
 * does not depend on the layer) and only the per-layer part is redone.
 */
typedef struct tutti_batch {
    uint32_t n_req;
    uint32_t n_obj;
    uint32_t n_blk;
    uint32_t plan_epoch;
    const uint32_t *hit_tokens; /* [n_req]     */
    const uint32_t *obj_start;  /* [n_req + 1] */
    const uint32_t *obj_slot;   /* [n_obj]     */
    const uint32_t *blk_start;  /* [n_req + 1] */
    const int32_t *block_ids;   /* [n_blk]     */
} tutti_batch_t;

/* I/O context (Section 3.2: "SGL address, GPU file offset, and length"): one
 * contiguous byte range of one storage device and the scatter-gather entries that
 * cover it.  sgl_first counts from the first entry of the build the context
 * belongs to. */
typedef struct tutti_sqe {
    uint64_t src_off; /* object-side byte offset on device `dev` (both directions) */
    uint64_t len;
    uint32_t sgl_first;
    uint32_t sgl_count;
    uint32_t dev;
    uint16_t opcode;
    uint16_t layer;
} tutti_sqe_t;

/* Scatter-gather entry, 16 bytes (Section 3.1: address 8 B, length 4 B, identifier
 * 4 B).  addr is the pool-side device address, id the pool block id.  A stored chunk that
 * several requests of the batch hit (Section 3.1: a chunk is shared by every request with
 * that prefix) is named once in its context; the entries of the second and later requests
 * carry TUTTI_SGL_FLAG_DUP in id: "the object bytes of the entry before this one", so the
 * walk over the context's byte range does not advance for them. */
#define TUTTI_SGL_FLAG_DUP 0x80000000u
typedef struct tutti_sgl {
    uint64_t addr;
    uint32_t len;
    uint32_t id;
} tutti_sgl_t;

/* Completion entry: the IOCB index the kernel writes to the CQ (Section 3.2, step
 * 3), with a status and the bytes it moved. */
typedef struct tutti_cqe {
    uint32_t iocb_idx;
    int32_t status;
    uint64_t bytes;
} tutti_cqe_t;

/* Read-back of one IOCB header (inspection / tests). */
typedef struct tutti_iocb_info {
    uint32_t iocb_idx;
    uint32_t ready;         /* 1 once its descriptors are published           */
    uint32_t num_ioctx;
    uint32_t opcode;
    uint32_t layer;
    int32_t status;
    uint32_t sgl_base;      /* arena index of the build's first entry         */
    uint32_t entry_first;   /* first entry of this IOCB, relative to sgl_base */
    uint32_t total_entries;
    uint32_t entry_len;     /* common entry length, 0 if lengths differ       */
    uint64_t bytes;
} tutti_iocb_info_t;

typedef struct tutti_ctx tutti_ctx_t;
typedef struct tutti_ring tutti_ring_t;

/* ------------------------------------------------------------------------- */
/* The five calls of the path                                                 */
/* ------------------------------------------------------------------------- */

/*
 * Object id -> (device, byte offset, length): sizes and strides of the object
 * store for a geometry (Section 3.1: a GPU file is 2 x L objects, one key and one
 * value object per layer; files are placed round-robin across devices).
 * Pure host function; both pointers are host memory.  TUTTI_EINVAL if a field is
 * zero, obj_tokens is not a multiple of block_tokens, token_bytes is not a multiple
 * of 16, n_devices > TUTTI_MAX_DEVICES or the layout is unknown.
 */
int tutti_obj_layout(const tutti_geom_t *geom, tutti_layout_t *out);

/*
 * Build one layer's I/O contexts on the GPU (Section 3.1 "block lookup and P2P
 * table lookup to generate a batch of lightweight GPU I/O contexts"; Section 3.2
 * step 2, get_iocb).  GPU threads turn (object slot, layer) into (device, offset,
 * length) items, order them by (device, offset, length), treat items that name
 * exactly the same bytes as one source (read once, TUTTI_SGL_FLAG_DUP), merge
 * exactly byte-adjacent sources into one context, emit one 16-byte SGL entry per
 * pool block in object byte order, pack contexts into IOCBs of ioctx_per_iocb
 * entries and publish them in the ring.  A context's len is the bytes it names in
 * the store; a completion's bytes are the bytes that landed (entries x length).
 *   batch        host pointer to the struct; its arrays are device pointers.
 *   first_iocb,  host out: indices of the reserved IOCBs, known without waiting
 *   n_iocb       for the GPU: ceil(2*n_obj / ioctx_per_iocb), at least 1 (or the
 *                count tutti_ring_set_iocb_bytes states).  IOCBs the build does
 *                not need are published with num_ioctx = 0.
 * Asynchronous on `stream`.  TUTTI_EAGAIN if the ring or the SGL arena has no
 * room (poll completed IOCBs first); TUTTI_EINVAL for layer >= n_layers, unknown
 * opcode, unregistered pool layer / store device, or a batch larger than the ring
 * was created for.  Bad batch contents (misaligned hit length, short rows, slot or
 * block id out of range) are found by the kernel: the IOCBs then carry that status,
 * move no bytes and complete with it.
 */
int tutti_build_sqes(tutti_ctx_t *ctx, tutti_ring_t *ring, const tutti_batch_t *batch,
                     uint32_t layer, uint32_t opcode, void *stream, uint32_t *first_iocb,
                     uint32_t *n_iocb);

/*
 * The same build for n_layers consecutive layers in ONE kernel launch (the batch is known
 * when the request arrives, so all its layers' contexts can be prepared ahead, Section 3.3
 * "When an inference request arrives, the runtime enqueues the corresponding read IOCBs").
 * Layer first_layer + k owns the IOCBs [*first_iocb + k * *iocbs_per_layer,
 * *first_iocb + (k + 1) * *iocbs_per_layer); the descriptors are exactly those of
 * tutti_build_sqes for that layer.  The reservation is one group: its SGL entries are
 * reusable once every IOCB of every layer has been polled.
 */
int tutti_build_sqes_layers(tutti_ctx_t *ctx, tutti_ring_t *ring, const tutti_batch_t *batch,
                            uint32_t first_layer, uint32_t n_layers, uint32_t opcode, void *stream,
                            uint32_t *first_iocb, uint32_t *iocbs_per_layer);

/*
 * Layer-wise Retrieve (Section 3.1; retrieve_layer of Section 3.4; issue_io of
 * Section 3.2 step 3): execute the READ IOCBs [first_iocb, first_iocb + n_iocb):
 * for every context, the bytes at its object-store range are scattered to the
 * pool addresses of its SGL entries.  sm_count = 0 runs on all SMs; otherwise
 * that many persistent CTAs (one per SM) claim the work, for use beside compute
 * kernels (Section 3.2 "SM Partitioning"; Section 3.3).  When the last byte of an
 * IOCB has landed, the kernel writes its index to the completion queue.
 * Asynchronous on `stream`; must be ordered after the build (same stream or an
 * event).  TUTTI_EINVAL if an index was not reserved, or has the other opcode.
 */
int tutti_kv_restore_layer(tutti_ctx_t *ctx, tutti_ring_t *ring, uint32_t first_iocb,
                           uint32_t n_iocb, uint32_t sm_count, void *stream);

/*
 * Layer-wise Store (store_layer of Section 3.4): the same transfer in the other
 * direction for WRITE IOCBs: pool blocks are gathered into the object-store
 * ranges.  Saving and restoring the same objects concurrently is the caller's
 * race (the paper orders them with CUDA events, Section 3.2 step 2).
 */
int tutti_kv_save_layer(tutti_ctx_t *ctx, tutti_ring_t *ring, uint32_t first_iocb,
                        uint32_t n_iocb, uint32_t sm_count, void *stream);

/*
 * wait_cqe (Section 3.2 step 4): look in the completion queue for one IOCB index.
 * timeout_ns = 0 never blocks.  Returns TUTTI_OK and fills *out (host pointer)
 * when the IOCB has completed — out->status carries a device-side error, if any;
 * TUTTI_EAGAIN when it has not completed within the timeout; TUTTI_EINVAL when
 * the index is not a live reservation.  A successful poll releases the IOCB (and,
 * once all IOCBs of its build are polled, the build's SGL entries) for reuse.
 */
int tutti_ring_poll(tutti_ring_t *ring, uint32_t iocb_idx, tutti_cqe_t *out, uint64_t timeout_ns);

/*
 * wait_cqe for a run of IOCBs (a layer's, or a whole pass's): polls first_iocb,
 * first_iocb + 1, ... in order, as tutti_ring_poll does, with one budget of timeout_ns for
 * all of them (0 never blocks).  TUTTI_OK when all n_iocb have completed (and are released);
 * otherwise the code of the poll that stopped the walk (TUTTI_EAGAIN: that IOCB has not
 * completed in time; TUTTI_EINVAL: not a live index) — the IOCBs before it were consumed, so
 * the caller resumes at first_iocb + *n_done.  Host out (each may be NULL): *bytes_total sum
 * of the completions' bytes, *first_error status of the first completion that carried one
 * (0 if none), *n_done completions consumed by this call.
 */
int tutti_ring_poll_range(tutti_ring_t *ring, uint32_t first_iocb, uint32_t n_iocb,
                          uint64_t *bytes_total, int32_t *first_error, uint32_t *n_done,
                          uint64_t timeout_ns);

/*
 * GPU-side dependency on one IOCB (Section 3.2: once enqueued, "GPU-side dependency
 * tracking" orders I/O and compute without the CPU): everything enqueued on `stream`
 * after this call starts only once IOCB iocb_idx has completed — for instance a layer's
 * attention behind that layer's restore, while the copy launch that carries it is still
 * busy with later layers.  Implemented as a stream wait on the IOCB's state word; no
 * kernel, no SM, no host involvement.  The copy launch that executes the IOCB
 * (tutti_kv_restore_layer / tutti_kv_save_layer) must already have been enqueued: for any
 * other index the call returns TUTTI_EAGAIN and enqueues nothing, so a stream can never be
 * left waiting for a completion that no kernel will produce (every wait inside the copy
 * kernels is bounded, so an issued IOCB always completes).  A completion with an error
 * status also releases the stream; read the status with tutti_ring_poll.  The wait is also
 * satisfied if the ring slot has already been reused by a later IOCB when the stream gets
 * there.  TUTTI_EINVAL if the index is not a live reservation; TUTTI_ECUDA if the driver has
 * no stream memory operations.
 */
int tutti_stream_wait_iocb(tutti_ring_t *ring, uint32_t iocb_idx, void *stream);

/* ------------------------------------------------------------------------- */
/* Lifecycle                                                                  */
/* ------------------------------------------------------------------------- */

/* Create a context for `geom` on CUDA device `device` (host call; allocates the
 * small registration tables).  TUTTI_ECUDA if no usable device. */
int tutti_ctx_create(const tutti_geom_t *geom, int device, tutti_ctx_t **out);
int tutti_ctx_destroy(tutti_ctx_t *ctx);

/* Register layer `layer` of the pre-allocated paged KV pool (Section 3.4: "register
 * the pre-allocated KV memory block pool").  Block b's K bytes start at k_base +
 * b * block_stride, its V bytes at v_base + b * block_stride (device pointers,
 * 16-byte aligned, block_stride a multiple of 16 and >= block_bytes).  Layers may
 * share memory.  The caller keeps ownership. */
int tutti_pool_register(tutti_ctx_t *ctx, uint32_t layer, void *k_base, void *v_base,
                        uint64_t block_stride, uint64_t n_blocks);

/* Register the region of storage device `dev`: `base` is a device pointer (HBM,
 * or the device alias of pinned mapped host memory for TUTTI_STORE_HOST_PINNED),
 * 16-byte aligned, `bytes` >= layout.dev_bytes. */
int tutti_store_register(tutti_ctx_t *ctx, uint32_t dev, void *base, uint64_t bytes, uint32_t kind);

int tutti_set_option(tutti_ctx_t *ctx, uint32_t option, uint64_t value);

/* init_queue(depth) (Section 3.2 step 1): a submission ring of `depth` IOCBs (a
 * power of two) of ioctx_per_iocb contexts each, a completion queue of the same
 * depth in pinned host memory, an SGL arena of sgl_capacity entries and plan
 * scratch for batches of up to max_items = 2 * n_obj items.  All memory the
 * per-layer path needs is allocated here. */
int tutti_ring_create(tutti_ctx_t *ctx, uint32_t depth, uint32_t ioctx_per_iocb,
                      uint32_t sgl_capacity, uint32_t max_items, tutti_ring_t **out);
int tutti_ring_destroy(tutti_ring_t *ring);

/* IOCBs of equal work (Section 3.2: the paper's IOCB is a uniform batch of 2048 equal I/O
 * contexts, which is what lets Section 3.3 profile kernel time against the IOCB count).  Here
 * contexts are coalesced runs of very different length, so by default an IOCB (ioctx_per_iocb
 * contexts) is not a unit of time.  With bytes != 0, builds made afterwards on this ring cut
 * IOCBs by bytes instead: IOCB k of a build takes the scatter-gather entries from entry
 * k * (bytes / block_bytes) to entry (k + 1) * (bytes / block_bytes), each boundary moved back
 * so that a TUTTI_SGL_FLAG_DUP entry stays with the entry it repeats; a context that crosses
 * a boundary is cut there into two.  A build then reserves ceil(2 * n_blk * block_bytes /
 * bytes) IOCBs per layer.  bytes / block_bytes must be 1..ioctx_per_iocb (TUTTI_EINVAL);
 * bytes = 0 goes back to IOCBs of ioctx_per_iocb contexts. */
int tutti_ring_set_iocb_bytes(tutti_ring_t *ring, uint64_t bytes);

/*
 * Staged transfers over the host link.  Kernels that read or write pinned host memory directly
 * (TUTTI_STORE_HOST_PINNED, zero-copy) cross the link in the SMs' 128-byte transactions; the
 * copy engines use larger ones and get ~8 % more one way and ~25 % more with both directions
 * busy.  The staged path lets them carry the bytes: a layer's contexts (Section 3.2: file offset
 * + length each) are copied as they are, one cudaMemcpyAsync per context, between the store and
 * a staging buffer in HBM that holds them packed in context order, and the scatter / gather
 * between that buffer and the paged pool stays with the kernels.  Host work per layer is
 * O(contexts), never O(blocks).
 *
 *   tutti_stage_plan        once per batch (plan_epoch != 0): runs the plan on `stream` if the
 *                           ring does not hold it, waits for it and keeps the batch's contexts
 *                           on the host.  A context of at least min_ctx_bytes is staged; a
 *                           smaller one keeps its entries pointing into the store and is moved
 *                           by the kernels alone (a copy engine pays a fixed start-up per copy:
 *                           below about 2 MiB per copy the zero-copy path is the faster one);
 *                           0 stages every context.  Host out: *n_ctx contexts, *n_staged of
 *                           them staged, *bytes_per_layer the staging bytes a layer needs (the
 *                           distinct object bytes of the staged contexts).  Blocks the host: a
 *                           per-request call, not a per-layer one.
 *   tutti_stage_copy_layer  enqueues on `stream` the copies of layer `layer`: store -> staging
 *                           for TUTTI_OP_READ, staging -> store for TUTTI_OP_WRITE.  `stage` is a
 *                           device pointer to at least *bytes_per_layer bytes, 16-byte aligned,
 *                           owned by the caller.  Works for HBM and pinned-host stores alike.
 *   tutti_build_sqes_staged tutti_build_sqes for one layer with the object side of every entry
 *                           of a staged context pointing into `stage` (contexts still carry the
 *                           store offsets).
 *                           The IOCBs are then executed with tutti_kv_restore_layer (after the
 *                           copies into `stage`) or tutti_kv_save_layer (before the copies out
 *                           of it); ordering between copies and kernels is the caller's (stream
 *                           order or events).
 * TUTTI_EINVAL if the batch is not the one tutti_stage_plan saw, or `stage` is too small.
 */
int tutti_stage_plan(tutti_ctx_t *ctx, tutti_ring_t *ring, const tutti_batch_t *batch,
                     uint64_t min_ctx_bytes, void *stream, uint32_t *n_ctx, uint32_t *n_staged,
                     uint64_t *bytes_per_layer);
int tutti_stage_copy_layer(tutti_ctx_t *ctx, tutti_ring_t *ring, uint32_t layer, uint32_t opcode,
                           void *stage, uint64_t stage_bytes, void *stream);
int tutti_build_sqes_staged(tutti_ctx_t *ctx, tutti_ring_t *ring, const tutti_batch_t *batch,
                            uint32_t layer, uint32_t opcode, void *stage, uint64_t stage_bytes,
                            void *stream, uint32_t *first_iocb, uint32_t *n_iocb);

/* get_iocb(nums) for descriptors prepared by the CPU (the paper's own split,
 * Section 3.2: "CPU-prepared, GPU-executed"): reserve n IOCBs and n_sgl arena
 * entries without building anything. */
int tutti_ring_reserve(tutti_ring_t *ring, uint32_t n_iocb, uint32_t n_sgl, uint32_t *first_iocb);

/* Fill one reserved IOCB from host arrays and publish it: sqes[n_sqe] (sgl_first
 * relative to sgl[0]) and sgl[n_sgl] are host pointers, copied before the call
 * returns.  Entry lengths may differ.  `sgl_offset` places this IOCB's entries
 * inside the reservation made by tutti_ring_reserve. */
int tutti_ring_fill_host(tutti_ctx_t *ctx, tutti_ring_t *ring, uint32_t iocb_idx,
                         const tutti_sqe_t *sqes, uint32_t n_sqe, const tutti_sgl_t *sgl,
                         uint32_t n_sgl, uint32_t sgl_offset, void *stream);

/* Inspection (synchronises the device; not for the per-layer path): header, and up
 * to max_sqes contexts, of a live IOCB into host memory; its SGL entries. */
int tutti_ring_read_iocb(tutti_ring_t *ring, uint32_t iocb_idx, tutti_iocb_info_t *info,
                         tutti_sqe_t *sqes, uint32_t max_sqes);
int tutti_ring_read_sgl(tutti_ring_t *ring, uint32_t iocb_idx, tutti_sgl_t *sgl,
                        uint32_t max_entries, uint32_t *n_entries);

/* Counters since ring creation (host pointers): kernels launched by this ring's
 * calls, host calls made on the per-layer path. */
int tutti_ring_stats(tutti_ring_t *ring, uint64_t *kernel_launches, uint64_t *host_calls);

/* Inspection (synchronises the device): the SM id every CTA of the ring's most recent copy
 * launch ran on, smids[0 .. min(*n_ctas, max_ctas)) in CTA order; *n_ctas is the launch's CTA
 * count.  A capped launch (sm_count > 0) has exactly sm_count CTAs on sm_count distinct SMs
 * (Section 3.2 "SM Partitioning"), with either copy engine and on any stream. */
int tutti_ring_last_launch_sms(tutti_ring_t *ring, uint32_t *smids, uint32_t max_ctas,
                               uint32_t *n_ctas);

/* SM partition for the capped mode (Section 3.2 "SM Partitioning For Accurate
 * I/O": a compute domain and an I/O control domain isolated with green contexts).
 * Splits the device's SMs into `io_sms` (rounded up to the hardware granularity)
 * and the rest; returns one stream in each partition and the SM counts obtained.
 * TUTTI_ECUDA if the driver refuses green contexts. */
int tutti_sm_partition_create(tutti_ctx_t *ctx, uint32_t io_sms, void **io_stream,
                              void **compute_stream, uint32_t *io_sms_got,
                              uint32_t *compute_sms_got);
int tutti_sm_partition_destroy(tutti_ctx_t *ctx);

/*
 * (No counterpart in the paper.)  Build and restore one layer without allocating
 * anything.  Some callers must not call cudaMalloc: code that runs after a serving
 * engine has handed the whole HBM budget to its own pools, or inside a section where
 * allocator calls are forbidden.  They cannot create a ring, so this call keeps what
 * a ring would hold — one IOCB with its contexts, SGL entries and plan arrays — in a
 * fixed device array inside the library (about 2 MiB, held by every GPU that loads
 * the library until the process exits) and runs the same kernels on it.
 *   geom, batch      host pointers; the batch arrays are device pointers, as for
 *                    tutti_build_sqes.  Limits: 2 * n_obj <= 4096 and
 *                    2 * n_blk <= 65536; a larger batch returns TUTTI_EINVAL.
 *   k_base, v_base,  the pool layer to restore into (device pointers, 16-byte
 *   block_stride,    aligned), as for tutti_pool_register.
 *   n_blocks
 *   store_base,      host arrays [geom->n_devices]: device pointer and size of every
 *   store_bytes      storage device's region (HBM).
 *   cqe_out          where the completion entry {iocb_idx = 0, status, bytes} is
 *                    copied when the layer is done: device memory, or pinned host
 *                    memory.  Valid once `stream` has reached that point.  If the copy
 *                    kernel could not post a completion, status reads TUTTI_ETIMEDOUT.
 * Asynchronous on `stream`; completion is observed through the stream (there is no
 * completion queue here: a pinned CQ would have to be allocated).  The call issues
 * no cudaMalloc / cudaFree / cudaHostAlloc.  The first call on a device resolves the
 * address of the fixed array and sets kernel attributes; make that first call before
 * any stream capture begins.  All calls on a device share the array, which keeps the
 * previous call's contents (the call clears the words that must start at zero): two
 * calls whose kernels overlap on the GPU — different streams without ordering — race.
 */
int tutti_kv_restore_layer_noalloc(const tutti_geom_t *geom, int device, uint32_t layer,
                                   const tutti_batch_t *batch, void *k_base, void *v_base,
                                   uint64_t block_stride, uint64_t n_blocks,
                                   void *const *store_base, const uint64_t *store_bytes,
                                   tutti_cqe_t *cqe_out, void *stream);

/* ------------------------------------------------------------------------- */
/* Slack-aware I/O scheduler (Section 3.3).  Pure host logic.                  */
/* ------------------------------------------------------------------------- */
#define TUTTI_PHASE_PREFILL 0
#define TUTTI_PHASE_DECODE 1

typedef struct tutti_sched tutti_sched_t;

/* One kernel launch the scheduler asks for: IOCBs [first_iocb, first_iocb + n_iocb)
 * with tutti_kv_restore_layer / tutti_kv_save_layer on sm_count SMs (0 = all).
 * est_us is the profiled time of the whole read (or write) group the launch opens. */
typedef struct tutti_launch {
    uint32_t opcode;
    uint32_t first_iocb;
    uint32_t n_iocb;
    uint32_t sm_count;
    uint32_t layer; /* layer of the first IOCB */
    float est_us;
} tutti_launch_t;

/* The lookup table is indexed by input length and prefix length in steps of
 * token_step tokens ("the token length of a single warp", Section 3.3). */
int tutti_sched_create(uint32_t n_layers, uint32_t token_step, uint32_t max_input_tokens,
                       uint32_t max_prefix_tokens, tutti_sched_t **out);
int tutti_sched_destroy(tutti_sched_t *sched);
/* Offline profile of the model: duration and free-SM budget of a layer's slack window. */
int tutti_sched_set_slack(tutti_sched_t *sched, uint32_t l_input, uint32_t l_prefix,
                          float slack_us, uint32_t sm_budget);
int tutti_sched_set_decode_slack(tutti_sched_t *sched, float slack_us, uint32_t sm_budget);
/* Offline profile of the I/O kernels: time of one launch of n_iocb IOCBs on sm_count SMs.
 * Other counts are interpolated linearly (extrapolated beyond the last point); an
 * unprofiled SM count uses the largest profiled one that is not larger. */
int tutti_sched_set_io_time(tutti_sched_t *sched, uint32_t opcode, uint32_t sm_count,
                            uint32_t n_iocb, float us);
int tutti_sched_io_time(const tutti_sched_t *sched, uint32_t opcode, uint32_t sm_count,
                        uint32_t n_iocb, float *us);
/* The profiling pass itself (Section 3.3 "offline profiling ... kernel time and SM occupancy
 * vs IOCB count"; Section 3.4: done once at warm-up).  For every SM count in sm_counts[0..n_sm)
 * (0 = all SMs) it times launches of 1, 2, 4, ... and all of the IOCBs that one layer's build
 * of `batch` fills, with CUDA events on `stream` (minimum of `reps` launches per point), and
 * enters the times into the scheduler's I/O table.  opcode TUTTI_OP_READ times
 * tutti_kv_restore_layer, TUTTI_OP_WRITE tutti_kv_save_layer.  The transfers really run:
 * layer `layer` of the pool (READ) or the batch's objects of that layer (WRITE) are
 * overwritten as by any restore / save.  Blocks the host until done: a warm-up call, not for
 * the per-layer path.  With IOCBs cut by bytes (tutti_ring_set_iocb_bytes) every IOCB is the
 * same work and the table is exact; otherwise it is an average over unequal IOCBs.
 * *n_points (may be NULL): table entries written. */
int tutti_sched_profile(tutti_ctx_t *ctx, tutti_ring_t *ring, tutti_sched_t *sched,
                        const tutti_batch_t *batch, uint32_t layer, uint32_t opcode,
                        const uint32_t *sm_counts, uint32_t n_sm, uint32_t reps, void *stream,
                        uint32_t *n_points);
/* Queue built IOCBs: reads when a request arrives, writes when a layer's KV is produced. */
int tutti_sched_enqueue(tutti_sched_t *sched, uint32_t opcode, uint32_t layer, uint32_t first_iocb,
                        uint32_t n_iocb);
/* Decide what to launch before `layer` begins (prefill) or in a decode step: reads first —
 * as many as fit the window, at least those of layers <= layer — then writes if window
 * is left; the rest stays queued.  Launches are written to out[0..*n_out).  TUTTI_EAGAIN
 * (nothing lost: *n_out is the count needed) if max_out is too small. */
int tutti_sched_next(tutti_sched_t *sched, uint32_t phase, uint32_t layer, uint32_t l_input,
                     uint32_t l_prefix, tutti_launch_t *out, uint32_t max_out, uint32_t *n_out);
int tutti_sched_pending(const tutti_sched_t *sched, uint32_t *reads, uint32_t *writes);

/* ------------------------------------------------------------------------- */
/* CPU-side GPU-file pool (Section 3.1 "Scalable GPU File Pool").  Host only.  */
/* ------------------------------------------------------------------------- */
typedef struct tutti_filepool tutti_filepool_t;

/* Every object slot exists from the start and is free.  Keys are 64-bit hashes of a
 * chunk's token prefix (computed by the engine). */
int tutti_filepool_create(uint64_t n_slots, tutti_filepool_t **out);
int tutti_filepool_destroy(tutti_filepool_t *pool);
/* Slot for a chunk that is about to be saved: the slot it already has (*was_present = 1,
 * shared by every request with that prefix), else the free slot with the lowest id, else
 * the slot of the least recently used unpinned chunk (evicted).  TUTTI_EAGAIN when every
 * slot is pinned. */
int tutti_filepool_insert(tutti_filepool_t *pool, uint64_t key, uint32_t *slot, int *was_present);
int tutti_filepool_lookup(tutti_filepool_t *pool, uint64_t key, uint32_t *slot); /* or TUTTI_ENOENT */
/* Longest stored prefix of a request's chunk keys: slots[0..*n_hit) are filled in chunk
 * order (ready to be a row of tutti_batch_t.obj_slot).  pin != 0 pins every hit slot
 * until tutti_filepool_pin(slot, -1). */
int tutti_filepool_match_prefix(tutti_filepool_t *pool, const uint64_t *keys, uint32_t n_keys,
                                uint32_t *slots, uint32_t *n_hit, int pin);
int tutti_filepool_pin(tutti_filepool_t *pool, uint32_t slot, int delta);
int tutti_filepool_remove(tutti_filepool_t *pool, uint64_t key); /* TUTTI_EAGAIN while pinned */
int tutti_filepool_stats(const tutti_filepool_t *pool, uint64_t *used, uint64_t *free_slots,
                         uint64_t *hits, uint64_t *misses, uint64_t *evictions);

/* Host-side ring accounting on its own (no GPU involved; used by CPU tests):
 * the reservation / release bookkeeping that tutti_build_sqes and tutti_ring_poll
 * apply to IOCB indices and SGL arena ranges. */
typedef struct tutti_hostring tutti_hostring_t;
tutti_hostring_t *tutti_hostring_create(uint32_t depth, uint32_t sgl_capacity);
void tutti_hostring_destroy(tutti_hostring_t *h);
int tutti_hostring_reserve(tutti_hostring_t *h, uint32_t n_iocb, uint32_t n_sgl,
                           uint32_t *first_iocb, uint32_t *sgl_base);
int tutti_hostring_release(tutti_hostring_t *h, uint32_t iocb_idx); /* IOCB polled */
int tutti_hostring_cancel_last(tutti_hostring_t *h, uint32_t first_iocb); /* undo the newest reserve */
int tutti_hostring_live(const tutti_hostring_t *h, uint32_t *iocbs, uint32_t *sgl_entries);

const char *tutti_strerror(int code);
/* Text of the last CUDA failure seen by the calling thread (valid until its next failure). */
const char *tutti_last_cuda_error(void);
uint32_t tutti_version(void);

#ifdef __cplusplus
}
#endif
#endif /* TUTTI_H_ */
