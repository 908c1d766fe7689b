/*
 * pdkv -- block-free transfer of paged KVCache between a prefill pool and a
 * decode pool on one GPU (C ABI).
 *
 * The operations follow P/D-Serve, Sec. 3.5 "Block-free D2D KVCache Transfer":
 * the sender organises a request's discrete KV blocks into one contiguous
 * buffer ("Contiguous Buffer at Sender"), the bytes move as a whole, and the
 * receiver restores discrete blocks from them ("RecvScatter at Receiver").
 * Both sides manage HBM in fixed-size blocks (Sec. 2.3 "Block-fixed
 * Management").  Here both pools live in the same GPU's memory, so a fused
 * blocks-to-blocks call exists beside pack and unpack, and the block-by-block
 * transfer the paper argues against (Sec. 2.3 "Unnecessary Controls") is kept
 * as a timed baseline.
 *
 * Conventions
 *   - Every function returns 0 (PDKV_OK) or a negative pdkv_status.  Nothing
 *     throws, aborts or exits.  pdkv_strerror() names a status; after
 *     PDKV_ERR_CUDA it also carries the CUDA error string of the calling thread.
 *   - "device" pointers are CUDA device addresses on the pool's device; "host"
 *     pointers are ordinary process memory.  The library borrows pools, buffers
 *     and streams from the caller and never frees them.  It owns only a plan's
 *     small device arrays (tile lists), freed by pdkv_plan_destroy().
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *     stream).  pack / unpack / transfer only enqueue work: no allocation, no
 *     host<->device copy, no synchronisation; after one call outside capture
 *     they can be recorded into a CUDA graph (e.g. the per-layer sequence of a
 *     model) and replayed.
 *   - A plan is immutable once created and may be used from any thread: it
 *     carries its own copy of the launch tunables (pdkv_tune) as they stood at
 *     creation, so a later pdkv_tune() -- from this or another thread -- changes
 *     only plans created afterwards.  (pdkv_plan_autotune / pdkv_plan_set_shape
 *     are the two calls that modify a plan; they are set-up calls and must not
 *     run beside launches of the same plan.)
 *   - Elements are opaque: `elem_bytes` bytes are moved bit for bit (NaN
 *     payloads and -0 survive).
 *
 * Pool layouts (b = block id, tt = token slot inside the block)
 *   PDKV_LAYOUT_BLOCK_MAJOR  [block][layer][K/V][token][head][dim]
 *       elem = ((((b*L + l)*2 + c)*B + tt)*H + h)*D + d
 *   PDKV_LAYOUT_LAYER_MAJOR  [layer][K/V][block][head][token][dim]
 *       elem = ((((l*2 + c)*NB + b)*H + h)*B + tt)*D + d
 *
 * Contiguous buffer (Sec. 3.5: the K and V tensors of consecutive layers lie
 * back to back; a layer's offset and length follow from prompt length, hidden
 * size and precision): requests are concatenated in batch order without padding; inside
 * request r the order is [layer][K/V][kept token][head][dim].  With n_r kept
 * tokens, layer l of request r is the byte range
 *       [ off_r + l*2*n_r*H*D*E ,  + 2*n_r*H*D*E ),
 * where off_r is the exclusive prefix sum of 2*L*n_q*H*D*E over earlier
 * requests q.  A layer range [layer_begin, layer_end) touches only those
 * ranges, at the same offsets as a whole-model call.
 *
 * Skip mask: entry j of a request's decode table may be marked resident
 * (shared prefix already on the decode side).  Token t is kept iff entry
 * t / skip_granule_tokens is unmarked; marked blocks are neither packed nor
 * written.  rank_r(t) is the number of kept tokens before t.
 */
#ifndef PDKV_H
#define PDKV_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct pdkv_pool pdkv_pool; /* opaque: geometry + borrowed device base */
typedef struct pdkv_plan pdkv_plan; /* opaque: validated batch + device tile lists */
typedef struct pdkv_queue pdkv_queue; /* opaque: receive slots for asynchronous retrieval */

enum pdkv_layout {
    PDKV_LAYOUT_BLOCK_MAJOR = 0,
    PDKV_LAYOUT_LAYER_MAJOR = 1
};

enum pdkv_status {
    PDKV_OK = 0,
    PDKV_ERR_INVALID_ARG = -1,      /* NULL, negative count, bad layer range, misaligned base */
    PDKV_ERR_GEOMETRY = -2,         /* non-positive sizes; pools disagree on L/H/D/E */
    PDKV_ERR_TABLE = -3,            /* block id out of range, table too short, duplicate decode block */
    PDKV_ERR_BUFFER_TOO_SMALL = -4, /* contiguous buffer smaller than the plan needs */
    PDKV_ERR_CUDA = -5,             /* a CUDA runtime call failed */
    PDKV_ERR_DEVICE_BOUNDS = -6,    /* bounds-checked kernels refused an access (debug option) */
    PDKV_ERR_NOMEM = -7,            /* host allocation failed */
    PDKV_ERR_LIMIT = -8,            /* batch larger than pdkv_transfer_noalloc's built-in scratch */
    PDKV_ERR_BUSY = -9              /* pdkv_queue_submit: every receive slot is taken */
};

enum pdkv_op {
    PDKV_OP_PACK = 0,
    PDKV_OP_UNPACK = 1,
    PDKV_OP_TRANSFER = 2
};

/* Geometry of one block-fixed pool (Sec. 2.3 "Block-fixed Management"). */
typedef struct {
    int32_t layout;       /* enum pdkv_layout */
    int32_t num_layers;   /* L */
    int32_t num_kv_heads; /* H */
    int32_t head_dim;     /* D */
    int32_t elem_bytes;   /* E: 1, 2, 4 or 8 */
    int32_t block_tokens; /* B, any positive value */
    int64_t num_blocks;   /* NB */
} pdkv_pool_desc;

/* One transfer batch.  All arrays are host memory, read only during
 * pdkv_plan_create() (they are copied).  Tables are CSR: request r owns
 * entries [off[r], off[r+1]); it needs at least ceil(seq_len[r] / B) of them
 * and extra entries are ignored.  src_* may be NULL when the plan has no
 * prefill pool, dst_tbl may be NULL when it has no decode pool; dst_tbl_off is
 * still required when dst_skip is given, because the mask is parallel to the
 * decode table. */
typedef struct {
    int32_t n_req;
    const int32_t *seq_len;     /* [n_req] prompt tokens */
    const int64_t *src_tbl_off; /* [n_req+1] */
    const int32_t *src_tbl;     /* prefill block ids; duplicates allowed */
    const int64_t *dst_tbl_off; /* [n_req+1] */
    const int32_t *dst_tbl;     /* decode block ids; a used id may appear once */
    const uint8_t *dst_skip;    /* parallel to dst_tbl; NULL = keep everything */
} pdkv_batch_desc;

/* Bytes the caller must allocate for a pool of this geometry (0 if invalid). */
size_t pdkv_pool_bytes(const pdkv_pool_desc *desc);

/* Wrap caller-owned device memory as a pool.  `dev_base` (device) must be
 * 16-byte aligned and hold at least pdkv_pool_bytes() bytes on CUDA device
 * `device`.  The pool keeps the pointer; it never frees or touches the memory.
 * Errors: INVALID_ARG, GEOMETRY, NOMEM. */
int pdkv_pool_create(const pdkv_pool_desc *desc, void *dev_base, size_t bytes,
                     int device, pdkv_pool **out);
int pdkv_pool_destroy(pdkv_pool *pool);

/* Validate a batch against the pools and build the device-side tile lists --
 * the single-GPU counterpart of the one low-cost meta exchange that precedes a
 * transfer (Sec. 3.5).  `src` or `dst` may be NULL for a pack-only or
 * unpack-only plan (not both).  `skip_granule_tokens` must equal the decode
 * block size when `dst` is given; it is only free for pack-only plans (<= 0
 * selects it from `dst`).  The two pools must not overlap in memory (there is
 * no in-place re-blocking), nor may the contiguous buffer later passed to
 * pack / unpack overlap the pool it is paired with: INVALID_ARG.  One small
 * host->device copy is enqueued on `stream`
 * and the call waits for it; later calls on other streams are therefore safe.
 * Errors: INVALID_ARG, GEOMETRY, TABLE, CUDA, NOMEM; *out is NULL on error. */
int pdkv_plan_create(const pdkv_pool *src, const pdkv_pool *dst,
                     int32_t skip_granule_tokens, const pdkv_batch_desc *batch,
                     void *stream, pdkv_plan **out);
/* As pdkv_plan_create(), but the plan's device arrays (a 256-byte status area
 * and the tile lists) are placed in `workspace` (device, 16-byte aligned,
 * workspace_bytes long) instead of a cudaMalloc'ed block: creation then
 * allocates nothing on the device and pdkv_plan_destroy() frees nothing, which
 * takes cudaMalloc/cudaFree (about 0.3 ms each) off the path of engines that
 * build a plan per transfer.  The workspace belongs to the caller and must stay
 * untouched until the plan is destroyed.  `needed_bytes` (optional) receives
 * the size the batch needs; if the workspace is smaller the call returns
 * PDKV_ERR_BUFFER_TOO_SMALL and creates nothing.  workspace == NULL behaves
 * exactly like pdkv_plan_create(). */
int pdkv_plan_create_in(const pdkv_pool *src, const pdkv_pool *dst,
                        int32_t skip_granule_tokens, const pdkv_batch_desc *batch,
                        void *workspace, size_t workspace_bytes, size_t *needed_bytes,
                        void *stream, pdkv_plan **out);

/* Frees the plan and its device arrays.  Call it once the work enqueued with
 * the plan has completed (its kernels read the tile lists). */
int pdkv_plan_destroy(pdkv_plan *plan);

/* Optional: find the launch shape (threads per CTA, accesses in flight per thread,
 * CTAs per SM) of each operation by timing it on this batch.  The built-in
 * choice is tuned for Llama-shaped geometries (32 KiB tiles of 256-byte rows);
 * other head sizes, head counts or block sizes can run several percent -- for
 * 160-byte rows up to 30% -- faster with a shape that covers one of their tiles
 * in exactly one or two passes.  About ten candidate shapes are launched four
 * times each over all layers of the batch, for pack and unpack (only
 * if `buf` is given: device, at least pdkv_plan_buffer() bytes) and for
 * transfer; a shape replaces the built-in one only if it is more than 2.5%
 * faster.  With a block-major pool the strip skew (see "lc_skew") is also timed
 * the other way round than its stride rule decides, and kept on the same terms;
 * so is the other kernel for tiles that are transposed on the way (register copy
 * against staged transpose, see "variant"; pdkv_plan_launch_shape() shows the outcome).  The operations are the real ones: afterwards `buf` holds the packed
 * layers and the decode pool the transferred layers that were used for timing
 * (with an unpack-only plan `buf` must already hold a packed batch).  The
 * call synchronises `stream` repeatedly; it is meant for set-up time, once per
 * geometry: the result is kept in the plan and, unless "autotune_reuse" is 0,
 * remembered for every later plan of the process with the same pool
 * geometries and tile sizes.  Explicit "threads" / "unroll" tunables override
 * it.  Plans with small tiles (under 8 KiB) are left alone.  (No counterpart in
 * the paper.)  pdkv_plan_shape() reports what a plan uses (zeros: built-in;
 * lc_skew -1: by the stride rule, 0: none, > 0: that many strips).
 * Errors: INVALID_ARG, BUFFER_TOO_SMALL, CUDA. */
int pdkv_plan_autotune(pdkv_plan *plan, void *buf, size_t buf_bytes, void *stream);
int pdkv_plan_shape(const pdkv_plan *plan, int op, int32_t *threads, int32_t *unroll,
                    int32_t *ctas_per_sm, int32_t *lc_skew);
/* Pin the launch shape of one operation of this plan by hand (threads: multiple of
 * 32 up to 1024, clamped to what the register budget allows; unroll: 1, 2, 4 or 8;
 * ctas_per_sm: 1..32); all three zero returns to the built-in choice.  Not
 * thread-safe against launches that use the plan at the same time.
 * Errors: INVALID_ARG. */
int pdkv_plan_set_shape(pdkv_plan *plan, int op, int32_t threads, int32_t unroll,
                        int32_t ctas_per_sm);

/* Size of the contiguous buffer in bytes and, optionally, the host array of
 * n_req+1 request offsets off_r (owned by the plan, valid until destroy). */
int pdkv_plan_buffer(const pdkv_plan *plan, size_t *total_bytes,
                     const int64_t **req_off_bytes);

/* Algorithmic traffic of one whole-model call of `op` (enum pdkv_op):
 * payload bytes read, and payload plus zero-padding bytes written.  Tile
 * metadata is not counted. */
int pdkv_plan_traffic(const pdkv_plan *plan, int op, uint64_t *bytes_read,
                      uint64_t *bytes_written);

/* Sender side, Sec. 3.5 "Contiguous Buffer at Sender": gather every kept token
 * of layers [layer_begin, layer_end) from the prefill pool into `buf` (device,
 * 16-byte aligned, buf_bytes >= pdkv_plan_buffer()).  Bytes of `buf` outside
 * the addressed layer ranges keep their value.
 * Errors: INVALID_ARG, BUFFER_TOO_SMALL, CUDA. */
int pdkv_pack(const pdkv_plan *plan, void *buf, size_t buf_bytes,
              int layer_begin, int layer_end, void *stream);

/* Receiver side, Sec. 3.5 "RecvScatter at Receiver": restore decode blocks of
 * layers [layer_begin, layer_end) from `buf`, then zero the token slots past
 * the prompt's end in each request's last decode block (unless that block is
 * marked resident).  All other bytes of the decode pool are left untouched. */
int pdkv_unpack(const pdkv_plan *plan, const void *buf, size_t buf_bytes,
                int layer_begin, int layer_end, void *stream);

/* Fused blocks-to-blocks: same decode pool image as pdkv_pack followed by
 * pdkv_unpack, without materialising the buffer.  (No counterpart in the
 * paper, whose two pools sit on different devices.) */
int pdkv_transfer(const pdkv_plan *plan, int layer_begin, int layer_end, void *stream);

/* Fused transfer for callers that must not allocate device memory.  (The paper
 * has no counterpart; this is a deployment convenience.)
 *
 * Who needs it: a serving engine that hands all of HBM to its own block
 * allocator at start-up, a process running under a frozen memory pool, or code
 * on a path where cudaMalloc's implicit device-wide synchronisation is not
 * acceptable.  Such callers cannot use pdkv_plan_create(), which allocates the
 * plan's tile list with cudaMalloc.  Here the tile list lives in a fixed array
 * of PDKV_NOALLOC_SCRATCH_BYTES that is part of the library image: every GPU on
 * which the library is used holds those bytes until the process exits, and no
 * cudaMalloc, cudaFree or other allocating CUDA or framework routine is called
 * (host-side bookkeeping uses ordinary heap memory).
 *
 * Arguments are those of pdkv_plan_create() + pdkv_transfer(): two pools, one
 * batch (host arrays, read during the call), a layer range and a stream.  The
 * decode pool receives exactly what pdkv_transfer() would write.
 *
 * Limits and caveats
 *   - The batch may need at most PDKV_NOALLOC_MAX_TILES tiles (see
 *     pdkv_plan_tiles(); roughly kept_tokens * H*D*E / "tile_bytes", plus one
 *     per block boundary); beyond that PDKV_ERR_LIMIT is returned and nothing
 *     is enqueued.  Raise "tile_bytes" or split the batch.
 *   - The first call on each device looks up the device address of the scratch
 *     array (with that device current) and loads the library's device image;
 *     make it once at start-up, before HBM is handed to the engine's allocator.
 *   - The call stages the tile list from host memory that it frees on return,
 *     so it cannot be recorded: when `stream` is capturing it returns
 *     INVALID_ARG and enqueues nothing.  Graph users need plans
 *     (pdkv_plan_create_in places one in caller-owned memory).
 *   - Launch shape, work order and strip skew come from the same chooser as
 *     pdkv_transfer() with the tunables as they stand at the call; "variant"
 *     and "debug_bounds" are not honoured (register-copy kernel, no checks).
 *   - Every call on a device reuses the same scratch, which still holds the
 *     previous call's tiles; the call rewrites what it needs (including the
 *     words that must start at zero) on `stream` before its kernel runs.  Two
 *     calls whose GPU work can overlap (different streams without an ordering
 *     between them) race on it, and so do two host threads that enqueue on the
 *     same stream at the same time (their clear / copy / kernel steps may
 *     interleave): order them, or use plans.
 *   - The tile list is copied from pageable host memory, so the call may block
 *     until earlier work on `stream` has finished.
 * Errors: INVALID_ARG, GEOMETRY, TABLE, LIMIT, CUDA, NOMEM. */
#define PDKV_NOALLOC_MAX_TILES 32768
#define PDKV_NOALLOC_SCRATCH_BYTES (256 + PDKV_NOALLOC_MAX_TILES * 24)
int pdkv_transfer_noalloc(const pdkv_pool *src, const pdkv_pool *dst,
                          const pdkv_batch_desc *batch, int layer_begin, int layer_end,
                          void *stream);

/* Baseline: the block-by-block transfer that Sec. 2.3 describes as the natural
 * consequence of block-fixed pools, one copy or one kernel launch per prefill block issued from a host loop.
 * Same result as pdkv_transfer over all layers. */
int pdkv_transfer_blockwise(const pdkv_plan *plan, void *stream);

/* The fused transfer of layers [layer_begin, layer_end) issued as plain device copies
 * (cudaMemcpyAsync per prefill block, 2-D copies and memsets for a partial last block)
 * instead of a kernel, for plans whose two pools are both block-major with the same
 * block size: there a block's layer range is one contiguous byte range on either side.
 * Same decode pool image as pdkv_transfer().  Such copies may be served by the GPU's copy
 * engines and then take no SM from kernels that run beside them -- the no-interference
 * form of the per-layer trigger (Sec. 3.5) -- at the price of one host call per block,
 * the control cost Sec. 2.3 describes.
 * Errors: INVALID_ARG, GEOMETRY (other layouts or unequal block sizes), CUDA. */
int pdkv_transfer_copies(const pdkv_plan *plan, int layer_begin, int layer_end, void *stream);

/* Host-resident pools.  `host_src_pool` / `host_dst_pool` (host; pinned memory
 * makes the copies asynchronous) are byte images of the prefill / decode pool
 * with the pool's own geometry.  pdkv_upload_blocks() copies every prefill
 * block that holds at least one kept token of the batch into the device pool
 * at the same offsets; pdkv_download_blocks() copies every decode block the
 * batch writes back out.  Consecutive block ids travel as one (pitched) copy;
 * other bytes of either image are not touched.  Both only enqueue on
 * `stream`.  With pack / unpack / transfer in between, this is the whole path
 * for a caller whose KV lives in host memory.  (No counterpart in Sec. 3.5,
 * which moves device to device; the paper's discussion section mentions a
 * host-memory KV pool as orthogonal work.)
 * pdkv_plan_block_bytes() reports the bytes each of the two calls moves.
 * Errors: INVALID_ARG, CUDA. */
int pdkv_upload_blocks(const pdkv_plan *plan, const void *host_src_pool, void *stream);
int pdkv_download_blocks(const pdkv_plan *plan, void *host_dst_pool, void *stream);
int pdkv_plan_block_bytes(const pdkv_plan *plan, uint64_t *src_bytes, uint64_t *dst_bytes);

/* Asynchronous retrieval, Sec. 3.5: the decode side has little room for
 * incoming KVCache, so the space forms a small queue of `capacity` (1..64)
 * receive slots; retrieval runs concurrently with decoding and a completed
 * request triggers the next retrieval, on demand.
 *
 *   pdkv_queue_create   one non-blocking stream and one event per slot on
 *                       `device`; the pools are borrowed until destroy.
 *   pdkv_queue_submit   takes a free slot, builds the plan for `batch` (host
 *                       arrays, read during the call) and enqueues the fused
 *                       transfer over all layers on the slot's stream --
 *                       preceded by pdkv_upload_blocks() if `host_src_pool` is
 *                       given and followed by pdkv_download_blocks() if
 *                       `host_dst_pool` is given (either may be NULL).  A slot's
 *                       stream is ordered after nothing the caller has enqueued:
 *                       pass in `wait_event` (a cudaEvent_t as void*, or NULL) an
 *                       event recorded after the work that produces the prefill
 *                       blocks and after the last reader of the decode blocks
 *                       about to be overwritten -- the slot waits for it on the
 *                       device -- or synchronise with that work on the host
 *                       before the call.  Returns a ticket.  If every slot is taken it returns PDKV_ERR_BUSY at
 *                       once and enqueues nothing: nothing waits inside the library,
 *                       the caller retries when a request completes.
 *   pdkv_queue_poll     *done = 1 once the slot's transfer has finished (its
 *                       decode blocks are valid for the next decode iteration).
 *   pdkv_queue_wait     blocks the calling thread until then.
 *   pdkv_queue_release  hands the slot back (waits for the transfer if it is
 *                       still running); the ticket becomes invalid.
 *   pdkv_queue_stats    capacity, slots in use, accepted and rejected submits.
 * Concurrent tickets must write disjoint decode blocks (the caller's block
 * allocator guarantees that).  Calls on one queue are serialised by a mutex.
 * Errors: INVALID_ARG (unknown ticket, bad arguments), BUSY, and whatever
 * pdkv_plan_create / pdkv_transfer return. */
int pdkv_queue_create(const pdkv_pool *src, const pdkv_pool *dst, int device, int capacity,
                      pdkv_queue **out);
int pdkv_queue_submit(pdkv_queue *queue, const pdkv_batch_desc *batch, const void *host_src_pool,
                      void *host_dst_pool, void *wait_event, int64_t *ticket);
int pdkv_queue_poll(pdkv_queue *queue, int64_t ticket, int *done);
int pdkv_queue_wait(pdkv_queue *queue, int64_t ticket);
int pdkv_queue_release(pdkv_queue *queue, int64_t ticket);
int pdkv_queue_stats(const pdkv_queue *queue, int *capacity, int *in_use, int64_t *submitted,
                     int64_t *rejected);
int pdkv_queue_destroy(pdkv_queue *queue);

/* SM partition for the per-layer trigger (Sec. 3.5: the transfer of layer l runs while
 * layer l+1 computes, and as an operator it must not hold the other operators up).
 * pdkv_sm_partition_create() splits the SMs of `device` into a transfer share of
 * about `transfer_sms` (the driver rounds it up to its granularity, 8 on sm_90 and
 * later) and the rest, as two CUDA green contexts of this process, each with one
 * non-blocking stream: kernels enqueued on stream 0 (`which` = 0) run only on the
 * transfer SMs, kernels on stream 1 only on the others, so neither waits for a CTA
 * slot of the other.  Streams belong to the partition; use them like any
 * cudaStream_t.  A pack / unpack / transfer call given a partition's stream sizes
 * its persistent grid to that partition's SMs ("ctas_per_sm" CTAs on each) by itself.
 * Nothing outlasts the process and no device setting changes.  (No counterpart in
 * the paper, whose transfer engine is not the compute device.)
 * Errors: INVALID_ARG, NOMEM, CUDA (driver without green contexts, or a split the
 * device refuses). */
typedef struct pdkv_sm_partition pdkv_sm_partition;
int pdkv_sm_partition_create(int device, int transfer_sms, pdkv_sm_partition **out);
int pdkv_sm_partition_info(const pdkv_sm_partition *partition, int *transfer_sms, int *compute_sms);
int pdkv_sm_partition_stream(const pdkv_sm_partition *partition, int which, void **stream);
int pdkv_sm_partition_destroy(pdkv_sm_partition *partition);

/* Number of GPU operations (kernel launches + memcpys) one call of `op`
 * enqueues; op = 3 asks about pdkv_transfer_blockwise. */
int pdkv_plan_launches(const pdkv_plan *plan, int op, int64_t *launches);

/* One entry of a plan's tile list, for inspection and host-side tests: `ntok`
 * consecutive kept tokens of one request lying inside one block on every paged
 * side.  Offsets are bytes from the side's base for layer 0 / K; (l, c) adds
 * (2*l + c) times the side's per-(l,c) stride, which for the contiguous buffer
 * is n_kept*H*D*E.  src_off < 0 marks a zero-fill tile (tail slots). */
typedef struct {
    int64_t src_off;
    int64_t dst_off;
    int32_t ntok;
    int32_t n_kept;
} pdkv_tile;

/* Host copy of the tile list of `op`, owned by the plan. */
int pdkv_plan_tiles(const pdkv_plan *plan, int op, const pdkv_tile **tiles, int64_t *n_tiles);

/* Synchronise `stream` and report the plan's device status word: PDKV_OK,
 * PDKV_ERR_DEVICE_BOUNDS (with "debug_bounds": an access was refused and
 * skipped; with "variant" 1: a bounded wait on a bulk copy gave up and the
 * kernel returned early) or PDKV_ERR_CUDA. */
int pdkv_plan_status(const pdkv_plan *plan, void *stream);

/* What a plan will launch for `op` over layers [layer_begin, layer_end): the
 * result of the library's chooser (class of copy, tile sizes, stride rule,
 * autotuned or pinned shape) applied to the tunables frozen in the plan.  Works
 * on host-only ("dry_run") plans too.  pdkv_plan_option() reads one frozen
 * tunable by its pdkv_tune() key.  Errors: INVALID_ARG. */
typedef struct {
    int32_t threads, unroll, ctas_per_sm, group_threads, vec_bytes, max_ctas;
    int32_t lc_skew, lc_skew_shift, lc_fastest, chunked, src_order, variant, debug_bounds;
} pdkv_launch_shape;
int pdkv_plan_launch_shape(const pdkv_plan *plan, int op, int layer_begin, int layer_end,
                           pdkv_launch_shape *out);
int pdkv_plan_option(const pdkv_plan *plan, const char *key, int64_t *value);

/* Process-wide tunables: the defaults of plans created afterwards.  pdkv_plan_create()
 * copies them into the plan (pdkv_transfer_noalloc() reads them at the call); changing
 * them never affects a plan that already exists.
 *   "tile_bytes"     target bytes moved per tile (default 32768)
 *   "ctas_per_sm"    persistent CTAs per SM; 0 (default) = automatic: 2, or 3 for row-permuting
 *                    copies of 12-16 KiB tiles (which then run 256 threads x 2 accesses)
 *   "max_ctas"       cap on the grid size, 0 = none (default).  A small grid
 *                    leaves most SMs to other kernels of the process at a
 *                    proportionally lower copy rate
 *   "threads"        threads per CTA, multiple of 32, clamped to what the register
 *                    budget of the chosen variant allows; 0 = automatic (default)
 *   "unroll"         independent accesses in flight per thread: 1, 2, 4, 8;
 *                    0 = automatic (default).  Automatic means 512 threads x 1
 *                    access for flat copies (token-major on both sides) and for
 *                    batches of small tiles, 256 threads x 4 for full-tile
 *                    copies with a head-major side
 *   "group_threads"  threads that cooperate on one work item (a CTA hosts
 *                    threads / group_threads independent groups); 0 = automatic
 *                    (default): sized so that the plan's mean tile is covered in
 *                    one or two passes, 32 at least
 *   "vec32"          1: use 32-byte accesses when rows and bases allow (default 1)
 *   "lc_fastest"     1: consecutive work items walk the (layer, K/V) strips of
 *                    one tile; 0: they walk the tiles of one strip (default 0)
 *   "lc_skew"        with "lc_fastest" 0, one sweep of the grid moves the same
 *                    (layer, K/V) strip of every tile.  A skew S (a power of two)
 *                    lets tile t take strip (s + ((t >> "lc_skew_shift") mod S))
 *                    mod n_strips in sweep s instead, so that neighbouring blocks
 *                    are read at different offsets.  0: off; -1 (default):
 *                    automatic -- 16 for calls that read (else write) a block-major
 *                    pool whose block stride is a power of two times a multiple of
 *                    3, 5 or 17 (B200's DRAM handles same-offset accesses at such strides
 *                    2-12% slower), off otherwise; the register-copy kernels
 *                    honour it, the bulk-copy variants ignore it
 *   "lc_skew_shift"  used with an explicit "lc_skew": tiles whose index agrees above
 *                    this many low bits share a skew (keep the tiles of one prefill
 *                    block together); chosen automatically with "lc_skew" -1
 *   "chunked"        1: each CTA takes one contiguous run of work items instead
 *                    of every gridDim-th one (default 0)
 *   "src_order"      order in which the threads of a CTA walk the rows of a tile whose
 *                    two sides differ in order (one token-major, one head-major): 0 in
 *                    the order of the side written, 1 of the side read, -1 (default)
 *                    automatic: read order unless a row (D*E bytes) is a multiple of 256
 *                    bytes (measured: lone reads of other row sizes cost 3-13%, and rows that
 *                    are not whole 64-byte sector pairs fetch more DRAM bytes than they use)
 *   "debug_bounds"   1: kernels range-check every access and skip bad ones
 *   "debug_shrink"   with "debug_bounds": pretend each side is N bytes shorter, so
 *                    that the refusal path can be exercised on valid memory
 *   "variant"        kernel family.  -1 (default): chosen per call -- the register copy (0),
 *                    except that tiles going from a token-major side to a head-major one in
 *                    rows of more than 128 bytes that are not multiples of 256, 24 KiB or more
 *                    per tile, run the staged transpose (3).  0: register copy.  1: bulk async copies (TMA)
 *                    through shared memory, one warp per CTA; used when rows are multiples
 *                    of 16 bytes and a tile fits a stage, else variant 0 runs.  2: as 1, and
 *                    tiles whose two sides differ in order (one token-major, one head-major)
 *                    are moved with tiled TMA loads or stores through a tensor map of the
 *                    token-major side (one per head instead of one bulk copy per row) when
 *                    the geometry meets the TMA rules.  3: staged transpose for tiles whose
 *                    two sides differ in order: bulk loads (TMA) fetch the tile in the order
 *                    of the side that is read into a ring of shared-memory stages, all
 *                    threads of the CTA store it in the order of the side that is written,
 *                    so both sides see contiguous runs; other tiles run variant 0
 *   "stages"         variants 1 to 3: shared-memory stages per CTA, 2..16 (default 3);
 *                    stages x "tile_bytes" must fit in 220 KiB
 *   "autotune_reuse" 1 (default): a new plan starts with the shapes that an earlier
 *                    pdkv_plan_autotune() found for the same geometry
 *   "dry_run"        1: pdkv_plan_create builds host-only plans (no CUDA call is
 *                    made; the plan can be inspected but not launched)
 * Unknown keys or out-of-range values give INVALID_ARG. */
int pdkv_tune(const char *key, int64_t value);
int pdkv_tune_get(const char *key, int64_t *value);

const char *pdkv_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* PDKV_H */
