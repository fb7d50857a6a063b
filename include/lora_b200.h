/*
 * lora_b200 -- unmerged multi-adapter LoRA forward for NVIDIA B200 (sm_100a).
 *
 *     y[t, :] = y_base[t, :] + s_i * (x[t, :] . A_i) . B_i ,      i = slot_idx[t]
 *
 * A LoRA adapter is a pair of low-rank matrices per adapted projection whose
 * activations are added to the output of the backbone projection (paper
 * Section 2.2).  Serving systems keep the adapters unmerged so that hundreds of
 * them share one backbone, run several of them inside one batch, hold them in a
 * statically reserved GPU region of A_max slots with one uniform footprint
 * S_max each, and swap missing ones in from CPU memory (paper Sections 1, 2.2
 * and the adapter-cache / Lat_load stage of Section 5, Eq. 1).  This library is
 * that per-projection computation and the slot pool around it:
 *
 *   lora_pool_create      the A_max x S_max slot pool in caller-owned device memory
 *   lora_pool_load_slot   side-stream swap-in of one adapter from pinned host memory
 *   lora_build_segments   integer metadata: tokens grouped by adapter slot, cut in tiles
 *   lora_bgmv_apply       decode batches (one token per request)
 *   lora_sgmv_apply       prefill / chunked-prefill batches (per-adapter segments)
 *
 * Conventions
 *  - plain C ABI; every call returns a lora_status_t; nothing aborts, traps or resets a device;
 *  - "dev" pointers are device memory, "host" pointers are host memory; all buffers are owned
 *    by the caller and must stay valid until the work queued on the stream has finished;
 *  - streams are cudaStream_t values passed as void*; all GPU work is asynchronous on the
 *    stream given; the library never synchronises a device and never allocates device memory;
 *  - bf16 tensors are row-major with a leading dimension in ELEMENTS; base pointers must be
 *    16-byte aligned and every d_in, d_out and leading dimension a multiple of 8;
 *  - arithmetic: bf16 inputs, fp32 accumulation, one round-to-nearest-even to bf16 at the store;
 *  - a pool handle keeps host-side state (slot table copy, events, tensor maps, the shapes of the
 *    metadata tables built through it) and is not thread-safe: calls on one pool come from one
 *    host thread at a time.  Different pools are independent.
 */
#ifndef LORA_B200_H
#define LORA_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    LORA_OK = 0,
    LORA_ERR_INVALID_ARG = 1,      /* null pointer, bad enum, misaligned or overlapping buffers */
    LORA_ERR_SHAPE = 2,            /* dimension not a multiple of 8, negative sizes */
    LORA_ERR_SLOT_RANGE = 3,       /* slot >= num_slots or < 0 */
    LORA_ERR_RANK = 4,             /* rank < 1 or rank > r_max */
    LORA_ERR_NOT_LOADED = 5,       /* operation needs an occupied slot (slot policy calls) */
    LORA_ERR_BUSY = 6,             /* every candidate slot is pinned by an in-flight batch */
    LORA_ERR_BUFFER_TOO_SMALL = 7, /* caller buffer smaller than the matching *_bytes query */
    LORA_ERR_NOT_PINNED = 8,       /* host adapter memory is pageable */
    LORA_ERR_CUDA = 9,             /* a CUDA runtime call failed: see lora_last_cuda_error() */
    LORA_ERR_TIMEOUT = 10          /* a bounded device-side wait expired (lora_pool_check_status) */
} lora_status_t;

const char *lora_status_string(lora_status_t s);
/* cudaError_t value of the most recent failing runtime call made by this thread's last call. */
int32_t lora_last_cuda_error(void);
/* Number of kernels this library has launched since it was loaded (all pools, all threads). */
int64_t lora_launch_count(void);

/* ----------------------------------------------------------------------------------------
 * Slot pool (paper Section 2.2: a fixed region for adapter weights, at most A_max adapters
 * loaded at once, every adapter given the same maximum footprint S_max).
 * num_slots = A_max; r_max = the rank that S_max is sized for.
 * -------------------------------------------------------------------------------------- */
typedef struct lora_pool lora_pool_t;

typedef struct {
    int32_t d_in;    /* input width of the adapted projection  (multiple of 8) */
    int32_t d_out;   /* output width of the adapted projection (multiple of 8) */
} lora_target_t;

typedef struct {
    int32_t device;               /* CUDA device ordinal the pool lives on */
    int32_t num_slots;            /* A_max, 1 .. 8192 */
    int32_t r_max;                /* largest rank a slot can hold, 1 .. 64 */
    int32_t num_targets;          /* adapted projections (e.g. 7 per layer x 32 layers) */
    const lora_target_t *targets; /* host, [num_targets]; copied */
    void *device_buf;             /* dev, 256-byte aligned, >= lora_pool_bytes(); caller-owned */
    size_t device_buf_bytes;
} lora_pool_desc_t;

/* Bytes of device memory a pool of this shape needs (control block with the slot table and the
 * targets' tensor maps + transpose staging + num_slots slots of r_max rows for every target's
 * A and B).  device_buf is ignored. */
lora_status_t lora_pool_bytes(const lora_pool_desc_t *desc, size_t *bytes);

/* Creates the host handle and clears the pool's control block (slot table: all slots empty;
 * status words: zero).  Synchronous: returns after the clear has completed.  The handle is
 * owned by the library; the device memory stays the caller's and must outlive the handle. */
lora_status_t lora_pool_create(const lora_pool_desc_t *desc, lora_pool_t **out);
lora_status_t lora_pool_destroy(lora_pool_t *pool);

enum { LORA_A_DIN_MAJOR = 0,   /* A given as [d_in, rank] row-major (the formula's orientation) */
       LORA_A_RANK_MAJOR = 1,  /* A given as [rank, d_in] row-major (already in slot layout)    */
       LORA_PACKED = 2         /* A[0] is ONE pinned buffer (16-byte aligned) holding, for every
                                  target in order, A as [rank, d_in] then B as [rank, d_out]; the
                                  other pointers are ignored.  With rank == r_max this is the slot's
                                  own layout and the swap-in is a single DMA. */ };

typedef struct {
    int32_t rank;            /* 1 .. r_max */
    float scale;             /* s_i */
    const void *const *A;    /* host, [num_targets] pointers to pinned bf16 matrices, see a_layout */
    const void *const *B;    /* host, [num_targets] pointers to pinned bf16 [rank, d_out] row-major */
    int32_t a_layout;        /* LORA_A_DIN_MAJOR, LORA_A_RANK_MAJOR or LORA_PACKED */
    int32_t trust_pinned;    /* non-zero: skip the per-pointer pinned-memory check */
} lora_adapter_host_t;

/*
 * Swap one adapter into a slot (paper Section 5: the adapter-cache stage loads missing
 * adapters from CPU memory; its cost is Lat_load in Eq. 1).  Queues on load_stream:
 *   wait until everything queued so far on compute_stream has finished (the slot may still be
 *   read), mark the slot empty, copy A and B for every target, zero the padding rows
 *   rank .. r_max - 1, mark the slot occupied with (rank, scale), record the slot's ready event.
 * Inside a slot every matrix is stored rank-major: A as [r_max, d_in], B as [r_max, d_out],
 * rows 0 .. rank-1 meaningful, the rest zero.  LORA_A_DIN_MAJOR input is transposed on the device.
 * Host matrices must stay valid until the ready event has fired (lora_pool_acquire + stream
 * completion, or a synchronise on load_stream).  compute_stream may be NULL when no reader
 * can be in flight.  All loads of one pool go through ONE load stream (LORA_A_DIN_MAJOR input
 * passes through a staging area of the pool that consecutive loads reuse in stream order).
 * On an argument error (every code below but CUDA) the slot is left untouched; after a CUDA error
 * in the middle of the sequence the slot is empty on the device and in the host's view.
 * Errors: INVALID_ARG, SLOT_RANGE, RANK, NOT_PINNED, CUDA.
 */
lora_status_t lora_pool_load_slot(lora_pool_t *pool, int32_t slot, const lora_adapter_host_t *adapter,
                                  void *load_stream, void *compute_stream);

/* Marks a slot empty (same ordering as a load: waits for compute_stream's queued readers). */
lora_status_t lora_pool_evict_slot(lora_pool_t *pool, int32_t slot, void *load_stream,
                                   void *compute_stream);

/* Makes compute_stream wait for the ready events of these slots (host array of n slot ids).
 * Slots that were never loaded are skipped.  Errors: SLOT_RANGE, CUDA. */
lora_status_t lora_pool_acquire(lora_pool_t *pool, const int32_t *slots_host, int32_t n,
                                void *compute_stream);

/* Copies one slot's stored matrices of one target back to host memory (A_host: [r_max, d_in],
 * B_host: [r_max, d_out], bf16) on `stream`; either pointer may be NULL.  For inspection. */
lora_status_t lora_pool_read_slot(lora_pool_t *pool, int32_t slot, int32_t target,
                                  void *A_host, void *B_host, void *stream);

/* Host-side view of a slot as of the last load/evict call: rank (0 when empty) and scale. */
lora_status_t lora_pool_slot_info(const lora_pool_t *pool, int32_t slot, int32_t *rank, float *scale);

/* Device status words, copied asynchronously to host_out[4] (pinned host memory) on `stream`:
 * [0] tokens whose slot id was neither -1 nor an occupied slot (accumulated; such tokens are
 * treated as -1), [1] expired device-side waits, [2..3] reserved. */
lora_status_t lora_pool_poll_status(lora_pool_t *pool, int32_t *host_out, void *stream);
lora_status_t lora_pool_reset_status(lora_pool_t *pool, void *stream);

/* The one call that waits: copies the status words back on `stream`, synchronises that stream and
 * returns LORA_ERR_TIMEOUT when word 1 is non-zero (some block of some kernel gave up a bounded
 * wait and stored no result for its rows: the outputs of the applies queued since the last reset
 * are not to be trusted), LORA_OK otherwise.  words_out (host, [4]) may be NULL.  The apply calls
 * themselves are asynchronous and cannot report this; call it wherever a step's results are
 * consumed on the host, or once per step in a server loop. */
lora_status_t lora_pool_check_status(lora_pool_t *pool, void *stream, int32_t *words_out);

/* Exercises the time-out path without disturbing anything: launches ONE block that polls an
 * mbarrier nobody completes, `polls` times (1 .. 2^20), then records the expiry in status word 1
 * exactly as the apply kernels do and returns without writing *witness_dev (dev int32, may be
 * NULL; it is written only if the wait had succeeded).  For tests and for monitoring code that
 * wants to see its own alarm fire. */
lora_status_t lora_pool_selftest_wait_expiry(lora_pool_t *pool, int32_t polls, int32_t *witness_dev,
                                             void *stream);

/* Tuning knobs, for measurement (0 = the default behaviour for every key):
 *   key 0  apply path: 1 = two-phase CUDA-core kernels with the fp32 workspace
 *   key 1  fused kernel: blocks per cluster (1, 2, 4, 8)
 *   key 2  programmatic dependent launch of the fused kernel: 2 = never
 *   key 3  fused kernel: upper bound on the clusters in the grid
 *   key 4  tensor-core kernels of lora_sgmv_apply: 1 = never, 2 = whenever they apply (read by
 *          lora_build_segments, which writes their tile list, and by the apply)
 *   key 5  fused kernel: stages of the shared-memory ring (2 .. 4)
 *   key 6  lora_sgmv_apply: 1 = the tiles the tensor-core kernels leave over run after them on the
 *          caller's stream, not beside them on the pool's own stream
 *   key 7  segment builder: 1 = one warp per slot also for long batches
 *   key 8  tensor-core expand of lora_sgmv_apply: blocks per SM in its grid (0 = the default, 8)
 *   key 9  fused kernel: share (1 .. 99 %) of the resident clusters one launch may take
 *   key 10 1 = decode batches take the general fused kernel, not the decode kernel
 *   key 11 when a fused kernel lets its successor on the stream become resident: 1 = only at its
 *          end, 2 = at its start (default: at its start for launches of fewer than four projections)
 * Keys outside 0 .. 15 -> INVALID_ARG. */
lora_status_t lora_pool_set_tuning(lora_pool_t *pool, int32_t key, int32_t value);

/* ----------------------------------------------------------------------------------------
 * Slot policy and pool sizing (paper Section 1: adapters move between CPU and GPU memory
 * according to their usage; Section 2.2: A_max slots of one footprint S_max; Section 5: the
 * adapter-cache stage of a step loads what the scheduled batch needs).  Host-side bookkeeping
 * only: no CUDA call is made, and a policy object is independent of any pool.  Adapter ids are
 * the caller's non-negative 64-bit keys.  "Least recently used" follows a logical clock advanced
 * by every use, so decisions are a deterministic function of the call sequence.  A pinned slot
 * (pin count > 0: an in-flight batch's metadata references it) is never chosen as a victim.
 * Not thread-safe.
 * -------------------------------------------------------------------------------------- */
typedef struct lora_policy lora_policy_t;
lora_status_t lora_policy_create(int32_t num_slots, lora_policy_t **out);
lora_status_t lora_policy_destroy(lora_policy_t *policy);
/* *slot_out = the slot holding the adapter, or -1. */
lora_status_t lora_policy_lookup(const lora_policy_t *policy, int64_t adapter, int32_t *slot_out);
/* What a slot holds (-1: empty) and its pin count; either pointer may be NULL. */
lora_status_t lora_policy_slot(const lora_policy_t *policy, int32_t slot, int64_t *adapter_out,
                               int32_t *pins_out);
/* Marks the slot most recently used.  Errors: SLOT_RANGE, NOT_LOADED (empty slot). */
lora_status_t lora_policy_touch(lora_policy_t *policy, int32_t slot);
/* Pin / unpin the n slots of a host array (a slot named twice is pinned twice).  All or nothing.
 * Errors: SLOT_RANGE, NOT_LOADED (pin of an empty slot), INVALID_ARG (unpin below zero). */
lora_status_t lora_policy_pin(lora_policy_t *policy, const int32_t *slots_host, int32_t n);
lora_status_t lora_policy_unpin(lora_policy_t *policy, const int32_t *slots_host, int32_t n);
/* The slot to fill next: the lowest empty unpinned slot, else the unpinned slot used longest ago
 * (ties: lowest index); *evicted_out (may be NULL) = the adapter it holds now, or -1.  Changes
 * nothing.  Errors: BUSY (every slot is pinned). */
lora_status_t lora_policy_choose_victim(const lora_policy_t *policy, int32_t *slot_out,
                                        int64_t *evicted_out);
/* Records that `adapter` now lives in `slot` (after lora_pool_load_slot), replacing what was
 * there, and marks it used.  Errors: SLOT_RANGE, BUSY (slot pinned), INVALID_ARG (the adapter is
 * resident in another slot). */
lora_status_t lora_policy_assign(lora_policy_t *policy, int32_t slot, int64_t adapter);
/* Records that the slot is empty (after lora_pool_evict_slot).  Errors: NOT_LOADED, BUSY. */
lora_status_t lora_policy_release(lora_policy_t *policy, int32_t slot);
/* The adapter-cache stage for one batch: adapters[i] is request i's adapter (-1: none).
 * Writes slot_idx_out[i] (host, [n]; -1 for requests without adapter) and the loads the caller
 * has to queue with lora_pool_load_slot before the batch's metadata is built: miss_slots_out[k],
 * miss_adapters_out[k], k < *n_miss_out, in order of first appearance in the batch.  Victims are
 * chosen as by lora_policy_choose_victim among slots the batch itself does not use; every slot of
 * the batch is marked used.  On error nothing has changed.
 * Errors: BUSY (more distinct adapters than slots that are free or may be evicted: the scheduler
 * has to defer requests, the A_max limit of paper Section 5), BUFFER_TOO_SMALL (miss_cap). */
lora_status_t lora_policy_admit(lora_policy_t *policy, const int64_t *adapters, int32_t n,
                                int32_t *slot_idx_out, int32_t *miss_slots_out,
                                int64_t *miss_adapters_out, int32_t miss_cap, int32_t *n_miss_out);
/* Counters since creation: distinct resident adapters found per batch, loads asked for, adapters
 * displaced.  Any pointer may be NULL. */
lora_status_t lora_policy_stats(const lora_policy_t *policy, int64_t *hits, int64_t *misses,
                                int64_t *evictions);

/* Sizing: the largest num_slots (A_max) whose pool fits in bytes_budget for these targets at this
 * r_max (S_max), and the bytes one more slot costs.  Errors: BUFFER_TOO_SMALL (not even one slot),
 * plus those of lora_pool_bytes. */
lora_status_t lora_pool_plan(size_t bytes_budget, const lora_target_t *targets, int32_t num_targets,
                             int32_t r_max, int32_t *num_slots_out, size_t *bytes_per_slot_out);

/* ----------------------------------------------------------------------------------------
 * Segment metadata (several adapters are served inside one batch, paper Section 2.2; each
 * request names its adapter, Section 5): a stable group-by-slot of the batch's tokens.
 *
 * Output buffer `meta_dev`, all int32, in this order (N = num_slots,
 * cap_seg = min(T, N), cap_tile = cap_seg + T / tile_m):
 *   header[16]   {T, n_active, n_invalid, n_seg, n_tile, tile_m, long_min, N, cap_seg, cap_tile, 0..}
 *   perm[T]      active tokens ordered by (slot, token id), then the other tokens ascending
 *   seg_slot[cap_seg], seg_start[cap_seg + 1], seg_rank[cap_seg], seg_flags[cap_seg]
 *                flags bit0: the segment's tokens are consecutive ids; bit1: length >= long_min
 *   tile_seg[cap_tile], tile_row0[cap_tile], tile_rows[cap_tile]
 *                each segment cut into pieces of at most tile_m rows (positions in perm)
 *   (then words private to the library: one flag word per tile, and from the next 16-byte
 *    boundary a 4-word record per
 *    tile, a 4-word record plus 16 row ids per piece of at most 16 rows of a tile, and the
 *    list of the tiles lora_sgmv_apply gives to its tensor-core kernels (written by a second
 *    small launch when the batch qualifies for them); lora_segments_bytes counts them)
 * Unused entries are -1.  A token is active iff its slot id names an occupied slot; a token
 * that is neither active nor -1 is invalid (counted in header and in the pool's status word 0).
 * The result is an exact integer function of its inputs.
 * -------------------------------------------------------------------------------------- */
lora_status_t lora_segments_bytes(int32_t T, int32_t num_slots, int32_t tile_m, size_t *bytes);

/* slot_idx_dev: dev int32 [T]; meta_dev: dev, 16-byte aligned, meta_bytes >= lora_segments_bytes.
 * tile_m in 1 .. 128, long_min >= 1.  T == 0 writes an empty table.  Uses the slot table as it is
 * on the device when the kernel runs.  Errors: INVALID_ARG, SHAPE, BUFFER_TOO_SMALL, CUDA. */
lora_status_t lora_build_segments(lora_pool_t *pool, const int32_t *slot_idx_dev, int32_t T,
                                  int32_t tile_m, int32_t long_min,
                                  void *meta_dev, size_t meta_bytes, void *stream);

/* ----------------------------------------------------------------------------------------
 * The forward itself.  x: bf16 [T, d_in]; y_base: bf16 [T, d_out] (the backbone projection's
 * output, computed by the caller); y: bf16 [T, d_out], either exactly y_base (in place) or
 * not overlapping it.  Tokens without an active slot get y = y_base bit for bit.  Row t of y
 * depends only on row t of x and y_base, the token's slot and the pool.
 * workspace: dev scratch of >= lora_workspace_bytes(pool, T) bytes (fp32 partial products
 * v = x . A_i between the two phases of the tensor-core and two-phase kernels; the fused
 * kernels keep v on chip), contents undefined afterwards; calls sharing a workspace must be ordered on
 * one stream.
 * Ordering: every apply is ordered behind the lora_build_segments call that wrote its table.
 * Later applies on the same table may start reading the table and the pool (never x or y_base)
 * while the kernel queued before them on the stream is still running, so nothing queued between
 * two applies may write the table or the pool without an event or a rebuild in between (slot
 * loads go through lora_pool_load_slot / lora_pool_acquire, which order themselves).
 * T == 0 returns LORA_OK without launching.
 * Errors: INVALID_ARG, SHAPE, SLOT_RANGE (target), BUFFER_TOO_SMALL, CUDA.
 * -------------------------------------------------------------------------------------- */
lora_status_t lora_workspace_bytes(const lora_pool_t *pool, int32_t T_max, size_t *bytes);

/* Decode batches.  meta_dev_or_null: metadata built from the same slot_idx_dev (tile_m <= 16)
 * so that each adapter's matrices are fetched once per group of tokens; NULL = index per token. */
lora_status_t lora_bgmv_apply(lora_pool_t *pool, int32_t target,
                              const void *x, int64_t ldx,
                              const void *y_base, int64_t ldyb,
                              void *y, int64_t ldy,
                              const int32_t *slot_idx_dev, int32_t T,
                              const void *meta_dev_or_null,
                              void *workspace, size_t workspace_bytes, void *stream);

/*
 * Several projections of ONE decode batch in one launch (paper Section 2.2: the adapters of a
 * batch are served together through kernel-level work; Section 8.1: the models carry LoRA on all
 * their attention and MLP projections): q/k/v, or gate/up, or all seven adapted projections of a
 * layer when the caller has their inputs ready.  Every item is what one lora_bgmv_apply call would
 * take; all items share the batch (slot_idx_dev, T) and its grouped metadata, which is required.
 * The items must be independent: no item's y may overlap another item's x, y_base or y (an item's
 * own y may equal its y_base); items may share x.  The launch walks the units of item 0 first,
 * then item 1, ...: list wide projections first for the best balance.  Results are bit-identical
 * to n_items separate lora_bgmv_apply calls.
 * n_items in 1 .. LORA_MULTI_MAX.  Errors: those of lora_bgmv_apply, per item.
 */
#define LORA_MULTI_MAX 8
typedef struct {
    int32_t target;
    const void *x;       int64_t ldx;    /* dev bf16 [T, d_in]  */
    const void *y_base;  int64_t ldyb;   /* dev bf16 [T, d_out] */
    void *y;             int64_t ldy;    /* dev bf16 [T, d_out] */
} lora_apply_item_t;
lora_status_t lora_bgmv_apply_multi(lora_pool_t *pool, const lora_apply_item_t *items, int32_t n_items,
                                    const int32_t *slot_idx_dev, int32_t T, const void *meta_dev,
                                    void *workspace, size_t workspace_bytes, void *stream);

/*
 * lora_bgmv_apply for callers that cannot hand over a workspace (the paper has no counterpart;
 * this is a convenience of the library).  Some hosts of this code may not allocate device
 * memory at the point where they call it: a serving engine that has already given all free HBM
 * to its KV cache and adapter pool, a plug-in running inside another framework's memory
 * manager, code on a latency path where an allocation (or the implicit synchronisation of a
 * free) is not acceptable.  For them the fp32 scratch between the shrink and expand phases is a
 * fixed array of LORA_STATIC_SCRATCH_BYTES inside the library image; every GPU that loads the
 * library holds that much memory until the process exits.
 *  - Same arguments and results as lora_bgmv_apply minus the workspace; it always runs the
 *    two-phase CUDA-core kernels.  It allocates and frees nothing.
 *  - Limit: 32 * T * bucket(r_max) <= LORA_STATIC_SCRATCH_BYTES, bucket = r_max rounded up to
 *    8, 16, 32 or 64 (T <= 4096 at r_max 16, T <= 1024 at r_max 64); beyond it the call returns
 *    LORA_ERR_BUFFER_TOO_SMALL and launches nothing.
 *  - The first call on each device looks up the array's device address; make that call before
 *    starting any stream capture.
 *  - All calls on a device share the one array, and it keeps whatever the last call left there
 *    (the kernels overwrite every entry they later read, so nothing is cleared).  Two calls
 *    that can overlap on the GPU (different streams without an ordering between them) race on
 *    it: keep such calls on one stream or order them with events.
 */
#define LORA_STATIC_SCRATCH_BYTES (2u * 1024u * 1024u)
lora_status_t lora_bgmv_apply_static(lora_pool_t *pool, int32_t target,
                                     const void *x, int64_t ldx,
                                     const void *y_base, int64_t ldyb,
                                     void *y, int64_t ldy,
                                     const int32_t *slot_idx_dev, int32_t T,
                                     const void *meta_dev_or_null, void *stream);

/* Prefill / chunked-prefill batches.  meta_dev: metadata built for this batch (any tile_m).
 * With tile_m = 128 and a batch of at least 4096 tokens, tiles that are runs of 32 .. 128
 * consecutive tokens take the tcgen05 kernels (split-K partials in `workspace`); every other tile,
 * and every tile of a shorter batch, takes the fused kernel that also serves lora_bgmv_apply.
 * When both kinds are present the fused kernel runs on a stream the pool owns, forked from
 * `stream` by an event at the call and joined back into it before the call returns, so work
 * enqueued on `stream` afterwards is ordered behind all of it (this also holds inside a stream
 * capture: the pool's stream joins the capture and leaves it within the call). */
lora_status_t lora_sgmv_apply(lora_pool_t *pool, int32_t target,
                              const void *x, int64_t ldx,
                              const void *y_base, int64_t ldyb,
                              void *y, int64_t ldy,
                              const void *meta_dev, int32_t T,
                              void *workspace, size_t workspace_bytes, void *stream);

/* ----------------------------------------------------------------------------------------
 * One layer step from HOST buffers: copies x, y_base and slot_idx (pinned host memory) to the
 * caller's device staging buffers, builds the metadata, applies, and copies y back, all on
 * `stream`.  kind: 0 = BGMV, 1 = SGMV.  y_host is complete when the stream has drained.
 * -------------------------------------------------------------------------------------- */
typedef struct {
    void *x_dev;            /* >= T * d_in  bf16 */
    void *y_base_dev;       /* >= T * d_out bf16 */
    void *y_dev;            /* >= T * d_out bf16 (may equal y_base_dev) */
    int32_t *slot_idx_dev;  /* >= T int32 */
    void *meta_dev;         size_t meta_bytes;
    void *workspace;        size_t workspace_bytes;
} lora_step_buffers_t;

lora_status_t lora_apply_host(lora_pool_t *pool, int32_t target, int32_t kind,
                              const void *x_host, const void *y_base_host, void *y_host,
                              const int32_t *slot_idx_host, int32_t T,
                              int32_t tile_m, int32_t long_min,
                              const lora_step_buffers_t *dev, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* LORA_B200_H */
