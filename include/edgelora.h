/*
 * edgelora.h -- C ABI of the B200 (sm_100a) batch LoRA inference library.
 *
 * One operation sits behind this boundary: a LoRA-augmented linear layer over a
 * mixed batch of T tokens in which every token names its own adapter,
 *
 *     y[t] = W x[t] + s_a * B_a (A_a x[t]),   a = adapter_id[t],   a = -1 => y[t] = W x[t]
 *
 * (paper Section 3.4 "Batch LoRA Inference", the displayed batch equation; adapter shapes
 * A: r x h_in, B: h_out x r from Section 2.1).  Adapters live in a pool of fixed-size
 * blocks reserved once (Section 3.3 "pre-allocated memory pool", Section 4.2); a token's
 * adapter id is the index of the block ("slot") that holds its adapter.
 *
 * Conventions
 *   - All matrices are row-major bfloat16 (uint16 bit patterns).  Accumulation is fp32,
 *     outputs are rounded to nearest-even bfloat16.  Ids are int32.
 *   - "dev" pointers are CUDA device pointers on the current device, "host" pointers are
 *     ordinary host memory.  The caller owns W, x, ids and y; the pool owns the slot
 *     memory (unless the caller lends an arena), its staging buffers, workspaces, side
 *     stream and events.
 *   - Every function returns an int: EDGELORA_OK (0) or a negative edgelora_status.
 *     Nothing throws or aborts across this boundary.  There is no CPU fallback: without
 *     a CUDA device every compute entry point returns EDGELORA_ERR_CUDA.
 *   - Conditions only the GPU can see (an id outside [-1, n_slots), an id that names an
 *     empty slot) never trap: that token is computed base-only, a bit is set in a device
 *     status word, and edgelora_pool_sync_status() reports it.
 *   - Shape limits: h_in % 8 == 0, h_out % 8 == 0, 1 <= max_rank <= 64 (rounded up to a
 *     multiple of 16 internally), n_slots <= 65534, T <= max_tokens <= 32768.
 */
#ifndef EDGELORA_H_
#define EDGELORA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  EDGELORA_OK = 0,
  EDGELORA_ERR_INVALID_ARG = -1,
  EDGELORA_ERR_BAD_SLOT = -2,
  EDGELORA_ERR_RANK_TOO_LARGE = -3,
  EDGELORA_ERR_ARENA_TOO_SMALL = -4,
  EDGELORA_ERR_CUDA = -5,
  EDGELORA_ERR_BAD_ADAPTER_ID = -6,
  EDGELORA_ERR_SLOT_EMPTY = -7,
  EDGELORA_ERR_TIMEOUT = -8,
  EDGELORA_ERR_TOO_MANY_TOKENS = -9,
  EDGELORA_ERR_CACHE_FULL = -10,
  EDGELORA_ERR_BOUNDS = -11
} edgelora_status;

/* Bits of the device status word returned by edgelora_pool_sync_status(). */
#define EDGELORA_STATUS_BAD_ADAPTER_ID 0x1u /* an id outside [-1, n_slots) was seen     */
#define EDGELORA_STATUS_SLOT_EMPTY 0x2u     /* an id named a slot with nothing loaded   */
#define EDGELORA_STATUS_TIMEOUT 0x4u        /* a bounded in-kernel wait gave up         */
#define EDGELORA_STATUS_BOUNDS 0x8u         /* checked build only: a kernel met an index outside
                                               its array and skipped the access            */

typedef struct edgelora_pool edgelora_pool_t; /* opaque, owned by the library */
typedef struct edgelora_plan edgelora_plan_t; /* opaque, owned by the library */

/* Pool geometry for ONE linear site (one W shape).  Section 3.3: the pool is a set of
 * fixed blocks, each the size of one adapter; here a block holds A padded to
 * [max_rank][h_in] and B padded to [h_out][max_rank]. */
typedef struct {
  int32_t h_in;       /* input width of the linear site                                  */
  int32_t h_out;      /* output width                                                    */
  int32_t n_slots;    /* number of blocks S                                              */
  int32_t max_rank;   /* largest adapter rank a block can hold                           */
  int32_t max_tokens; /* largest T of a call; 0 => 8192.  Sizes the workspaces.          */
  uint32_t flags;     /* EDGELORA_FLAG_*                                                 */
  void *arena_dev;    /* optional caller-owned device memory for the slot blocks, 256-byte
                         aligned; NULL => the library allocates and owns it              */
  size_t arena_bytes; /* size of arena_dev; ignored when arena_dev is NULL               */
} edgelora_pool_config;

#define EDGELORA_FLAG_NONE 0u
/* The pool keeps every adapter's A in Q8_0 in device memory (Section 5.1: adapters are stored in
 * Q8_0), 34/64 of the bfloat16 bytes, which are the bytes that bound a many-adapter decode step; B
 * stays bfloat16.  Such a pool needs h_in % 256 == 0, takes adapters through
 * edgelora_pool_load_slot_q8 only, and serves decode batches (T <= 256) only: the shrink kernel
 * decodes the blocks as it streams them.  Other calls return EDGELORA_ERR_INVALID_ARG. */
#define EDGELORA_FLAG_A_Q8 1u

/* Options for edgelora_pool_set_option(). */
#define EDGELORA_OPT_REGIME 1    /* 0 auto (T <= 256 => decode), 1 force decode, 2 force prefill */
#define EDGELORA_OPT_PROFILE 2   /* 1 => bracket every kernel with CUDA events (slower)          */
#define EDGELORA_OPT_PDL 3       /* programmatic dependent launch: 0 off; 1 (default) between the
                                    kernels of one call; 2 also lets the first kernel of a call
                                    start under the tail of earlier work on the stream -- only
                                    valid when W, x and the ids of a call are not produced by the
                                    call before it (independent sites / batches)                  */
#define EDGELORA_OPT_DECODE_SPLITS 4 /* tuning: K splits per W row tile in decode, 0 = automatic  */
#define EDGELORA_OPT_SHRINK_ITEMS 5  /* tuning: work items the decode shrink aims for, 0 = auto   */
#define EDGELORA_OPT_GATHER_SPLITS 7 /* tuning: K splits of the tensor-core gather shrink in decode, 0 = chosen
                                        on the device from the number of adapters the batch touches  */
#define EDGELORA_OPT_GATHER_MIN_T 8  /* tuning: decode batches above this many tokens use the routing
                                        kernel + tensor-core gather shrink, the others the single shrink
                                        kernel with the routing inside.  Default 256: every decode batch
                                        takes the single kernel (it is the faster one as measured)   */
#define EDGELORA_OPT_SHRINK_DEPTH 9  /* tuning: ring depth of the decode shrink for batches above 64 tokens:
                                        2 (default, two CTAs per SM) or 4 (one CTA per SM); 0 = default */
#define EDGELORA_OPT_FUSED_DECODE 10 /* 1 (default): batches of at most 64 tokens take one launch, the shrink
                                        on otherwise idle warps of the base product's grid; 0: two launches.
                                        The CTAs of such a launch wait (bounded) for one another, so all of
                                        them must be resident at once: the library checks that against the
                                        device's occupancy figure.  Set 0 for pools whose calls run at the
                                        same time as another pool's on a stream of different priority: two
                                        such grids could each hold SMs the other needs, and the wait would
                                        end in EDGELORA_ERR_TIMEOUT */
#define EDGELORA_OPT_WAIT_CYCLES 6   /* limit of every bounded in-kernel wait of the layer, in units
                                        of 1024 SM clock cycles; 0 = default (about two seconds).
                                        A wait that runs out raises EDGELORA_STATUS_TIMEOUT           */

/* Bytes of device memory the slot blocks need for this geometry (what arena_bytes must
 * be at least).  Host-only arithmetic. */
int edgelora_pool_bytes_required(const edgelora_pool_config *cfg, size_t *bytes_out);

/* Section 3.3 / 4.2: reserve every block once, at initialisation.  Allocates the slot
 * blocks (unless an arena is lent), the slot table, pinned staging buffers, a side
 * stream, events and the per-call workspaces.  All slots start empty. */
int edgelora_pool_create(const edgelora_pool_config *cfg, edgelora_pool_t **pool_out);

/* Section 3.3: "when a new adapter is required it is assigned to a free block".
 * Copies adapter (A_host [rank][h_in], B_host [h_out][rank], dense bf16) into block
 * `slot`, asynchronously: the data is first copied into pinned staging (so the caller may
 * free A_host / B_host on return), then moved with cudaMemcpyAsync on the pool's side
 * stream.  The copy waits for the last edgelora_lora_linear call issued before it, and
 * later edgelora_lora_linear calls (on any stream) wait for the copy, so a call never sees a
 * half-written block; the caller must not reload a slot that ids of a still-queued call refer
 * to.  When several streams run calls of one pool, the copy waits only for the most recent
 * call: order the others yourself.
 * CUDA graphs: a call issued while its stream is being captured records neither of these
 * waits (an event wait inside a graph would name a load that is long gone at replay).  The
 * owner of a graph therefore calls edgelora_pool_wait_loads before capturing and before any
 * replay that follows a load, and synchronises the replays' stream before reloading a slot
 * their ids use.
 * rank must be in [1, max_rank]; scale is s_a. */
int edgelora_pool_load_slot(edgelora_pool_t *pool, int32_t slot, int32_t rank, float scale,
                            const uint16_t *A_host, const uint16_t *B_host);

/* The same load without the copy into the library's staging buffer, for adapters the caller keeps in
 * page-locked host memory in the block's own layout (Section 3.3: adapters that are not resident
 * wait in host memory; a server that pins that memory once swaps at the speed of the link instead
 * of the speed of a host memcpy).  rank must equal the pool's padded rank (16, 32 or 64), A_pinned
 * is [rank][h_in], B_pinned [h_out][rank].  Unlike edgelora_pool_load_slot the buffers must stay
 * valid and unchanged until edgelora_pool_wait_loads (or a later layer call's completion).
 * EDGELORA_ERR_INVALID_ARG when the memory is not page-locked or the rank is not the padded one. */
int edgelora_pool_load_slot_pinned(edgelora_pool_t *pool, int32_t slot, int32_t rank, float scale,
                                   const uint16_t *A_pinned, const uint16_t *B_pinned);

/* Section 5.1 ("All LoRA adapters are quantized using the Q8_0 format"): the same load for an
 * adapter stored in Q8_0, the published block format of 34 bytes per 32 consecutive values of a
 * row: a half-precision scale d (2 bytes, little endian) followed by 32 signed bytes q, value
 * d * q.  A_q8 is [rank][h_in / 32] blocks (h_in % 32 == 0), B_q8 is [h_out][ceil(rank / 32)]
 * blocks whose entries past `rank` are ignored.  The 8-bit form crosses to the device (about half
 * the bytes of the bfloat16 form) and is converted there, on the pool's side stream, into the
 * block's bfloat16 layout (each value rounded to nearest even), so the layer calls are unchanged.
 * Ordering, ownership and errors as for edgelora_pool_load_slot; the first call allocates a
 * device scratch for one adapter. */
int edgelora_pool_load_slot_q8(edgelora_pool_t *pool, int32_t slot, int32_t rank, float scale,
                               const void *A_q8, const void *B_q8);

/* Section 4.2: an evicted adapter's block returns to the pool.  Marks `slot` empty
 * (asynchronously, ordered like a load). */
int edgelora_pool_evict_slot(edgelora_pool_t *pool, int32_t slot);

/* Blocks the host until every load / evict issued so far has landed in device memory. */
int edgelora_pool_wait_loads(edgelora_pool_t *pool);

/* Section 3.4: the batched layer.  W_dev [h_out][h_in], x_dev [T][h_in],
 * adapter_id_dev [T] (slot index or -1), y_dev [T][h_out]; all device memory, 16-byte
 * aligned.  Enqueues, on `stream` (a cudaStream_t; NULL = legacy default stream):
 * routing plan -> shrink (z = s_a A_a x) -> base product W x on the tensor cores with
 * the expand B_a z accumulated into the same tile (z rounded to bfloat16 for it) -> y written
 * once.  Asynchronous; no host synchronisation, no
 * allocation.  T == 0 is a no-op.  x_dev / y_dev must not alias.  Calls of one pool share its
 * workspaces: they must not overlap on the GPU (one stream, or ordered by events). */
int edgelora_lora_linear(edgelora_pool_t *pool, const void *W_dev, const void *x_dev,
                         const int32_t *adapter_id_dev, int32_t T, void *y_dev, void *stream);

/* Same layer with HOST buffers: copies x and ids to the device through pinned staging,
 * runs the layer, copies y back and synchronises `stream` before returning.  W stays a
 * device pointer (weights are resident model state, like the pool). */
int edgelora_lora_linear_host(edgelora_pool_t *pool, const void *W_dev, const uint16_t *x_host,
                              const int32_t *adapter_id_host, int32_t T, uint16_t *y_host,
                              void *stream);

/* The same, pipelined: returns as soon as the copies and the layer are enqueued.  x_host,
 * adapter_id_host and y_host should be page-locked (otherwise the copies still complete but do
 * not overlap) and must stay valid and untouched until edgelora_pool_host_sync returns.  The
 * library keeps two sets of device mirrors and two copy streams: the copy-in of call i + 1 and
 * the copy-out of call i - 1 run beside the layer of call i (which runs on `stream`).  Calls of
 * one pool are issued from one thread.  (Serving loop of Section 3.4: a batch is formed while
 * the previous one computes.) */
int edgelora_lora_linear_host_async(edgelora_pool_t *pool, const void *W_dev, const uint16_t *x_host,
                                    const int32_t *adapter_id_host, int32_t T, uint16_t *y_host,
                                    void *stream);

/* Blocks until every y_host of earlier edgelora_lora_linear_host_async calls is complete. */
int edgelora_pool_host_sync(edgelora_pool_t *pool);

/* Routing plan (Section 3.4 "u-batch" grouping; Section 4.3 "maps adapter IDs to sample
 * indices ... scattered back to their original positions").  A plan depends only on the
 * ids, so one plan can serve every linear site that sees the same batch. */
int edgelora_plan_create(int32_t max_tokens, int32_t n_slots, edgelora_plan_t **plan_out);
int edgelora_plan_destroy(edgelora_plan_t *plan);
/* Builds the plan for adapter_id_dev[T] on `stream` (asynchronous). */
int edgelora_plan_build(edgelora_plan_t *plan, const int32_t *adapter_id_dev, int32_t T,
                        void *stream);
/* Copies the last built plan to host arrays (synchronises `stream`).  Any array may be
 * NULL.  Sizes: ids_valid[T], perm[T], group_start[T+1], group_adapter[T],
 * seg_start[T+1], seg_adapter[T]; counts_out = {n_groups, n_segments}.
 *   segments: maximal runs of equal id in token order;
 *   groups  : ids ascending with -1 first, token order kept inside a group. */
int edgelora_plan_export(edgelora_plan_t *plan, void *stream, int32_t *ids_valid,
                         int32_t *perm, int32_t *group_start, int32_t *group_adapter,
                         int32_t *seg_start, int32_t *seg_adapter, int32_t counts_out[2]);
/* The layer with a plan built beforehand by edgelora_plan_build on the same stream for
 * the same ids (plan.n_slots must equal the pool's). */
int edgelora_lora_linear_planned(edgelora_pool_t *pool, edgelora_plan_t *plan, const void *W_dev,
                                 const void *x_dev, int32_t T, void *y_dev, void *stream);
/* The pool's own plan object (the one edgelora_lora_linear builds each call). */
int edgelora_pool_plan(edgelora_pool_t *pool, edgelora_plan_t **plan_out);
/* Status word of a plan built with edgelora_plan_build (an id outside [-1, n_slots) raises
 * EDGELORA_STATUS_BAD_ADAPTER_ID there, not in the pools that later use the plan): synchronises
 * `stream`, returns the bits in *bits_out (may be NULL), clears them; return value as for
 * edgelora_pool_sync_status. */
int edgelora_plan_sync_status(edgelora_plan_t *plan, void *stream, uint32_t *bits_out);

/* ---- A set of linear sites over one batch (Section 3.4: every LoRA-augmented layer of the model
 * sees the same mixed batch; Section 4.3: the id -> sample mapping is worked out once).  Site i is
 * (pools[i], W_dev[i]) and reads input number input_of_site[i] (sites with the same input width
 * may share an input, e.g. q/k/v/o/gate/up of a decoder layer); all pools have the same n_slots
 * and max_tokens >= the set's.  A run builds ONE routing plan from the ids and evaluates the sites
 * in order; the sites are independent given their inputs, so in batches above 256 tokens the
 * shrink of site i + 1 is issued with the kernels of site i and only the first site's shrink stands
 * alone.  The set borrows the pools and W (the caller keeps them alive) and owns its plan and the
 * device mirrors of the host-buffer call.  One thread at a time per set; runs of one set (and of
 * its pools) must not overlap on the GPU. */
typedef struct edgelora_siteset edgelora_siteset_t;
int edgelora_siteset_create(int32_t n_sites, edgelora_pool_t *const *pools, const void *const *W_dev,
                            const int32_t *input_of_site, int32_t n_inputs, int32_t max_tokens,
                            edgelora_siteset_t **set_out);
int edgelora_siteset_destroy(edgelora_siteset_t *set);
/* x_dev [n_inputs] device pointers ([T][width of that input] bf16), adapter_id_dev [T],
 * y_dev [n_sites] device pointers ([T][h_out of that site]); asynchronous on `stream`. */
int edgelora_siteset_run(edgelora_siteset_t *set, const void *const *x_dev, const int32_t *adapter_id_dev,
                         int32_t T, void *const *y_dev, void *stream);
/* The same with HOST buffers (page-locked for full copy speed): copies the inputs and the ids to
 * the device, runs the set, copies back y of every site whose y_host entry is not NULL (the others
 * stay on the device and are overwritten by the next site of the same width) and synchronises
 * `stream` before returning.  Allocates its device mirrors on first use.  Copies that the running
 * sites do not wait for (a result that is complete, an input that only later sites read) go through
 * a second stream of the set's own, beside the kernels; that stream is synchronised too. */
int edgelora_siteset_run_host(edgelora_siteset_t *set, const uint16_t *const *x_host,
                              const int32_t *adapter_id_host, int32_t T, uint16_t *const *y_host,
                              void *stream);
/* The set's plan object (for edgelora_plan_export / edgelora_plan_sync_status). */
int edgelora_siteset_plan(edgelora_siteset_t *set, edgelora_plan_t **plan_out);

/* No counterpart in the paper: a routing-plan builder for callers that cannot allocate.
 *
 * Some hosts of this library may not call cudaMalloc on the path where they need a plan: a
 * serving loop that has handed all device memory to its own arena at start-up, code running
 * inside a region where allocation would synchronise the device or is simply forbidden by the
 * embedding runtime.  For them this entry point builds the same plan as edgelora_plan_build but
 * keeps the kernel's working arrays in a fixed array that is part of the library image (about
 * 100 KB on every GPU that loads the library, for the life of the process).  It calls no
 * cudaMalloc / cudaFree and no allocating library routine; the caller passes every output.
 *
 *   adapter_id_dev [T]     ids as for edgelora_lora_linear (device)
 *   ids_valid_dev, perm_dev, group_adapter_dev, seg_adapter_dev   [T]   int32, device, written
 *   group_start_dev, seg_start_dev                                [T+1] int32, device, written
 *   info_dev [4]           {n_groups, n_segments, status bits (EDGELORA_STATUS_*), 0}, device
 * Array meanings are those of edgelora_plan_export.  Asynchronous on `stream`.
 *
 * Limits and rules: T <= EDGELORA_PLAN_STATIC_MAX_TOKENS, otherwise
 * EDGELORA_ERR_TOO_MANY_TOKENS and nothing is launched.  The first call on each device looks up
 * the device address of the built-in array (with that device current); make that first call
 * outside any stream capture.  All calls on a device share the one array, and it keeps what the
 * last call left in it, so two calls whose kernels may overlap on the GPU (different streams with
 * no ordering between them) race: order them on one stream or with events. */
#define EDGELORA_PLAN_STATIC_MAX_TOKENS 4096
int edgelora_plan_build_static(const int32_t *adapter_id_dev, int32_t T, int32_t n_slots,
                               int32_t *ids_valid_dev, int32_t *perm_dev, int32_t *group_start_dev,
                               int32_t *group_adapter_dev, int32_t *seg_start_dev,
                               int32_t *seg_adapter_dev, int32_t *info_dev, void *stream);

/* Synchronises the device work issued through this pool, returns the status bits
 * accumulated since the last call in *bits_out and clears them.  The return value is
 * EDGELORA_OK, or the error matching the most severe bit. */
int edgelora_pool_sync_status(edgelora_pool_t *pool, uint32_t *bits_out);

int edgelora_pool_set_option(edgelora_pool_t *pool, int32_t option, int32_t value);

/* Self-test of the time-out path.  Enqueues on `stream` a one-thread kernel that waits, with the
 * pool's wait limit, on a shared-memory barrier nothing arrives at; the wait runs out, the kernel
 * raises EDGELORA_STATUS_TIMEOUT in the pool's status word and returns.  Nothing else is touched
 * and the context stays usable: edgelora_pool_sync_status then reports EDGELORA_ERR_TIMEOUT once.
 * Only with EDGELORA_OPT_WAIT_CYCLES lowered to at most 16384 (16 M cycles); otherwise
 * EDGELORA_ERR_INVALID_ARG and nothing is launched. */
int edgelora_pool_selftest_wait(edgelora_pool_t *pool, void *stream);

/* Section 5.1, model table (base models stored in Q8_0 or Q4_0): decodes a base weight matrix kept in
 * one of the two published block formats into the bfloat16 matrix W [h_out][h_in] that the layer
 * calls take, on the device, so that the stored form is what crosses to the GPU (34/64 or 18/64 of
 * the bfloat16 bytes).  Both formats block 32 consecutive values of a row (h_in % 32 == 0), a
 * half-precision scale d first (little endian): Q8_0 has 32 signed bytes q after it, value d * q
 * (34 bytes); Q4_0 has 16 bytes, byte j holding value j in its low and value j + 16 in its high four
 * bits as codes c, value d * (c - 8) (18 bytes).  Each value is rounded to nearest even bfloat16.
 * W_blocks_dev: device memory, [h_out][h_in / 32] blocks, read only; W_dev: device memory the caller
 * owns, 16-byte aligned, written on `stream`.  EDGELORA_ERR_INVALID_ARG for an unknown format, a null
 * pointer or h_in % 32 != 0; EDGELORA_ERR_CUDA if the launch fails. */
#define EDGELORA_WEIGHTS_Q8_0 0
#define EDGELORA_WEIGHTS_Q4_0 1
int edgelora_weights_decode(int32_t format, const void *W_blocks_dev, int32_t h_out, int32_t h_in,
                            uint16_t *W_dev, void *stream);

/* The checked build of the library (compiled with -DEDGELORA_CHECKED, for finding memory errors
 * where no memory-checking tool can be run; the paper has no counterpart).  It differs in two ways.
 * The kernels test the indices they read from device memory (adapter ids in the routing plan's lists,
 * token indices, tile descriptors, ranks) against their arrays' sizes; a failed test skips the
 * access and raises EDGELORA_STATUS_BOUNDS, which edgelora_pool_sync_status reports as
 * EDGELORA_ERR_BOUNDS.  And every device buffer the library allocates has 256 guard bytes of a fixed
 * value in front and behind.
 *   edgelora_build_is_checked  1 for the checked build, 0 for the normal one.
 *   edgelora_check_guards      synchronises the current device and compares every guard zone on it
 *                              with its value: EDGELORA_OK, or EDGELORA_ERR_BOUNDS when a kernel or
 *                              copy wrote outside a buffer.  The normal build has no zones and
 *                              returns EDGELORA_OK. */
int edgelora_build_is_checked(void);
int edgelora_check_guards(void);

/* Launch bookkeeping for measurement.  info_out[0] = kernels launched by the last
 * edgelora_lora_linear call, [1] = regime used (1 decode, 2 prefill), [2] = grid of the
 * base-product kernel, [3] = split-K factor, [4] = pipeline stages, [5] = N tile,
 * [6] = total kernels launched through this pool, [7] = reserved. */
int edgelora_pool_last_launch(edgelora_pool_t *pool, int64_t info_out[8]);

/* With EDGELORA_OPT_PROFILE on: accumulated device time per kernel since the last reset,
 * from CUDA events on the launching stream (synchronises them).  ms_out / launches_out:
 * [0] plan, [1] shrink of small decode batches (routing inside), [2] shrink on the tensor cores
 * (segment and gather tiles), [3] base product (expand and combine included), [4] unused.  reset != 0 clears the accumulators afterwards. */
int edgelora_pool_kernel_times(edgelora_pool_t *pool, double ms_out[5], int64_t launches_out[5],
                               int32_t reset);

/* Releases everything the pool owns (never the caller's arena).  Synchronises first. */
int edgelora_pool_destroy(edgelora_pool_t *pool);

/* ---- Adapter memory manager (host side; Section 3.3 "adapter memory manager", Section 4.2:
 * recency list + set of resident adapters + stack of free blocks).  Decides which block of a
 * pool an adapter lives in; moves no bytes (the caller passes the block to
 * edgelora_pool_load_slot on a miss, which copies on the pool's side stream beside the layer
 * calls).  Keys are the caller's adapter ids (>= 0); blocks are slot indices 0 .. n_blocks-1.
 * Host memory only, no CUDA call; one thread at a time per cache. */
typedef struct edgelora_cache edgelora_cache_t;
#define EDGELORA_CACHE_LRU 0 /* evict the least recently used adapter (Section 4.2)              */
#define EDGELORA_CACHE_LFU 1 /* evict the least frequently used one (Section 3.3), ties by recency;
                                a use count restarts when an adapter returns after an eviction  */

int edgelora_cache_create(int32_t n_blocks, int32_t policy, edgelora_cache_t **cache_out);
int edgelora_cache_destroy(edgelora_cache_t *cache);

/* The block of `key`.  Resident: *hit_out = 1, recency and use count updated.  Not resident:
 * *hit_out = 0 and *slot_out is the block to load it into: the lowest free block while any is
 * free, otherwise the victim's, whose key goes to *evicted_key_out (-1 if nothing was evicted).
 * pin != 0 marks the adapter as held by a running request until edgelora_cache_release: held
 * adapters are never victims; EDGELORA_ERR_CACHE_FULL when every block is held.  hit_out and
 * evicted_key_out may be NULL. */
int edgelora_cache_acquire(edgelora_cache_t *cache, int64_t key, int32_t pin, int32_t *slot_out,
                           int32_t *hit_out, int64_t *evicted_key_out);
/* Cache-aware adapter selection (Algorithm 1 of the paper, Section 3.2): scores[j] is the
 * router's confidence for adapter j (host array, n entries, key = index).  Of the k best-scored
 * adapters, in descending order of score (equal scores: lower index first; scores are finite), the
 * first resident one is chosen; if none of them is resident the best-scored one is chosen and
 * admitted.  The choice goes to *key_out; the rest is edgelora_cache_acquire of that key. */
int edgelora_cache_select(edgelora_cache_t *cache, const float *scores, int32_t n, int32_t k,
                          int32_t pin, int64_t *key_out, int32_t *slot_out, int32_t *hit_out,
                          int64_t *evicted_key_out);
/* Section 4.2: "during server initialization, the memory cache is prefilled with random adapters".
 * Makes keys[0..n) (distinct, n <= n_blocks; which ones is the caller's draw) resident in an empty
 * cache, block i for keys[i] (the lowest free block each time), without holds, and leaves the hit /
 * miss counters at zero so that they describe the serving phase.  blocks_out may be NULL.  The
 * caller loads those adapters into the pools' slots. */
int edgelora_cache_prefill(edgelora_cache_t *cache, const int64_t *keys, int32_t n, int32_t *blocks_out);
/* Drops one hold on `key` (EDGELORA_ERR_INVALID_ARG if it has none). */
int edgelora_cache_release(edgelora_cache_t *cache, int64_t key);
/* Block of `key` or -1, without touching recency or counts. */
int edgelora_cache_lookup(const edgelora_cache_t *cache, int64_t key, int32_t *slot_out);
/* Counters since creation; any pointer may be NULL. */
int edgelora_cache_stats(const edgelora_cache_t *cache, int64_t *hits, int64_t *misses,
                         int64_t *evictions, int32_t *resident);

/* ---- Request batcher: the slot state machine of the server manager (Section 4 "Slot state
 * machine": idle -> adapter selection (Algorithm 1) -> prompt processing -> generation; slots in the
 * prompt or generation state are grouped into one batch per step; Section 5.1: gamma slots bound
 * the requests in flight, the rest queue).  Host memory only, no CUDA call; one thread per batcher.
 * The batcher borrows `cache` (whose blocks are the slots of the adapter pools) and holds a
 * request's adapter there until the request finishes.  Time is virtual and the caller's. */
typedef struct edgelora_batcher edgelora_batcher_t;
/* n_slots = gamma; max_batch_tokens >= n_slots bounds the tokens of one step (every generating
 * slot gives one token, the rest of the budget goes to prompts, which are cut and continued);
 * top_k = candidates per request. */
int edgelora_batcher_create(int32_t n_slots, int32_t max_batch_tokens, int32_t top_k,
                            edgelora_cache_t *cache, edgelora_batcher_t **batcher_out);
int edgelora_batcher_destroy(edgelora_batcher_t *batcher);
/* A request: arrival time in seconds (calls in ascending arrival order), prompt and output length in
 * tokens (>= 1), and the router's top_k adapters in descending order of confidence (host array). */
int edgelora_batcher_submit(edgelora_batcher_t *batcher, int64_t request_id, double arrival,
                            int32_t in_len, int32_t out_len, const int64_t *candidates);
/* Forms the next step's batch.  Admits arrived requests (arrival order, lowest idle slot first),
 * chooses their adapters (the first resident candidate, else the first candidate is loaded; the
 * choice is held until the request ends; a slot waits in the selection state while every block is
 * held), then lists the tokens: one per generating slot (slot order), then the prompt tokens of the
 * slots in the prompt state (slot order).  token_block[i] is the pool slot of token i's adapter,
 * token_slot[i] the batcher slot it belongs to (arrays of `capacity` >= max_batch_tokens entries);
 * load_key / load_block (n_slots entries each) name the adapters the caller must load into those
 * pool slots before running the step.  When nothing is in flight the clock jumps to the next
 * arrival.  Returns 1 with a batch, 0 when every submitted request is finished, or an error
 * (EDGELORA_ERR_CACHE_FULL: nothing runs and every block is held). */
int edgelora_batcher_next_batch(edgelora_batcher_t *batcher, int32_t capacity, int32_t *token_block,
                                int32_t *token_slot, int32_t *n_tokens_out, int32_t *n_decode_out,
                                int64_t *load_key, int32_t *load_block, int32_t *n_loads_out,
                                double *now_out);
/* The step handed out by the last edgelora_batcher_next_batch took `seconds`: the clock advances,
 * prompts move on, the step that ends a prompt also yields the request's first token, every
 * generating slot yields one token, finished requests leave their slot and release their adapter. */
int edgelora_batcher_complete_step(edgelora_batcher_t *batcher, double seconds);
/* The finished requests so far, in order of completion (any array may be NULL; capacity 0 only
 * returns the count): ids, arrival / first-token / finish times, the adapter used and whether it
 * was resident when chosen.  Section 5.1's metrics (throughput, average latency, average
 * first-token latency, SLO attainment) and Section 3.3's hit rate follow from these. */
int edgelora_batcher_finished(const edgelora_batcher_t *batcher, int32_t capacity, int64_t *request_id,
                              double *arrival, double *first_token, double *finish, int64_t *adapter,
                              int32_t *hit, int32_t *n_out);

/* Scoring head of the adapter router (Section 3.2: a score s_j in [0, 1] per adapter j for a
 * prompt): scores_dev[b][j] = sigmoid(sum_k Wr_dev[j][k] * h_dev[b][k] + bias_dev[j]).
 * Wr_dev [n][hidden] and h_dev [B][hidden] are bfloat16, row-major, 16-byte aligned device memory;
 * bias_dev [n] float32 or NULL; scores_dev [B][n] float32.  hidden is a multiple of 8, at most
 * 8192.  fp32 accumulation.  Enqueued on `stream`, asynchronous, no allocation; B == 0 is a
 * no-op.  The backbone pass that produces h and the training of the router are not part of this
 * library; the scores feed edgelora_cache_select after a copy to the host. */
int edgelora_router_scores(const void *Wr_dev, const float *bias_dev, const void *h_dev, int32_t B,
                           int32_t n, int32_t hidden, float *scores_dev, void *stream);

const char *edgelora_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* EDGELORA_H_ */
