/*
 * asynclm.h -- C ABI of the AsyncLM serving-step attention library for NVIDIA B200 (sm_100a).
 *
 * One serving step under AsyncLM's interrupt mechanism is one batched attention pass over a paged
 * KV cache.  Most sequences contribute a single decode query.  A sequence whose function call has
 * returned contributes a multi-token interrupt span: the paper inserts the interrupt block at the
 * end of the sequence's token stream and lets generation resume after it (Section 3.2,
 * "Triggering Interrupts"), and the interrupt manager appends all queued interrupts to the
 * generated tokens so that the next decoding step processes them (Section 5.3).  A sequence paused
 * by a trap (Section 3.2, "Waiting for interrupts") contributes no query at all.  The span is
 * appended in place; the cached context is not recomputed (the restart-and-recompute alternative is
 * Section 5.5).
 *
 * Per step the caller runs, on one CUDA stream:
 *     asynclm_plan       (host integer work + one async host->device copy of the plan)
 *     asynclm_kv_append  (scatter the new K/V rows into their page slots)
 *     asynclm_attn_mixed (attention of every new row over its sequence's pages)
 * or, instead of the last two, asynclm_step, which does both in one launch.
 * A plan depends only on the lengths and the page table, so a multi-layer model builds it once per
 * step and reuses it for every layer's pool.
 *
 * Conventions
 *   - bf16 tensors are passed as untyped device pointers; rows are contiguous and 16-byte aligned.
 *   - kv_pool layout: [num_pages][2 (0 = K, 1 = V)][num_kv_heads][page_size][head_dim] bf16.
 *   - Query heads [h*G, (h+1)*G), G = num_q_heads / num_kv_heads, share kv head h.
 *   - New token i of sequence b (0 <= i < q_len_b) sits at position ctx_b + i of the sequence and
 *     attends to positions 0 .. ctx_b + i (whole prior context; causal inside the span).
 *   - "device" / "host" below says where a pointer must live.  The library never allocates or
 *     frees device memory, never synchronises the stream and keeps no global mutable state other
 *     than per-device attributes cached on first use.
 *   - Every function returns an asynclm_status (0 = success, negative = error).  Nothing throws,
 *     aborts or traps; kernels never wait on one another.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 */
#ifndef ASYNCLM_H_
#define ASYNCLM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum asynclm_status {
    ASYNCLM_OK = 0,
    ASYNCLM_ERR_INVALID_ARG = -1,         /* NULL pointer, negative size, misaligned pointer   */
    ASYNCLM_ERR_UNSUPPORTED_SHAPE = -2,   /* head_dim / page_size / group outside the set below */
    ASYNCLM_ERR_PAGE_TABLE = -3,          /* too few pages for a sequence, or a page id out of
                                             [0, num_pages), or (if asked) a page written twice  */
    ASYNCLM_ERR_WORKSPACE_TOO_SMALL = -4,
    ASYNCLM_ERR_CUDA = -5,                /* a CUDA runtime call or a launch failed            */
    ASYNCLM_ERR_ARCH = -6,                /* current device is not compute capability 10.x     */
    ASYNCLM_ERR_DEVICE_STATUS = -7,       /* a kernel reported a bounded wait that ran out     */
    ASYNCLM_ERR_STATIC_SCRATCH_TOO_SMALL = -8  /* asynclm_attn_mixed_static: the plan's partial
                                             results exceed ASYNCLM_STATIC_SCRATCH_BYTES         */
} asynclm_status;

/* Supported: head_dim in {64, 128}; page_size = 16; num_q_heads / num_kv_heads in {1, 2, 4, 8}. */
typedef struct asynclm_shape {
    int32_t num_q_heads;
    int32_t num_kv_heads;
    int32_t head_dim;
    int32_t page_size;
    int64_t num_pages;    /* capacity of the pool; page ids are checked against it */
    float   sm_scale;     /* softmax scale; <= 0 selects 1/sqrt(head_dim) */
    int32_t reserved;     /* must be 0 */
} asynclm_shape;

/* Planner knobs; a zero field selects the default. */
typedef struct asynclm_plan_options {
    int32_t num_sms;          /* SM count to balance for; 0 = query the current device.  Must be
                                 given (> 0) when planning without a device workspace. */
    int32_t kv_chunk_tokens;  /* fixed split-KV chunk length (multiple of 64); 0 = chosen so that
                                 the work items roughly fill the machine; a value >= the longest
                                 context disables splitting */
    int32_t tensor_min_rows;  /* new tokens of a sequence use the span body (tcgen05 MMA, 128
                                 query rows to a tile) when G * q_len >= this; 0 = default: 32.
                                 Below it they use the warp body (warp-level MMA with the keys
                                 on the M axis, 8 / G tokens to a unit), which streams K/V at
                                 the memory rate for every supported G and is where decode
                                 rows always go by default.  INT32_MAX keeps every row on the
                                 warp body, like ASYNCLM_PLAN_NO_TENSOR_PATH */
    int32_t flags;            /* ASYNCLM_PLAN_* */
} asynclm_plan_options;

#define ASYNCLM_PLAN_REJECT_ALIASED_WRITES 1  /* error if two sequences append into one page */
#define ASYNCLM_PLAN_NO_TENSOR_PATH        2  /* keep every row on the warp body              */

/* Host-side description of one step's batch (all arrays on the host, int32). */
typedef struct asynclm_batch {
    int32_t        batch;          /* number of sequences B */
    const int32_t* q_indptr;       /* [B+1] CSR over new tokens; q_len_b = q_indptr[b+1]-q_indptr[b]:
                                      0 paused, 1 decode, > 1 interrupt append */
    const int32_t* kv_len_before;  /* [B] tokens of b already stored in its pages (ctx_b) */
    const int32_t* page_indptr;    /* [B+1] CSR over page_indices */
    const int32_t* page_indices;   /* logical page j of b lives in physical page
                                      page_indices[page_indptr[b] + j]; at least
                                      ceil((ctx_b + q_len_b) / page_size) entries per sequence,
                                      extra (pre-allocated) pages are allowed */
} asynclm_batch;

/* Opaque plan; it lives inside the caller's host workspace. */
typedef struct asynclm_plan_s asynclm_plan_t;

/* What the planner decided; filled by asynclm_plan_get_info. */
typedef struct asynclm_plan_info {
    int32_t total_q;          /* T = sum of q_len */
    int32_t num_units;        /* (sequence, kv head, query tile) units */
    int32_t num_items;        /* (unit, kv chunk) work items */
    int32_t num_split_units;  /* units whose keys were split into > 1 chunk */
    int32_t partial_rows;     /* rows of fp32 partial output held in the device workspace */
    int32_t kv_chunk_tokens;  /* chosen chunk length (INT32_MAX = unsplit) */
    int32_t num_ctas_cuda;    /* persistent CTAs that may run the warp body */
    int32_t num_ctas_tensor;  /* persistent CTAs that may run the span body */
    int32_t num_items_tensor; /* items routed to the span body */
    int32_t launches_append;  /* kernels asynclm_kv_append launches */
    int32_t launches_attn;    /* kernels asynclm_attn_mixed launches */
    int32_t num_sms;
    int64_t total_kv_tokens;  /* sum over active sequences of ctx_b + q_len_b */
    uint64_t device_bytes_used;
    uint64_t host_bytes_used;
} asynclm_plan_info;

/* One row of the plan's work list, for inspection and tests (asynclm_plan_get_items). */
typedef struct asynclm_item_view {
    int32_t seq;        /* sequence b */
    int32_t kv_head;
    int32_t tok0;       /* first new token of the unit, index i inside the sequence's span */
    int32_t ntok;       /* tokens of the span covered by the unit */
    int32_t kv0, kv1;   /* key positions [kv0, kv1) the item reads (before causal clipping) */
    int32_t path;       /* 0 = warp body, 1 = span body */
    int32_t cta;        /* persistent CTA that processes the item; -1 = handed out at run time to
                           whichever CTA is free (items are listed in hand-out order) */
} asynclm_item_view;

int asynclm_version(void);
const char* asynclm_strerror(int status);
/* Text of the CUDA error behind the calling thread's most recent ASYNCLM_ERR_CUDA from
   asynclm_kv_append / asynclm_attn_mixed / asynclm_attn_mixed_static ("no error" if there was
   none). */
const char* asynclm_last_cuda_error(void);

/*
 * Upper bounds on the workspaces asynclm_plan needs for any batch with at most max_batch
 * sequences, max_total_q new tokens and max_total_pages page-table entries.  The device workspace
 * holds the uploaded plan and the fp32 partial outputs of split-KV items.  opts may be NULL.
 */
int asynclm_plan_workspace_size(const asynclm_shape* shape, const asynclm_plan_options* opts,
                                int32_t max_batch, int32_t max_total_q, int64_t max_total_pages,
                                size_t* host_bytes, size_t* device_bytes);

/*
 * Build the plan for one step (the "next decoding step" of Section 5.3, seen from attention).
 *
 * Validates the batch, tiles every (sequence, kv head) into query tiles and page-aligned KV chunks
 * (long contexts are split; partial results are merged by log-sum-exp inside asynclm_attn_mixed),
 * and decides who runs what: span tiles are packed whole where possible, largest first, onto as
 * few persistent CTAs as a load limit allows (a span of two row tiles that does not fit is divided
 * by rows before it is cut by keys); decode rows and short spans are cut into chunks (long pieces
 * first, short ones from a few units at the end) that the CTAs take from a queue at run time, one
 * atomic add per chunk, so that no cost model has to predict how fast each SM streams.  Results do
 * not depend on which CTA ran which chunk: partial results are indexed by chunk and merged in
 * chunk order.  Then ONE host->device copy of the packed plan is enqueued on `stream`.
 *
 * A plan holds a few counters in its device workspace (queue position, arrivals per split unit)
 * that every launch leaves at zero; launches that use the same plan must therefore not overlap on
 * the GPU (use one stream, as the layers of a model do, or order them with events).
 *
 *   host_ws / host_bytes  host memory (16-byte aligned; pinned recommended) that must stay
 *                         untouched until the copy has completed and for as long as the plan is
 *                         used.
 *   dev_ws / dev_bytes    device memory (256-byte aligned) owned by the caller.  dev_ws == NULL
 *                         builds the plan on the host only (no CUDA call is made; opts->num_sms
 *                         must be set); such a plan can be inspected but not executed.
 *   out_plan              receives a pointer into host_ws.
 *
 * The batch arrays may be freed as soon as the call returns.  Errors: INVALID_ARG (NULL, negative
 * or non-monotone indptr), UNSUPPORTED_SHAPE, PAGE_TABLE, WORKSPACE_TOO_SMALL, ARCH, CUDA.
 */
int asynclm_plan(const asynclm_shape* shape, const asynclm_plan_options* opts,
                 const asynclm_batch* batch, void* host_ws, size_t host_bytes,
                 void* dev_ws, size_t dev_bytes, void* stream, asynclm_plan_t** out_plan);

int asynclm_plan_get_info(const asynclm_plan_t* plan, asynclm_plan_info* info);

/* Copies up to `capacity` items into `items` (host); returns the number of items, or < 0. */
int asynclm_plan_get_items(const asynclm_plan_t* plan, asynclm_item_view* items, int32_t capacity);

/*
 * Interrupt append (Section 3.2: the block is inserted at the end of the context).  For every new
 * token row r = q_indptr[b] + i and kv head h, copies the head_dim bf16 values of k_new[r][h] and
 * v_new[r][h] bit for bit into
 *     kv_pool[page_indices[page_indptr[b] + (ctx_b + i) / page_size]][0 | 1][h][(ctx_b + i) % page_size].
 * No other byte of the pool is written.
 *
 *   k_new, v_new  device, bf16 [T][num_kv_heads][head_dim]
 *   kv_pool       device, bf16, layout above
 * Errors: INVALID_ARG, CUDA.
 */
int asynclm_kv_append(const asynclm_plan_t* plan, const void* k_new, const void* v_new,
                      void* kv_pool, void* stream);

/*
 * asynclm_kv_append with the rotary position embedding fused in, as the layers of a Llama-family model
 * (the models of the paper's evaluation, Section 6) need it: the key row of new token i of sequence b
 * is rotated by its position ctx_b + i before it is stored (rotate-half pairs (j, j + d/2), angle
 * position * rope_theta^(-2j / head_dim)), the value row is copied bit for bit, and, if q_inout is
 * given, the step's query rows [T][num_q_heads][head_dim] are rotated in place by the same positions.
 * Angles and products are evaluated in fp64 and rounded once to bf16.  Slots as in asynclm_kv_append.
 * Errors: INVALID_ARG (also rope_theta <= 1), CUDA.
 */
int asynclm_kv_append_rope(const asynclm_plan_t* plan, const void* k_new, const void* v_new, void* kv_pool,
                           void* q_inout, double rope_theta, void* stream);

/*
 * Mixed decode + interrupt-append attention (Section 5.3: the appended tokens are processed in the
 * next decoding step, alongside the other sequences' single-token decodes).  Must follow
 * asynclm_kv_append on the same stream: the new rows are read back from the pages.  For every new
 * token row r = q_indptr[b] + i and query head hq (kv head hq / G):
 *     s_j  = sm_scale * <q[r][hq], K_j>            j = 0 .. ctx_b + i
 *     out[r][hq] = sum_j softmax(s)_j V_j          lse[r][hq] = ln sum_j exp(s_j)
 * with K_j, V_j read through the page table.  bf16 inputs, fp32 accumulation, bf16 output rounded
 * to nearest even.  Slots beyond a sequence's length and unreferenced pages are never allowed to
 * influence the result, whatever bit patterns they hold.
 *
 *   q    device, bf16 [T][num_q_heads][head_dim]
 *   out  device, bf16 [T][num_q_heads][head_dim]
 *   lse  device, fp32 [T][num_q_heads], natural log; may be NULL
 * The current device must be the one the plan was made on.
 * Errors: INVALID_ARG (also: another device is current), CUDA.
 */
int asynclm_attn_mixed(const asynclm_plan_t* plan, const void* q, const void* kv_pool,
                       void* out, float* lse, void* stream);

/*
 * The whole step in one call: asynclm_kv_append followed by asynclm_attn_mixed, with the same
 * arguments, results and bit-exact pool contents, but without a separate append launch.  The
 * interrupt block still goes to the end of the context first (Section 3.2) and is then processed
 * with the other sequences' decodes (Section 5.3): every work item of the attention kernel copies
 * the new K/V rows it is about to read into their page slots itself, right before it fetches the
 * pages that hold them, so no part of the kernel waits for another, and every new row is written
 * (each new token attends to itself).  Items that read the same new rows write the same bytes; for
 * a step with a span of more than 64 tokens (the trap handler's recompute, say) that duplication
 * would dominate, and the call runs the append as a kernel of its own instead.
 *
 *   q             device, bf16 [T][num_q_heads][head_dim]
 *   k_new, v_new  device, bf16 [T][num_kv_heads][head_dim]
 *   kv_pool       device, bf16, layout above; written (the new rows) and read
 *   out, lse      as in asynclm_attn_mixed
 * Errors: INVALID_ARG, CUDA.
 */
int asynclm_step(const asynclm_plan_t* plan, const void* q, const void* k_new, const void* v_new,
                 void* kv_pool, void* out, float* lse, void* stream);

/*
 * Reads the device status word of the plan's workspace (synchronises `stream`).  *host_out is 0
 * if no kernel reported a problem, otherwise a code naming the bounded wait that ran out (1-39).
 * A library built with -DASYNCLM_DEBUG (build.py --debug) also checks, on the device, every page id
 * it is about to turn into an address and reports the first bad one here instead of using it:
 * 41 the append's row slot, 42 a span tile's page, 43 a decode chunk's page, 44 the append inside
 * asynclm_step; the access is left out (span tiles get zeros, decode chunks read page 0), nothing
 * faults.  The ordinary build relies on asynclm_plan, which validates every id on the host.
 * Returns ASYNCLM_OK or ASYNCLM_ERR_DEVICE_STATUS / ASYNCLM_ERR_CUDA.
 */
int asynclm_last_device_status(const asynclm_plan_t* plan, void* stream, int32_t* host_out);

/*
 * Trap handler data path (Section 5.4, "Trap Handler": a sequence paused by a trap need not hold its
 * KV cache in GPU memory while it waits).  The swapped form of a sequence is its pages in logical
 * order, one contiguous image of n_pages * (2 * num_kv_heads * page_size * head_dim * 2) bytes.
 *
 * asynclm_kv_swap_out copies page page_ids[j] of the pool to page j of the image: one gather kernel
 * into `staging`, then ONE device->host copy of the whole image.  asynclm_kv_swap_in is the reverse,
 * into whatever pages the sequence is given then (page_ids must be distinct): one host->device copy,
 * one scatter kernel.  Both are bit copies and asynchronous on `stream`; no other byte of the pool or
 * of the image is written.  A model with several layers calls them once per layer's pool.
 *
 *   shape        head shape and pool capacity (page ids are checked against num_pages)
 *   page_ids     host, int32 [n_pages]; may be reused as soon as the call returns if it is pageable
 *                memory, and must stay untouched until the stream reaches the copy if it is pinned
 *   kv_pool      device, layout above
 *   staging      device, 256-byte aligned, asynclm_kv_swap_staging_bytes(shape, n_pages) bytes, owned
 *                by the caller (the library allocates nothing)
 *   host_image   host (pinned recommended), 16-byte aligned, n_pages * page bytes
 * Errors: INVALID_ARG, PAGE_TABLE (id outside the pool; duplicate id on swap-in), CUDA.
 */
size_t asynclm_kv_swap_staging_bytes(const asynclm_shape* shape, int32_t n_pages);
int asynclm_kv_swap_out(const asynclm_shape* shape, const int32_t* page_ids, int32_t n_pages,
                        const void* kv_pool, void* staging, void* host_image, void* stream);
int asynclm_kv_swap_in(const asynclm_shape* shape, const int32_t* page_ids, int32_t n_pages,
                       void* kv_pool, void* staging, const void* host_image, void* stream);

/*
 * Trap handler decision (Section 5.4; worked example in Section 6.4, "Trap handling strategy"): swap
 * time grows linearly and recompute time quadratically with the context length.  The cache is kept
 * in GPU memory if both exceed the estimated wait until the next interrupt; otherwise the cheaper of
 * the two is chosen.  Host arithmetic only.  "Recompute" is an asynclm_plan / asynclm_step over the
 * whole context with kv_len_before = 0; its cost model is fitted by the caller from measurements
 * (bench.py --trap prints one for the attention part).
 */
typedef struct asynclm_trap_model {
    double swap_fixed_us, swap_us_per_token;
    double recompute_fixed_us, recompute_us_per_token, recompute_us_per_token2;
} asynclm_trap_model;
#define ASYNCLM_TRAP_KEEP      0
#define ASYNCLM_TRAP_SWAP      1
#define ASYNCLM_TRAP_RECOMPUTE 2
int asynclm_trap_decide(const asynclm_trap_model* model, int32_t context_tokens, double wait_us,
                        int32_t* decision, double* swap_us, double* recompute_us);

/*
 * Token monitor's hook into next-token selection (Section 5.1, "Token Monitor"; CML is Section 3): for
 * every sequence b, the allowed token with the largest logit is chosen (the lowest id among equal
 * logits; a NaN logit is never chosen) and the sequence's CML state advances.  Allowed tokens by state:
 *     0 TEXT  outside a block : ordinary tokens, [CALL], [TRAP]
 *     1 CALL  after [CALL]    : ordinary tokens (identifier or the call itself), [HEAD], [END]
 *     2 BODY  after [HEAD]    : ordinary tokens, [END]
 *     3 TRAP  after [TRAP]    : [END] only          ([TRAP][END] is the whole trap)
 * [INTR] is allowed nowhere: interrupts are injected by the system (Section 3.2), never generated.
 * flags_out: ASYNCLM_MONITOR_CALL when this token closed a function-call block (the executor is to be
 * notified), ASYNCLM_MONITOR_TRAP when it closed a trap (the trap handler is), ASYNCLM_MONITOR_CRITICAL
 * while the sequence is inside a function-call block after this token (interrupts are deferred).
 * Greedy selection is this library's reading: the paper leaves the sampling rule to the model's
 * decoding settings.
 *
 *   logits      device, [batch][row_stride] of bf16 (dtype 0) or fp32 (dtype 1), 16-byte aligned rows
 *   tokens      the five CML token ids (distinct, inside the vocabulary)
 *   state_in    device, int32 [batch]; token_out / state_out / flags_out device, int32 [batch]
 *               (state_out may alias state_in)
 *   workspace   device, 16-byte aligned, asynclm_token_monitor_workspace_bytes(batch) bytes, owned by
 *               the caller and all zero before the first call; every call leaves it all zero again (the
 *               slices of a row meet there), so calls that share it must not overlap on the GPU
 * One kernel on `stream`; vocab * element size bytes are read per sequence; batch <= 65535.
 * Errors: INVALID_ARG, CUDA.
 */
typedef struct asynclm_cml_tokens {
    int32_t call, intr, trap, end, head;
} asynclm_cml_tokens;
#define ASYNCLM_DTYPE_BF16 0
#define ASYNCLM_DTYPE_F32  1
#define ASYNCLM_MONITOR_CALL     1
#define ASYNCLM_MONITOR_TRAP     2
#define ASYNCLM_MONITOR_CRITICAL 4
size_t asynclm_token_monitor_workspace_bytes(int32_t batch);
int asynclm_token_monitor_step(const void* logits, int32_t dtype, int32_t batch, int32_t vocab,
                               int64_t row_stride, const asynclm_cml_tokens* tokens,
                               const int32_t* state_in, int32_t* token_out, int32_t* state_out,
                               int32_t* flags_out, void* workspace, void* stream);

/*
 * Latency model (Section 6.3, "Latency Analysis", and Appendix A) for n independent function calls
 * with token-generation latency gen[i] > 0 and execution time exec[i] > 0 (any one unit of time):
 *     l_sync     = sum gen + sum exec                  calls generated and executed one after the other
 *     l_sync_par = sum gen + max exec                  generated in sequence, executed concurrently
 *     l_async    = max_i (gen[o_1] + .. + gen[o_i] + exec[o_i])   for the longest-execution-first order o,
 * which is the paper's max_f (E(f) + sum of G over pred(f)), and speedup_estimate = 1 + mean exec /
 * mean gen (Theorem 6.2).  lpt_order (host, [n], may be NULL) receives o.
 * asynclm_async_latency_of_order evaluates the same completion times for any generation order
 * (a permutation of 0..n-1); completion[i] (host, [n], may be NULL) is when call i returns, i.e.
 * when its interrupt becomes available.  Host arithmetic only.  Errors: INVALID_ARG.
 */
typedef struct asynclm_latency {
    double l_sync, l_sync_par, l_async, speedup_estimate;
} asynclm_latency;
int asynclm_latency_model(const double* gen, const double* exec, int32_t n, asynclm_latency* out,
                          int32_t* lpt_order);
int asynclm_async_latency_of_order(const double* gen, const double* exec, const int32_t* order, int32_t n,
                                   double* latency, double* completion);

/*
 * Measurement aid (no counterpart in the paper, none of the method's arithmetic): reads n_blocks
 * pairs of K/V blocks of the pool with plain 16-byte loads, as fast as the GPU can, so that the
 * attention kernels' rate can be held against a read-only ceiling for the same scattered blocks.
 *
 *   kv_pool          device, 16-byte aligned
 *   k_block_offsets  device, int64 [n_blocks]: byte offset of a K block (one page, one kv head)
 *   v_delta_bytes    distance from a K block to its V block (num_kv_heads * page_size * head_dim * 2)
 *   block_bytes      page_size * head_dim * 2
 *   sink             device, 4 bytes, left alone unless an XOR of all the data hits one chosen value
 * Errors: INVALID_ARG, CUDA.
 */
int asynclm_read_ceiling(const void* kv_pool, const int64_t* k_block_offsets, int64_t n_blocks,
                         int64_t v_delta_bytes, int32_t block_bytes, void* sink, void* stream);

/*
 * asynclm_attn_mixed with no caller-provided scratch (the paper has no counterpart to this call; it
 * exists for deployment reasons only).
 *
 * Some callers cannot allocate device memory for the library: a server that gave all of HBM to
 * its KV pool and weights at start-up, a plug-in that may not touch its host's memory pool, a
 * latency-critical loop in which cudaMalloc is banned because it can stall the device.  For them
 * the fp32 partial results of split contexts (the only scratch the attention kernels use) are kept
 * in a fixed array of ASYNCLM_STATIC_SCRATCH_BYTES that is compiled into the library; every GPU
 * that uses the library holds that array until the process exits.  The call itself performs no
 * allocation and no free, on the device or through any library.
 *
 * Arguments, results and numerics are exactly those of asynclm_attn_mixed, computed by the same
 * kernels.  The plan's device workspace is still the caller's (it holds the uploaded plan), but
 * the part of it reserved for partial results is left unused.
 *
 *   - A plan whose partial results need more than ASYNCLM_STATIC_SCRATCH_BYTES
 *     (align256(partial_rows * G * head_dim * 4) + align256(partial_rows * G * 4), with
 *     partial_rows from asynclm_plan_get_info) is refused with
 *     ASYNCLM_ERR_STATIC_SCRATCH_TOO_SMALL before anything is launched; plan with a longer
 *     kv_chunk_tokens, or use asynclm_attn_mixed.
 *   - The first call on each device looks up the array's device address (one
 *     cudaGetSymbolAddress with that device current).  Make that first call before starting any
 *     stream capture on that device, and while the device still has the array's size to spare: the
 *     driver may set the library image's data up only then.
 *   - All calls on a device share the one array, and it keeps whatever the previous call left in
 *     it.  Nothing in it has to start at zero: each call writes every partial row before reading
 *     it.  Two calls whose kernels may overlap on the GPU (different streams, or different threads
 *     or processes' streams of one process image) race on the array; run them on one stream or
 *     order them with events.
 * Errors: INVALID_ARG, STATIC_SCRATCH_TOO_SMALL, CUDA.
 */
#define ASYNCLM_STATIC_SCRATCH_BYTES (16u << 20)
int asynclm_attn_mixed_static(const asynclm_plan_t* plan, const void* q, const void* kv_pool,
                              void* out, float* lse, void* stream);
/* The compiled-in value of ASYNCLM_STATIC_SCRATCH_BYTES. */
size_t asynclm_static_scratch_bytes(void);

#ifdef __cplusplus
}
#endif
#endif /* ASYNCLM_H_ */
