/*
 * rollart.h -- C ABI of the B200 (sm_100a) paged-KV rollout-attention library.
 *
 * Scope.  The rollout stage of agentic RL advances many independent trajectories; each one
 * appends tokens to its own growing context (an observation from the environment, then the
 * tokens of the next action) while the inference worker runs one decode or prefill step after
 * another over the batch of requests it currently holds (paper Sec. 6.1, trajectory-level rollout
 * and step-wise command processing; Sec. 3.1: decoding is memory-bandwidth bound, observation
 * prefill compute bound).  This library is the attention
 * part of that engine step over a paged bf16 KV cache:
 *
 *   rollart_kv_append       write the new tokens' K/V rows into the trajectories' pages
 *   rollart_decode_attn     one new query token per trajectory attends to its whole context
 *   rollart_obs_chunk_attn  a chunk of new observation tokens attends to the cached prefix and,
 *                           causally, to itself
 *
 * The paper gives no formula for the step; the operation is standard scaled-dot-product softmax
 * attention with grouped query heads, defined precisely below.
 *
 * Conventions.
 *   - Plain C99 types only.  Pointers marked [device] are CUDA device pointers in the context's
 *     device; [host] are ordinary host pointers.  `stream` is a cudaStream_t passed as void*
 *     (NULL = the legacy default stream).
 *   - The caller owns every buffer it passes.  The library owns only what rollart_create
 *     allocates (one workspace, one status word, one pinned host word).
 *   - kv_append / decode_attn / obs_chunk_attn enqueue work on `stream` and return without
 *     synchronising and without allocating.  Errors the host can see (bad shapes, NULL pointers,
 *     workspace too small) are returned at once and nothing is enqueued.  Errors only the device
 *     can see (a page id outside the pool, a length that overruns its page-table row) make the
 *     kernel skip that access and record a code in the device status word, which
 *     rollart_check() fetches; a kernel never traps and every in-kernel wait is bounded.
 *   - A context is not thread safe; use one per host thread / stream.
 *   - head_dim must be 128; page_size 16, 32 or 64; num_q_heads a multiple of num_kv_heads with
 *     at most 16 query heads per kv head.  Anything else returns ROLLART_ERR_UNSUPPORTED.
 *
 * Data layout.
 *   pools       bf16 [num_pages][num_kv_heads][page_size][head_dim], K and V in separate pools,
 *               both 16-byte aligned (a (page, head) tile is one contiguous block)
 *   page_table  int32 [num_traj][max_pages_per_traj] row major; entry i of row t is the physical
 *               page of logical page i.  Entries at or beyond ceil(len/page_size) are never read.
 *   seq_lens    int32 [num_traj], tokens
 *   Token at logical position pos of trajectory t, kv head h:
 *               pool[page_table[t][pos / page_size]][h][pos % page_size][0..head_dim)
 *   Query head hq reads kv head hq / (num_q_heads / num_kv_heads).
 *   Slots that hold no live token (page tails, unowned pages) may contain anything, including
 *   NaN and Inf bit patterns; results never depend on them.
 */
#ifndef ROLLART_H_
#define ROLLART_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    ROLLART_OK = 0,
    ROLLART_ERR_INVALID_ARG = 1, /* NULL pointer, negative count, overlapping in/out buffers   */
    ROLLART_ERR_UNSUPPORTED = 2, /* head_dim, page_size or group size outside the supported set */
    ROLLART_ERR_WORKSPACE = 3,   /* the context's workspace is too small for this call         */
    ROLLART_ERR_CUDA = 4,        /* a CUDA runtime/driver call failed (see rollart_last_error) */
    ROLLART_ERR_BOUNDS = 5,      /* device saw a page id / length / trajectory id out of range */
    ROLLART_ERR_TIMEOUT = 6      /* a bounded in-kernel wait ran out                           */
} rollart_status;

typedef struct rollart_ctx rollart_ctx; /* opaque */

typedef struct {
    void *k_pool; /* [device] bf16 [num_pages][num_kv_heads][page_size][head_dim] */
    void *v_pool; /* [device] same shape */
    int32_t num_pages;
    int32_t page_size;
    int32_t num_kv_heads;
    int32_t head_dim;
} rollart_kv_pool;

typedef struct {
    const int32_t *page_table; /* [device] int32 [num_traj][max_pages_per_traj] */
    int32_t max_pages_per_traj;
    const int32_t *seq_lens; /* [device] int32 [num_traj] */
    int32_t num_traj;
} rollart_trajs;

/* Bytes of workspace that calls with at most max_items items (trajectories per call),
 * these head counts and contexts up to max_seq_len tokens need.  Pure host arithmetic. */
size_t rollart_workspace_size(int32_t max_items, int32_t num_q_heads, int32_t num_kv_heads, int32_t max_seq_len);

/* Creates a context on CUDA device `device` and allocates its workspace (workspace_bytes, may
 * be 0 if only kv_append is used).  *out [host] receives the context.  The only call that
 * allocates device memory; rollart_destroy frees it. */
rollart_status rollart_create(rollart_ctx **out, int device, size_t workspace_bytes);
rollart_status rollart_destroy(rollart_ctx *ctx);

/*
 * KV append (Sec. 6.1: every turn the trajectory's history grows by the observation and the
 * generated action; the engine step writes the new tokens' K/V into the cache before attending).
 *
 *   trajs->seq_lens   lengths BEFORE the append.
 *   traj_ids          [device] int32 [n_items], trajectory of item i; NULL = identity (item i is
 *                     trajectory i).  A trajectory may appear at most once per call.
 *   new_indptr        [device] int32 [n_items+1], item i appends rows new_indptr[i] ..
 *                     new_indptr[i+1]-1 of k_new / v_new; new_indptr[0] = 0,
 *                     new_indptr[n_items] = total_new (the host passes total_new as well).
 *   k_new, v_new      [device] bf16 [total_new][num_kv_heads][head_dim], 16-byte aligned.
 *   seq_lens_out      [device] int32 [num_traj] or NULL; entry traj_ids[i] receives len + n_i,
 *                     other entries are left alone.  Must not overlap trajs->seq_lens.
 *
 * Row r of item i lands at logical position len + r.  The pages covering the new positions must
 * already be present in the page table (page allocation is the caller's).  The copy is bit exact;
 * no other byte of the pools changes.  Device-side errors (ROLLART_ERR_BOUNDS): trajectory id out
 * of range, negative length, position beyond max_pages_per_traj * page_size, page id outside
 * [0, num_pages), a new_indptr that is not non-decreasing from 0 to total_new (a row that falls
 * outside its item's range): the offending row is skipped.
 */
rollart_status rollart_kv_append(rollart_ctx *ctx, const rollart_kv_pool *pool, const rollart_trajs *trajs,
                                 const int32_t *traj_ids, const int32_t *new_indptr, int32_t n_items,
                                 int32_t total_new, const void *k_new, const void *v_new, int32_t *seq_lens_out,
                                 void *stream);

/*
 * KV gather: the inverse of rollart_kv_append, for handing a trajectory's cache to another worker
 * (Sec. 6.3: with prefill/decode disaggregation the prefill worker's KV moves to a decode worker;
 * Sec. 6.1: a trajectory resumes on another inference worker).  Item i copies the first
 * n_i = out_indptr[i+1] - out_indptr[i] tokens of trajectory traj_ids[i] (NULL = identity) from its
 * pages into rows out_indptr[i] .. of k_out / v_out ([device] bf16 [total_rows][num_kv_heads][head_dim],
 * 16-byte aligned); the receiving side stores them with rollart_kv_append onto its own pages.
 * Bit copy.  n_i > seq_lens[t], a trajectory id or a page id out of range, and an out_indptr that is not
 * non-decreasing from 0 to total_rows are device-side ROLLART_ERR_BOUNDS errors; the offending rows are
 * left unwritten.
 */
rollart_status rollart_kv_gather(rollart_ctx *ctx, const rollart_kv_pool *pool, const rollart_trajs *trajs,
                                 const int32_t *traj_ids, const int32_t *out_indptr, int32_t n_items, int32_t total_rows,
                                 void *k_out, void *v_out, void *stream);

/*
 * Page bookkeeping between engine steps (Sec. 6.1: the inference worker processes ADD and ABORT commands
 * between steps; Sec. 6.2: trajectories that have become too stale are evicted).  The free pages are a
 * stack: free_pages [device] int32 [capacity] with *free_count [device] live entries, top at the end.
 *
 * rollart_pages_reserve: item i (trajectory traj_ids[i], NULL = identity) is about to grow by new_tokens[i]
 *   [device] tokens; it pops ceil((len + n) / page_size) - ceil(len / page_size) pages, items in order, and
 *   stores them in the next entries of its page-table row.  seq_lens is only read (rollart_kv_append moves
 *   the lengths).  A new trajectory is one with len = 0.
 * rollart_pages_release: item i pushes all pages of trajectory traj_ids[i] (logical order, items in order),
 *   sets those table entries to -1 and seq_lens[t] to 0.
 *
 * page_table is the same [num_traj][max_pages_per_traj] table the other calls read.  Both calls are
 * deterministic and all-or-nothing: if the stack is too small (or too full), a trajectory id or length is
 * out of range, or a row would overflow, nothing changes and ROLLART_ERR_BOUNDS is recorded for
 * rollart_check.  A trajectory may appear at most once per call.
 */
rollart_status rollart_pages_reserve(rollart_ctx *ctx, int32_t *free_pages, int32_t *free_count, int32_t page_size,
                                     int32_t *page_table, int32_t max_pages_per_traj, const int32_t *seq_lens,
                                     int32_t num_traj, const int32_t *traj_ids, const int32_t *new_tokens, int32_t n_items,
                                     void *stream);
rollart_status rollart_pages_release(rollart_ctx *ctx, int32_t *free_pages, int32_t *free_count, int32_t capacity,
                                     int32_t page_size, int32_t *page_table, int32_t max_pages_per_traj, int32_t *seq_lens,
                                     int32_t num_traj, const int32_t *traj_ids, int32_t n_items, void *stream);

/*
 * Stale eviction (Sec. 6.2, asynchronous bound alpha: with the agent LLM at version n, a trajectory in flight must
 * have been started by a version no older than n - alpha; trajectories outside this window are aborted before the
 * next batch is formed).  The caller keeps the version each trajectory was started under in start_version; this call
 * selects the stale ones on the device and returns their pages, so that the selection needs no round trip to the host:
 *
 *   stale(t)  =  seq_lens[t] > 0  and  start_version[t] < current_version - alpha          (alpha >= 0)
 *
 * The stale trajectories, in ascending order of t, are released exactly as rollart_pages_release would release that
 * list (pages pushed in logical order, table entries set to -1, seq_lens[t] set to 0).
 *   start_version   [device] int32 [num_traj]
 *   evicted_ids     [device] int32 [num_traj]: receives the released trajectories, in ascending order
 *   n_evicted       [device] int32: receives how many there are
 * Deterministic and all-or-nothing: if the stack cannot take the pages (capacity), or a length is negative or longer
 * than its table row, nothing changes, *n_evicted is set to 0 and ROLLART_ERR_BOUNDS is recorded for rollart_check.
 */
rollart_status rollart_pages_evict_stale(rollart_ctx *ctx, int32_t *free_pages, int32_t *free_count, int32_t capacity,
                                         int32_t page_size, int32_t *page_table, int32_t max_pages_per_traj, int32_t *seq_lens,
                                         int32_t num_traj, const int32_t *start_version, int32_t current_version, int32_t alpha,
                                         int32_t *evicted_ids, int32_t *n_evicted, void *stream);

/*
 * Decode attention (Sec. 3.1: the decoding phase is bound by reading the whole context once per
 * generated token).  For item i with trajectory t = traj_ids[i], L = seq_lens[t] (lengths AFTER
 * the append: the query attends to its own K/V), query head hq, kv head h = hq / g:
 *
 *   s_j = sm_scale * <q[i][hq], K_t[j][h]>,  j = 0..L-1
 *   out[i][hq] = sum_j softmax(s)_j * V_t[j][h]          (bf16, round to nearest even)
 *   lse[i][hq] = log sum_j exp(s_j)                       (fp32, natural log; optional)
 *
 *   q, out            [device] bf16 [n_items][num_q_heads][head_dim], 16-byte aligned.
 *   lse               [device] fp32 [n_items][num_q_heads] or NULL.
 *                     out and lse are only stored to, so either may also be page-locked host memory that the
 *                     device can address (cudaHostAlloc under unified addressing): the result then reaches the
 *                     host with the kernel's own stores and is readable once the stream has been synchronised.
 *                     The same holds for the fused and the fp8 decode calls below.
 *   max_seq_len       [host value] an upper bound on every L of this call; sizes the schedule and
 *                     the workspace check (values above max_pages_per_traj * page_size are
 *                     clamped to it).  A longer trajectory is reported as ROLLART_ERR_BOUNDS.
 *   L = 0 gives out = 0 and lse = -inf.
 * Arithmetic: bf16 operands, fp32 scores, softmax and accumulation; softmax weights are rounded
 * to bf16 before they multiply V.  The schedule (how contexts are split over thread blocks and
 * merged with a log-sum-exp combine) is a fixed function of the lengths, so reruns are bit
 * identical.
 */
rollart_status rollart_decode_attn(rollart_ctx *ctx, const rollart_kv_pool *pool, const rollart_trajs *trajs,
                                   const int32_t *traj_ids, int32_t n_items, int32_t max_seq_len, const void *q,
                                   int32_t num_q_heads, float sm_scale, void *out, float *lse, void *stream);

/*
 * Fused decode step: rollart_kv_append of one new token per item followed by rollart_decode_attn, in a single
 * kernel launch (the engine executes a decode step once per generated token, Sec. 6.1, so launches count).
 * trajs->seq_lens holds the lengths BEFORE the step; item i stores k_new[i] / v_new[i] ([device] bf16
 * [n_items][num_kv_heads][head_dim], 16-byte aligned) at position len of trajectory traj_ids[i] and its query
 * attends to all len + 1 keys.  max_seq_len bounds the lengths AFTER the step.  seq_lens_out ([device] int32
 * [num_traj] or NULL, must not overlap seq_lens) receives len + 1 for the trajectories named.  Results (pool
 * bytes, out, lse) are identical to the two separate calls.  Device-side errors as for the two calls, with one
 * difference: an item that the device rejects (its new position has no page-table entry, or len + 1 exceeds
 * max_seq_len) is skipped as a whole: its row is not stored, its seq_lens_out entry is left unwritten, its out row
 * is 0, so a trajectory that outgrows the bound of a captured decode loop stops advancing instead of leaving
 * unwritten rows behind.
 */
rollart_status rollart_append_decode_attn(rollart_ctx *ctx, const rollart_kv_pool *pool, const rollart_trajs *trajs,
                                          const int32_t *traj_ids, int32_t n_items, int32_t max_seq_len, const void *k_new,
                                          const void *v_new, const void *q, int32_t num_q_heads, float sm_scale, void *out,
                                          float *lse, int32_t *seq_lens_out, void *stream);

/*
 * The fused decode step driven from host buffers: q, k_new and v_new are [host] page-locked buffers (cudaHostAlloc /
 * cudaHostRegister), layouts as for rollart_append_decode_attn.  The call enqueues their copy into `staging`
 * (cudaMemcpyAsync on `stream`: one copy if the three buffers follow one another in host memory in the order q, k_new,
 * v_new, else three) and then the fused step from there.  `out` and `lse` may be device buffers or page-locked host
 * buffers (see rollart_decode_attn), so a whole step can go host -> device -> host inside this one call; the host may
 * read the result once the stream has been synchronised and may rewrite its input buffers from then on.
 *   staging   [device] 256-byte aligned, at least rollart_host_staging_size(n_items, num_q_heads, num_kv_heads)
 *             bytes; owned by the caller.  Too small: ROLLART_ERR_WORKSPACE, nothing is enqueued.
 * Pageable host buffers are not refused, but their copy is staged by the driver and the call may block until it is
 * done.  Everything else as for rollart_append_decode_attn.  Launches one kernel.
 */
size_t rollart_host_staging_size(int32_t n_items, int32_t num_q_heads, int32_t num_kv_heads);
rollart_status rollart_append_decode_attn_host(rollart_ctx *ctx, const rollart_kv_pool *pool, const rollart_trajs *trajs,
                                               const int32_t *traj_ids, int32_t n_items, int32_t max_seq_len,
                                               const void *k_new_host, const void *v_new_host, const void *q_host,
                                               int32_t num_q_heads, float sm_scale, void *out, float *lse,
                                               int32_t *seq_lens_out, void *staging, size_t staging_bytes, void *stream);

/*
 * fp8 KV pools.  Decoding is bound by reading the whole context once per generated token (Sec. 3.1), so a cache held
 * in 8 bits halves the bytes of a decode step.  The two calls below are rollart_kv_append and rollart_decode_attn for
 * pools whose elements are E4M3 codes (OCP 8-bit floating point: 1 sign, 4 exponent bits with bias 7, 3 mantissa
 * bits, no infinities, largest finite value 448): pool->k_pool / v_pool are [device] uint8
 * [num_pages][num_kv_heads][page_size][head_dim], 16-byte aligned, with one scale per pool and call: a key is
 * k_scale * value(code), a value is v_scale * value(code).  Both scales must be positive and finite.
 *
 * rollart_kv_append_fp8: arguments as rollart_kv_append; k_new / v_new are bf16.  Every element is stored as
 *   code = nearest E4M3 code (ties to even, magnitudes above 448 saturate to +-448) of x * (1 / scale), the
 *   reciprocal and the product each rounded to fp32.  No other byte of the pools changes.
 * rollart_decode_attn_fp8: arguments and result as rollart_decode_attn (q, out bf16; lse fp32) with
 *   s_j = sm_scale * k_scale * <q, value(K code)>, out = v_scale * sum_j softmax(s)_j * value(V code).
 *   Arithmetic: the codes and the query are converted to f16 (exact for the codes; a query element beyond the f16
 *   range, |q| > 65504, is not supported), fp32 scores, softmax and accumulation; softmax weights are rounded to f16
 *   before they multiply V.  Same schedule, same workspace, same errors as rollart_decode_attn.
 * rollart_append_decode_attn_fp8: rollart_kv_append_fp8 of one new token per item followed by
 *   rollart_decode_attn_fp8, in a single kernel launch; arguments as rollart_append_decode_attn plus the two scales.
 *   Pool bytes, out and lse are identical to the two separate calls.
 * rollart_kv_gather_fp8 / rollart_kv_append_fp8_codes: the hand-over of an fp8 cache to another worker (Sec. 6.3), as
 *   rollart_kv_gather / rollart_kv_append do it for bf16 pools.  The gather copies the codes of the first n_i tokens of
 *   each listed trajectory into k_out / v_out ([device] uint8 [total_rows][num_kv_heads][head_dim], 16-byte aligned);
 *   the append stores rows of codes (k_codes / v_codes, same layout) onto the receiving pool's pages.  Both are bit
 *   copies: the scales travel with the caller and must be the same on both sides.  Errors as for the bf16 calls.
 * The paper does not describe a cache format; the fp8 pool is this library's option.
 */
rollart_status rollart_kv_append_fp8(rollart_ctx *ctx, const rollart_kv_pool *pool, const rollart_trajs *trajs,
                                     const int32_t *traj_ids, const int32_t *new_indptr, int32_t n_items,
                                     int32_t total_new, const void *k_new, const void *v_new, float k_scale, float v_scale,
                                     int32_t *seq_lens_out, void *stream);
rollart_status rollart_decode_attn_fp8(rollart_ctx *ctx, const rollart_kv_pool *pool, const rollart_trajs *trajs,
                                       const int32_t *traj_ids, int32_t n_items, int32_t max_seq_len, const void *q,
                                       int32_t num_q_heads, float sm_scale, float k_scale, float v_scale, void *out,
                                       float *lse, void *stream);
rollart_status rollart_append_decode_attn_fp8(rollart_ctx *ctx, const rollart_kv_pool *pool, const rollart_trajs *trajs,
                                              const int32_t *traj_ids, int32_t n_items, int32_t max_seq_len,
                                              const void *k_new, const void *v_new, const void *q, int32_t num_q_heads,
                                              float sm_scale, float k_scale, float v_scale, void *out, float *lse,
                                              int32_t *seq_lens_out, void *stream);

rollart_status rollart_kv_gather_fp8(rollart_ctx *ctx, const rollart_kv_pool *pool, const rollart_trajs *trajs,
                                     const int32_t *traj_ids, const int32_t *out_indptr, int32_t n_items, int32_t total_rows,
                                     void *k_out, void *v_out, void *stream);

rollart_status rollart_kv_append_fp8_codes(rollart_ctx *ctx, const rollart_kv_pool *pool, const rollart_trajs *trajs,
                                           const int32_t *traj_ids, const int32_t *new_indptr, int32_t n_items,
                                           int32_t total_new, const void *k_codes, const void *v_codes,
                                           int32_t *seq_lens_out, void *stream);

/*
 * Group decode step: rollart_decode_attn for a batch whose items form groups that share a prompt prefix.
 * The paper trains with GRPO at a group size of 8 and runs the rollout engine with prefix caching (Sec. 7.1),
 * so the members of a group hold the same first tokens and, with prefix sharing, their page-table rows list
 * the same physical pages there.  Results are those of rollart_decode_attn (same definition of out and lse);
 * the shared pages are read once per group instead of once per member: the prefix part runs on the tensor
 * cores with the members' query rows stacked into one tile, the private remainder through the split-KV decode
 * kernel, and the two parts are merged from their log-sum-exps (fp32 partial results, one rounding to bf16).
 *
 *   group_indptr   [device] int32 [n_groups + 1]: group j holds items group_indptr[j] .. group_indptr[j+1]-1
 *                  (consecutive items of the batch; starts at 0, ends at n_items, non-decreasing).
 *   shared_lens    [device] int32 [n_groups]: tokens of the shared prefix; a whole number of pages (0 allowed),
 *                  not longer than any member's seq_lens entry.  For pages below shared_lens[j] / page_size the
 *                  members' page-table rows must hold identical entries.
 *   other arguments as for rollart_decode_attn.
 * Workspace: rollart_group_decode_workspace_size(...) bytes (more than rollart_workspace_size: it adds two
 * fp32 partial results per item); a smaller workspace returns ROLLART_ERR_WORKSPACE and launches nothing.
 * Device-side checks: a group_indptr that is not such a partition, a shared length that is not page aligned
 * or exceeds a member's length, and members whose rows differ on the shared pages are each reported as
 * ROLLART_ERR_BOUNDS (the results of that call are then undefined, memory outside out/lse is not touched).
 * Launches four kernels.  Groups of one member and shared_lens of 0 are valid (no saving).
 */
size_t rollart_group_decode_workspace_size(int32_t max_items, int32_t num_q_heads, int32_t num_kv_heads,
                                           int32_t max_seq_len);
rollart_status rollart_group_decode_attn(rollart_ctx *ctx, const rollart_kv_pool *pool, const rollart_trajs *trajs,
                                         const int32_t *traj_ids, int32_t n_items, const int32_t *group_indptr,
                                         const int32_t *shared_lens, int32_t n_groups, int32_t max_seq_len, const void *q,
                                         int32_t num_q_heads, float sm_scale, void *out, float *lse, void *stream);

/*
 * Group decode over fp8 pools: rollart_group_decode_attn with keys k_scale * value(code) and values
 * v_scale * value(code) (pools of E4M3 codes as for rollart_decode_attn_fp8).  The shared prefixes, one per group,
 * are expanded to bf16 into `scratch` for the tensor-core kernel (as rollart_obs_chunk_attn_fp8 does for whole
 * contexts); the private remainders are read as codes by the fp8 decode kernel.
 *   scratch   [device] 256-byte aligned, sized as for rollart_obs_chunk_attn_fp8 with the groups as items and the shared
 *             prefixes as their contexts (rollart_obs_chunk_fp8_scratch_size(n_groups, ...) always suffices); owned by
 *             the caller, contents undefined afterwards.
 * Workspace, checks and errors as for rollart_group_decode_attn; scratch errors as for rollart_obs_chunk_attn_fp8.
 * Launches six kernels.
 */
rollart_status rollart_group_decode_attn_fp8(rollart_ctx *ctx, const rollart_kv_pool *pool, const rollart_trajs *trajs,
                                             const int32_t *traj_ids, int32_t n_items, const int32_t *group_indptr,
                                             const int32_t *shared_lens, int32_t n_groups, int32_t max_seq_len, const void *q,
                                             int32_t num_q_heads, float sm_scale, float k_scale, float v_scale, void *out,
                                             float *lse, void *scratch, size_t scratch_bytes, void *stream);

/*
 * Observation-chunk attention (Sec. 2.1 / 3.1: many-turn tasks keep re-entering generation with
 * a longer history; with the prefix cached only the newly arrived observation tokens are
 * computed, a dense compute-bound block).  Item i owns query rows q_indptr[i] .. q_indptr[i+1]-1;
 * they are the LAST n_i tokens of trajectory t = traj_ids[i] (already appended; L = seq_lens[t]).
 * Row j (0-based within the chunk) sees keys 0 .. L - n_i + j: the whole prior context, and the
 * chunk causally including itself.  Same formula, layout of q/out/lse ([total_q][...]) and
 * arithmetic as rollart_decode_attn; n_i = 1 is exactly a decode step.  n_i > L is a
 * ROLLART_ERR_BOUNDS device error for that item.
 * Per 1024 items the call enqueues a 576-byte clear and two kernels: the first keeps, per query row, the largest
 * score among the row's first 128 keys as the reference of its exponentials for the whole row; a block of rows in which
 * some later score lies more than 64 powers of two above that reference (or is not finite) is marked in a bitmap that
 * belongs to the context and is computed again by the second kernel, which moves its reference as it goes; the other
 * blocks of the second kernel return at once.  Results do not depend on which kernel produced them beyond rounding.
 * One chunk call per context may be in flight (the bitmap, like the status word, is the context's).
 */
rollart_status rollart_obs_chunk_attn(rollart_ctx *ctx, const rollart_kv_pool *pool, const rollart_trajs *trajs,
                                      const int32_t *traj_ids, const int32_t *q_indptr, int32_t n_items,
                                      int32_t total_q, int32_t max_seq_len, const void *q, int32_t num_q_heads,
                                      float sm_scale, void *out, float *lse, void *stream);

/*
 * Observation-chunk attention over fp8 pools (pool->k_pool / v_pool hold E4M3 codes as for rollart_decode_attn_fp8;
 * the chunk's own tokens have been appended with rollart_kv_append_fp8).  Same rows, mask and formula as
 * rollart_obs_chunk_attn with keys k_scale * value(code) and values v_scale * value(code):
 *   s_j = sm_scale * k_scale * <q, value(K code)>,  out = v_scale * sum_j softmax(s)_j * value(V code).
 * This phase is bound by the tensor cores, not by reading the cache (Sec. 3.1), so the call first expands the listed
 * trajectories' contexts to bf16 (exact: every finite E4M3 value is a bf16 value) into `scratch` and then runs the
 * bf16 kernel over that copy; the expansion is one pass at the HBM rate, a few per cent of the attention.
 *   scratch        [device] 256-byte aligned; owned by the caller, contents undefined afterwards.  It holds two bf16
 *                  pools into which the items' pages are packed one after the other (a running sum of
 *                  ceil(L / page_size) taken on the device), plus a page table, lengths and offsets for them.
 *                  rollart_obs_chunk_fp8_scratch_size(n_items, num_kv_heads, page_size, max_seq_len) bytes always
 *                  suffice (every item at the bound); rollart_obs_chunk_fp8_scratch_size_for_pages(..., total_pages)
 *                  gives the size for a caller who knows a bound on the pages the listed contexts hold (its page
 *                  allocator does).  A buffer that cannot hold one page returns ROLLART_ERR_WORKSPACE and launches
 *                  nothing; one that turns out smaller than the contexts is a device-side ROLLART_ERR_WORKSPACE:
 *                  the items that do not fit are skipped (their rows of out are not written).
 *   other arguments, errors and arithmetic as for rollart_obs_chunk_attn (bf16 operands: here the exact code values).
 * Launches four kernels (plan, expansion, and the two of rollart_obs_chunk_attn).  A code of NaN in a live slot gives NaN results for the rows that see it, as a bf16 NaN would.
 */
size_t rollart_obs_chunk_fp8_scratch_size(int32_t n_items, int32_t num_kv_heads, int32_t page_size, int32_t max_seq_len);
size_t rollart_obs_chunk_fp8_scratch_size_for_pages(int32_t n_items, int32_t num_kv_heads, int32_t page_size,
                                                    int32_t max_seq_len, int64_t total_pages);
rollart_status rollart_obs_chunk_attn_fp8(rollart_ctx *ctx, const rollart_kv_pool *pool, const rollart_trajs *trajs,
                                          const int32_t *traj_ids, const int32_t *q_indptr, int32_t n_items,
                                          int32_t total_q, int32_t max_seq_len, const void *q, int32_t num_q_heads,
                                          float sm_scale, float k_scale, float v_scale, void *out, float *lse,
                                          void *scratch, size_t scratch_bytes, void *stream);

/*
 * Decode attention for callers that cannot allocate device memory.  The paper has no counterpart
 * to this call; it exists for the way the library gets embedded.
 *
 * Who needs it: a serving engine that has already handed every byte of device memory to its own
 * KV-cache pool, a plug-in running inside someone else's process under a "no cudaMalloc after
 * start-up" rule, or a latency-critical loop in which an allocation (which synchronises the
 * device and may fail) is not acceptable.  Such a caller cannot use rollart_create, because that
 * is where the regular path allocates its workspace.
 *
 * What it does: exactly what rollart_decode_attn does (same kernels, same arithmetic, same
 * meaning of every shared argument), without a context.  The partial results, the ticket counters
 * and a status word live in a fixed array of about 19.2 MB that is part of the library image.
 * The call performs no cudaMalloc / cudaFree and calls nothing that does.  The array itself is
 * not free, though: the CUDA runtime loads a library's kernels and fixed arrays when they are
 * first used, so the first call on a device (see below) is the moment at which that GPU gives up
 * the 19.2 MB, and it keeps them until the process exits.
 *
 *   device          CUDA device that owns every [device] pointer of the call.
 *   device_status   [device] int32[4] or NULL.  Cleared on `stream` at the start of the call;
 *                   afterwards word 0 holds 0 or the first device-side rollart_status
 *                   (ROLLART_ERR_BOUNDS / ROLLART_ERR_TIMEOUT), word 1 the offending value.  With
 *                   NULL, device-side errors are recorded inside the fixed array and not reported.
 *   err_buf/err_len [host] optional buffer that receives a NUL-terminated description whenever
 *                   the return value is not ROLLART_OK.
 *
 * Limits: n_items * num_kv_heads <= 2048 and n_items <= 512 per call.  A larger call returns
 * ROLLART_ERR_WORKSPACE with a message that states the limit, and launches nothing; split the
 * batch and call again.
 *
 * Sharing: all calls on one GPU, from every thread and stream, use the same array, and it keeps
 * what the previous call left in it.  The call itself clears the words that have to start at
 * zero (status and ticket counters); nothing else is read before it is written.  Two calls whose kernels overlap on the GPU
 * (different streams without an ordering between them) race on the array and give wrong
 * results: keep these calls on one stream, or order the streams with events.
 *
 * First call on a device: it looks up the device address of the array (cudaGetSymbolAddress,
 * with that device current) and raises the kernel's shared-memory limit; this is also when the
 * runtime places the array in device memory.  A call with n_items = 0 does exactly this set-up and
 * nothing else: it is the warm-up.  Make it at start-up, before the embedding program takes the
 * device's remaining memory for itself (afterwards the set-up can fail for lack of room: the call
 * then returns ROLLART_ERR_CUDA and says so in err_buf) and before any stream capture; later
 * calls only enqueue work on `stream`.
 */
rollart_status rollart_decode_attn_noalloc(int device, const rollart_kv_pool *pool, const rollart_trajs *trajs,
                                           const int32_t *traj_ids, int32_t n_items, int32_t max_seq_len, const void *q,
                                           int32_t num_q_heads, float sm_scale, void *out, float *lse,
                                           int32_t *device_status, void *stream, char *err_buf, size_t err_len);

/*
 * Diagnostic of the bounded waits (no counterpart in the paper).  Every in-kernel wait of this library (on a copy, on
 * the tensor core, on another role of the block) polls with a limit of about a second; when the limit runs out the
 * kernel records ROLLART_ERR_TIMEOUT, stops waiting and runs to its end, so a fault elsewhere cannot hang the GPU.
 * This call enqueues one thread block whose only thread waits, with that same bounded wait, on a barrier nothing
 * arrives at: it returns after about a second of GPU time and the next rollart_check returns ROLLART_ERR_TIMEOUT
 * (and clears it); the context is usable afterwards.  For health checks and for testing the error path.
 */
rollart_status rollart_selftest_bounded_wait(rollart_ctx *ctx, void *stream);

/* Synchronises `stream`, then returns and clears the device status word: ROLLART_OK, or the
 * first device-side error recorded since the last check (ROLLART_ERR_BOUNDS / _TIMEOUT), or
 * ROLLART_ERR_CUDA if the stream itself reports an error. */
rollart_status rollart_check(rollart_ctx *ctx, void *stream);

/* [host] NUL-terminated description of the last non-OK status returned for this context; valid
 * until the next call on it.  Never NULL. */
const char *rollart_last_error(rollart_ctx *ctx);

/* Number of kernels the library has launched through this context since it was created. */
int64_t rollart_launch_count(rollart_ctx *ctx);

#ifdef __cplusplus
}
#endif
#endif /* ROLLART_H_ */
