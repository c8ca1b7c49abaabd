/*
 * liba2sf -- C ABI of the A2SF KV-cache pruning hot path on one NVIDIA B200 (sm_100a).
 *
 * A2SF (Accumulative Attention Score with Forgetting Factor) keeps, per attention
 * head, a score for every cached token: the forgetting-weighted sum over query
 * steps of the softmax probability that token received (paper Eq. 5), and evicts
 * the lowest-scoring tokens so the cache never exceeds a fixed budget (Sec. 3.1,
 * Sec. 4.1).  This library computes, per (batch, head) unit:
 *
 *   prefill : causal attention over the prompt, the score of every prompt token,
 *             and the set of tokens that stay in the cache;
 *   decode  : one generation step over the pruned, slot-indexed cache -- attention,
 *             the score recurrence S <- alpha*S + a_t, the eviction of one token
 *             and the in-place insertion of the new one.
 *
 * Conventions
 *   - Positions, slots and rows are 0-based.  n = prompt length, d = head size,
 *     M = budget (cache slots per head), R = recent (newest positions that are
 *     never evicted), U = B*H units.
 *   - Unless an argument says "host", every data pointer is a DEVICE pointer owned
 *     by the caller; the library never frees caller memory.  Rows of q/k/v/out
 *     must be 16-byte aligned (base pointer and strides).
 *   - Calls enqueue work on `cuda_stream` (a cudaStream_t passed as void*; NULL is
 *     the default stream) and return without synchronising, except where stated.
 *     The cache's resident count and length live on the device, so a decode step
 *     has no host-side data-dependent control flow.
 *   - Every function returns an a2sf_status.  Invalid arguments are rejected on
 *     the host before anything is launched; nothing is dereferenced on the host.
 *   - There is no CPU fallback.
 */
#ifndef A2SF_H
#define A2SF_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum { A2SF_F32 = 0, A2SF_BF16 = 1, A2SF_F16 = 2 } a2sf_dtype;

typedef enum {
    A2SF_OK = 0,
    A2SF_ERR_INVALID_ARG = -1,   /* null / misaligned pointer, bad shape or policy        */
    A2SF_ERR_UNSUPPORTED = -2,   /* dtype or head size without a kernel                   */
    A2SF_ERR_CUDA = -3,          /* a CUDA runtime call failed                            */
    A2SF_ERR_TIMEOUT = -4,       /* a bounded device-side wait ran out (kernel gave up)   */
    A2SF_ERR_WORKSPACE = -5      /* workspace / buffer smaller than the *_bytes() figure  */
} a2sf_status;

/* Shape and policy of a call.  `scale` = 0 selects 1/sqrt(d).  `alpha` is the
 * forgetting factor of Eq. 5; the paper states 0 < alpha < 1 and also runs
 * alpha = 0 (Sec. 4.4); alpha = 1 is the plain accumulative score of H2O (Eq. 4).
 * Accepted: 0 <= alpha <= 1 with alpha^0 = 1.  1 <= budget <= A2SF_MAX_BUDGET (one unit's
 * logits of a generation step are held in one CTA's shared memory), 0 <= recent <= budget,
 * d in {64, 128}.  Anything else: A2SF_ERR_INVALID_ARG, or A2SF_ERR_UNSUPPORTED for a dtype,
 * head size or budget outside the supported set. */
#define A2SF_MAX_BUDGET 49152
typedef struct a2sf_params {
    int32_t B, H, d;
    int32_t dtype;               /* a2sf_dtype of q, k, v, out and the cache rows */
    int32_t budget, recent;
    float alpha;
    float scale;
    int32_t flags;               /* 0 or A2SF_FLAG_* */
    int32_t score_window;        /* 0, or W > 0: see a2sf_score_window_bound */
} a2sf_params;

/* Scoring pass: Eq. 5 weighs query row i with alpha^(n-1-i).  Once that weight is below
 * 2^-127 (2^-152 on the CUDA-core path) the fp32 term is exactly zero, so with this flag the
 * pass leaves those rows out: O(n * window) instead of O(n^2) work with bit-identical scores.
 * Off by default; alpha = 1 has no such rows. */
#define A2SF_FLAG_SKIP_ZERO_WEIGHT_ROWS 1

/* Truncated scoring pass.  With score_window = W > 0 the sum of Eq. 5 runs over the last W
 * query rows only, S_j = sum_{i >= max(j, n-W)} alpha^(n-1-i) P_ij: O(n * W) work.  Every
 * probability is at most 1, so each score falls short of the full sum by at most
 *     sum_{a=W}^{n-1} alpha^a = alpha^W (1 - alpha^(n-W)) / (1 - alpha)      (n - W for alpha = 1),
 * which this function returns (0 when W = 0 or W >= n).  The attention output and lse are not
 * affected.  Unlike A2SF_FLAG_SKIP_ZERO_WEIGHT_ROWS this changes the scores: the kept set may
 * differ wherever two scores are closer than the bound. */
double a2sf_score_window_bound(float alpha, int32_t n, int32_t score_window);

typedef struct a2sf_cache a2sf_cache;   /* opaque, owned by the library */

/* ---------------------------------------------------------------------------
 * Prefill (prompt phase).
 *
 * For every unit, with s_ij = scale * q_i . k_j for j <= i (causal mask: Eq. 3 sets
 * the probability of a later key to zero) and P = row softmax of s:
 *     out_i    = sum_j P_ij v_j
 *     lse_i    = log sum_{j<=i} exp(s_ij)
 *     scores_j = sum_{i>=j} alpha^(n-1-i) P_ij           (Eq. 5, Eq. 6: the sum ends
 *                                                         at the diagonal term)
 *     kept_idx = every position >= n-R plus, of the others, all but the n-M lowest
 *                under the order (score, position) ascending; ascending positions.
 *                If n <= M every position is kept.  (Sec. 3.1, Sec. 4.1)
 *
 * q, k, v, out : [B][H][n][d] in `dtype`, element strides stride_b/stride_h/stride_t,
 *                d contiguous; out uses the same strides.
 * scores       : [B][H][n] fp32, contiguous.      kept_idx: [B][H][min(n,M)] int32.
 * lse_opt      : [B][H][n] fp32 or NULL (then it lives in the workspace).
 * workspace    : device scratch of at least a2sf_prefill_workspace_bytes() bytes,
 *                256-byte aligned; contents undefined afterwards.
 * Errors: INVALID_ARG, UNSUPPORTED, WORKSPACE, CUDA (launch failure).
 * ------------------------------------------------------------------------- */
size_t a2sf_prefill_workspace_bytes(const a2sf_params *p, int32_t n);

int a2sf_prefill(const a2sf_params *p, int32_t n,
                 const void *q, const void *k, const void *v,
                 int64_t stride_b, int64_t stride_h, int64_t stride_t,
                 void *out, float *scores, int32_t *kept_idx, float *lse_opt,
                 void *workspace, size_t workspace_bytes, void *cuda_stream);

/* Scores and kept set only, from the log-sum-exp a prefill produced (the second
 * pass of the prefill alone).  Lets a sweep over alpha reuse one attention pass.
 * lse: [B][H][n] fp32 (input).  Other arguments as in a2sf_prefill; workspace may
 * be NULL when a2sf_rescore_workspace_bytes() is 0. */
size_t a2sf_rescore_workspace_bytes(const a2sf_params *p, int32_t n);

int a2sf_rescore(const a2sf_params *p, int32_t n,
                 const void *q, const void *k,
                 int64_t stride_b, int64_t stride_h, int64_t stride_t,
                 const float *lse, float *scores, int32_t *kept_idx,
                 void *workspace, size_t workspace_bytes, void *cuda_stream);

/* Selection alone (Sec. 3.1, Sec. 4.1): kept_idx from a given score vector, exactly the last
 * step of a2sf_prefill / a2sf_rescore -- every position >= n-R plus, of the others, all but the
 * n-M lowest under (score, position) ascending.  scores [B][H][n] fp32 (input, non-negative),
 * kept_idx [B][H][min(n,M)] int32 (output, ascending).  Lets a caller re-select under another
 * budget or recent window without recomputing scores. */
int a2sf_select(const a2sf_params *p, int32_t n, const float *scores, int32_t *kept_idx,
                void *cuda_stream);

/* Per-head forgetting factors (the paper's Limitation section suggests a distinct factor per
 * layer and head instead of one uniform value).  `alphas` is a DEVICE array [B][H] fp32, one
 * factor per unit; p->alpha is ignored.  Values outside [0, 1] (or NaN) cannot be rejected on
 * the host and are clamped into [0, 1] on the device.  Everything else as in a2sf_prefill /
 * a2sf_rescore. */
int a2sf_prefill_per_head(const a2sf_params *p, int32_t n,
                          const void *q, const void *k, const void *v,
                          int64_t stride_b, int64_t stride_h, int64_t stride_t,
                          const float *alphas,
                          void *out, float *scores, int32_t *kept_idx, float *lse_opt,
                          void *workspace, size_t workspace_bytes, void *cuda_stream);

int a2sf_rescore_per_head(const a2sf_params *p, int32_t n,
                          const void *q, const void *k,
                          int64_t stride_b, int64_t stride_h, int64_t stride_t,
                          const float *lse, const float *alphas,
                          float *scores, int32_t *kept_idx,
                          void *workspace, size_t workspace_bytes, void *cuda_stream);

/* Same as a2sf_prefill with HOST buffers: q, k, v, out contiguous [B][H][n][d];
 * scores, kept_idx as above, all in host memory (pinned memory makes the copies
 * asynchronous).  Inputs are copied to the device workspace, results copied back,
 * and the call returns after the stream has drained.  The device copies of k, v,
 * scores and kept_idx stay valid in the workspace for a2sf_cache_load: their
 * addresses are returned through dev_k, dev_v, dev_scores, dev_kept (any may be NULL).
 * With two or more batch rows the work is pipelined over chunks of rows on two internal
 * streams (created once per device on first use and kept): they start after what is already
 * queued on cuda_stream, and cuda_stream (and the call) continues only when they have drained.
 * Chunked calls on one device are serialised against each other. */
size_t a2sf_prefill_host_workspace_bytes(const a2sf_params *p, int32_t n);

int a2sf_prefill_host(const a2sf_params *p, int32_t n,
                      const void *q_host, const void *k_host, const void *v_host,
                      void *out_host, float *scores_host, int32_t *kept_idx_host,
                      void *workspace, size_t workspace_bytes,
                      void **dev_k, void **dev_v, float **dev_scores, int32_t **dev_kept,
                      void *cuda_stream);

/* Prefill without any allocation, for callers that cannot call cudaMalloc (an
 * engine whose own allocator owns the device, a plugin that only sees one layer's
 * tensors, a loop that must not hit an allocation's implicit synchronisation).
 * The paper has no counterpart: this is the same computation as a2sf_prefill, with
 * the per-row log-sum-exp scratch held in a fixed 4 MiB array inside the library's
 * device image (every GPU that loads the library carries it until the process
 * exits).  It runs the same kernels as a2sf_prefill except that, having no workspace
 * for an fp16 copy of V, bf16 storage multiplies P V with two bf16 terms.
 *   - Limit: B*H*n <= a2sf_prefill_static_scratch_max_rows() (1,048,576); larger
 *     calls return A2SF_ERR_WORKSPACE and launch nothing.
 *   - The first call on each device looks up the array's device address (a short
 *     host-side driver query with that device current); make that first call
 *     before starting any stream capture.
 *   - All calls on a device share the one array, which keeps the previous call's
 *     contents.  Each call overwrites every row it later reads, so nothing needs
 *     clearing, but two calls that overlap on the GPU (different streams without an
 *     event between them) race on it: keep them ordered.
 *   - It calls no cudaMalloc / cudaFree and takes no workspace; the log-sum-exp is
 *     not returned.  Other arguments, results and errors are those of a2sf_prefill. */
size_t a2sf_prefill_static_scratch_max_rows(void);

int a2sf_prefill_static_scratch(const a2sf_params *p, int32_t n,
                                const void *q, const void *k, const void *v,
                                int64_t stride_b, int64_t stride_h, int64_t stride_t,
                                void *out, float *scores, int32_t *kept_idx, void *cuda_stream);

/* ---------------------------------------------------------------------------
 * The pruned cache.  Per unit: K and V rows [M][d] in `dtype`, scores [M] fp32,
 * positions [M] int32 (slot -> token position, -1 = empty), the resident count and
 * the number of tokens seen so far.  Slot order carries no meaning (softmax . V is
 * permutation invariant); positions exist for recency and the tie-break.
 *
 * a2sf_cache_create: `device_mem` NULL -> the library allocates a2sf_cache_bytes()
 * with cudaMalloc and frees it in a2sf_cache_destroy; otherwise it adopts the
 * caller's buffer (256-byte aligned, at least a2sf_cache_bytes(); WORKSPACE if
 * smaller), which the caller frees after destroy.  The cache starts empty.
 * Creation synchronises the device (it is not on the hot path).
 * ------------------------------------------------------------------------- */
size_t a2sf_cache_bytes(const a2sf_params *p);

int a2sf_cache_create(const a2sf_params *p, void *device_mem, size_t bytes, a2sf_cache **cache);

int a2sf_cache_destroy(a2sf_cache *cache);

/* Initial cache from a prefill: slot s <- token kept_idx[s] (its K and V row, score
 * and position); count = min(n, M); length = n; remaining slots emptied.
 * k, v: [B][H][n][d] with the given strides; scores [B][H][n]; kept_idx [B][H][min(n,M)]. */
int a2sf_cache_load(a2sf_cache *cache, int32_t n, const void *k, const void *v,
                    int64_t stride_b, int64_t stride_h, int64_t stride_t,
                    const float *scores, const int32_t *kept_idx, void *cuda_stream);

/* ---------------------------------------------------------------------------
 * One generation step for every unit, fused in one kernel (Eq. 5 as a recurrence;
 * Sec. 3.1 eviction; the softmax runs over the pruned cache plus the new token,
 * cf. Sec. 2.2 on the changed denominator):
 *   a      = softmax over { scale*q.K[slot] : slot < count } and scale*q.k_new
 *   out    = sum_slot a_slot V[slot] + a_self v_new
 *   S[slot] <- alpha*S[slot] + a_slot,   S_new = a_self
 *   count < M : the new token goes to slot `count`; evicted_slot = -1.
 *   count = M : among the slots whose position is <= p - R (p = position of the new
 *               token) -- and the new token itself iff R = 0 -- the minimum under
 *               (S, position) is vacated and the new K/V/score/position are written
 *               there in place; evicted_slot = that slot, or -2 if the new token was
 *               the minimum (cache left as it was, apart from the updated scores).
 *   length += 1.
 * q, k_new, v_new, out: [B][H][d] contiguous in the cache's dtype; evicted_slot
 * [B][H] int32.  alpha overrides the value given at creation.
 * Steps on one cache must be ordered (same stream, or events between streams).
 * ------------------------------------------------------------------------- */
int a2sf_decode_step(a2sf_cache *cache, float alpha,
                     const void *q, const void *k_new, const void *v_new,
                     void *out, int32_t *evicted_slot, void *cuda_stream);

/* The same step with one forgetting factor per unit: `alphas` is a DEVICE array [B][H] fp32
 * (clamped into [0, 1] on the device).  See a2sf_prefill_per_head. */
int a2sf_decode_step_per_head(a2sf_cache *cache, const float *alphas,
                              const void *q, const void *k_new, const void *v_new,
                              void *out, int32_t *evicted_slot, void *cuda_stream);

/* The same step with HOST buffers.  Page-locked (pinned, mapped) buffers are read and written
 * by the step kernel directly over the bus; for any other host memory q, k_new, v_new are
 * copied into staging rows inside the cache, the step runs, out and evicted_slot are copied
 * back.  Either way the call returns after the stream has drained, with the results in place. */
int a2sf_decode_step_host(a2sf_cache *cache, float alpha,
                          const void *q_host, const void *k_new_host, const void *v_new_host,
                          void *out_host, int32_t *evicted_slot_host, void *cuda_stream);

/* Several tokens appended in one call (a draft that was accepted, a prompt continued in
 * chunks): exactly `steps` generation steps in order, token t taking row t of q, k_new,
 * v_new and writing row t of out -- DEVICE [B][H][steps][d] with element strides as in
 * a2sf_prefill.  evicted_opt: DEVICE [steps][B][H] int32 or NULL.  Runs as `steps` launches;
 * the result is bit-identical to calling a2sf_decode_step `steps` times. */
int a2sf_decode_multi(a2sf_cache *cache, float alpha, int32_t steps,
                      const void *q, const void *k_new, const void *v_new,
                      int64_t stride_b, int64_t stride_h, int64_t stride_t,
                      void *out, int32_t *evicted_opt, void *cuda_stream);

/* ---------------------------------------------------------------------------
 * Grouped query heads (GQA / MQA): `group` query heads share one K/V head, hence one pruned
 * cache.  The paper scores tokens per head and leaves grouping open (Limitation section);
 * the rule here: a token's score is the SUM over the group's query heads of Eq. 5, and one
 * selection / one eviction per K/V head serves the whole group.  a2sf_params.H counts K/V
 * heads; the query tensors have H * group heads, head h*group + g reading K/V head h.
 *
 * a2sf_prefill_group: q, out DEVICE [B][H*group][n][d] (q strides), k, v DEVICE [B][H][n][d]
 * (kv strides), scores [B][H][n] fp32 (summed over the group), kept_idx [B][H][min(n,budget)],
 * lse_opt [B][H*group][n] or NULL.  flags and score_window must be 0.  Workspace as for
 * a2sf_prefill, size from a2sf_prefill_group_workspace_bytes (0 = invalid arguments).
 *
 * a2sf_decode_step_group: the generation step for a cache built from those scores
 * (a2sf_cache_load).  q, out DEVICE [B][H*group][d] contiguous; k_new, v_new DEVICE [B][H][d];
 * evicted_slot [B][H].  Each query head attends over the cached tokens and the new one; the
 * cached scores become alpha * S + sum_g a_g, the new token's score sum_g a_g,self; eviction as
 * in a2sf_decode_step.  A2SF_ERR_UNSUPPORTED when group > A2SF_MAX_GROUP or (group + 2) * budget
 * is too large for one CTA's shared memory (about 47,000 for d = 128, group = 8).  For 16-bit
 * storage the products of the group run on the tensor cores (fp32 accumulation).
 * ------------------------------------------------------------------------- */
#define A2SF_MAX_GROUP 8
size_t a2sf_prefill_group_workspace_bytes(const a2sf_params *p, int32_t group, int32_t n);
int a2sf_prefill_group(const a2sf_params *p, int32_t group, int32_t n,
                       const void *q, int64_t q_stride_b, int64_t q_stride_h, int64_t q_stride_t,
                       const void *k, const void *v,
                       int64_t kv_stride_b, int64_t kv_stride_h, int64_t kv_stride_t,
                       void *out, float *scores, int32_t *kept_idx, float *lse_opt,
                       void *workspace, size_t workspace_bytes, void *cuda_stream);
int a2sf_decode_step_group(a2sf_cache *cache, int32_t group, float alpha,
                           const void *q, const void *k_new, const void *v_new,
                           void *out, int32_t *evicted_slot, void *cuda_stream);

/* Empties the cache (count = length = 0, scores 0, positions -1), asynchronously. */
int a2sf_cache_reset(a2sf_cache *cache, void *cuda_stream);

/* ---------------------------------------------------------------------------
 * Streamed prompt: the cache is pruned WHILE the prompt is processed, row by row, the way
 * the paper's mask figures (Sec. 3.2, Sec. 4.3) draw it: token i attends only to what
 * is left of tokens 0..i-1, scores follow Eq. 5 as a recurrence and one token leaves per row
 * once the budget is full.  This is NOT a2sf_prefill followed by a2sf_cache_load (dense causal
 * attention, one selection at the end): the two give the same result only while n <= budget.
 *
 * Exactly: a2sf_cache_reset, then a2sf_decode_multi over the n prompt tokens (the generation
 * step with (q_i, k_i, v_i), out_i written to row i of `out`): n launches of the step kernel.
 * q, k, v, out: DEVICE [B][H][n][d] with the strides of a2sf_prefill.  evicted_opt: DEVICE
 * [n][B][H] int32 (each row as a2sf_decode_step's evicted_slot) or NULL.  On return (the work
 * is queued on the stream) the cache holds the pruned prompt and generation continues with
 * a2sf_decode_step.
 * ------------------------------------------------------------------------- */
int a2sf_prefill_streaming(a2sf_cache *cache, float alpha, int32_t n,
                           const void *q, const void *k, const void *v,
                           int64_t stride_b, int64_t stride_h, int64_t stride_t,
                           void *out, int32_t *evicted_opt, void *cuda_stream);

/* ---------------------------------------------------------------------------
 * Similarity with the ideal mask (Sec. 4.3: the mask figure and the similarity table).
 *
 * Runs a2sf_prefill_streaming and, for every row i, compares the attention the policy
 * actually uses -- the softmax over the cached tokens and token i itself -- with the ideal
 * row: the softmax over the budget + 1 largest logits of ALL tokens 0..i (equal logits: the
 * lower position first), i.e. the best any policy with that many tokens could do.
 *     cos_out[b][h][i] = <a_i, p_i> / (|a_i| |p_i|),   both rows as length-(i+1) vectors.
 * Rows i <= budget see every token and give 1.  Averaging (over rows, heads) is the caller's.
 * q, k, v, out, evicted_opt as in a2sf_prefill_streaming; cos_out DEVICE [B][H][n] fp32.
 * workspace: DEVICE, 256-byte aligned, a2sf_ideal_similarity_workspace_bytes (0 = invalid
 * arguments).  n <= A2SF_IDEAL_SIMILARITY_MAX_N (a row's logits are held in shared memory).
 * A diagnostic, not a hot path: 1 + 2n launches, O(n^2 d) CUDA-core work per unit.
 * ------------------------------------------------------------------------- */
#define A2SF_IDEAL_SIMILARITY_MAX_N 32768
size_t a2sf_ideal_similarity_workspace_bytes(const a2sf_params *p, int32_t n);
int a2sf_ideal_similarity(a2sf_cache *cache, float alpha, int32_t n,
                          const void *q, const void *k, const void *v,
                          int64_t stride_b, int64_t stride_h, int64_t stride_t,
                          void *out, float *cos_out, int32_t *evicted_opt,
                          void *workspace, size_t workspace_bytes, void *cuda_stream);

/* Snapshot / restore of the whole cache state into / from caller DEVICE buffers:
 * k, v [B][H][M][d] dtype; scores [B][H][M] fp32; pos [B][H][M] int32; count, len
 * [B][H] int32.  Any pointer may be NULL to skip that part. */
int a2sf_cache_export(const a2sf_cache *cache, void *k, void *v, float *scores,
                      int32_t *pos, int32_t *count, int32_t *len, void *cuda_stream);

int a2sf_cache_import(a2sf_cache *cache, const void *k, const void *v, const float *scores,
                      const int32_t *pos, const int32_t *count, const int32_t *len,
                      void *cuda_stream);

/* Number of kernels this library has launched in the calling process so far. */
int64_t a2sf_kernel_launch_count(void);

/* Synchronises the stream and returns the sticky device-side status (A2SF_OK, or
 * A2SF_ERR_TIMEOUT if a kernel abandoned a bounded wait), then clears it.  While the
 * status is set the tensor-core prefill kernels return without working, so results
 * of calls made after a timeout and before this call are undefined. */
int a2sf_last_device_status(void *cuda_stream);

/* Self-test of the device-side failure path (the paper has no counterpart; a test hook, not
 * part of the method).  Every wait inside the kernels of this library is bounded: a wait that
 * runs out poisons its CTA, the kernel unwinds and raises the sticky status that
 * a2sf_last_device_status reports.  This call exercises exactly that, harmlessly: it launches one
 * CTA whose first thread waits -- through the library's own bounded wait, with `limit_cycles`
 * SM clocks as the limit -- on a barrier at which nobody ever arrives, then raises the status
 * word of the tensor-core prefill kernels (which = 0) or of the generation-step kernels
 * (which = 1).  Nothing traps and nothing waits without a bound.
 *   report : DEVICE int64[4], written by the kernel: [0] 1 if the wait reported failure,
 *            [1] SM clocks the wait took, [2] SM clocks of a second wait in the same CTA (it
 *            returns at once because the CTA is poisoned), [3] 1 if that second wait failed too.
 *   limit_cycles in [1, A2SF_SELFTEST_MAX_WAIT_CYCLES]; INVALID_ARG otherwise.
 * Afterwards a2sf_last_device_status returns A2SF_ERR_TIMEOUT once, then A2SF_OK. */
#define A2SF_SELFTEST_MAX_WAIT_CYCLES 2000000000ll
int a2sf_selftest_bounded_wait(int32_t which, int64_t limit_cycles, int64_t *report, void *cuda_stream);

/* Bounds-checked debug library (built with -DA2SF_DEBUG as liba2sf_debug.so; the paper has no
 * counterpart).  In it every slot, position, tile-row and ring-stage index that addresses global
 * or shared memory inside a kernel is range-checked; a violation is counted, the first one is
 * recorded, and the offending access is skipped (nothing traps).  a2sf_debug_build returns 1 in
 * that library and 0 in the release one.  a2sf_debug_violations synchronises the stream, writes
 * to the HOST array report[4] = { violations since the last call, (kernel id << 32) | source
 * line of the first one, its index, its bound } and clears the record; the release library
 * always reports zeros. */
int a2sf_debug_build(void);
int a2sf_debug_violations(int64_t *report, void *cuda_stream);

const char *a2sf_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* A2SF_H */
