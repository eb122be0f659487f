/*
 * sgbv.h -- C ABI of the batched multi-draft greedy block verification step (SpecTr-GBV).
 *
 * One call verifies, for every batch row, K i.i.d. draft blocks of gamma tokens against the
 * target model's distributions and returns the accepted block and one extra token
 * (Algorithm 1 of the paper with Eqs. 2, 3 and 4).  The draft and target model forwards are
 * not part of this library: their logits are inputs.
 *
 * Tensor layouts (row-major, last index contiguous; "device" = CUDA device memory of the
 * current device, "host" = ordinary or pinned host memory):
 *   target_logits [B, K, gamma+1, V]   row (b,k,i): target logits after the first i tokens of
 *                                      draft k, i = 0..gamma (the paper's q(. | x_k^{i}))
 *   draft_logits  [B, K, gamma,   V]   row (b,k,i): draft logits after the same prefix
 *                                      (the paper's p(. | x_k^{i})), i = 0..gamma-1
 *   draft_tokens  [B, K, gamma]        int32, token i of draft k, 0 <= token < V
 *   uniforms      [B, K*gamma + 1]     float32 in [0,1): entry k*gamma + (i-1) is the uniform eta of
 *                                      the Bernoulli trial on the length-i sub-block of draft k
 *                                      in Algorithm 1; the last entry draws the extra token by
 *                                      inverse CDF
 *   out_accept_len [B]                 int32 tau in 0..gamma, or -1 if the row was flagged invalid
 *   out_draft_idx  [B]                 int32 accepted draft f in 0..K-1, -1 when tau == 0
 *   out_tokens     [B, gamma+1]        int32: the tau accepted tokens, then the extra token y at
 *                                      index tau, then -1 padding
 * Probabilities are softmax(logits / temperature) of each row (one temperature for both models).
 *
 * Ownership: every pointer is owned by the caller; the library neither frees nor keeps it past
 * the call.  Device entry points only enqueue work on `stream` (a cudaStream_t passed as void*;
 * NULL = the legacy default stream) and return without synchronising: outputs are valid once the
 * stream has been synchronised.
 *
 * Errors: the return value is SGBV_OK or a negative SGBV_ERR_* code found on the host before
 * anything is launched (nothing has been written then).  Conditions found on the device never
 * trap: they set per-row bits in the status array (SGBV_STATUS_*), and a row flagged
 * TOKEN_RANGE or NONFINITE_LOGIT gets tau = f = -1 and tokens = -1.  There is no CPU fallback.
 */
#ifndef SGBV_H_
#define SGBV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SGBV_OK 0
#define SGBV_ERR_NULL (-1)        /* a required pointer is NULL */
#define SGBV_ERR_SHAPE (-2)       /* B,K,gamma,V < 1, K > 64, gamma > 64, V > 2^22, unknown dtype */
#define SGBV_ERR_TEMPERATURE (-3) /* temperature <= 0 or not finite */
#define SGBV_ERR_ALIGN (-4)       /* a pointer is not aligned to its element size */
#define SGBV_ERR_WORKSPACE (-5)   /* caller workspace too small or misaligned (256 B) */
#define SGBV_ERR_CUDA (-6)        /* a CUDA runtime call failed (allocation, copy, launch) */

#define SGBV_STATUS_TOKEN_RANGE 1         /* a draft token of the row is outside [0,V) */
#define SGBV_STATUS_NONFINITE_LOGIT 2     /* NaN/+inf logit, or a row with no finite logit, among the rows read */
#define SGBV_STATUS_DEGENERATE_RESIDUAL 4 /* Eq. 4 had zero total mass; y was drawn from q of that row */

#define SGBV_STATUS_TIMEOUT 8             /* a bounded device-side wait expired; the row's outputs are -1 */

#define SGBV_DTYPE_F32 0
#define SGBV_DTYPE_BF16 1

/* Bytes of device scratch one call of the given shape needs (for sgbv_verify_ex). */
int sgbv_workspace_bytes(int B, int K, int gamma, int V, int dtype, size_t *out_bytes);

/*
 * The verify step on float32 logits (problem statement and Algorithm 1; Eqs. 2-4).
 * All tensor pointers are device pointers.  Scratch comes from a per-device buffer that the
 * library grows with cudaMalloc when a larger shape is first seen (so the first call of a
 * shape is not stream-capturable; later ones allocate nothing).  Calls that use that buffer on
 * one device must be ordered with respect to one another (one stream, or events between streams):
 * they share it, and every call leaves part of it prepared for the next one (whatever their
 * shapes, eager or replayed from a CUDA graph).  A CUDA graph captured on that buffer holds its
 * address: a later call of a larger shape reallocates the buffer and invalidates such graphs, so
 * call the largest shape first, or pass a workspace of your own to sgbv_verify_ex.  The kernels are launched with programmatic stream serialisation:
 * for batches of at most 16 rows the first kernel of a call may be scheduled while the kernel
 * ahead of it in the stream is still running; it touches no global memory until that kernel has
 * completed, so the caller sees ordinary stream order.
 */
int sgbv_verify(const float *target_logits, const float *draft_logits, const int32_t *draft_tokens,
                const float *uniforms, int B, int K, int gamma, int V, float temperature,
                int32_t *out_accept_len, int32_t *out_draft_idx, int32_t *out_tokens, void *stream);

/* Same with bfloat16 logits (raw 16-bit patterns), widened to float32 inside the kernels. */
int sgbv_verify_bf16(const uint16_t *target_logits, const uint16_t *draft_logits,
                     const int32_t *draft_tokens, const float *uniforms, int B, int K, int gamma,
                     int V, float temperature, int32_t *out_accept_len, int32_t *out_draft_idx,
                     int32_t *out_tokens, void *stream);

/*
 * Extended form: caller-provided scratch and diagnostics (device pointers).
 *   dtype           SGBV_DTYPE_F32 or SGBV_DTYPE_BF16 (element type of the two logit tensors)
 *   workspace       >= sgbv_workspace_bytes(...) bytes, 256-byte aligned, or NULL to use the
 *                   library's own per-device buffer
 *   out_h           [B,K,gamma] float64 or NULL: acceptance weight of the length-i sub-block at
 *                   index i-1 (Eq. 2 for i < gamma, Eq. 3 for i = gamma), clamped to [0,1]
 *   out_resmass     [B,K,gamma] float64 or NULL: S_i = sum_x q(x^i,x)(1-min{p(x^i,x)/q(x^i,x),1})^K,
 *                   i = 0..gamma-1 (the vocabulary sum of Eq. 2 = normaliser of Eq. 4)
 *   out_status      [B] int32 or NULL: SGBV_STATUS_* bits
 */
int sgbv_verify_ex(const void *target_logits, const void *draft_logits, int dtype,
                   const int32_t *draft_tokens, const float *uniforms, int B, int K, int gamma, int V,
                   float temperature, int32_t *out_accept_len, int32_t *out_draft_idx,
                   int32_t *out_tokens, void *workspace, size_t workspace_bytes, double *out_h,
                   double *out_resmass, int32_t *out_status, void *stream);

/*
 * Host-buffer form: every tensor pointer is a HOST pointer (pinned memory makes the copies
 * asynchronous).  Copies the inputs to device staging buffers owned by the library, runs the
 * verify step on `stream`, copies the three outputs (and out_status if not NULL) back and
 * synchronises the stream before returning.  All calls on one device share one staging buffer
 * (grown with cudaMalloc when a larger shape is first seen): callers on the same device must be
 * serialised with respect to one another.
 */
int sgbv_verify_host(const void *target_logits, const void *draft_logits, int dtype,
                     const int32_t *draft_tokens, const float *uniforms, int B, int K, int gamma,
                     int V, float temperature, int32_t *out_accept_len, int32_t *out_draft_idx,
                     int32_t *out_tokens, int32_t *out_status, void *stream);

/*
 * One position of the distribution modification that follows a verify step which stopped short
 * (Algorithm 2; Theorem 4.2 needs it for the law of a whole decode).  With s = everything emitted so
 * far in the modified region (the accepted block, the extra token, the tokens drawn here before),
 * the next token comes from
 *   q_new(x) = q(s,x) (1 - min{p(s,x)/q(s,x), 1})^K / sum_x' q(s,x') (1 - min{p(s,x')/q(s,x'), 1})^K
 * with JOINT probabilities q(s,x) = q(s) q(x|s), p(s,x) = p(s) p(x|s): Eq. 4's weights with the ratio
 * p(s)/q(s) carried in instead of built from a draft.  Per batch row the call draws that token by
 * inverse CDF and appends it to the carried logs.  All pointers are device pointers.
 *   target_logits [B,V], draft_logits [B,V]   logits of this position given s (dtype as in sgbv_verify_ex)
 *   log_a, log_b  [B] float64                 log q(s), log p(s); 0 for an empty s
 *   uniforms      [B] float32 in [0,1)        one per row, for the inverse CDF
 *   K                                          the number of drafts of the decode (the exponent above)
 *   out_token     [B] int32                   the drawn token, -1 if the row was flagged invalid
 *   out_log_a, out_log_b [B] float64          log q(s,token), log p(s,token) (may alias log_a, log_b)
 *   out_resmass   [B] float64 or NULL         sum_x q(x|s)(1 - min{(p(s)/q(s)) p(x|s)/q(x|s), 1})^K, the normaliser over q(s)
 *   out_status    [B] int32 or NULL           SGBV_STATUS_* bits; zero total mass draws from q(.|s), flagged
 *                                             DEGENERATE_RESIDUAL
 *   workspace                                  >= sgbv_workspace_bytes(B, 1, 1, V, dtype) bytes, 256-byte aligned,
 *                                              or NULL for the library's per-device buffer (see sgbv_verify)
 * Errors as for sgbv_verify_ex.
 */
int sgbv_modify(const void *target_logits, const void *draft_logits, int dtype, const double *log_a,
                const double *log_b, const float *uniforms, int B, int K, int V, float temperature,
                int32_t *out_token, double *out_log_a, double *out_log_b, double *out_resmass,
                int32_t *out_status, void *workspace, size_t workspace_bytes, void *stream);

/*
 * Comparison verifiers of the paper's Section 3 behind the same boundary (device pointers, layouts and
 * error behaviour as sgbv_verify_ex; workspace >= sgbv_workspace_bytes(B,K,gamma,V,dtype) or NULL).  They
 * serve the verification-cost comparison of the paper's Table 2 and are not tuned like the block verifier.
 *
 * sgbv_verify_kseq: SpecTr's position-wise K-SEQ (Section 3.2).  At every position the drafts that still match
 * the accepted prefix (n of them, n = K at first) are tried in order; draft k's token x is accepted if
 * eta < min{1, q(x)/(rho p(x))}, rho in [1,n] the root of 1 - (1 - beta(rho))^n = rho beta(rho) with
 * beta(rho) = sum_x min{p(x), q(x)/rho}; the first accepted token extends the prefix.  If none is accepted the
 * extra token comes from norm(max{q - rho p, 0}); after gamma accepted positions from the target row after
 * the block.  uniforms[b, k*gamma + i] is eta of draft k at position i (0-based), the last entry draws the
 * extra token.
 *   out_rho         [B,gamma] float64 or NULL: rho of every position reached, NaN elsewhere
 *   out_accept_prob [B,K,gamma] float64 or NULL: acceptance probability of every token tried, NaN elsewhere
 * sgbv_verify_token: token-level speculative sampling (Section 3.1) = K-SEQ with one draft (rho = 1);
 *   tensors without the K axis: target [B,gamma+1,V], draft [B,gamma,V], tokens [B,gamma], uniforms [B,gamma+1].
 * sgbv_verify_gbv: single-draft greedy block verification (Section 3.3) = the block verifier with K = 1; same
 *   tensors as sgbv_verify_token; out_accept_prob [B,gamma] or NULL holds the sub-block weights alpha(x^i).
 */
int sgbv_verify_kseq(const void *target_logits, const void *draft_logits, int dtype, const int32_t *draft_tokens,
                     const float *uniforms, int B, int K, int gamma, int V, float temperature,
                     int32_t *out_accept_len, int32_t *out_tokens, double *out_rho, double *out_accept_prob,
                     int32_t *out_status, void *workspace, size_t workspace_bytes, void *stream);
int sgbv_verify_token(const void *target_logits, const void *draft_logits, int dtype, const int32_t *draft_tokens,
                      const float *uniforms, int B, int gamma, int V, float temperature, int32_t *out_accept_len,
                      int32_t *out_tokens, double *out_accept_prob, int32_t *out_status, void *workspace,
                      size_t workspace_bytes, void *stream);
int sgbv_verify_gbv(const void *target_logits, const void *draft_logits, int dtype, const int32_t *draft_tokens,
                    const float *uniforms, int B, int gamma, int V, float temperature, int32_t *out_accept_len,
                    int32_t *out_tokens, double *out_accept_prob, int32_t *out_status, void *workspace,
                    size_t workspace_bytes, void *stream);

/*
 * Draft-token draw (Algorithm 3: "sample x_1^L, ..., x_K^L ~ p i.i.d."; the draft model produces one position's
 * logits at a time, so the unit is one token per logit row): token r is drawn from softmax(logits[r]/temperature) by
 * inverse CDF (ascending vocabulary index, first x whose cumulative mass exceeds u times the total), softmax and
 * draw fused in one pass over the row.  Device pointers.
 *   logits      [N,V] (dtype as in sgbv_verify_ex), one row per (batch row, draft) at the position being drafted
 *   uniforms    [N] float32 in [0,1)
 *   out_token   [N] int32, -1 for a row with NaN/+inf or without a finite logit
 *   out_logprob [N] float64 or NULL: log softmax of the drawn token
 *   out_status  [N] int32 or NULL: SGBV_STATUS_NONFINITE_LOGIT
 *   workspace   >= sgbv_workspace_bytes(N, 1, 1, V, dtype) bytes, 256-byte aligned, or NULL (library buffer)
 */
int sgbv_draw_tokens(const void *logits, int dtype, const float *uniforms, int N, int V, float temperature,
                     int32_t *out_token, double *out_logprob, int32_t *out_status, void *workspace,
                     size_t workspace_bytes, void *stream);

/*
 * Vocabulary-sharded verify step (no counterpart in the paper, which verifies on one device; the results are those
 * of Algorithm 1 on the whole vocabulary).  Rank r of n_ranks holds the logits of the vocabulary range
 * [v_begin_r, v_begin_r + shard_V_r), the ranges ascending with the rank and covering [0,V) without gaps, as a
 * tensor-parallel output layer leaves them:
 *   target_shard [B,K,gamma+1,shard_V], draft_shard [B,K,gamma,shard_V] row-major, dtype as in sgbv_verify_ex;
 * draft_tokens [B,K,gamma] (global ids) and uniforms [B,K*gamma+1] are the same on every rank.  All pointers are
 * device pointers.  The step is four local calls with three exchanges between them, which the CALLER performs with
 * its collective library (the Python binding uses torch.distributed); no call waits for another rank:
 *   sgbv_shard_stats   -> out_stats [B,K,gamma+1,8] float32: per row the shard's (max, sum of exponentials relative
 *                         to it) of the target and the draft row, the token's two logits if the shard holds it, flags
 *     exchange 1: all-gather the records in rank order -> stats_all [n_ranks,B,K,gamma+1,8]
 *   sgbv_shard_sums    -> normalisers and the ratios c_i of Eq. 2 from stats_all (identical on every rank), the
 *                         vocabulary sums of Eq. 2 and Eq. 4 over the shard; out_sums [B,K,gamma,3] float64
 *     exchange 2: all-gather -> sums_all [n_ranks,B,K,gamma,3]
 *   sgbv_shard_decide  -> Eq. 2 / Eq. 3 and the scan of Algorithm 1 from the shards' sums added in rank order:
 *                         identical out_accept_len, out_draft_idx, out_h, out_resmass, out_status on every rank;
 *                         out_tokens holds the accepted prefix and -1 elsewhere.  The inverse CDF of the extra token
 *                         (Eq. 4, or the target row) is split in rank order: which rank's range holds it, and where
 *                         inside that rank's share of the mass (kept in the workspace)
 *   sgbv_shard_draw    -> the owning rank finds the token inside its shard and writes its global id into
 *                         tokens[b, accept_len]; the other ranks leave -1 there
 *     exchange 3: max-all-reduce of tokens [B,gamma+1]
 * workspace: >= sgbv_shard_workspace_bytes(B,K,gamma,shard_V,dtype) bytes, 256-byte aligned, the caller's, and the
 * same buffer for the three calls of a step that take one (it carries the row records, the cell sums and the plan).
 * The flat parts of stats_all and sums_all must be the ranks' outputs in rank order; n_ranks <= 64.
 * Return codes as sgbv_verify_ex; per-row status bits as there (a token id outside [0,V), NaN/+inf in any shard).
 */
int sgbv_shard_workspace_bytes(int B, int K, int gamma, int shard_V, int dtype, size_t *out_bytes);
int sgbv_shard_stats(const void *target_shard, const void *draft_shard, int dtype, const int32_t *draft_tokens, int B,
                     int K, int gamma, int shard_V, int v_begin, int V, float temperature, float *out_stats,
                     void *stream);
int sgbv_shard_sums(const void *target_shard, const void *draft_shard, int dtype, int B, int K, int gamma, int shard_V,
                    float temperature, const float *stats_all, int n_ranks, void *workspace, size_t workspace_bytes,
                    double *out_sums, void *stream);
int sgbv_shard_decide(const int32_t *draft_tokens, const float *uniforms, int B, int K, int gamma, int shard_V,
                      float temperature, const float *stats_all, const double *sums_all, int n_ranks, void *workspace,
                      size_t workspace_bytes, int32_t *out_accept_len, int32_t *out_draft_idx, int32_t *out_tokens,
                      double *out_h, double *out_resmass, int32_t *out_status, void *stream);
int sgbv_shard_draw(const void *target_shard, const void *draft_shard, int dtype, int B, int K, int gamma, int shard_V,
                    int v_begin, float temperature, int rank, void *workspace, size_t workspace_bytes, int32_t *tokens,
                    void *stream);

/*
 * Allocation-free form of sgbv_verify_ex (the paper has no counterpart: this entry point exists
 * for deployment, not for the method).
 *
 * Who needs it: a serving process that hands all free device memory to its own pool or KV cache
 * at start-up cannot count on a later cudaMalloc succeeding, and a latency-critical decode loop
 * cannot afford the device-wide synchronisation a cudaMalloc or cudaFree implies.  This call
 * never allocates or frees: not with cudaMalloc/cudaFree, not through any library routine.
 *
 * Where the scratch lives: in a fixed array of SGBV_STATIC_SCRATCH_BYTES that is part of the
 * library's device image; every GPU that loads the library holds it until the process exits.
 * A shape whose sgbv_workspace_bytes(...) exceeds that size is refused with SGBV_ERR_WORKSPACE
 * and nothing is launched.
 *
 * First call on a device: resolves the array's device address (once per device, with that
 * device current); with CUDA's lazy module loading this is also when the driver loads the part of
 * the library that holds the array and reserves its bytes, and the first launch of each kernel
 * variant (shape, dtype, K) loads its code the same way.  So make one small call per variant that
 * will be used at start-up: before the caller's pool takes the rest of the device memory, and
 * before starting any stream capture.
 *
 * Sharing: all calls on a device use the same array, and it keeps the previous call's contents;
 * the call clears what has to start at zero itself.  Two calls that overlap on the GPU (different
 * streams, or the same shape from two threads) race on it: serialise them.
 *
 * Arguments, results and error codes are those of sgbv_verify_ex without the workspace pair.
 */
#define SGBV_STATIC_SCRATCH_BYTES (32u * 1024u * 1024u)
int sgbv_verify_static(const void *target_logits, const void *draft_logits, int dtype,
                       const int32_t *draft_tokens, const float *uniforms, int B, int K, int gamma, int V,
                       float temperature, int32_t *out_accept_len, int32_t *out_draft_idx,
                       int32_t *out_tokens, double *out_h, double *out_resmass, int32_t *out_status,
                       void *stream);

/* Number of kernel launches the last successful call on this thread enqueued. */
int sgbv_last_launch_count(void);

/* Name of the kernel that streamed the logits in the last successful call on this thread
 * (the one sgbv_profile_begin/_end time). Never NULL. */
const char *sgbv_last_main_kernel(void);

/*
 * Measurement support (not part of the method): between sgbv_profile_begin(n) and
 * sgbv_profile_end, each of the next n verify calls records a CUDA event pair on its stream
 * around the kernel that moves the logits (the one a memory roofline is quoted for).
 * sgbv_profile_end waits for those events, returns their summed elapsed time in milliseconds
 * and the number of recorded calls, and releases the events.  Not thread-safe.
 */
int sgbv_profile_begin(int max_records);
int sgbv_profile_end(double *out_total_ms, int *out_records);

/*
 * Tuning knobs for experiments (process-wide, not thread-safe; 0 restores the automatic choice):
 *   "path"         1 = always the generic two-sweep kernels, 2 = the fused single-read kernel or fail
 *   "cluster"      CTAs per cluster of the fused kernel (1..8)
 *   "max_clusters" cap on the number of resident clusters it launches
 *   "walk"         1 = a cluster of the fused kernel walks whole draft chains, 2 = single rows
 *   "aux"          where the two extra vocabulary sums that Eq. 2 may need for a row with p(x^i) < q(x^i) are worked out:
 *                  1 = in the fused kernel, for every such row; 2 = in two small kernels behind it, for the rows that
 *                  need them (one more read of a few per cent of the rows); 0 = the second for steps of 1 GB of logits
 *                  or more, else the first.  The row walk always works them out itself.
 * and two for the failure-detection test (a bounded device-side wait that runs out, see SGBV_STATUS_TIMEOUT):
 *   "poll_us"      limit, in microseconds, of the row walk's wait for a ratio published by another cluster
 *   "withhold"     1 = the first row of every chain does not publish its ratio
 * Returns SGBV_ERR_SHAPE for an unknown name or a value out of range.
 */
int sgbv_set_option(const char *name, int value);

/* Human-readable name of a return code. Never NULL. */
const char *sgbv_status_string(int code);

#ifdef __cplusplus
}
#endif
#endif /* SGBV_H_ */
