/*
 * difr.h -- C ABI of the B200 token-scoring library (libdifr.so).
 *
 * The library re-scores, on one sm_100a GPU, every claimed output token of a
 * logged LLM response the way the verification server of "Verifying LLM
 * Inference to Detect Model Weight Exfiltration" does: the final hidden state
 * of each position goes through the LM head, and the logits are turned into
 * the Fixed-Seed Sampling Likelihood estimators of Sec. "Classification using
 * the Fixed-Seed Sampling Likelihood Policy" with the sampling seed shared with
 * the inference server.  Logits are never written to memory.
 *
 * Entry points
 *   scoring      difr_score_gm, difr_score_ipt, difr_score_both (one pass over the logits);
 *                difr_score_gm_filtered, difr_score_ipt_filtered (the generation's top-k / top-p
 *                filter, s competitors: one contraction, two passes over the logits); difr_score_gm_static (no caller workspace)
 *   decisions    difr_detect (threshold, three risk classes with the raw-logit rank, per-sequence
 *                pooling), difr_admissible (sizes of the admissible sets), difr_exfiltratable_bits
 *   randomness   difr_expand_seeds (seeds that also depend on the context)
 *   sizes        difr_workspace_bytes, difr_filtered_workspace_bytes
 *   aids         difr_logits, difr_philox, difr_selftest_wait, difr_debug_plan_override,
 *                difr_status_string, difr_version
 *
 * Conventions
 *   - Plain C linkage, no exceptions, no global state visible to the caller.
 *     Host threads may call concurrently (each with its own workspace; see
 *     difr_score_gm_static for the one exception).
 *   - Every pointer is a DEVICE pointer owned by the caller unless it says
 *     "host"; the caller keeps all buffers alive until `stream` has passed the
 *     call.  The library allocates no device memory and never synchronises
 *     the stream; all work is enqueued on `stream` (kernels and a few small
 *     cudaMemsetAsync on the workspace).  Two calls may run at the same time
 *     only with separate workspaces.
 *   - The return value reports what the host can detect (bad arguments,
 *     alignment, workspace size, wrong architecture, launch failure).  What
 *     only the device can detect is reported in `row_status` and
 *     `device_status`.
 *   - Randomness RO(seed || i) (Sec. "Sampling From Large Language Models") is
 *     Philox-4x32-10 with key = (seed low word, seed high word) and counter =
 *     (id >> 2, i, stream, 0); vocabulary id `id` takes output word id & 3.
 *     stream 0 is the Gumbel noise, stream 1 the single uniform of the
 *     inverse-probability-transform sampler (id 0).  A 32-bit word x becomes
 *     u = ((x >> 9) + 1/2) 2^-23 and G = -ln(-ln u) for Gumbel noise, and
 *     mu = (x + 1/2) 2^-32 for the IPT uniform.
 */
#ifndef DIFR_H_
#define DIFR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct CUstream_st* difr_stream_t; /* a cudaStream_t */

typedef enum {
  DIFR_OK = 0,
  DIFR_ERR_INVALID_ARG = -1, /* null required pointer, non-positive size, bad scalar  */
  DIFR_ERR_SHAPE = -2,       /* d not a multiple of 8, V < 2, T > 2^30, d > 2^20 ...  */
  DIFR_ERR_ALIGN = -3,       /* h, W or workspace not 16-byte aligned                 */
  DIFR_ERR_WORKSPACE = -4,   /* workspace missing or smaller than difr_workspace_bytes */
  DIFR_ERR_CUDA = -5,        /* a CUDA runtime/driver call failed                     */
  DIFR_ERR_ARCH = -6,        /* current device is not compute capability 10.x         */
  DIFR_ERR_TIMEOUT = -7      /* device_status only: a bounded device-side wait ran out */
} difr_status;

/* Per-sequence pooled statistics written by difr_detect. */
typedef struct {
  int32_t n_flagged; /* rows with score < threshold (or NaN)                      */
  int32_t n_match;   /* rows whose claimed token is the verifier's own sample      */
  float sum;         /* sum of the scores (summed log-likelihood)                  */
  float min;         /* smallest non-NaN score; +inf for an empty sequence         */
} difr_seq_stats;

/*
 * Estimator parameters and outputs of one scoring call.  Arrays are device
 * pointers of T elements; optional ones may be NULL.
 */
typedef struct {
  float sigma; /* width of the Gaussian noise model: raw-logit units for
                  difr_score_gm, probability (CDF) units for difr_score_ipt; > 0 */
  float eps;   /* floor inside the logarithm; >= 0 (1e-12 is customary)          */
  float* score;       /* required. ln(pi + eps) (Token-DiFR) / ln(mass + eps) (IPT)  */
  float* margin;      /* GM: A = y[t*] - max_{v != t*} y[v], y = l + Temp*G.  A >= +0
                         means exact match; -0.0 encodes a tie lost to a lower id;
                         -inf for an out-of-range claim.  Unused by IPT.           */
  int32_t* argmax;    /* GM: the verifier's own Gumbel-max token (ties: lowest id) */
  int32_t* runner_up; /* GM: id of the second largest y                            */
  float* lse;         /* ln sum_v exp(l_v / Temp); NaN when Temp == 0              */
  float* p_claimed;   /* IPT: softmax probability of the claimed token            */
  float* cdf_lo;      /* IPT: a = sum_{v < t*} p_v                                 */
  float* u;           /* IPT: the uniform mu of this row                           */
  uint32_t* row_status; /* bit0: claimed id outside [0, V); bit1: non-finite logits (the
                           scores of such a row are NaN, which difr_detect flags);
                           bit2: candidate list overflow (difr_score_gm_filtered);
                           bit3: unusable per-row temperature or filter values; bit4: the nucleus holds more
                           ids than the filtered calls resolve (128); bit5: more than 64 ids lie within
                           fp32 rounding of the claimed logit (rank) or of a bound (difr_admissible):
                           the integer leaves the unlisted ones out                           */
  void* workspace;      /* >= difr_workspace_bytes(T, d, V) bytes, 16-byte aligned;
                           contents are scratch, overwritten by every call         */
  size_t workspace_bytes;
  int32_t* device_status; /* [1] optional. Sticky: a kernel writes DIFR_ERR_TIMEOUT
                             here if a bounded wait ran out; never cleared         */
  void* event_fused_start; /* optional cudaEvent_t (host handles): recorded on `stream` */
  void* event_fused_stop;  /* right before / after the fused GEMM+epilogue kernel, so a
                              caller can time that kernel apart from the finalize pass */
  /* -- members added in version 200; zero them when unused -- */
  int32_t* rank;     /* GM, optional: raw-logit rank of the claimed token, #{v != t* : l_v > l_t*}
                        (0 = largest logit; V for an out-of-range claim), Sec. "Problems with FSSL
                        Estimators and Logit-Rank as a Solution".  An exact integer: the fused kernel
                        counts the fp32 logits that exceed l_t* by more than the tensor cores' rounding
                        and lists the ids it cannot decide (at most 64 per row; row_status bit 5 on
                        overflow), which the finalize kernel compares in fp64.  Asking for it adds one
                        gather pass and two compares per logit.                                  */
  float* y_max;      /* GM, optional: y = l + Temp*G of the verifier's own sample (the largest) */
  float* y_second;   /* GM, optional: the second largest y                                     */
  float sigma_ipt;   /* difr_score_both only: noise width of the IPT estimator (CDF units), > 0 */
  float* score_ipt;  /* difr_score_both only, required there: ln(mass + eps)                   */
  float* cutoff;     /* difr_score_*_filtered only, optional: the filter's cutoff per row      */
  const float* temperatures; /* difr_score_gm / _ipt / _both, optional: [T] one sampling temperature per
                        row (requests with their own sampling parameters in one batch); when given, the
                        `temperature` argument is ignored.  A row whose value is negative, not finite, or
                        zero where the IPT score is asked for gets a NaN score and row_status bit 3.
                        The filtered calls take it too (there a row needs a temperature > 0).       */
} difr_out;

/* Scratch bytes a scoring call needs for T rows, hidden size d, vocabulary V.
 * Returns 0 for sizes the library rejects. */
size_t difr_workspace_bytes(int64_t T, int64_t d, int64_t V);

/*
 * Token-DiFR, the Gumbel-max estimator (Alg. "Token-DiFR", with the paper's
 * default Gaussian noise, one active competitor and no top-k/top-p filter;
 * Sec. "Gumbel-Max Scoring Function").
 *
 * For every row r: logits l = h[r,:] . W^T (bf16 inputs, fp32 accumulation on
 * the tensor cores), Gumbel noise G regenerated from (seeds[r], positions[r]),
 * y = l + temperature * G; the claimed token's margin A over its strongest
 * competitor is re-evaluated in fp64 and scored as
 * ln(Phi(A / (sigma sqrt 2)) + eps).  The same pass yields the exact-match
 * replay of Sec. "Sampled-Token Verification via Exact Matching" (argmax,
 * margin >= 0) and the log-sum-exp of l / temperature.
 *
 *   h          bf16 [T, d] row-major; h[r,:] is the hidden state that predicts token r
 *   W          bf16 [V, d] row-major LM-head matrix
 *   tokens     int32 [T] claimed ids (any value; out of range => maximally suspicious)
 *   seeds      uint64 [T], positions uint32 [T]: RO(seed || i) per row
 *   temperature  >= 0 (0: greedy replay, y = l)
 *   0 <= T <= 2^30, 0 < d <= 2^20 with d % 8 == 0, 2 <= V <= 2^31 - 1024
 * Errors: see difr_status.  T == 0 returns DIFR_OK without launching.
 */
difr_status difr_score_gm(const void* h, const void* W, const int32_t* tokens, const uint64_t* seeds,
                          const uint32_t* positions, float temperature, int64_t T, int64_t d, int64_t V,
                          difr_out* out, difr_stream_t stream);

/*
 * Token-IPT-DiFR, the inverse-probability-transform estimator (Alg.
 * "Token-IPT-DiFR"; Sec. "Inverse Probability Transform Scoring Function").
 *
 * Same arguments.  Per row: p = softmax(l / temperature), [a, b] the claimed
 * token's interval of the cumulative distribution in vocabulary-id order, mu the
 * row's uniform, score = ln(Phi((b - mu)/sigma) - Phi((a - mu)/sigma) + eps).
 * Requires temperature > 0.  Writes score, lse, p_claimed, cdf_lo, u,
 * row_status; margin/argmax/runner_up are left untouched.
 * Accuracy: the softmax sums come from the tensor cores' fp32 logits (the claimed token's own term is replaced by
 * its fp64 value), so a and b carry a relative error of about 1e-7 for unit-scale logits and up to 3e-5 for
 * logits of magnitude 200; the score's error is that times |a - mu| / sigma^2.  Measured against the fp64
 * oracle: within 2e-5 for unit-variance logits at d = 5120 and within 7e-4 for logits reaching +-200, for
 * sigma from 1 down to 0.01; below sigma = 0.01 the 2e-3 tolerance is no longer assured for such heads.
 */
difr_status difr_score_ipt(const void* h, const void* W, const int32_t* tokens, const uint64_t* seeds,
                           const uint32_t* positions, float temperature, int64_t T, int64_t d, int64_t V,
                           difr_out* out, difr_stream_t stream);

/*
 * difr_score_gm without a workspace: for callers that cannot allocate.
 * (The paper has no counterpart; this is a property of the library only.)
 *
 * Some hosts of this library hand it input and output buffers but have no way
 * to obtain scratch memory of their own: a plugin running inside another
 * framework's memory pool that may not call cudaMalloc behind its back, a
 * process whose device memory was carved up in advance, a caller replaying a
 * fixed sequence of launches that must not contain an allocation.  For them this
 * entry point computes exactly what difr_score_gm computes, with the partial
 * records kept in an array of DIFR_STATIC_SCRATCH_BYTES that is part of the
 * library's device image.  Every GPU that loads the library holds that array
 * until the process exits.
 *
 *   - out->workspace and out->workspace_bytes are ignored; all other arguments and
 *     outputs are those of difr_score_gm.
 *   - Returns DIFR_ERR_WORKSPACE, launching nothing, when
 *     difr_workspace_bytes(T, d, V) exceeds DIFR_STATIC_SCRATCH_BYTES.
 *   - Calls no cudaMalloc, cudaFree or other allocating routine.
 *   - The first call on each device looks up the array's device address (the
 *     device must be current); make that first call before starting any stream
 *     capture.
 *   - All calls on a device share the one array, and it keeps what the last
 *     call left there.  The one word that has to start at zero (the work counter
 *     behind the records) is cleared on the stream by every call; the records
 *     themselves are overwritten before they are read.  Two calls that overlap on the GPU (different
 *     streams, no ordering between them) race on it and give wrong scores;
 *     serialise them, or use difr_score_gm with separate workspaces.
 */
#define DIFR_STATIC_SCRATCH_BYTES (16u << 20)
difr_status difr_score_gm_static(const void* h, const void* W, const int32_t* tokens, const uint64_t* seeds,
                                 const uint32_t* positions, float temperature, int64_t T, int64_t d, int64_t V,
                                 difr_out* out, difr_stream_t stream);

/*
 * Both estimators from one pass over the logits (the fused kernel keeps the
 * statistics of both anyway): everything difr_score_gm writes, with sigma in
 * raw-logit units, plus score_ipt / p_claimed / cdf_lo / u of difr_score_ipt
 * with out->sigma_ipt.  Requires temperature > 0 and out->score_ipt.
 */
difr_status difr_score_both(const void* h, const void* W, const int32_t* tokens, const uint64_t* seeds,
                            const uint32_t* positions, float temperature, int64_t T, int64_t d, int64_t V,
                            difr_out* out, difr_stream_t stream);

/*
 * Token-DiFR in full (Alg. "Token-DiFR"): the sampling filter's cutoff, the
 * B_i terms and an active subset of s competitors,
 *
 *   pi = E_{x ~ N(0, sigma^2)} [ 1{l_t* + x > cutoff} prod_{i in S} Phi(max(x + A_i, B_i) / sigma) ],
 *
 * S = the s ids with the largest y = l + Temp*G other than t*, A_i = y_t* - y_i,
 * B_i = cutoff - l_i, score = ln(pi + eps).  `cutoff` is the smallest logit that
 * survives the filter: the top_k largest logits are kept, then, among those,
 * the shortest prefix in descending order whose renormalised softmax(l / Temp)
 * mass reaches top_p.  The expectation is evaluated by Gauss-Legendre quadrature
 * (512 nodes over the range that carries the mass), not by sampling.
 *
 *   filter->top_k  0: no top-k; otherwise >= 1 (a top_k >= V filters nothing)
 *   filter->top_p  in (0, 1]; 1: no nucleus.  With no top-k in front of it the nucleus is the
 *                  shortest prefix that holds top_p of the whole row's softmax mass.
 *   Filters of any size: with one policy for the whole call (no *_rows arrays), a top_k above 128 or a
 *   nucleus over the whole vocabulary is resolved exactly by a selection over the rows' logits, which the
 *   first pass then also writes to the workspace (fp32, up to 2 GiB: a call with more rows than that holds
 *   is worked off block by block); the selection walks each row three or four times.  Per-row policies
 *   (the *_rows arrays) are by default resolved among each row's 128 largest logits: a row's top_k must be
 *   <= 128 (or >= V), and a row whose whole-vocabulary nucleus holds more than 128 ids gets row_status
 *   bit 4 and the 128th largest logit as cutoff.  The host cannot see the rows' values, so the caller says
 *   when they may go beyond that: filter->any_size != 0 sends every row of a per-row call through the
 *   selection (same cost as above, same results where both paths apply).
 *   filter->s      1..8
 *   filter->min_p  in [0, 1]; 0: none.  min-p (Sec. "Sampling From Large Language Models") keeps the ids whose
 *                  probability is at least min_p times the largest one, i.e. whose logit reaches
 *                  l_max + Temp ln(min_p); that bound is the value a (perturbed) logit has to reach to
 *                  survive, so the cutoff is the larger of it and the top-k / top-p cutoff.  l_max is
 *                  re-evaluated in fp64.
 *   temperature > 0
 *   Requests with their own sampling parameters in one batch: filter->top_k_rows, filter->top_p_rows
 *   and out->temperatures give one value per row; a row whose values are outside the ranges above
 *   gets a NaN score and row_status bit 3 (the scalars are checked on the host, DIFR_ERR_INVALID_ARG).
 *   out->workspace needs difr_filtered_workspace_bytes(T, d, V) bytes
 *
 * Everything difr_score_gm writes is written as there (margin, argmax, runner_up,
 * lse, y_max, y_second, and `rank`, counted during the second pass); `score` holds
 * the full estimator and out->cutoff, if given, the cutoff per row (-inf: no
 * filter).  Two passes over the logits, one contraction: the scoring pass, which
 * also stores the fp32 logits in the workspace (up to 2 GiB; a call with more rows
 * than that holds is worked off block by block), then a pass over the stored logits that
 * collects, per row, the ids that can be among the s + 2 best or among the top_k
 * logits (6 KB of list per row, or 12 V bytes per row for vocabularies below 16384 ids,
 * where every id is listed; row_status bit 2 marks a row whose list
 * overflowed, which takes hundreds of logits within rounding of the top_k-th).
 * With s = 1 and no filter the result equals difr_score_gm's up to quadrature
 * error (< 1e-6 in the score).
 */
typedef struct {
  int32_t top_k;
  float top_p;
  int32_t s;
  /* -- members added in version 210; zero them when unused -- */
  const int32_t* top_k_rows; /* device [T], optional: one top_k per row (top_k is then ignored)            */
  const float* top_p_rows;   /* device [T], optional: one top_p per row (top_p is then ignored)            */
  /* -- members added in version 220; zero them when unused -- */
  float min_p;               /* in [0, 1]; 0: no min-p filter                                               */
  const float* min_p_rows;   /* device [T], optional: one min_p per row (min_p is then ignored)            */
  /* -- member added in version 221; zero it when unused -- */
  int32_t any_size;          /* with *_rows arrays: non-zero resolves every row by the selection over its   */
                             /* logits (no limit of 128 ids); ignored when there is one policy for the call */
} difr_filter;
size_t difr_filtered_workspace_bytes(int64_t T, int64_t d, int64_t V);
difr_status difr_score_gm_filtered(const void* h, const void* W, const int32_t* tokens, const uint64_t* seeds,
                                   const uint32_t* positions, float temperature, int64_t T, int64_t d, int64_t V,
                                   const difr_filter* filter, difr_out* out, difr_stream_t stream);

/*
 * Token-IPT-DiFR with the generation's sampling filter (Alg. "Token-IPT-DiFR":
 * the token probabilities include the same temperature / top-k / nucleus
 * policy as generation): p is softmax(l / Temp) restricted to the ids that
 * survive the filter (as in difr_score_gm_filtered: the top_k largest logits,
 * then the shortest prefix whose renormalised mass reaches top_p) and
 * renormalised; [a, b] is the claimed token's interval of that distribution's
 * CDF in vocabulary-id order; a claimed id the filter removed has p = 0 and
 * scores ln(eps).
 *
 *   filter->top_k and filter->top_p as in difr_score_gm_filtered (any size with one policy for the call:
 *   the selection also sums the kept ids' masses; per-row policies within the 128 largest logits);
 *   filter->top_p in (0, 1]; filter->min_p in [0, 1] (the ids that reach l_max + Temp ln(min_p); any number of them
 *   with one policy for the call, else resolved among the 128 largest logits with row_status bit 4 when more
 *   survive); filter->s is ignored; per-row values
 *   as in difr_score_gm_filtered (a row whose own policy filters nothing keeps the unfiltered score)
 *   temperature > 0; out->workspace needs difr_filtered_workspace_bytes(T, d, V)
 * Writes score, p_claimed, cdf_lo, u, row_status, out->cutoff (optional) and
 * lse (of the unfiltered logits).  Two passes over the logits (one contraction), the second
 * without noise.
 */
difr_status difr_score_ipt_filtered(const void* h, const void* W, const int32_t* tokens, const uint64_t* seeds,
                                    const uint32_t* positions, float temperature, int64_t T, int64_t d, int64_t V,
                                    const difr_filter* filter, difr_out* out, difr_stream_t stream);

/*
 * Sizes of the admissible sets A_t(tau) = { i : FSSL_t(i) >= tau } (Sec.
 * "Empirical Results"), the quantity behind the paper's information bound
 * sum_t log2 |A_t(tau)|, for the Token-DiFR score with one competitor.
 *
 * For id i != the verifier's own sample the score is ln(Phi((y_i - y_max) /
 * (sigma sqrt 2)) + eps), so i is admissible iff y_i >= y_max + A(tau) with
 * A(tau) = sigma sqrt 2 Phi^-1(e^tau - eps); the sample itself is admissible iff
 * the score of its margin y_max - y_second reaches tau.  The call makes a second
 * pass over the logits (same tensor-core main loop, noise regenerated, two
 * compares per logit and threshold) and needs the outputs of a difr_score_gm call
 * on the same h, W, seeds, positions and temperature: argmax, runner_up, y_max,
 * y_second.
 *
 *   taus       host pointer, n_tau thresholds, 1 <= n_tau <= 4
 *   runner_up  int32 [T], nullable: with it the sample's own margin is re-evaluated in fp64, without it
 *              taken from the fp32 values y_max - y_second
 *   counts     int32 [n_tau, T] (device): |A_t(taus[j])| in counts[j*T + t]
 *   row_status uint32 [T], nullable: bit 5 marks a row with more than 64 undecided ids (see below)
 *   workspace  >= difr_workspace_bytes(T, d, V), scratch
 * The counts are integers decided exactly: the pass evaluates y in fp32, counts the ids that clear the bound by
 * more than fp32's error there (about 4e-4 * max(1, Temp)), lists the ids inside that band (at most 64 per
 * row) and a last kernel scores each listed id as the claim in fp64 against tau itself.  A row whose list
 * overflows (thousands of ids within 1e-3 of a bound: thresholds that cut through the bulk of the
 * vocabulary) gets bit 5 and a count that leaves the unlisted ids out.
 */
difr_status difr_admissible(const void* h, const void* W, const uint64_t* seeds, const uint32_t* positions,
                            float temperature, int64_t T, int64_t d, int64_t V, const int32_t* argmax,
                            const int32_t* runner_up, const float* y_max, const float* y_second, float sigma,
                            float eps, const float* taus, int32_t n_tau, int32_t* counts, uint32_t* row_status,
                            void* workspace, size_t workspace_bytes, int32_t* device_status, difr_stream_t stream);

/*
 * Per-token exfiltratable information (displayed cases of Sec. "Problems with
 * FSSL Estimators and Logit-Rank as a Solution"): log2 |A_t| for a safe token,
 * log2 R for a suspicious one, log2 V for a dangerous one, summed per sequence.
 *
 *   classes     uint8 [T]: 0 safe, 1 suspicious, 2 dangerous (the flags of difr_detect)
 *   counts      int32 [T]: |A_t(tau)| from difr_admissible (0 counts as no information)
 *   rank_cutoff R >= 1, V >= 1
 *   bits        float [T], nullable; seq_bits float [n_seq] (or [1]), nullable
 */
difr_status difr_exfiltratable_bits(const uint8_t* classes, const int32_t* counts, int32_t rank_cutoff, int64_t V,
                                    const int32_t* seq_offsets, int64_t n_seq, int64_t T, float* bits,
                                    float* seq_bits, difr_stream_t stream);

/*
 * Threshold detection and pooling (Sec. "Classification via Thresholding":
 * flag t iff FSSL(t) < tau; per-sequence match count as in Alg. "Sampled token
 * verification via prefill").
 *
 *   scores      float [T]
 *   threshold   tau; a score equal to tau is safe, NaN is flagged
 *   margins     float [T], nullable: rows without a sign bit count as matches
 *   ranks, rank_cutoff   nullable / ignored when NULL: with raw-logit ranks (difr_out.rank, counted
 *               from 0) a flagged row whose claimed token is not among the R = rank_cutoff largest
 *               logits (rank >= R) gets flag 2 (Alg. "Per-Token Risk Classification via GLS and
 *               Rank": 0 safe, 1 suspicious, 2 dangerous).  With R = 1 only the top-ranked token
 *               can be suspicious; a suspicious token is one of R ids, hence log2 R bits
 *               (appendix "Logit-Rank Ablations").  The algorithm prints the test as rank > R,
 *               which is this rule for a rank counted from 1.
 *   seq_offsets int32 [n_seq + 1] ascending row offsets, nullable => one sequence [0, T)
 *   flags       uint8 [T], nullable: 0 safe, 1 flagged (suspicious), 2 dangerous
 *   seq_stats   difr_seq_stats [n_seq] (or [1]), nullable
 */
difr_status difr_detect(const float* scores, float threshold, const float* margins, const int32_t* ranks,
                        int32_t rank_cutoff, const int32_t* seq_offsets, int64_t n_seq, int64_t T,
                        uint8_t* flags, difr_seq_stats* seq_stats, difr_stream_t stream);

/*
 * Sequential randomness expansion RO(seed || i || context) (footnote to the
 * definition of honest sampling, Sec. "Sampling From Large Language Models";
 * first further measure of Sec. "Message-Sampling Secure Seed Expansion"): per-row
 * seeds that make the noise of a row depend on the prompt and on every claimed
 * token before it, to be passed as `seeds` to the scoring calls (both servers
 * expand the same way).  The paper fixes no hash; the library's is
 *
 *   e(j, t) = words 0,1 of Philox-4x32-10(counter (j, t, 0, 1), key (0x243F6A88, 0x85A308D3))
 *   c_r     = prompt_hashes[q] + sum_{j < r - o_q} e(j, tokens[o_q + j])   (mod 2^64)
 *   expanded[r] = words 0,1 of Philox-4x32-10(counter (c_r low, c_r high, 0, 2), key seeds[r])
 *
 * with q the sequence of row r, o_q = seq_offsets[q] its first row, t the token
 * as an unsigned 32-bit value and "words 0,1" = word 0 + 2^32 word 1.  A 64-bit
 * sum of pseudo-random words is no collision-resistant hash: a deployment that
 * needs one hashes on its own side and passes the result as prompt_hashes or
 * directly as seeds.
 *
 *   seeds         uint64 [T]; tokens int32 [T] (the claimed ids, any value)
 *   seq_offsets   int32 [n_seq + 1], non-decreasing from 0 to T, or NULL: one sequence [0, T)
 *   prompt_hashes uint64 [n_seq] (or [1]), or NULL for zeros
 *   expanded      uint64 [T]; may be the same array as seeds.  Rows outside every
 *                 sequence are left untouched.
 * T, n_seq < 2^31.  T == 0 returns DIFR_OK without launching.
 */
difr_status difr_expand_seeds(const uint64_t* seeds, const int32_t* tokens, const int32_t* seq_offsets,
                              int64_t n_seq, const uint64_t* prompt_hashes, int64_t T, uint64_t* expanded,
                              difr_stream_t stream);

/*
 * Validation aid, not part of the scoring path: writes the fp32 logits
 * l[r, v] = h[r,:] . W[v,:] computed by the same tensor-core main loop to
 * `logits` (float [T, V] row-major).  Meant for small shapes.
 */
difr_status difr_logits(const void* h, const void* W, int64_t T, int64_t d, int64_t V, float* logits,
                        int32_t* device_status, difr_stream_t stream);

/*
 * Validation aid: the library's own Philox-4x32-10 block for n counters.
 * ctr uint32 [n, 4], key uint32 [n, 2] -> out uint32 [n, 4] (device pointers).
 */
difr_status difr_philox(const uint32_t* ctr, const uint32_t* key, int64_t n, uint32_t* out, difr_stream_t stream);

/*
 * Validation aid: exercises the bounded wait every kernel of the library uses.  One warp waits on a barrier
 * that nothing arrives at; after `limit_cycles` SM clocks (1 .. 1e9, i.e. well under a second) the wait must
 * give up.  status2 (device, int32 [2]) receives {DIFR_ERR_TIMEOUT, 1} when it did; the kernel ends normally
 * either way and the context stays usable.
 */
difr_status difr_selftest_wait(int32_t* status2, int64_t limit_cycles, difr_stream_t stream);

/*
 * Validation aid: overrides the work planner's choices for every later call of the process (0 = the planner's
 * own value): the number of vocabulary strips, the number of 256-row tiles per raster group, and the megabytes
 * of h per raster group the planner aims at.  Results do not depend on these values (tests sweep them to show
 * it); speed and the workspace size do, so query difr_workspace_bytes again after changing them, and do not
 * change them while a call is being issued on another thread.  Not meant for production use.
 */
difr_status difr_debug_plan_override(int32_t strips, int32_t group, int32_t l2_mb);

const char* difr_status_string(difr_status status); /* host pointer to a static string */
int difr_version(void);

#ifdef __cplusplus
}
#endif
#endif /* DIFR_H_ */
