/*
 * difr_oracle.c -- TEST INFRASTRUCTURE, not the product.
 *
 * A plain, slow, fp64 CPU statement of what the verifier's scoring path
 * computes, written from the paper's algorithms so that a reader can check
 * it by eye.  It shares no code with the CUDA path and must only be used by
 * the tests, the smoke check and the CPU-baseline leg of the benchmark.
 *
 *   logits          : l[r,v] = sum_k h[r,k] * W[v,k]           (the last op of the prefill in
 *                     Alg. "Sampled token verification via prefill")
 *   randomness      : RO(seed || i) := Philox-4x32-10 (Salmon et al., SC'11),
 *                     key = (seed lo, seed hi), counter = (id>>2, i, tag, 0)
 *   Gumbel noise    : G = -ln(-ln u), u in (0,1)              (Sec. "Gumbel-Max Trick")
 *   Gumbel-max      : argmax_v l_v + Temp * G_v               (Alg. "Gumbel-Max Sampler",
 *                     in the log-probability form of the text; Alg. Token-DiFR ranks
 *                     its active subset by the same l_i + T * G_i)
 *   Token-DiFR      : A = l_t* - l_c + Temp (G_t* - G_c), one competitor (s = 1),
 *                     Gaussian noise of std sigma on every logit, no top-k/top-p
 *                     filter: pi = E_x[ Phi((x + A)/sigma) ] = Phi(A / (sigma sqrt 2))
 *                     score = ln(pi + eps)                    (Alg. Token-DiFR)
 *   softmax         : p_v = exp(l_v/Temp - lse)               (Sec. "Sampling From LLMs")
 *   Token-IPT-DiFR  : mu = Uniform(RO(seed||i)); [a,b] = CDF interval of t*;
 *                     mass = Phi((b-mu)/sigma) - Phi((a-mu)/sigma);
 *                     score = ln(mass + eps)                  (Alg. Token-IPT-DiFR)
 *   IPT sampler     : min{ v : C_v > u }                      (Alg. "IPT Sampler")
 *   detection       : flag iff score < tau                    (Sec. "Classification via
 *                     Thresholding"); per-sequence match count (Alg. prefill verification)
 *   risk classes    : safe / suspicious / dangerous from the score and the raw-logit rank
 *                     (Alg. "Per-Token Risk Classification via GLS and Rank")
 *   admissible set  : A_t(tau) = { i : FSSL_t(i) >= tau }, the score each vocabulary id
 *                     would get if it were the claim          (Sec. "Empirical Results")
 *   exfiltratable information : log2 |A_t| / log2 R / log2 |V| by class, summed per
 *                     sequence                               (Sec. "Problems with FSSL
 *                     Estimators and Logit-Rank as a Solution", displayed cases)
 *
 * Parity pins (tests, -m "not gpu"): Philox against the cuRAND host generator;
 * Gumbel-max sampler against softmax frequencies (chi-square); honest tokens
 * give margin >= 0; closed form against a literal Monte-Carlo of the fixed-seed
 * posterior; lse against scipy; IPT mass against mpmath quadrature and the
 * telescoping identity; the admissible set against re-scoring every id as the
 * claim; the information formula against hand-worked cases.  Absolute score values on realistic model data are
 * "parity unpinned": the paper prints no worked numeric example.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_OK 0
#define ORACLE_ERR_ARG -1
#define ORACLE_ERR_MEM -2

/* ------------------------------------------------------------------ bf16 */
static double bf16_to_double(uint16_t b) {
  uint32_t u = (uint32_t)b << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return (double)f;
}

/* ---------------------------------------------------------------- Philox */
/* Philox-4x32-10 as published: ten rounds; each round multiplies words 0 and 2
 * by two fixed odd constants, mixes the high halves with words 1, 3 and the
 * key, and the key grows by two Weyl constants between rounds. */
void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  const uint64_t mul_a = 0xD2511F53u, mul_b = 0xCD9E8D57u;
  const uint32_t weyl_a = 0x9E3779B9u, weyl_b = 0xBB67AE85u;
  uint32_t x0 = ctr[0], x1 = ctr[1], x2 = ctr[2], x3 = ctr[3];
  uint32_t ka = key[0], kb = key[1];
  for (int round = 0; round < 10; ++round) {
    uint64_t pa = mul_a * (uint64_t)x0;
    uint64_t pb = mul_b * (uint64_t)x2;
    uint32_t n0 = (uint32_t)(pb >> 32) ^ x1 ^ ka;
    uint32_t n1 = (uint32_t)pb;
    uint32_t n2 = (uint32_t)(pa >> 32) ^ x3 ^ kb;
    uint32_t n3 = (uint32_t)pa;
    x0 = n0; x1 = n1; x2 = n2; x3 = n3;
    ka += weyl_a;
    kb += weyl_b;
  }
  out[0] = x0; out[1] = x1; out[2] = x2; out[3] = x3;
}

/* The 32-bit word that RO(seed || position) assigns to noise id `id` in stream
 * `tag` (0: Gumbel noise over the vocabulary, 1: the IPT uniform). */
uint32_t oracle_ro_word(uint64_t seed, uint32_t position, uint32_t tag, uint32_t id) {
  uint32_t ctr[4] = {id >> 2, position, tag, 0u};
  uint32_t key[2] = {(uint32_t)(seed & 0xffffffffu), (uint32_t)(seed >> 32)};
  uint32_t out[4];
  oracle_philox4x32_10(ctr, key, out);
  return out[id & 3u];
}

/* u = (k + 1/2) 2^-23 with k the top 23 bits: strictly inside (0,1). */
double oracle_uniform23(uint32_t word) { return ((double)(word >> 9) + 0.5) * (1.0 / 8388608.0); }

/* mu = (x + 1/2) 2^-32 for the single IPT draw of a row. */
double oracle_uniform32(uint32_t word) { return ((double)word + 0.5) * (1.0 / 4294967296.0); }

double oracle_gumbel(uint32_t word) { return -log(-log(oracle_uniform23(word))); }

double oracle_gumbel_noise(uint64_t seed, uint32_t position, uint32_t id) {
  return oracle_gumbel(oracle_ro_word(seed, position, 0u, id));
}

/* The whole row of Gumbel noise, ids 0..V-1. */
void oracle_gumbel_row(uint64_t seed, uint32_t position, int64_t V, double* out) {
  for (int64_t v = 0; v < V; ++v) out[v] = oracle_gumbel_noise(seed, position, (uint32_t)v);
}

double oracle_ipt_uniform(uint64_t seed, uint32_t position) {
  return oracle_uniform32(oracle_ro_word(seed, position, 1u, 0u));
}

/* ------------------------------------------------------------- Gaussian */
static double std_normal_cdf(double z) { return 0.5 * erfc(-z / sqrt(2.0)); }

/* Phi(zb) - Phi(za) for za <= zb, taking the tail on whichever side avoids
 * cancellation. */
static double normal_interval_mass(double za, double zb) {
  const double r2 = sqrt(2.0);
  if (za >= 0.0) return 0.5 * (erfc(za / r2) - erfc(zb / r2));
  if (zb <= 0.0) return 0.5 * (erfc(-zb / r2) - erfc(-za / r2));
  return 1.0 - 0.5 * erfc(zb / r2) - 0.5 * erfc(-za / r2);
}

double oracle_normal_cdf(double z) { return std_normal_cdf(z); }
double oracle_normal_interval_mass(double za, double zb) { return normal_interval_mass(za, zb); }

/* Token-DiFR with one competitor and Gaussian noise: pi = Phi(A/(sigma sqrt2)). */
double oracle_gm_pi(double A, double sigma) { return std_normal_cdf(A / (sigma * sqrt(2.0))); }
double oracle_gm_score(double A, double sigma, double eps) { return log(oracle_gm_pi(A, sigma) + eps); }

/* ---------------------------------------------------------------- logits */
/* l[v] = sum_k h[k] W[v,k], natural order, one accumulator. */
static void row_logits(const uint16_t* h_row, const uint16_t* W, int64_t d, int64_t V, double* hd,
                       double* logit) {
  for (int64_t k = 0; k < d; ++k) hd[k] = bf16_to_double(h_row[k]);
  for (int64_t v = 0; v < V; ++v) {
    const uint16_t* w = W + v * d;
    double acc = 0.0;
    for (int64_t k = 0; k < d; ++k) acc += hd[k] * bf16_to_double(w[k]);
    logit[v] = acc;
  }
}

int oracle_logits(const uint16_t* h, const uint16_t* W, int64_t T, int64_t d, int64_t V, double* out) {
  if (!h || !W || !out || T < 0 || d <= 0 || V <= 0) return ORACLE_ERR_ARG;
  int err = 0;
#pragma omp parallel
  {
    double* hd = (double*)malloc((size_t)d * sizeof(double));
    if (!hd) {
#pragma omp atomic write
      err = 1;
    }
#pragma omp barrier
    if (!err) {
#pragma omp for schedule(dynamic, 1)
      for (int64_t r = 0; r < T; ++r) row_logits(h + r * d, W, d, V, hd, out + r * V);
    }
    free(hd);
  }
  return err ? ORACLE_ERR_MEM : ORACLE_OK;
}

static double log_sum_exp_scaled(const double* logit, int64_t V, double inv_temp) {
  double mx = -INFINITY;
  for (int64_t v = 0; v < V; ++v)
    if (logit[v] * inv_temp > mx) mx = logit[v] * inv_temp;
  double s = 0.0;
  for (int64_t v = 0; v < V; ++v) s += exp(logit[v] * inv_temp - mx);
  return mx + log(s);
}

/* ---------------------------------------------------------- Token-DiFR */
typedef struct {
  double* score;       /* [T] ln(pi + eps)                                       */
  double* margin;      /* [T] A = y[t*] - max_{v != t*} y[v]; -0.0 when A == 0
                              and t* loses the lowest-id tie-break              */
  int32_t* argmax;     /* [T] verifier's own Gumbel-max token (tie -> lowest id) */
  int32_t* runner_up;  /* [T] id of the second largest y                         */
  double* top2_margin; /* [T] y_(1) - y_(2)                                      */
  double* lse;         /* [T] ln sum_v exp(l_v / Temp); NaN when Temp == 0       */
  double* y_claimed;   /* [T] y[t*]  (NaN for an out-of-range claim)             */
  double* logit_claimed; /* [T] l[t*]                                            */
  int32_t* rank;       /* [T] #{v : l_v > l_t*}  (raw-logit rank, 0 = largest)   */
  int32_t* match;      /* [T] 1 iff argmax == t*                                 */
  uint32_t* row_status; /* [T] bit0: claim outside [0,V); bit1: non-finite logit */
  double* top23_margin; /* [T] y_(2) - y_(3); +inf when V < 3                     */
} oracle_gm_out;

/* One row of Token-DiFR from its logits.  y[V] is scratch.  noise_id (nullable):
 * vocabulary id v draws the noise of id noise_id[v]; used only by the
 * permutation-invariance check. */
static void gm_row(const double* logit, double* y, int64_t V, int64_t t, uint64_t seed, uint32_t position,
                   double temperature, double sigma, double eps, const int32_t* noise_id, int64_t r,
                   oracle_gm_out* out) {
  uint32_t status = 0;
  for (int64_t v = 0; v < V; ++v) {
    uint32_t id = noise_id ? (uint32_t)noise_id[v] : (uint32_t)v;
    double G = oracle_gumbel_noise(seed, position, id);
    y[v] = logit[v] + temperature * G;
    if (!isfinite(logit[v])) status |= 2u;
  }
  /* largest and second largest, ties to the lowest id */
  int64_t i1 = -1, i2 = -1;
  for (int64_t v = 0; v < V; ++v) {
    if (i1 < 0 || y[v] > y[i1]) {
      i2 = i1;
      i1 = v;
    } else if (i2 < 0 || y[v] > y[i2]) {
      i2 = v;
    }
  }
  int in_range = (t >= 0 && t < V);
  if (!in_range) status |= 1u;
  double A, score;
  if (in_range) {
    int64_t c = (t == i1) ? i2 : i1; /* strongest competitor */
    A = y[t] - y[c];
    if (A == 0.0 && t > c) A = -0.0;
    score = oracle_gm_score(A, sigma, eps);
  } else {
    A = -INFINITY;
    score = log(eps);
  }
  if (out->score) out->score[r] = score;
  if (out->margin) out->margin[r] = A;
  if (out->argmax) out->argmax[r] = (int32_t)i1;
  if (out->runner_up) out->runner_up[r] = (int32_t)i2;
  if (out->top2_margin) out->top2_margin[r] = y[i1] - y[i2];
  if (out->top23_margin) {
    double third = -INFINITY;
    for (int64_t v = 0; v < V; ++v)
      if (v != i1 && v != i2 && y[v] > third) third = y[v];
    out->top23_margin[r] = y[i2] - third;
  }
  if (out->lse) out->lse[r] = temperature > 0.0 ? log_sum_exp_scaled(logit, V, 1.0 / temperature) : NAN;
  if (out->y_claimed) out->y_claimed[r] = in_range ? y[t] : NAN;
  if (out->logit_claimed) out->logit_claimed[r] = in_range ? logit[t] : NAN;
  if (out->rank) {
    int32_t rank = (int32_t)V;
    if (in_range) {
      rank = 0;
      for (int64_t v = 0; v < V; ++v) rank += (logit[v] > logit[t]);
    }
    out->rank[r] = rank;
  }
  if (out->match) out->match[r] = in_range && (t == i1);
  if (out->row_status) out->row_status[r] = status;
}

int oracle_score_gm(const uint16_t* h, const uint16_t* W, const int32_t* tokens, const uint64_t* seeds,
                    const uint32_t* positions, double temperature, double sigma, double eps, int64_t T,
                    int64_t d, int64_t V, const int32_t* noise_id, oracle_gm_out* out) {
  if (!h || !W || !tokens || !seeds || !positions || !out || T < 0 || d <= 0 || V < 2) return ORACLE_ERR_ARG;
  if (!(sigma > 0.0) || !(eps >= 0.0) || !(temperature >= 0.0)) return ORACLE_ERR_ARG;
  int err = 0;
#pragma omp parallel
  {
    double* hd = (double*)malloc((size_t)d * sizeof(double));
    double* logit = (double*)malloc((size_t)V * sizeof(double));
    double* y = (double*)malloc((size_t)V * sizeof(double));
    if (!hd || !logit || !y) {
#pragma omp atomic write
      err = 1;
    }
#pragma omp barrier
    if (!err) {
#pragma omp for schedule(dynamic, 1)
      for (int64_t r = 0; r < T; ++r) {
        row_logits(h + r * d, W, d, V, hd, logit);
        gm_row(logit, y, V, tokens[r], seeds[r], positions[r], temperature, sigma, eps, noise_id, r, out);
      }
    }
    free(hd);
    free(logit);
    free(y);
  }
  return err ? ORACLE_ERR_MEM : ORACLE_OK;
}

/* ------------------------------------------------------ Token-IPT-DiFR */
typedef struct {
  double* score;     /* [T] ln(mass + eps)                                   */
  double* p_claimed; /* [T] p[t*]                                            */
  double* cdf_lo;    /* [T] a = sum_{v < t*} p_v                              */
  double* u;         /* [T] mu                                               */
  double* lse;       /* [T]                                                  */
  double* mass;      /* [T]                                                  */
  int32_t* sampled;  /* [T] Alg. IPT sampler with the same mu: min{v: C_v>mu} */
  uint32_t* row_status;
} oracle_ipt_out;

/* Alg. Token-IPT-DiFR's last steps: the Gaussian of width sigma centred on mu,
 * integrated over the claimed token's CDF interval [a, b], and its log-score. */
double oracle_ipt_mass(double a, double b, double mu, double sigma) {
  return normal_interval_mass((a - mu) / sigma, (b - mu) / sigma);
}
double oracle_ipt_score(double a, double b, double mu, double sigma, double eps) {
  return log(oracle_ipt_mass(a, b, mu, sigma) + eps);
}

/* One row of Token-IPT-DiFR from its logits.  p[V] is scratch. */
static void ipt_row(const double* logit, double* p, int64_t V, int64_t t, uint64_t seed, uint32_t position,
                    double temperature, double sigma, double eps, int64_t r, oracle_ipt_out* out) {
  uint32_t status = 0;
  for (int64_t v = 0; v < V; ++v)
    if (!isfinite(logit[v])) status |= 2u;
  const double inv_temp = 1.0 / temperature;
  double lse = log_sum_exp_scaled(logit, V, inv_temp);
  for (int64_t v = 0; v < V; ++v) p[v] = exp(logit[v] * inv_temp - lse);
  double mu = oracle_ipt_uniform(seed, position);
  /* the IPT sampler: first id whose cumulative mass exceeds mu */
  int64_t sampled = V - 1;
  {
    double C = 0.0;
    for (int64_t v = 0; v < V; ++v) {
      C += p[v];
      if (C > mu) {
        sampled = v;
        break;
      }
    }
  }
  int in_range = (t >= 0 && t < V);
  if (!in_range) status |= 1u;
  double a = NAN, pt = NAN, mass = 0.0, score = log(eps);
  if (in_range) {
    a = 0.0;
    for (int64_t v = 0; v < t; ++v) a += p[v];
    pt = p[t];
    double b = a + pt;
    mass = oracle_ipt_mass(a, b, mu, sigma);
    score = oracle_ipt_score(a, b, mu, sigma, eps);
  }
  if (out->score) out->score[r] = score;
  if (out->p_claimed) out->p_claimed[r] = pt;
  if (out->cdf_lo) out->cdf_lo[r] = a;
  if (out->u) out->u[r] = mu;
  if (out->lse) out->lse[r] = lse;
  if (out->mass) out->mass[r] = mass;
  if (out->sampled) out->sampled[r] = (int32_t)sampled;
  if (out->row_status) out->row_status[r] = status;
}

int oracle_score_ipt(const uint16_t* h, const uint16_t* W, const int32_t* tokens, const uint64_t* seeds,
                     const uint32_t* positions, double temperature, double sigma, double eps, int64_t T,
                     int64_t d, int64_t V, oracle_ipt_out* out) {
  if (!h || !W || !tokens || !seeds || !positions || !out || T < 0 || d <= 0 || V < 1) return ORACLE_ERR_ARG;
  if (!(sigma > 0.0) || !(eps >= 0.0) || !(temperature > 0.0)) return ORACLE_ERR_ARG;
  int err = 0;
#pragma omp parallel
  {
    double* hd = (double*)malloc((size_t)d * sizeof(double));
    double* logit = (double*)malloc((size_t)V * sizeof(double));
    double* p = (double*)malloc((size_t)V * sizeof(double));
    if (!hd || !logit || !p) {
#pragma omp atomic write
      err = 1;
    }
#pragma omp barrier
    if (!err) {
#pragma omp for schedule(dynamic, 1)
      for (int64_t r = 0; r < T; ++r) {
        row_logits(h + r * d, W, d, V, hd, logit);
        ipt_row(logit, p, V, tokens[r], seeds[r], positions[r], temperature, sigma, eps, r, out);
      }
    }
    free(hd);
    free(logit);
    free(p);
  }
  return err ? ORACLE_ERR_MEM : ORACLE_OK;
}

/* Both estimators from one evaluation of each row's logits: exactly what
 * oracle_score_gm (claims tokens_gm, width sigma_gm) and oracle_score_ipt (claims
 * tokens_ipt, width sigma_ipt) would write, row by row.  It exists so that
 * stored expected values for the large workloads cost one contraction per row
 * instead of two. */
int oracle_score_both(const uint16_t* h, const uint16_t* W, const int32_t* tokens_gm, const int32_t* tokens_ipt,
                      const uint64_t* seeds, const uint32_t* positions, double temperature, double sigma_gm,
                      double sigma_ipt, double eps, int64_t T, int64_t d, int64_t V, oracle_gm_out* gm,
                      oracle_ipt_out* ipt) {
  if (!h || !W || !tokens_gm || !tokens_ipt || !seeds || !positions || !gm || !ipt || T < 0 || d <= 0 || V < 2)
    return ORACLE_ERR_ARG;
  if (!(sigma_gm > 0.0) || !(sigma_ipt > 0.0) || !(eps >= 0.0) || !(temperature > 0.0)) return ORACLE_ERR_ARG;
  int err = 0;
#pragma omp parallel
  {
    double* hd = (double*)malloc((size_t)d * sizeof(double));
    double* logit = (double*)malloc((size_t)V * sizeof(double));
    double* scratch = (double*)malloc((size_t)V * sizeof(double));
    if (!hd || !logit || !scratch) {
#pragma omp atomic write
      err = 1;
    }
#pragma omp barrier
    if (!err) {
#pragma omp for schedule(dynamic, 1)
      for (int64_t r = 0; r < T; ++r) {
        row_logits(h + r * d, W, d, V, hd, logit);
        gm_row(logit, scratch, V, tokens_gm[r], seeds[r], positions[r], temperature, sigma_gm, eps, NULL, r, gm);
        ipt_row(logit, scratch, V, tokens_ipt[r], seeds[r], positions[r], temperature, sigma_ipt, eps, r, ipt);
      }
    }
    free(hd);
    free(logit);
    free(scratch);
  }
  return err ? ORACLE_ERR_MEM : ORACLE_OK;
}

/* ------------------------------------------------------------- detection */
typedef struct {
  int32_t n_flagged;
  int32_t n_match;
  double sum; /* NaN if any score is NaN */
  double min; /* over the non-NaN scores; +inf for an empty sequence */
} oracle_seq_stats;

/* flag iff score < tau (NaN counts as flagged); a row matches iff its margin
 * does not carry a sign bit (see oracle_gm_out.margin). seq_offsets nullable
 * => one sequence [0,T). */
int oracle_detect(const double* scores, double threshold, const double* margins, const int32_t* seq_offsets,
                  int64_t n_seq, int64_t T, uint8_t* flags, oracle_seq_stats* stats) {
  if (!scores || T < 0 || n_seq < 0) return ORACLE_ERR_ARG;
  for (int64_t r = 0; r < T; ++r)
    if (flags) flags[r] = (scores[r] < threshold || isnan(scores[r])) ? 1 : 0;
  if (!stats) return ORACLE_OK;
  int64_t one[2] = {0, T};
  int64_t ns = seq_offsets ? n_seq : 1;
  for (int64_t s = 0; s < ns; ++s) {
    int64_t lo = seq_offsets ? seq_offsets[s] : one[0];
    int64_t hi = seq_offsets ? seq_offsets[s + 1] : one[1];
    if (lo < 0 || hi > T || lo > hi) return ORACLE_ERR_ARG;
    oracle_seq_stats st = {0, 0, 0.0, INFINITY};
    for (int64_t r = lo; r < hi; ++r) {
      st.n_flagged += (scores[r] < threshold || isnan(scores[r]));
      if (margins) st.n_match += (!isnan(margins[r]) && !signbit(margins[r]));
      st.sum += scores[r];
      if (scores[r] < st.min) st.min = scores[r]; /* NaN never compares below */
    }
    stats[s] = st;
  }
  return ORACLE_OK;
}

/* ------------------------------------------------------- risk classes */
/* Alg. "Per-Token Risk Classification via GLS and Rank": 0 safe if score >= tau;
 * otherwise suspicious (1) if the claimed token is among the R largest raw logits,
 * else dangerous (2).  `ranks` are 0-based (0 = largest logit, the convention of
 * the paper's rank histograms), so "among the R largest" is rank < R: with cutoff 1
 * only the top-ranked token can be suspicious and with cutoff 4 the top four, which
 * is what makes log2 R the information a suspicious token can carry (appendix
 * "Logit-Rank Ablations").  The algorithm's printed test "rank > R" is the same rule
 * for a rank counted from 1.  A NaN score is not >= tau.  ranks nullable => classes
 * 0/1 only. */
int oracle_classify(const double* scores, double threshold, const int32_t* ranks, int32_t rank_cutoff, int64_t T,
                    uint8_t* classes) {
  if (!scores || !classes || T < 0) return ORACLE_ERR_ARG;
  for (int64_t r = 0; r < T; ++r) {
    if (scores[r] >= threshold) {
      classes[r] = 0;
    } else if (ranks && ranks[r] >= rank_cutoff) {
      classes[r] = 2;
    } else {
      classes[r] = 1;
    }
  }
  return ORACLE_OK;
}

/* ----------------------------------------------------- admissible sets */
/* |A_t(tau)| for every row: each vocabulary id i is scored as if it were the
 * claimed token (Token-DiFR, one competitor: the best other id under the row's
 * regenerated noise) and counted when that score is >= tau. */
int oracle_admissible_count(const uint16_t* h, const uint16_t* W, const uint64_t* seeds, const uint32_t* positions,
                            double temperature, double sigma, double eps, double tau, int64_t T, int64_t d,
                            int64_t V, int32_t* counts) {
  if (!h || !W || !seeds || !positions || !counts || T < 0 || d <= 0 || V < 2) return ORACLE_ERR_ARG;
  if (!(sigma > 0.0) || !(eps >= 0.0) || !(temperature >= 0.0)) return ORACLE_ERR_ARG;
  int err = 0;
#pragma omp parallel
  {
    double* hd = (double*)malloc((size_t)d * sizeof(double));
    double* logit = (double*)malloc((size_t)V * sizeof(double));
    double* y = (double*)malloc((size_t)V * sizeof(double));
    if (!hd || !logit || !y) {
#pragma omp atomic write
      err = 1;
    }
#pragma omp barrier
    if (!err) {
#pragma omp for schedule(dynamic, 1)
      for (int64_t r = 0; r < T; ++r) {
        row_logits(h + r * d, W, d, V, hd, logit);
        for (int64_t v = 0; v < V; ++v) y[v] = logit[v] + temperature * oracle_gumbel_noise(seeds[r], positions[r], (uint32_t)v);
        int64_t i1 = -1, i2 = -1;
        for (int64_t v = 0; v < V; ++v) {
          if (i1 < 0 || y[v] > y[i1]) {
            i2 = i1;
            i1 = v;
          } else if (i2 < 0 || y[v] > y[i2]) {
            i2 = v;
          }
        }
        int32_t n = 0;
        for (int64_t i = 0; i < V; ++i) {
          int64_t c = (i == i1) ? i2 : i1;
          double A = y[i] - y[c];
          if (oracle_gm_score(A, sigma, eps) >= tau) ++n;
        }
        counts[r] = n;
      }
    }
    free(hd);
    free(logit);
    free(y);
  }
  return err ? ORACLE_ERR_MEM : ORACLE_OK;
}

/* ------------------------------------------- exfiltratable information */
/* Per token: log2 |A_t| if safe, log2 R if suspicious, log2 |V| if dangerous
 * (the displayed cases of Sec. "Problems with FSSL Estimators ..."); bits[r]
 * nullable, seq_bits[s] = sum over the sequence's rows.  An empty admissible set
 * (count 0) carries no information: 0 bits. */
int oracle_exfiltratable_bits(const uint8_t* classes, const int32_t* counts, int32_t rank_cutoff, int64_t V,
                              const int32_t* seq_offsets, int64_t n_seq, int64_t T, double* bits,
                              double* seq_bits) {
  if (!classes || !counts || T < 0 || n_seq < 0 || V < 1 || rank_cutoff < 1) return ORACLE_ERR_ARG;
  int64_t ns = seq_offsets ? n_seq : 1;
  for (int64_t s = 0; s < ns; ++s) {
    int64_t lo = seq_offsets ? seq_offsets[s] : 0;
    int64_t hi = seq_offsets ? seq_offsets[s + 1] : T;
    if (lo < 0 || hi > T || lo > hi) return ORACLE_ERR_ARG;
    double total = 0.0;
    for (int64_t r = lo; r < hi; ++r) {
      double b;
      if (classes[r] == 0) {
        b = counts[r] > 0 ? log2((double)counts[r]) : 0.0;
      } else if (classes[r] == 1) {
        b = log2((double)rank_cutoff);
      } else {
        b = log2((double)V);
      }
      if (bits) bits[r] = b;
      total += b;
    }
    if (seq_bits) seq_bits[s] = total;
  }
  return ORACLE_OK;
}

int oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}
