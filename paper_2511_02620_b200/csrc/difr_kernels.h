// Parameter blocks and launchers of the three kernels (host-visible part).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "difr_device.cuh"

namespace difr {

constexpr int kStatusTimeout = -7;  // DIFR_ERR_TIMEOUT

struct K1Params {
  const int32_t* tokens;
  const uint64_t* seeds;
  const uint32_t* positions;
  const float* temperatures;  // [T], nullable: per-row temperature in place of c1 / neg_tl2
  const float* bounds;  // [5][T_pad]: planes 0..3 claimed logits (rank mode) or bounds on y' (counting modes), each
                        // raised by the fp32 rounding allowance; plane 4 the width of the undecided band below
  BandEntry* band_list;  // rank / counting modes: [T_pad][band_cap] ids inside a band, for the exact decision
  int* band_count;       // [T_pad], zeroed before the launch; may end above band_cap (overflow)
  int band_cap;
  void* cand_list;      // collect mode: [T][cand_cap] records {int32 id, float l, float y'}
  int* cand_count;      // collect mode: [T], zeroed before the launch; may end above cand_cap (overflow)
  int cand_cap;
  Partial* partials;  // [T_pad][S]: a row's records side by side (the finalize kernels read them a row at a time)
  float* logits_out;  // dump mode only
  int32_t* device_status;
  int* row_floor;     // Gumbel-max scoring modes, nullable: [T_pad] per-row lower bounds of the second largest key
                      // (order-preserving integers), every byte preset to 0x80 (a value below every key)
  int* rank_out;      // Collect mode, nullable: [T] zeroed counters that receive the claimed tokens' raw-logit ranks
  int* unit_counter;  // zeroed before the launch: units are handed out in order on demand; null: round robin
  int T, d, V;
  int T_pad, m_tiles, n_tiles, k_steps;
  int S, Gm, n_units;
  float c1;       // log2(e) / Temp  (0 when Temp == 0)
  float neg_tl2;  // -Temp * ln 2
};

struct K2Params {
  const uint16_t* h;
  const uint16_t* W;
  const int32_t* tokens;
  const uint64_t* seeds;
  const uint32_t* positions;
  const Partial* partials;
  int n_slots, T_pad;
  int T, d, V;
  const float* temperatures;  // [T], nullable: per-row temperature in place of `temperature` / `c1`
  int ipt;  // 0: Token-DiFR (Gumbel-max), 1: Token-IPT-DiFR, 2: both (IPT score to score_ipt with sigma_ipt)
  int tok_logit_in_records;  // the records' last words add up to the bits of the claimed token's fp32 logit
  float sigma_ipt;
  float* score_ipt;
  int32_t* rank;
  const BandEntry* band_list;  // rank mode: the ids the fused kernel could not decide in fp32 (nullable)
  const int* band_count;
  int band_cap;
  float* y_max;
  float* y_second;
  float temperature, sigma, eps;
  float c1;  // log2(e) / Temp as used by the fused kernel
  float* score;
  float* margin;
  int32_t* argmax;
  int32_t* runner_up;
  float* lse;
  float* p_claimed;
  float* cdf_lo;
  float* u;
  uint32_t* row_status;
};

struct K3Params {
  const float* scores;
  const float* margins;
  const int32_t* ranks;
  const int32_t* seq_offsets;
  float threshold;
  int32_t rank_cutoff;
  int64_t n_seq, T;
  uint8_t* flags;
  void* seq_stats;
};

// mode: 0 Gumbel-max epilogue, 1 softmax statistics only, 2 logits dump, 3 Gumbel-max + raw-logit rank,
// 4 / 5 count the ids whose noisy logit reaches one / four per-row bounds, 6 Gumbel-max + the strips' two
// largest 16-id group maxima (word 7 of the record), 7 collect the ids that reach the row's bounds on y' / l,
// 8 softmax statistics + group maxima, 9 collect by raw logit only.
cudaError_t launch_k1(int mode, const CUtensorMap& tmap_h, const CUtensorMap& tmap_w, const K1Params& p, int grid,
                      cudaStream_t stream);
// The collecting modes (7, 9) over logits the first pass stored: [T][V] fp32, p as for launch_k1.
cudaError_t launch_collect_from_logits(int mode, const K1Params& p, const float* logits, cudaStream_t stream);  // grid: number of CTAs, two per pair
int k1_max_resident_pairs();  // CTA pairs of the fused kernel the current device keeps resident at once
cudaError_t launch_k2(const K2Params& p, cudaStream_t stream);
cudaError_t launch_k3(const K3Params& p, cudaStream_t stream);

// Claimed logits l[r, tokens[r]] plus the tensor cores' rounding allowance into hi[r] (+inf for an id outside
// [0, V)) and the width of the undecided band below it into width[r]: one warp per row.
cudaError_t launch_claimed_logits(const uint16_t* h, const uint16_t* W, const int32_t* tokens, int T, int d, int V,
                                  float* hi, float* width, cudaStream_t stream);

// Counting pass of the admissible sets.
struct CountParams {
  const uint16_t* h;
  const uint16_t* W;
  const uint64_t* seeds;
  const uint32_t* positions;
  const Partial* partials;  // records of the counting modes: four int32 counts each
  int n_slots, T_pad, T, d, V, n_tau;
  const int32_t* argmax;
  const int32_t* runner_up;  // nullable: without it the sample's own margin is taken from y_max - y_second in fp32
  const float* y_max;
  const float* y_second;
  float temperature, sigma, eps;
  float a_tau[4];   // A(tau_j): id i != argmax is admissible iff y_i - y_max >= A(tau_j)
  float taus[4];
  float y_shift;    // the fused kernel ranks y' = y + y_shift
  float* bounds;    // [5][T_pad] out: bounds on y' (raised by the fp32 allowance), band width in plane 4
  const BandEntry* band_list;
  const int* band_count;
  int band_cap;
  int32_t* counts;  // [n_tau][T] out
  uint32_t* row_status;  // nullable out: bit 5 = the row's list of undecided ids overflowed
};
cudaError_t launch_count_bounds(const CountParams& p, cudaStream_t stream);
cudaError_t launch_count_finalize(const CountParams& p, cudaStream_t stream);

// Full Token-DiFR estimator: bounds for the collecting pass and the finalize over the candidate lists.
struct FilterParams {
  const uint16_t* h;
  const uint16_t* W;
  const int32_t* tokens;
  const uint64_t* seeds;
  const uint32_t* positions;
  const Partial* partials;  // records of the first pass (mode GmFilter)
  int n_slots, T_pad, T, d, V;
  float temperature, sigma, eps, c1;
  int top_k;    // as the caller gave it (0 or >= V: no top-k); one per row in top_k_rows when that is given
  float top_p;  // 1: no nucleus; one per row in top_p_rows when that is given
  const int32_t* top_k_rows;   // nullable
  const float* top_p_rows;     // nullable
  float min_p;                 // 0: no min-p; one per row in min_p_rows when that is given
  const float* min_p_rows;     // nullable
  const float* temperatures;   // nullable: one temperature per row (then `temperature` and `c1` are unused)
  int ipt;      // the IPT estimator's finalize: a row without any filter keeps the first pass's outputs
  int s;        // competitors in the active subset
  float* bounds;  // [3][T_pad]: on y', on the raw logit; claimed logits (when the rank is wanted)
  const Candidate* cand_list;
  const int* cand_count;
  int cand_cap;
  float* score;
  float* cutoff;  // nullable
  int32_t* rank;  // nullable: counted by the collecting pass; the finalize sets V for an out-of-range claim
  uint32_t* row_status;
  float* p_claimed;  // IPT finalize only, nullable
  float* cdf_lo;
  float* u;
  // filters of any size (one policy for the whole call): the kept prefix found by select_cutoff; null otherwise
  const int* sel_cut_id;
  const int* sel_top_id;
  const int* sel_kept_n;  // negative: the min-p bound ended the prefix
  const double* sel_z;
  const double* sel_below;
  const double* sel_mine;
};
cudaError_t launch_filter_bounds(const FilterParams& p, cudaStream_t stream);
cudaError_t launch_filtered_finalize(const FilterParams& p, cudaStream_t stream);
cudaError_t launch_ipt_filtered_finalize(const FilterParams& p, cudaStream_t stream);
cudaError_t launch_ipt_select_finalize(const FilterParams& p, cudaStream_t stream);

// Filters of any size: exact length and last id of the kept prefix from a block of rows' fp32 logits.
struct SelectParams {
  const float* logits;   // [rows][V]: the logits of rows row0 .. row0 + rows - 1
  int rows, V, row0;
  const int32_t* tokens;       // [T]
  const float* temperatures;   // [T], nullable
  float temperature;
  int top_k;      // 0 or >= V: none
  float top_p;    // 1: none
  float min_p;    // 0: none
  const int32_t* top_k_rows;  // [T], nullable: one value per row in place of the scalar; a value outside its
  const float* top_p_rows;    //      range acts as "none" here (the finalize kernels mark such a row)
  const float* min_p_rows;
  int* cut_id;    // [T] out: the last kept id in the order (logit descending, id ascending)
  int* top_id;    // [T] out: the id of the largest logit (lowest id among equals)
  int* kept_n;    // [T] out: how many ids are kept; negated when the min-p bound ended the prefix
  int want_sums;       // non-zero: also sum the kept ids' masses (one more walk over the row)
  double* kept_z;      // [T] out: mass of the kept ids, of those below the claimed id, of the claimed id if kept,
  double* kept_below;  //         all in units of 2^-40 of the row's largest term
  double* kept_mine;
  uint32_t* row_status;  // nullable: bit 4 when more than 256 ids tie exactly at the cutoff
};
cudaError_t launch_select_cutoff(const SelectParams& p, cudaStream_t stream);

struct BitsParams {
  const uint8_t* classes;
  const int32_t* counts;
  const int32_t* seq_offsets;
  int64_t n_seq, T;
  float log2_r, log2_v;
  float* bits;
  float* seq_bits;
};
cudaError_t launch_bits(const BitsParams& p, cudaStream_t stream);
cudaError_t launch_wait_selftest(int32_t* status, long long limit_cycles, cudaStream_t stream);
cudaError_t launch_expand_seeds(const uint64_t* seeds, const int32_t* tokens, const int32_t* seq_offsets,
                                const uint64_t* prompt_hashes, long long n_seq, long long T, uint64_t* expanded,
                                cudaStream_t stream);
cudaError_t launch_philox(const uint32_t* ctr, const uint32_t* key, int64_t n, uint32_t* out, cudaStream_t stream);

}  // namespace difr
