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
  Partial* partials;  // [n_slots][T_pad]
  float* logits_out;  // dump mode only
  int32_t* device_status;
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
  int ipt;  // 0: Token-DiFR (Gumbel-max), 1: Token-IPT-DiFR
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

// mode: 0 Gumbel-max epilogue, 1 softmax statistics only, 2 logits dump.
cudaError_t launch_k1(int mode, const CUtensorMap& tmap_h, const CUtensorMap& tmap_w, const K1Params& p, int grid,
                      cudaStream_t stream);  // grid: number of CTAs, two per pair
int k1_max_resident_pairs();  // CTA pairs of the fused kernel the current device keeps resident at once
cudaError_t launch_k2(const K2Params& p, cudaStream_t stream);
cudaError_t launch_k3(const K3Params& p, cudaStream_t stream);
cudaError_t launch_philox(const uint32_t* ctr, const uint32_t* key, int64_t n, uint32_t* out, cudaStream_t stream);

}  // namespace difr
