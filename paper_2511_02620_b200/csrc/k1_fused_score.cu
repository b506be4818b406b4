// K1: LM-head contraction fused with the scoring epilogue.
//
//   logits l[r, v] = sum_k h[r, k] W[v, k]   -- tcgen05.mma (bf16 x bf16 -> fp32 in TMEM),
//                                               operands staged in shared memory by TMA
//   epilogue                                 -- reads the accumulator with tcgen05.ld and, without ever
//                                               storing a logit, regenerates the Gumbel noise of
//                                               (seed, position, vocabulary id), keeps the running
//                                               top-2 of y = l + Temp*G, the running log-sum-exp of
//                                               l/Temp and the exponential mass below the claimed id
//
// CTAs run as persistent pairs (a cluster of two, one CTA per SM).  A pair owns a
// 256 x 256 logit tile: each CTA loads its own 128 rows of h and its own 128 of
// the tile's 256 rows of W, and one thread of the pair's first CTA issues
// tcgen05.mma.cta_group::2, which reads both CTAs' shared memory and writes rows
// 0..127 of the accumulator to the first CTA's TMEM and rows 128..255 to the
// second's.  Per 256 x 256 x 64 step each SM therefore fills 32 KB of shared
// memory instead of the 48 KB a lone 128 x 256 tile needs.
//
// Warp roles in each CTA: warp 0 issues the TMA loads, warp 1 (first CTA only)
// issues the MMAs, warp 2 owns the TMEM allocation, warps 4..11 are the epilogue
// (two warpgroups, one per 128-column half of the CTA's 128 x 256 accumulator).
// Two accumulator stages (all 512 TMEM columns) let the epilogue of tile n
// overlap the MMAs of tile n + 1.  A work unit is (256-row tile, vocabulary
// strip); its running statistics stay in registers across the strip and leave
// as one 32-byte partial record per (row, strip, column half).
#include <cuda.h>
#include <cuda_runtime.h>
#include <math_constants.h>
#include <string.h>

#include "difr_device.cuh"
#include "difr_kernels.h"
#include "difr_plan.h"

namespace difr {

constexpr int kStages = 6;
constexpr int kABytes = kBM * kBK * 2;         // 16 KB: this CTA's 128 rows of h
constexpr int kBBytes = (kBN / 2) * kBK * 2;   // 16 KB: this CTA's 128 of the tile's 256 rows of W
constexpr int kStageBytes = kABytes + kBBytes;
constexpr int kAccStages = 2;
constexpr int kThreads = 384;
constexpr int kEpiWarp0 = 4;
constexpr int kEpiWarps = 8;
constexpr int kTmemCols = 512;
constexpr int kBarBytes = 256;
constexpr int kSmemBytes = kStages * kStageBytes + kBarBytes + 1024;  // + slack for 1024-byte alignment
constexpr float kMasked = -3.0e38f;  // stands in for -inf on padded vocabulary columns (keeps keys finite)

enum : int { kModeGm = 0, kModeIpt = 1, kModeDump = 2 };

struct Unit {
  int m, n0, n1, strip;  // m: 256-row tile of the pair
};

__device__ __forceinline__ Unit decode_unit(const K1Params& p, int u) {
  const int per_group = p.Gm * p.S;
  const int g = u / per_group;
  const int rem = u - g * per_group;
  const int m_base = g * p.Gm;
  const int cnt = min(p.Gm, p.m_tiles - m_base);
  Unit w;
  w.strip = rem / cnt;
  w.m = m_base + rem % cnt;
  w.n0 = (int)(((long long)w.strip * p.n_tiles) / p.S);
  w.n1 = (int)(((long long)(w.strip + 1) * p.n_tiles) / p.S);
  return w;
}

// ---------------------------------------------------------- running statistics
struct RowStats {
  float m1, m2;        // top-2 keys of y' (low 5 mantissa bits carry the column within its chunk)
  int i1, i2;          // their vocabulary ids
  float lmax;          // running max of z = l * c1
  float lsum, lsum_c;  // compensated sum of 2^(z - lmax)
  float lpre, lpre_c;  // the same restricted to ids below the claimed one
};

__device__ __forceinline__ void stats_init(RowStats& s) {
  s.m1 = s.m2 = -CUDART_INF_F;
  s.i1 = s.i2 = -1;
  s.lmax = -CUDART_INF_F;
  s.lsum = s.lsum_c = s.lpre = s.lpre_c = 0.f;
}

// sum += x with the rounding error carried in comp (Neumaier).
__device__ __forceinline__ void comp_add(float& sum, float& comp, float x) {
  float t = sum + x;
  comp += (fabsf(sum) >= fabsf(x)) ? ((sum - t) + x) : ((x - t) + sum);
  sum = t;
}

// One chunk of 32 consecutive vocabulary ids [base, base + 32) of one row.
template <int MODE>
__device__ __forceinline__ void process_chunk(uint32_t (&raw)[32], int base, int V, int tok, float c1,
                                              float neg_tl2, const RowNoise& rn, RowStats& s) {
  float l[32];
#pragma unroll
  for (int j = 0; j < 32; ++j) l[j] = __uint_as_float(raw[j]);
  if (base + 32 > V) {  // padded columns of the last tile (uniform over the warp)
#pragma unroll
    for (int j = 0; j < 32; ++j)
      if (base + j >= V) l[j] = kMasked;
  }

  // ---- softmax statistics (online log-sum-exp in base 2)
  {
    float cm = fmax3(l[0], l[1], l[2]);
#pragma unroll
    for (int j = 3; j + 1 < 32; j += 2) cm = fmax3(cm, l[j], l[j + 1]);
    cm = fmaxf(cm, l[31]);
    const float new_max = fmaxf(s.lmax, cm * c1);
    const float scale = ex2_approx(s.lmax - new_max);  // 0 on the first chunk
    s.lsum *= scale; s.lsum_c *= scale;
    s.lpre *= scale; s.lpre_c *= scale;
    s.lmax = new_max;
    const float shift = -new_max;
    float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
    for (int j = 0; j < 32; j += 4) {
      a0 += ex2_approx(fmaf(l[j + 0], c1, shift));
      a1 += ex2_approx(fmaf(l[j + 1], c1, shift));
      a2 += ex2_approx(fmaf(l[j + 2], c1, shift));
      a3 += ex2_approx(fmaf(l[j + 3], c1, shift));
    }
    const float cs = (a0 + a1) + (a2 + a3);
    comp_add(s.lsum, s.lsum_c, cs);
    const int tl = tok - base;  // ids below the claimed one: all, none, or the first tl of this chunk
    if (tl >= 32) {
      comp_add(s.lpre, s.lpre_c, cs);
    } else if (tl > 0) {
      float ps = 0.f;
#pragma unroll
      for (int j = 0; j < 32; ++j)
        if (j < tl) ps += ex2_approx(fmaf(l[j], c1, shift));
      comp_add(s.lpre, s.lpre_c, ps);
    }
  }

  // ---- Gumbel-max replay: top-2 of y' = l - Temp*ln2 * log2(-log2 u)
  if (MODE == kModeGm) {
    float c1k = -CUDART_INF_F, c2k = -CUDART_INF_F;
#pragma unroll
    for (int j = 0; j < 32; j += 4) {
      uint32_t x[4];
      row_noise_block(rn, (uint32_t)(base + j) >> 2, x);
      float key[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const float u = __uint_as_float(0x3F800000u | (x[q] >> 9)) - 0.99999994f;  // ((x>>9) + 1/2) 2^-23, exact
        const float e2 = -lg2_approx(u);                                           // -log2 u = E / ln 2
        const float y = fmaf(lg2_approx(e2), neg_tl2, l[j + q]);
        key[q] = __uint_as_float((__float_as_uint(y) & ~31u) | (uint32_t)(j + q));
      }
      // u within 2^-11 of one: -log2 u loses relative accuracy, redo those with a series for -ln(1 - w)
      const uint32_t xm = max(max(x[0], x[1]), max(x[2], x[3]));
      if (xm >= 0xFFE00000u) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          if (x[q] >= 0xFFE00000u) {
            const float w = __uint_as_float(0x3F800000u | ((~x[q]) >> 9)) - 0.99999994f;  // 1 - u, exact
            const float E = w * fmaf(w, fmaf(w, 0.33333334f, 0.5f), 1.0f);
            const float y = fmaf(lg2_approx(E * 1.4426950408889634f), neg_tl2, l[j + q]);
            key[q] = __uint_as_float((__float_as_uint(y) & ~31u) | (uint32_t)(j + q));
          }
        }
      }
      const float h1 = fmaxf(key[0], key[1]), l1 = fminf(key[0], key[1]);
      const float h2 = fmaxf(key[2], key[3]), l2 = fminf(key[2], key[3]);
      const float t1 = fmaxf(h1, h2);
      const float t2 = fmax3(fminf(h1, h2), l1, l2);
      const float n2 = fmax3(fminf(c1k, t1), c2k, t2);
      c1k = fmaxf(c1k, t1);
      c2k = n2;
    }
    // merge the chunk's top-2 into the running top-2 (earlier ids win ties)
    const int g1 = base + (int)(__float_as_uint(c1k) & 31u);
    const int g2 = base + (int)(__float_as_uint(c2k) & 31u);
    if (c1k > s.m1) {
      const bool q = c2k > s.m1;
      s.m2 = q ? c2k : s.m1;
      s.i2 = q ? g2 : s.i1;
      s.m1 = c1k;
      s.i1 = g1;
    } else if (c1k > s.m2) {
      s.m2 = c1k;
      s.i2 = g1;
    }
  }
}

template <int MODE>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
k1_fused_score(const __grid_constant__ CUtensorMap tmap_h, const __grid_constant__ CUtensorMap tmap_w,
               const K1Params p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t smem_base = (raw_addr + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (smem_base - raw_addr);

  // Both CTAs of a pair lay out their barriers at the same offsets.
  //   full[s]      first CTA's copy is used: 1 arrival (its producer) + the bytes of both CTAs' loads
  //   empty[s]     each CTA's own copy: 1 arrival, the MMA thread's commit delivered to both CTAs
  //   acc_full[a]  each CTA's own copy: 1 arrival, the commit after a tile's last MMA, delivered to both
  //   acc_empty[a] first CTA's copy is used: one arrival per epilogue warp of both CTAs
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kStages * kStageBytes);
  const uint32_t bar0 = smem_base + kStages * kStageBytes;
  auto full_bar = [&](int s) { return bar0 + 8u * (uint32_t)s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (uint32_t)(kStages + s); };
  auto acc_full_bar = [&](int a) { return bar0 + 8u * (uint32_t)(2 * kStages + a); };
  auto acc_empty_bar = [&](int a) { return bar0 + 8u * (uint32_t)(2 * kStages + kAccStages + a); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kStages + 2 * kAccStages);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t cta = cluster_ctarank();  // 0: the pair's first CTA (issues the MMAs), 1: its partner
  const int pair = blockIdx.x >> 1;
  const int n_pairs = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < kAccStages; ++a) {
      mbar_init(acc_full_bar(a), 1);
      mbar_init(acc_empty_bar(a), 2 * kEpiWarps);
    }
    *abort_flag = 0;
    mbar_fence_init();
    tma_prefetch_desc(&tmap_h);
    tma_prefetch_desc(&tmap_w);
  }
  if (warp == 2) {
    tmem_alloc_pair(smem_u32(tmem_slot), kTmemCols);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  __syncthreads();
  cluster_arrive();  // the partner's barriers are initialised and its TMEM allocated before anyone signals them
  cluster_wait();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      // a CTA re-reads its h tile for every vocabulary tile of the strip: keep it in L2;
      // a W tile is read by the pairs of one raster group at about the same time, then never again soon
      const uint64_t keep = l2_policy_evict_last(), stream = l2_policy_evict_first();
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int u = pair; u < p.n_units && ok; u += n_pairs) {
        const Unit w = decode_unit(p, u);
        const int row0 = w.m * kPairM + (int)cta * kBM;
        for (int n = w.n0; n < w.n1 && ok; ++n) {
          const int wrow0 = n * kBN + (int)cta * (kBN / 2);
          for (int k = 0; k < p.k_steps; ++k) {
            if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
            if (cta == 0) mbar_arrive_expect_tx(full_bar(stage), 2u * kStageBytes);
            const uint32_t full0 = map_to_cta(full_bar(stage), 0);
            const uint32_t a_dst = smem_base + (uint32_t)stage * kStageBytes;
            tma_load_2d_pair(a_dst, &tmap_h, k * kBK, row0, full0, keep);
            tma_load_2d_pair(a_dst + kABytes, &tmap_w, k * kBK, wrow0, full0, stream);
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
          }
        }
      }
    }
  } else if (warp == 1) {
    // -------------------------------------------------------------- MMA issuer
    if (cta == 0 && lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(kPairM, kBN);
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true;
      for (int u = pair; u < p.n_units && ok; u += n_pairs) {
        const Unit w = decode_unit(p, u);
        for (int n = w.n0; n < w.n1 && ok; ++n) {
          if (!mbar_wait(acc_empty_bar(acc), acc_phase ^ 1u, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t d_tmem = tmem_base + (uint32_t)(acc * kBN);
          for (int k = 0; k < p.k_steps; ++k) {
            if (!mbar_wait(full_bar(stage), phase, abort_flag)) { ok = false; break; }
            tc_fence_after();
            const uint32_t a_src = smem_base + (uint32_t)stage * kStageBytes;
            const uint64_t a_desc = umma_desc_k_major_sw128(a_src);
            const uint64_t b_desc = umma_desc_k_major_sw128(a_src + kABytes);
#pragma unroll
            for (int kk = 0; kk < kBK / 16; ++kk) {
              // 16 bf16 = 32 bytes further along K inside the 128-byte swizzled row: +2 in 16-byte units
              umma_bf16_pair(d_tmem, a_desc + (uint64_t)(2 * kk), b_desc + (uint64_t)(2 * kk), idesc,
                             (uint32_t)((k | kk) != 0));
            }
            umma_commit_pair(empty_bar(stage), 3);  // frees the stage in both CTAs once these MMAs have read it
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
          }
          if (ok) umma_commit_pair(acc_full_bar(acc), 3);
          if (++acc == kAccStages) { acc = 0; acc_phase ^= 1u; }
        }
      }
    }
  } else if (warp >= kEpiWarp0) {
    // ---------------------------------------------------------------- epilogue
    const int ew = warp - kEpiWarp0;
    const int quarter = ew & 3;  // == warp % 4: the TMEM lane quarter this warp may read
    const int half = ew >> 2;    // which 128 columns of the tile
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    for (int u = pair; u < p.n_units && ok; u += n_pairs) {
      const Unit w = decode_unit(p, u);
      const int row = w.m * kPairM + (int)cta * kBM + quarter * 32 + lane;
      const bool valid = row < p.T;
      RowNoise rn;
      RowStats st;
      stats_init(st);
      int tok = -1;
      if (MODE != kModeDump) {
        uint64_t seed = 0;
        uint32_t pos = 0;
        if (valid) {
          tok = p.tokens[row];
          seed = p.seeds[row];
          pos = p.positions[row];
        }
        if (MODE == kModeGm) row_noise_init(rn, seed, pos);
      }
      for (int n = w.n0; n < w.n1; ++n) {
        if (!mbar_wait(acc_full_bar(acc), acc_phase, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const int col0 = n * kBN + half * (kBN / 2);
#pragma unroll 1
        for (int c = 0; c < (kBN / 2) / 32; ++c) {
          const int base = col0 + c * 32;
          if (base >= p.V) break;
          uint32_t raw[32];
          __syncwarp();
          tmem_ld_32x32(tmem_base + lane_addr + (uint32_t)(acc * kBN + half * (kBN / 2) + c * 32), raw);
          tmem_ld_wait();
          if (MODE == kModeDump) {
            if (valid) {
              float* dst = p.logits_out + (size_t)row * (size_t)p.V + base;
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (base + j < p.V) dst[j] = __uint_as_float(raw[j]);
            }
          } else {
            process_chunk<MODE>(raw, base, p.V, tok, p.c1, p.neg_tl2, rn, st);
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(map_to_cta(acc_empty_bar(acc), 0));
        if (++acc == kAccStages) { acc = 0; acc_phase ^= 1u; }
      }
      if (MODE != kModeDump && valid && ok) {
        Partial out;
        out.m1 = st.m1; out.i1 = st.i1; out.m2 = st.m2; out.i2 = st.i2;
        out.lse2_max = st.lmax;
        out.lse2_sum = st.lsum + st.lsum_c;
        out.prefix2 = st.lpre + st.lpre_c;
        out.reserved = 0.f;
        Partial* dst = p.partials + (size_t)(w.strip * 2 + half) * (size_t)p.T_pad + row;
        const float4* src = reinterpret_cast<const float4*>(&out);
        reinterpret_cast<float4*>(dst)[0] = src[0];
        reinterpret_cast<float4*>(dst)[1] = src[1];
      }
    }
  }

  __syncwarp();
  if (*abort_flag) {
    // a wait ran out somewhere: give copies and MMAs still in flight time to land before TMEM is released
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000LL) { }
  }
  tc_fence_before();
  __syncthreads();
  // Neither CTA may leave while the other can still signal its barriers or while MMAs
  // issued by the first CTA can still touch the partner's shared memory and TMEM.
  cluster_arrive();
  cluster_wait();
  if (warp == 2) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, kTmemCols);
  }
  if (threadIdx.x == 0 && *abort_flag && p.device_status != nullptr) *p.device_status = kStatusTimeout;
}

// ------------------------------------------------------------------ launcher
template <int MODE>
static cudaError_t launch_mode(const CUtensorMap& th, const CUtensorMap& tw, const K1Params& p, int grid,
                               cudaStream_t stream) {
  cudaError_t e = cudaFuncSetAttribute(k1_fused_score<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
  if (e != cudaSuccess) return e;
  k1_fused_score<MODE><<<grid, kThreads, kSmemBytes, stream>>>(th, tw, p);  // grid: two CTAs per pair
  return cudaGetLastError();
}

// Number of CTA pairs the device keeps resident at once (one CTA per SM, pairs on adjacent SMs).
template <int MODE>
static int max_pairs_mode() {
  if (cudaFuncSetAttribute(k1_fused_score<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) !=
      cudaSuccess)
    return 0;
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof cfg);
  cfg.gridDim = dim3(2 * 148, 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = kSmemBytes;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeClusterDimension;
  attr.val.clusterDim.x = 2;
  attr.val.clusterDim.y = 1;
  attr.val.clusterDim.z = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, k1_fused_score<MODE>, &cfg) != cudaSuccess) return 0;
  return n;
}

int k1_max_resident_pairs() { return max_pairs_mode<kModeGm>(); }

cudaError_t launch_k1(int mode, const CUtensorMap& tmap_h, const CUtensorMap& tmap_w, const K1Params& p, int grid,
                      cudaStream_t stream) {
  switch (mode) {
    case kModeGm: return launch_mode<kModeGm>(tmap_h, tmap_w, p, grid, stream);
    case kModeIpt: return launch_mode<kModeIpt>(tmap_h, tmap_w, p, grid, stream);
    case kModeDump: return launch_mode<kModeDump>(tmap_h, tmap_w, p, grid, stream);
  }
  return cudaErrorInvalidValue;
}

}  // namespace difr
