// K2: split-V finalize.  One warp per row merges the row's partial records with
// warp shuffles, re-evaluates in fp64 the few logits the score depends on (the
// claimed token and every Gumbel-max candidate whose key lies within the fused
// kernel's ranking noise of the second largest: gathered rows of W against the
// row of h), ranks them exactly, and turns the margin (Token-DiFR) or the CDF
// interval (Token-IPT-DiFR) into the log-score.
#include <cuda_runtime.h>
#include <math_constants.h>

#include "difr_device.cuh"
#include "difr_kernels.h"

namespace difr {

constexpr int kK2Warps = 8;

struct Merged {
  float m1, m2;
  int i1, i2;
  double lmax, lsum, lpre;  // base-2 log-sum-exp state
  int larger;               // ids whose logit exceeds the claimed one (rank mode)
};

__device__ __forceinline__ bool beats(float v, int i, float w, int j) {
  // candidate (v, i) ranks ahead of (w, j); absent candidates carry id -1
  if (i < 0) return false;
  if (j < 0) return true;
  return v > w || (v == w && i < j);
}

__device__ __forceinline__ void top2_insert(Merged& a, float v, int i) {
  if (beats(v, i, a.m1, a.i1)) {
    a.m2 = a.m1; a.i2 = a.i1;
    a.m1 = v; a.i1 = i;
  } else if (beats(v, i, a.m2, a.i2)) {
    a.m2 = v; a.i2 = i;
  }
}

__device__ __forceinline__ void lse_merge(Merged& a, double bmax, double bsum, double bpre) {
  if (bmax == -CUDART_INF) return;
  if (a.lmax == -CUDART_INF) {
    a.lmax = bmax; a.lsum = bsum; a.lpre = bpre;
    return;
  }
  const double m = fmax(a.lmax, bmax);
  const double fa = exp2(a.lmax - m), fb = exp2(bmax - m);
  a.lsum = a.lsum * fa + bsum * fb;
  a.lpre = a.lpre * fa + bpre * fb;
  a.lmax = m;
}

// Phi(zb) - Phi(za), za <= zb, evaluated in the tail that avoids cancellation.
__device__ __forceinline__ double normal_interval(double za, double zb) {
  const double r = 0.70710678118654752440;
  if (za >= 0.0) return 0.5 * (erfc(za * r) - erfc(zb * r));
  if (zb <= 0.0) return 0.5 * (erfc(-zb * r) - erfc(-za * r));
  return 1.0 - 0.5 * erfc(zb * r) - 0.5 * erfc(-za * r);
}

__global__ void __launch_bounds__(kK2Warps * 32, 4) k2_finalize(const K2Params p) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row = blockIdx.x * kK2Warps + warp;
  if (row >= p.T) return;  // whole warps leave together

  // ---- merge the row's partial records
  Merged acc;
  acc.m1 = acc.m2 = -CUDART_INF_F;
  acc.i1 = acc.i2 = -1;
  acc.lmax = -CUDART_INF;
  acc.lsum = acc.lpre = 0.0;
  acc.larger = 0;
  uint32_t tie_bits = 0u;  // bit j: this lane's record of slot lane + 32 j carries the fused kernel's tie mark
  for (int slot = lane; slot < p.n_slots; slot += 32) {
    const float4* src = reinterpret_cast<const float4*>(p.partials + (size_t)row * (size_t)p.n_slots + slot);
    const float4 a = src[0], b = src[1];
    top2_insert(acc, a.x, __float_as_int(a.y));
    top2_insert(acc, a.z, __float_as_int(a.w));
    lse_merge(acc, (double)b.x, (double)fabsf(b.y), (double)b.z);  // (the sign bit of the sum is the tie mark)
    if (signbit(b.y) && slot < 1024) tie_bits |= 1u << (slot >> 5);
    acc.larger += __float_as_int(b.w);
  }
#pragma unroll
  for (int m = 16; m >= 1; m >>= 1) {
    const float o1 = __shfl_xor_sync(0xffffffffu, acc.m1, m), o2 = __shfl_xor_sync(0xffffffffu, acc.m2, m);
    const int j1 = __shfl_xor_sync(0xffffffffu, acc.i1, m), j2 = __shfl_xor_sync(0xffffffffu, acc.i2, m);
    const double om = shfl_xor_double(acc.lmax, m), os = shfl_xor_double(acc.lsum, m),
                 op = shfl_xor_double(acc.lpre, m);
    top2_insert(acc, o1, j1);
    top2_insert(acc, o2, j2);
    lse_merge(acc, om, os, op);
    acc.larger += __shfl_xor_sync(0xffffffffu, acc.larger, m);
  }
  // (every lane now holds the same merged state up to the order of the lse additions; use lane 0's)
  acc.lmax = __hiloint2double(__shfl_sync(0xffffffffu, __double2hiint(acc.lmax), 0),
                              __shfl_sync(0xffffffffu, __double2loint(acc.lmax), 0));
  acc.lsum = __hiloint2double(__shfl_sync(0xffffffffu, __double2hiint(acc.lsum), 0),
                              __shfl_sync(0xffffffffu, __double2loint(acc.lsum), 0));
  acc.lpre = __hiloint2double(__shfl_sync(0xffffffffu, __double2hiint(acc.lpre), 0),
                              __shfl_sync(0xffffffffu, __double2loint(acc.lpre), 0));

  const int tok = p.tokens[row];
  const uint64_t seed = p.seeds[row];
  const uint32_t pos = p.positions[row];
  const bool tok_ok = tok >= 0 && tok < p.V;
  const uint16_t* hrow = p.h + (size_t)row * (size_t)p.d;
  // the call's temperature, or the row's own (then c1 is rebuilt exactly as the fused kernel built it)
  float temp_f = p.temperature, c1_f = p.c1;
  if (p.temperatures != nullptr) {
    temp_f = p.temperatures[row];
    c1_f = temp_f > 0.f ? 1.4426950408889634f / temp_f : 0.f;
  }
  const double temp = (double)temp_f;
  const double sigma = (double)p.sigma, eps = (double)p.eps;
  uint32_t status = tok_ok ? 0u : 1u;

  const double ln2 = 0.69314718055994530942;
  const bool lse_finite = isfinite(acc.lmax) && isfinite(acc.lsum) && acc.lsum > 0.0;
  if (!lse_finite) status |= 2u;
  const bool temp_bad = !(temp_f >= 0.f) || isinf(temp_f) || (p.ipt != 0 && temp_f == 0.f);
  if (temp_bad) status |= 8u;
  double lse = (temp_f > 0.f) ? (acc.lmax + log2(acc.lsum)) * ln2 : CUDART_NAN;

  // ---- exact (fp64) values.  Token-DiFR: y = l + Temp * G of the claimed token and of every candidate that can
  // be among the two largest.  The fused kernel ranks by fp32 keys whose error (tensor-core accumulation,
  // lg2.approx in the noise, the index bits in the low mantissa) is bounded by `noise`; an id whose exact y is
  // among the two largest has a key within 2 * noise of the second largest key, so every candidate of the strips'
  // records inside that window is re-evaluated and the two largest are taken exactly (ties: lowest id).  The dot
  // products go three at a time (the claimed token and, normally, the two candidates) with their loads in flight
  // together.
  double l_tok = 0.0, yt = -CUDART_INF;
  double yb1 = -CUDART_INF, yb2 = -CUDART_INF;
  int ib1 = -1, ib2 = -1;
  auto place = [&](double y, int id) {
    if (id == ib1 || id == ib2) return;  // (a group that is walked whole can bring an id a second time)
    if (ib1 < 0 || y > yb1 || (y == yb1 && id < ib1)) {
      yb2 = yb1; ib2 = ib1;
      yb1 = y; ib1 = id;
    } else if (ib2 < 0 || y > yb2 || (y == yb2 && id < ib2)) {
      yb2 = y; ib2 = id;
    }
  };
  int pend[3] = {-1, -1, -1};
  int n_pend = 0;
  auto flush = [&]() {
    if (n_pend == 0) return;
    double l[3];
    warp_dot3(hrow, pend[0] >= 0 ? p.W + (size_t)pend[0] * (size_t)p.d : nullptr,
              pend[1] >= 0 ? p.W + (size_t)pend[1] * (size_t)p.d : nullptr,
              pend[2] >= 0 ? p.W + (size_t)pend[2] * (size_t)p.d : nullptr, p.d, lane, l);
#pragma unroll
    for (int i = 0; i < 3; ++i) {
      if (pend[i] < 0) continue;
      const double y = (p.ipt != 1) ? l[i] + temp * gumbel_exact(seed, pos, (uint32_t)pend[i]) : 0.0;
      if (pend[i] == tok) { l_tok = l[i]; yt = y; }
      if (p.ipt != 1) place(y, pend[i]);
      pend[i] = -1;
    }
    n_pend = 0;
  };
  auto push = [&](int id) {
    if (n_pend == 0) pend[0] = id; else if (n_pend == 1) pend[1] = id; else pend[2] = id;
    if (++n_pend == 3) flush();
  };
  if (tok_ok) push(tok);
  if (p.ipt != 1) {
    const float noise = 3e-4f * temp_f + 1e-4f + 3.9e-6f * fabsf(acc.m2);
    const float window = acc.m2 - 2.f * noise;  // -inf when there is no second candidate: everything qualifies
    for (int base = 0; base < p.n_slots; base += 32) {
      const int slot = base + lane;
      float4 a = make_float4(-CUDART_INF_F, __int_as_float(-1), -CUDART_INF_F, __int_as_float(-1));
      bool tie_mark = false;
      if (slot < p.n_slots) {
        const float4* src = reinterpret_cast<const float4*>(p.partials + (size_t)row * (size_t)p.n_slots + slot);
        a = src[0];
        tie_mark = base < 1024 ? ((tie_bits >> (base >> 5)) & 1u) != 0u : signbit(src[1].y);
      }
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const float key = e ? a.z : a.x;
        const int id = __float_as_int(e ? a.w : a.y);
        unsigned todo = __ballot_sync(0xffffffffu, id >= 0 && id < p.V && !(key < window));
        const unsigned marked = __ballot_sync(0xffffffffu, tie_mark);
        while (todo) {
          const int src_lane = __ffs(todo) - 1;
          todo &= todo - 1;
          const int cid = __shfl_sync(0xffffffffu, id, src_lane);
          if ((marked >> src_lane) & 1u) {
            // this strip ranked equal keys inside a 16-id group by column, not by id: every id of the
            // candidate's group is a candidate
            const int g0 = cid & ~15;
            for (int v = g0; v < g0 + 16 && v < p.V; ++v)
              if (v != tok) push(v);
          } else if (cid != tok) {
            push(cid);
          }
        }
      }
    }
  }
  flush();

  // The softmax sums come from the tensor cores' fp32 logits, the claimed token's own logit from the fp64 dot
  // product: where the claimed token carries much of the mass, the rounding of its fp32 logit (1e-5 of a unit
  // per ten units of magnitude) would go straight into p[t*].  The fused kernel sent that fp32 logit along;
  // its term of the sum is replaced by the exact one.
  if (p.tok_logit_in_records && tok_ok && acc.larger != 0 && temp_f > 0.f && isfinite(acc.lmax)) {
    const double l_fp32 = (double)__int_as_float(acc.larger);
    const double c1d = (double)c1_f;
    const double swapped = acc.lsum - exp2(l_fp32 * c1d - acc.lmax) + exp2(l_tok * c1d - acc.lmax);
    if (swapped > 0.0 && isfinite(swapped)) {
      acc.lsum = swapped;
      lse = (acc.lmax + log2(acc.lsum)) * ln2;
    }
  }

  // raw-logit rank: the fused kernel counted the ids whose fp32 logit is above the claimed one by more than the
  // tensor cores' rounding; the ids it could not decide are on the row's list and are decided here in fp64
  if (p.rank != nullptr && p.band_count != nullptr && tok_ok) {
    const int n_found = p.band_count[row];
    const int n_band = n_found < p.band_cap ? n_found : p.band_cap;
    if (n_found > p.band_cap) status |= 32u;
    const BandEntry* list = p.band_list + (size_t)row * (size_t)p.band_cap;
    for (int e = 0; e < n_band; e += 3) {
      double l[3];
      const int i0 = list[e].id, i1 = e + 1 < n_band ? list[e + 1].id : -1, i2 = e + 2 < n_band ? list[e + 2].id : -1;
      warp_dot3(hrow, p.W + (size_t)i0 * (size_t)p.d, i1 >= 0 ? p.W + (size_t)i1 * (size_t)p.d : nullptr,
                i2 >= 0 ? p.W + (size_t)i2 * (size_t)p.d : nullptr, p.d, lane, l);
      acc.larger += (l[0] > l_tok) ? 1 : 0;
      acc.larger += (i1 >= 0 && l[1] > l_tok) ? 1 : 0;
      acc.larger += (i2 >= 0 && l[2] > l_tok) ? 1 : 0;
    }
  }

  if (p.ipt != 1) {
    if (lane == 0) {
      double A = -CUDART_INF;
      if (tok_ok) {
        // strongest competitor: the best id that is not the claimed token
        const int c = (ib1 != tok) ? ib1 : ib2;
        const double yc = (ib1 != tok) ? yb1 : yb2;
        A = (c >= 0) ? yt - yc : CUDART_INF;
        if (A == 0.0 && tok > c) A = -0.0;
      }
      const double pi = 0.5 * erfc(-A / (2.0 * sigma));  // Phi(A / (sigma sqrt 2))
      double score = tok_ok ? log(pi + eps) : log(eps);
      if (temp_bad || !lse_finite) score = CUDART_NAN;  // a row with a non-finite logit is never scored as safe
      p.score[row] = (float)score;
      if (p.margin) p.margin[row] = (float)A;
      if (p.argmax) p.argmax[row] = ib1;
      if (p.runner_up) p.runner_up[row] = ib2;
      if (p.lse) p.lse[row] = (float)lse;
      if (p.row_status) p.row_status[row] = status;
      if (p.rank) p.rank[row] = tok_ok ? acc.larger : p.V;
      if (p.y_max) p.y_max[row] = (float)yb1;
      if (p.y_second) p.y_second[row] = (float)yb2;
    }
  }
  if (p.ipt != 0) {
    // ---- Token-IPT-DiFR
    if (lane == 0) {
      uint32_t x[4];
      philox4x32_10(0u, pos, 1u, 0u, (uint32_t)seed, (uint32_t)(seed >> 32), x);
      const double mu = ((double)x[0] + 0.5) * (1.0 / 4294967296.0);
      double score = log(eps), pt = CUDART_NAN, a = CUDART_NAN;
      if (tok_ok) {
        const double c1d = (double)c1_f;  // log2(e) / Temp, the very factor the fused kernel scaled its logits by
        pt = exp2(l_tok * c1d - acc.lmax) / acc.lsum;
        a = acc.lpre / acc.lsum;
        const double b = a + pt;
        const double sg = (p.ipt == 2) ? (double)p.sigma_ipt : sigma;
        const double mass = normal_interval((a - mu) / sg, (b - mu) / sg);
        score = log(mass + eps);
      }
      if (temp_bad || !lse_finite) score = CUDART_NAN;
      (p.ipt == 2 ? p.score_ipt : p.score)[row] = (float)score;
      if (p.lse) p.lse[row] = (float)lse;
      if (p.p_claimed) p.p_claimed[row] = (float)pt;
      if (p.cdf_lo) p.cdf_lo[row] = (float)a;
      if (p.u) p.u[row] = (float)mu;
      if (p.row_status) p.row_status[row] = status;
    }
  }
}

cudaError_t launch_k2(const K2Params& p, cudaStream_t stream) {
  const int blocks = (p.T + kK2Warps - 1) / kK2Warps;
  k2_finalize<<<blocks, kK2Warps * 32, 0, stream>>>(p);
  return cudaGetLastError();
}

// --------------------------------------------------------- claimed logits
// What the fused kernel's rank mode compares every fp32 logit with: the claimed token's logit l[r, tokens[r]]
// (fp64 dot product) raised by `allow`, a bound on the rounding of a tensor-core logit of that size, and the
// width 2 * allow of the band below in which fp32 cannot tell "larger" from "smaller".  The tensor cores add
// the d / 16 partial products of a logit in fp32 with truncation: at most one unit in the last place of the
// running sum per step.  +inf / 0 for an id outside [0, V): nothing counts.
__global__ void __launch_bounds__(kK2Warps * 32)
claimed_logits(const uint16_t* h, const uint16_t* W, const int32_t* tokens, int T, int d, int V, float* hi,
               float* width) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row = blockIdx.x * kK2Warps + warp;
  if (row >= T) return;
  const int tok = tokens[row];
  float v = CUDART_INF_F, w = 0.f;
  if (tok >= 0 && tok < V) {
    const double l = warp_dot(h + (size_t)row * (size_t)d, W + (size_t)tok * (size_t)d, d, lane);
    const double allow = 1.1920928955078125e-7 * ((double)(d / 16) + 32.0) * (fabs(l) + 2.0);
    v = (float)(l + allow);
    w = (float)(2.0 * allow);
    if (!isfinite(v)) { v = CUDART_INF_F; w = 0.f; }
  }
  if (lane == 0) {
    hi[row] = v;
    width[row] = w;
  }
}

cudaError_t launch_claimed_logits(const uint16_t* h, const uint16_t* W, const int32_t* tokens, int T, int d, int V,
                                  float* hi, float* width, cudaStream_t stream) {
  const int blocks = (T + kK2Warps - 1) / kK2Warps;
  claimed_logits<<<blocks, kK2Warps * 32, 0, stream>>>(h, W, tokens, T, d, V, hi, width);
  return cudaGetLastError();
}

// ------------------------------------------------------- admissible sets
// Id i != argmax is admissible at threshold j iff y_i >= y_max + A(tau_j).  The counting pass sees fp32 values
// y' = y + y_shift whose noise term comes from lg2.approx: it counts the ids whose y' is above the bound by more
// than that error (bound + allow) and lists the ids inside the band of width 2 * allow below; unused thresholds
// get +inf (nothing counts, nothing is listed).
__global__ void count_bounds(const CountParams p) {
  const int row = blockIdx.x * blockDim.x + threadIdx.x;
  if (row >= p.T) return;
  const float ymax = p.y_max[row];
  float top = 0.f;  // the largest finite |bound| of the row
  float b[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    b[j] = CUDART_INF_F;
    if (j < p.n_tau) {
      // -inf (everything admissible) must stay above the value that masks padded vocabulary columns
      b[j] = fmaxf(ymax + p.a_tau[j] + p.y_shift, -1.0e38f);
      if (isnan(b[j])) b[j] = CUDART_INF_F;
      if (b[j] > -1.0e38f && b[j] < CUDART_INF_F) top = fmaxf(top, fabsf(b[j]));
    }
  }
  const float allow = 3e-4f * p.temperature + 1e-4f + 3.9e-6f * top;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const bool open = !(b[j] > -1.0e38f) || !(b[j] < CUDART_INF_F);  // everything or nothing: no band to decide
    p.bounds[(size_t)j * (size_t)p.T_pad + row] = open ? b[j] : b[j] + allow;
  }
  p.bounds[(size_t)kBandPlane * (size_t)p.T_pad + row] = 2.f * allow;
}

// The Token-DiFR score of a claim with margin A (one competitor, Gaussian noise): ln(Phi(A / (sigma sqrt 2)) + eps).
__device__ __forceinline__ double gm_score_of_margin(double A, double sigma, double eps) {
  return log(0.5 * erfc(-A / (2.0 * sigma)) + eps);
}

// One warp per row: sums the strips' counts, decides the listed ids exactly (fp64 logit and noise, the score of
// the id as the claim against tau itself), and adds the verifier's own sample, which the counting pass leaves
// out and which is admissible iff the score of its margin over the runner-up reaches tau.
__global__ void __launch_bounds__(kK2Warps * 32) count_finalize(const CountParams p) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row = blockIdx.x * kK2Warps + warp;
  if (row >= p.T) return;
  int c[4] = {0, 0, 0, 0};
  for (int slot = lane; slot < p.n_slots; slot += 32) {
    const int4 a = *reinterpret_cast<const int4*>(p.partials + (size_t)row * (size_t)p.n_slots + slot);
    c[0] += a.x; c[1] += a.y; c[2] += a.z; c[3] += a.w;
  }
#pragma unroll
  for (int m = 16; m >= 1; m >>= 1) {
#pragma unroll
    for (int j = 0; j < 4; ++j) c[j] += __shfl_xor_sync(0xffffffffu, c[j], m);
  }
  const uint64_t seed = p.seeds[row];
  const uint32_t pos = p.positions[row];
  const uint16_t* hrow = p.h + (size_t)row * (size_t)p.d;
  const double temp = (double)p.temperature, sigma = (double)p.sigma, eps = (double)p.eps;
  const int best = p.argmax[row];
  const bool best_ok = best >= 0 && best < p.V;
  // exact y of the verifier's own sample (and of the runner-up when its id is known)
  double y_best = (double)p.y_max[row], y_second = (double)p.y_second[row];
  if (best_ok) y_best = warp_dot(hrow, p.W + (size_t)best * (size_t)p.d, p.d, lane) + temp * gumbel_exact(seed, pos, (uint32_t)best);
  if (p.runner_up != nullptr) {
    const int second = p.runner_up[row];
    if (second >= 0 && second < p.V)
      y_second = warp_dot(hrow, p.W + (size_t)second * (size_t)p.d, p.d, lane) + temp * gumbel_exact(seed, pos, (uint32_t)second);
  }
  uint32_t status = 0;
  if (p.band_count != nullptr) {
    const int n_found = p.band_count[row];
    const int n_band = n_found < p.band_cap ? n_found : p.band_cap;
    if (n_found > p.band_cap) status |= 32u;
    const BandEntry* list = p.band_list + (size_t)row * (size_t)p.band_cap;
    for (int e = 0; e < n_band; ++e) {
      const int id = list[e].id;
      const float yf = list[e].v;  // the fp32 y' the counting pass saw
      const double y = warp_dot(hrow, p.W + (size_t)id * (size_t)p.d, p.d, lane) + temp * gumbel_exact(seed, pos, (uint32_t)id);
      const double score = gm_score_of_margin(y - y_best, sigma, eps);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        if (j < p.n_tau) {
          const float hi = p.bounds[(size_t)j * (size_t)p.T_pad + row];
          const float w = p.bounds[(size_t)kBandPlane * (size_t)p.T_pad + row];
          // (ids at or above hi were counted by the pass, ids below the band are surely inadmissible)
          if (!(yf >= hi) && (yf + w >= hi) && score >= (double)p.taus[j]) ++c[j];
        }
      }
    }
  }
  if (lane == 0) {
    const double top_score = gm_score_of_margin(y_best - y_second, sigma, eps);
    for (int j = 0; j < p.n_tau; ++j)
      p.counts[(size_t)j * (size_t)p.T + row] = c[j] + ((top_score >= (double)p.taus[j]) ? 1 : 0);
    if (p.row_status != nullptr) p.row_status[row] = status;
  }
}

cudaError_t launch_count_bounds(const CountParams& p, cudaStream_t stream) {
  count_bounds<<<(p.T + 255) / 256, 256, 0, stream>>>(p);
  return cudaGetLastError();
}
cudaError_t launch_count_finalize(const CountParams& p, cudaStream_t stream) {
  count_finalize<<<(p.T + kK2Warps - 1) / kK2Warps, kK2Warps * 32, 0, stream>>>(p);
  return cudaGetLastError();
}

// --------------------------------------------------- bounded-wait self-test
// One warp waits on a barrier that nothing ever arrives at, with a short limit: the wait must give up, raise the
// abort flag and let the kernel end normally.  status[0] = kStatusTimeout if it did, status[1] = the abort flag.
__global__ void wait_selftest(int32_t* status, long long limit_cycles) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_flag = 0;
    mbar_fence_init();
  }
  __syncthreads();
  const bool completed = mbar_wait(smem_u32(&bar), 0u, &abort_flag, limit_cycles);
  __syncthreads();
  if (threadIdx.x == 0) {
    status[0] = completed ? 0 : kStatusTimeout;
    status[1] = abort_flag;
  }
}

cudaError_t launch_wait_selftest(int32_t* status, long long limit_cycles, cudaStream_t stream) {
  wait_selftest<<<1, 32, 0, stream>>>(status, limit_cycles);
  return cudaGetLastError();
}

// --------------------------------------------------------- Philox validation
__global__ void philox_blocks(const uint32_t* ctr, const uint32_t* key, int64_t n, uint32_t* out) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const uint32_t c0 = ctr[4 * i], c1 = ctr[4 * i + 1], c2 = ctr[4 * i + 2], c3 = ctr[4 * i + 3];
  const uint32_t k0 = key[2 * i], k1 = key[2 * i + 1];
  uint32_t x[4];
  if (c2 == 0u && c3 == 0u) {
    // the per-row form the scoring epilogue uses
    RowNoise rn;
    row_noise_init(rn, ((uint64_t)k1 << 32) | k0, c1);
    row_noise_block(rn, c0, x);
  } else {
    philox4x32_10(c0, c1, c2, c3, k0, k1, x);
  }
  out[4 * i] = x[0]; out[4 * i + 1] = x[1]; out[4 * i + 2] = x[2]; out[4 * i + 3] = x[3];
}

cudaError_t launch_philox(const uint32_t* ctr, const uint32_t* key, int64_t n, uint32_t* out, cudaStream_t stream) {
  if (n <= 0) return cudaSuccess;
  const int threads = 128;
  philox_blocks<<<(unsigned)((n + threads - 1) / threads), threads, 0, stream>>>(ctr, key, n, out);
  return cudaGetLastError();
}

}  // namespace difr
