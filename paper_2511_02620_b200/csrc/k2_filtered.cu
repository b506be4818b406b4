// Finalize kernels of the full Token-DiFR estimator (Alg. Token-DiFR with the top-k / top-p cutoff, the B_i
// terms and an active subset of s competitors):
//   filter_bounds      from the first pass's partial records, per row: a lower bound of the (s+3)-th largest
//                      y' and of the top_k-th largest raw logit -- what the collecting pass compares against
//   filtered_finalize  from the row's candidate list: the cutoff (top-k, then the nucleus inside it), the
//                      s + 2 best competitors by y', their exact logits and noise in fp64, and the expectation
//                      E_x[ 1{l_t + x > cutoff} prod_i Phi(max(x + A_i, B_i) / sigma) ] by composite
//                      Gauss-Legendre quadrature (one panel per lane).
#include <cuda_runtime.h>
#include <math_constants.h>

#include "difr_device.cuh"
#include "difr_kernels.h"

namespace difr {

constexpr int kFWarps = 4;
constexpr int kMaxK = 128;       // top_k limit (the nucleus is resolved inside the top k)
constexpr int kChunks = kMaxK / 32;  // sorted ranks held per lane
constexpr int kMaxCand = 10;     // s + 2 with s <= 8
constexpr int kGlOrder = 16;

// Nodes and weights of the 16-point Gauss-Legendre rule on [-1, 1] (roots of the Legendre polynomial P_16,
// weights 2 / ((1 - x^2) P_16'(x)^2)), to double precision.
__constant__ double c_gl_x[kGlOrder] = {
    -0.98940093499164994, -0.9445750230732326,  -0.86563120238783176, -0.755404408355003,
    -0.61787624440264377, -0.45801677765722737, -0.28160355077925892, -0.095012509837637441,
    0.095012509837637441, 0.28160355077925892,  0.45801677765722737,  0.61787624440264377,
    0.755404408355003,    0.86563120238783176,  0.9445750230732326,   0.98940093499164994};
__constant__ double c_gl_w[kGlOrder] = {
    0.027152459411754176, 0.062253523938647456, 0.095158511682492605, 0.12462897125553407,
    0.14959598881657671,  0.16915651939500265,  0.18260341504492364,  0.18945061045506864,
    0.18945061045506864,  0.18260341504492364,  0.16915651939500265,  0.14959598881657671,
    0.12462897125553407,  0.095158511682492605, 0.062253523938647456, 0.027152459411754176};

// n-th largest (n >= 1) of the values the warp holds, eight per lane; -inf when there are fewer than n.
__device__ __forceinline__ float warp_nth_largest(float (&v)[8], int n, int lane) {
  float result = -CUDART_INF_F;
  for (int it = 0; it < n; ++it) {
    float lm = v[0];
#pragma unroll
    for (int e = 1; e < 8; ++e) lm = fmaxf(lm, v[e]);
    float wm = lm;
#pragma unroll
    for (int m = 16; m >= 1; m >>= 1) wm = fmaxf(wm, __shfl_xor_sync(0xffffffffu, wm, m));
    result = wm;
    if (wm == -CUDART_INF_F) break;
    const unsigned holders = __ballot_sync(0xffffffffu, lm == wm);
    if (lane == __ffs(holders) - 1) {  // one instance leaves
      bool gone = false;
#pragma unroll
      for (int e = 0; e < 8; ++e)
        if (!gone && v[e] == wm) { v[e] = -CUDART_INF_F; gone = true; }
    }
  }
  return result;
}

// The sampling policy of one row, normalised: the call's scalars or the row's own values.
struct RowPolicy {
  float temperature, c1, top_p, min_p;
  int top_k;         // ids resolved by logit rank: the top-k, or kMaxK for a nucleus over the whole vocabulary or
                     // a min-p set; 1 when only the largest logit is needed (min-p bound); 0: none
  int nucleus_full;  // the nucleus takes its mass from the whole row (no top-k in front of it)
  bool by_rank;      // a top-k or a nucleus is in effect: the cutoff by rank is one of the resolved logits
  bool none;         // no filter at all
  bool bad;          // unusable values: the row's score is NaN and row_status bit 3 is set
};

__device__ __forceinline__ RowPolicy row_policy(const FilterParams& p, int row) {
  RowPolicy r;
  r.temperature = p.temperatures != nullptr ? p.temperatures[row] : p.temperature;
  r.c1 = p.temperatures != nullptr ? (r.temperature > 0.f ? 1.4426950408889634f / r.temperature : 0.f) : p.c1;
  int k = p.top_k_rows != nullptr ? p.top_k_rows[row] : p.top_k;
  r.top_p = p.top_p_rows != nullptr ? p.top_p_rows[row] : p.top_p;
  r.min_p = p.min_p_rows != nullptr ? p.min_p_rows[row] : p.min_p;
  r.bad = !(r.temperature > 0.f) || isinf(r.temperature) || k < 0 || !(r.top_p > 0.f) || !(r.top_p <= 1.f) ||
          !(r.min_p >= 0.f) || !(r.min_p <= 1.f);
  if (k > p.V) k = p.V;
  const bool selected = p.sel_cut_id != nullptr;  // every row's kept prefix was resolved by the selection kernel
  if (k > kMaxK && k < p.V && !selected) r.bad = true;
  const bool whole = k < 1 || k >= p.V;  // no top-k in effect
  r.nucleus_full = (whole && r.top_p < 1.f) ? 1 : 0;
  r.by_rank = !whole || r.nucleus_full;
  r.none = whole && !(r.top_p < 1.f) && !(r.min_p > 0.f);
  if (r.nucleus_full) k = kMaxK < p.V ? kMaxK : p.V;
  else if (whole) {
    k = (p.ipt && p.V <= kMaxK) ? p.V : 0;
    // min-p alone: the IPT estimator needs the surviving ids (resolved among the largest kMaxK), Token-DiFR
    // only the largest logit
    if (r.min_p > 0.f) k = p.ipt ? (kMaxK < p.V ? kMaxK : p.V) : (k > 1 ? k : 1);
  }
  if (selected && !r.bad) {
    // the cutoff by rank comes from the selection: only the min-p bound still needs the largest logit here
    k = (r.min_p > 0.f && !p.ipt) ? 1 : 0;
    r.nucleus_full = 0;
  }
  if (r.bad) { k = 0; r.nucleus_full = 0; r.by_rank = false; r.none = false; }
  r.top_k = k;
  return r;
}

// The min-p bound l_max + Temp ln(min_p) with l_max in fp64: the sorted list's first ranks whose fp32 logit lies
// within rounding of the largest are all re-evaluated, the largest exact value counts.  Whole warp.
__device__ __forceinline__ double min_p_bound_exact(const FilterParams& p, const RowPolicy& rp, int row, int lane,
                                                    const float* sl, const int* sid, int k_eff) {
  const uint16_t* hrow = p.h + (size_t)row * (size_t)p.d;
  double l_max = -CUDART_INF;
  const float near = sl[0] - 1e-4f * fmaxf(1.f, fabsf(sl[0]));
  for (int r = 0; r < k_eff && r < 8; ++r) {
    if (r > 0 && sl[r] < near) break;
    l_max = fmax(l_max, warp_dot(hrow, p.W + (size_t)sid[r] * (size_t)p.d, p.d, lane));
  }
  return l_max + (double)rp.temperature * log((double)rp.min_p);
}

// Softmax mass of the whole row in units of 2^(c1 * l0), from the first pass's records: sum_v 2^(c1 (l_v - l0)).
// The same value in every lane.
__device__ __forceinline__ double row_mass_relative(const FilterParams& p, int row, int lane, double l0, double c1) {
  double lmax = -CUDART_INF, lsum = 0.0;
  for (int slot = lane; slot < p.n_slots; slot += 32) {
    const float4* src = reinterpret_cast<const float4*>(p.partials + (size_t)row * (size_t)p.n_slots + slot);
    const float4 b = src[1];
    const double bm = (double)b.x, bs = (double)fabsf(b.y);  // (the sign bit is the fused kernel's tie mark)
    if (bm == -CUDART_INF) continue;
    if (bm > lmax) { lsum = lsum * exp2(lmax - bm) + bs; lmax = bm; }
    else lsum += bs * exp2(bm - lmax);
  }
  double wmax = lmax;
#pragma unroll
  for (int m = 16; m >= 1; m >>= 1) wmax = fmax(wmax, shfl_xor_double(wmax, m));
  double part = (lmax == -CUDART_INF) ? 0.0 : lsum * exp2(lmax - wmax);
#pragma unroll
  for (int m = 16; m >= 1; m >>= 1) part += shfl_xor_double(part, m);
  part = __hiloint2double(__shfl_sync(0xffffffffu, __double2hiint(part), 0),
                          __shfl_sync(0xffffffffu, __double2loint(part), 0));
  return part * exp2(wmax - l0 * c1);
}

// The row's k_eff largest logits stand sorted (descending) in sl[].  Returns the rank of the last id the row's
// nucleus keeps (k_eff - 1 when top_p = 1): the shortest prefix whose softmax mass reaches top_p of the top-k's
// renormalised mass, or of the whole row's when no top-k stands in front.  e[c]: unnormalised mass
// 2^(c1 (l - l0)) of rank 32 c + lane.  Whole warp.
__device__ __forceinline__ int nucleus_last_rank(const FilterParams& p, const RowPolicy& rp, int row, int lane,
                                                 const float* sl, int k_eff, double (&e)[kChunks],
                                                 uint32_t& status_bits) {
  const double c1 = (double)rp.c1, l0 = (double)sl[0];
#pragma unroll
  for (int c = 0; c < kChunks; ++c)
    e[c] = (32 * c + lane < k_eff) ? exp2(((double)sl[32 * c + lane] - l0) * c1) : 0.0;
  int last = k_eff - 1;
  if (rp.top_p < 1.f) {
    // inclusive scan over the ranks: inside each chunk of 32 by shuffles, then the chunks' totals carried over
    double cum[kChunks];
    double carry = 0.0;
#pragma unroll
    for (int c = 0; c < kChunks; ++c) {
      double v = e[c];
#pragma unroll
      for (int m = 1; m < 32; m <<= 1) {
        const double up = __hiloint2double(__shfl_up_sync(0xffffffffu, __double2hiint(v), m),
                                           __shfl_up_sync(0xffffffffu, __double2loint(v), m));
        if (lane >= m) v += up;
      }
      cum[c] = v + carry;
      carry = __hiloint2double(__shfl_sync(0xffffffffu, __double2hiint(cum[c]), 31),
                               __shfl_sync(0xffffffffu, __double2loint(cum[c]), 31));
    }
    const double total = carry;
    const double need = (double)rp.top_p * (rp.nucleus_full ? row_mass_relative(p, row, lane, l0, c1) : total);
    bool found = false;
#pragma unroll
    for (int c = 0; c < kChunks; ++c) {
      const unsigned m = __ballot_sync(0xffffffffu, 32 * c + lane < k_eff && cum[c] >= need);
      if (!found && m) {
        last = 32 * c + __ffs(m) - 1;
        found = true;
      }
    }
    if (!found && rp.nucleus_full && k_eff < p.V) status_bits |= 16u;  // the nucleus holds more ids than were resolved
  }
  return last;
}

__global__ void __launch_bounds__(kFWarps * 32) filter_bounds(const FilterParams p) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row = blockIdx.x * kFWarps + warp;
  if (row >= p.T) return;
  const RowPolicy rp = row_policy(p, row);
  // up to 128 strips: four records per lane, two values of each kind per record
  float yk[8], zk[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) yk[e] = zk[e] = -CUDART_INF_F;
#pragma unroll
  for (int t = 0; t < 4; ++t) {
    const int slot = lane + 32 * t;
    if (slot < p.n_slots) {
      const float4* src = reinterpret_cast<const float4*>(p.partials + (size_t)row * (size_t)p.n_slots + slot);
      const float4 a = src[0], b = src[1];
      if (__float_as_int(a.y) >= 0) yk[2 * t] = a.x;
      if (__float_as_int(a.w) >= 0) yk[2 * t + 1] = a.z;
      zk[2 * t] = b.x;
      zk[2 * t + 1] = b.w;
    }
  }
  // Any subset's n-th largest is a lower bound of the whole row's n-th largest.  s competitors are refined out of
  // s + 2, and the claimed token may sit among them: s + 3.  A little is taken off for the index bits stored in
  // the keys and for the rounding of z = l * c1.
  float by = (p.s > 0) ? -CUDART_INF_F : CUDART_INF_F;  // s == 0: no competitors wanted (IPT estimator)
  float bl = CUDART_INF_F;
  if (p.n_slots <= 128) {
    if (p.s > 0) {
      const float ky = warp_nth_largest(yk, p.s + 3, lane);
      if (ky > -CUDART_INF_F) by = ky - 1e-4f * fmaxf(1.f, fabsf(ky));
    }
    if (rp.top_k > 0) {
      const float kz = warp_nth_largest(zk, rp.top_k, lane);
      bl = -CUDART_INF_F;
      if (kz > -CUDART_INF_F) {
        const float l = kz / rp.c1;
        bl = l - 1e-5f * fmaxf(1.f, fabsf(l));
      }
    }
  } else if (rp.top_k > 0) {
    bl = -CUDART_INF_F;
  }
  if (rp.bad) { by = CUDART_INF_F; bl = CUDART_INF_F; }  // nothing is collected for a row that cannot be scored
  if (lane == 0) {
    p.bounds[row] = by;
    p.bounds[(size_t)p.T_pad + row] = bl;
    // no raw-logit rank unless the claimed-logit kernel overwrites these two
    p.bounds[(size_t)2 * (size_t)p.T_pad + row] = CUDART_INF_F;
    p.bounds[(size_t)kBandPlane * (size_t)p.T_pad + row] = 0.f;
  }
}

// The k-th largest (k >= 1) logit, or y' among the entries that are not the claimed token, of a candidate list
// (band-only entries left out); -inf when there are fewer than k.  Bisection on keys that order like the floats:
// the largest key that at least k entries reach.  Whole warp; every lane gets the value.
__device__ __forceinline__ float warp_kth_largest(const Candidate* list, int n, int k, bool by_y, int tok, int lane) {
  auto key_of = [](float f) {
    const uint32_t b = __float_as_uint(f);
    return b ^ ((b >> 31) ? 0xFFFFFFFFu : 0x80000000u);
  };
  uint32_t lo = 0u, hi = 0xFFFFFFFFu;  // invariant: count(key >= lo) >= k (or lo == 0)
  int total = 0;
  for (int i = lane; i < n; i += 32) total += (list[i].id >= 0 && (!by_y || list[i].id != tok)) ? 1 : 0;
#pragma unroll
  for (int m = 16; m >= 1; m >>= 1) total += __shfl_xor_sync(0xffffffffu, total, m);
  if (total < k) return -CUDART_INF_F;
  while (lo < hi) {
    const uint32_t mid = lo + (hi - lo) / 2u + 1u;  // upper middle: the loop ends with lo == hi
    int c = 0;
    for (int i = lane; i < n; i += 32) {
      const Candidate ci = list[i];
      if (ci.id < 0 || (by_y && ci.id == tok)) continue;
      c += key_of(by_y ? ci.y : ci.l) >= mid ? 1 : 0;
    }
#pragma unroll
    for (int m = 16; m >= 1; m >>= 1) c += __shfl_xor_sync(0xffffffffu, c, m);
    if (c >= k) lo = mid; else hi = mid - 1u;
  }
  const uint32_t b = lo ^ ((lo >> 31) ? 0x80000000u : 0xFFFFFFFFu);
  return __uint_as_float(b);
}

__global__ void __launch_bounds__(kFWarps * 32) filtered_finalize(const FilterParams p) {
  __shared__ float sm_l[kFWarps][kMaxK];
  __shared__ int sm_id[kFWarps][kMaxK];
  __shared__ int sm_cand[kFWarps][kMaxCand];
  __shared__ float sm_cand_y[kFWarps][kMaxCand];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row = blockIdx.x * kFWarps + warp;
  if (row >= p.T) return;
  const int tok = p.tokens[row];
  const bool tok_ok = tok >= 0 && tok < p.V;
  const Candidate* list = p.cand_list + (size_t)row * (size_t)p.cand_cap;
  const int n_found = p.cand_count[row];
  const int n = n_found < p.cand_cap ? n_found : p.cand_cap;
  uint32_t status_bits = (n_found > p.cand_cap) ? 4u : 0u;
  if (p.rank != nullptr && !tok_ok && lane == 0) p.rank[row] = p.V;  // as in the plain call
  const RowPolicy rp = row_policy(p, row);
  // (the first pass's finalize leaves NaN for a row with a non-finite logit: such a row stays unscored)
  const bool unscored = isnan(p.score[row]);
  if (rp.bad || unscored) {
    if (lane == 0) {
      p.score[row] = CUDART_NAN_F;
      if (p.cutoff) p.cutoff[row] = CUDART_NAN_F;
      if (p.row_status && rp.bad) p.row_status[row] |= 8u;
    }
    return;
  }

  const int k_eff = (rp.top_k > 0) ? (rp.top_k < n ? rp.top_k : n) : 0;
  // (entries with the sign bit set were kept for the rank's exact decision only: they take no part in the filter
  // or among the competitors, where the same id may stand a second time as an ordinary entry)
  int n_others = 0;  // ordinary entries that are not the claimed token
  for (int i = lane; i < n; i += 32) n_others += (list[i].id >= 0 && list[i].id != tok) ? 1 : 0;
#pragma unroll
  for (int m = 16; m >= 1; m >>= 1) n_others += __shfl_xor_sync(0xffffffffu, n_others, m);
  // The s competitors are the exact best s; the list ranks by the fused kernel's fp32 y'.  Taken for exact
  // re-evaluation: the first s + 2 by that ranking, and beyond them every entry within the keys' error of the
  // s-th (up to kMaxCand in all), so that near-ties at the edge of the active subset are decided in fp64.
  const int want = p.s + 2;
  const int n_top = n_others < kMaxCand ? n_others : kMaxCand;  // entries whose rank by y' is kept
  int n_cand = n_others < want ? n_others : want;

  // ---- order statistics of the list: rank by raw logit (the filter) and by y' (the competitors).
  // A long list (vocabularies below 64 tiles list every id) is first cut down: the k_eff-th largest logit and the
  // n_top-th largest y' are found by bisection on order-preserving keys (32 counting sweeps), and only entries
  // that reach one of them are ranked against the list.
  float need_l = -CUDART_INF_F, need_y = -CUDART_INF_F;
  if (n > 256) {
    need_l = k_eff > 0 ? warp_kth_largest(list, n, k_eff, false, tok, lane) : CUDART_INF_F;
    need_y = n_top > 0 ? warp_kth_largest(list, n, n_top, true, tok, lane) : CUDART_INF_F;
  }
  double cutoff = -CUDART_INF;
  int cut_rank = -1;
  for (int j = 0; j < n; ++j) {
    const Candidate cj = list[j];
    if (cj.id < 0) continue;  // (uniform over the warp)
    if (n > 256 && !(cj.l >= need_l) && !(cj.y >= need_y)) continue;
    int rl = 0, ry = 0;
    for (int i = lane; i < n; i += 32) {
      const Candidate ci = list[i];
      if (ci.id < 0) continue;
      rl += (ci.l > cj.l || (ci.l == cj.l && ci.id < cj.id)) ? 1 : 0;
      ry += (ci.id != tok && (ci.y > cj.y || (ci.y == cj.y && ci.id < cj.id))) ? 1 : 0;
    }
#pragma unroll
    for (int m = 16; m >= 1; m >>= 1) {
      rl += __shfl_xor_sync(0xffffffffu, rl, m);
      ry += __shfl_xor_sync(0xffffffffu, ry, m);
    }
    if (lane == 0) {
      if (rl < k_eff) { sm_l[warp][rl] = cj.l; sm_id[warp][rl] = cj.id; }
      if (cj.id != tok && ry < n_top) { sm_cand[warp][ry] = cj.id; sm_cand_y[warp][ry] = cj.y; }
    }
  }
  __syncwarp();
  if (n_top > n_cand && p.s <= n_top) {
    const float ys = sm_cand_y[warp][p.s - 1];
    const float edge = ys - 2.f * (3e-4f * rp.temperature + 1e-4f + 3.9e-6f * fabsf(ys));
    while (n_cand < n_top && sm_cand_y[warp][n_cand] >= edge) ++n_cand;
  }
  if (p.sel_cut_id != nullptr && rp.by_rank) {
    // a filter of any size: the last kept id was found by the selection over the row's logits
    const int cid = p.sel_cut_id[row];
    if (cid >= 0 && cid < p.V)
      cutoff = warp_dot(p.h + (size_t)row * (size_t)p.d, p.W + (size_t)cid * (size_t)p.d, p.d, lane);
  } else if (k_eff > 0 && rp.by_rank) {
    double e[kChunks];
    cut_rank = nucleus_last_rank(p, rp, row, lane, sm_l[warp], k_eff, e, status_bits);
    // the cutoff is that id's logit: re-evaluated in fp64 like every other logit the score depends on
    cutoff = warp_dot(p.h + (size_t)row * (size_t)p.d, p.W + (size_t)sm_id[warp][cut_rank] * (size_t)p.d, p.d, lane);
  }
  // min-p: a logit survives iff it reaches l_max + Temp ln(min_p); the stricter of the two bounds is the cutoff
  if (k_eff > 0 && rp.min_p > 0.f)
    cutoff = fmax(cutoff, min_p_bound_exact(p, rp, row, lane, sm_l[warp], sm_id[warp], k_eff));

  double score = log((double)p.eps);
  if (tok_ok) {
    const uint64_t seed = p.seeds[row];
    const uint32_t pos = p.positions[row];
    const uint16_t* hrow = p.h + (size_t)row * (size_t)p.d;
    const double temp = (double)rp.temperature, sigma = (double)p.sigma;
    const double l_t = warp_dot(hrow, p.W + (size_t)tok * (size_t)p.d, p.d, lane);
    const double y_t = l_t + temp * gumbel_exact(seed, pos, (uint32_t)tok);
    if (p.rank != nullptr) {
      // the collecting pass counted the logits surely above the claimed one; the ids it could not decide in
      // fp32 stand in the list with the sign bit set and are decided here in fp64
      int extra = 0;
      for (int i = 0; i < n; ++i) {
        const int id = list[i].id;
        if (id >= 0) continue;
        const double l = warp_dot(hrow, p.W + (size_t)(id & 0x7fffffff) * (size_t)p.d, p.d, lane);
        extra += (l > l_t) ? 1 : 0;
      }
      if (lane == 0 && extra != 0) atomicAdd(p.rank + row, extra);
    }
    // exact logits and noisy logits of the s + 2 candidates; then the s best of them
    double cl[kMaxCand], cy[kMaxCand];
    int cid[kMaxCand];
#pragma unroll
    for (int c = 0; c < kMaxCand; ++c) {
      cl[c] = 0.0; cy[c] = -CUDART_INF; cid[c] = 0x7fffffff;
      if (c < n_cand) {
        const int id = sm_cand[warp][c];
        cid[c] = id;
        cl[c] = warp_dot(hrow, p.W + (size_t)id * (size_t)p.d, p.d, lane);
        cy[c] = cl[c] + temp * gumbel_exact(seed, pos, (uint32_t)id);
      }
    }
    // selection sort, descending y, ties to the lower id (kMaxCand is tiny; every lane does the same)
#pragma unroll
    for (int a = 0; a < kMaxCand - 1; ++a) {
#pragma unroll
      for (int b = a + 1; b < kMaxCand; ++b) {
        const bool swap = cy[b] > cy[a] || (cy[b] == cy[a] && cid[b] < cid[a]);
        if (swap) {
          const double ty = cy[a]; cy[a] = cy[b]; cy[b] = ty;
          const double tl = cl[a]; cl[a] = cl[b]; cl[b] = tl;
          const int ti = cid[a]; cid[a] = cid[b]; cid[b] = ti;
        }
      }
    }
    const int s_eff = p.s < n_cand ? p.s : n_cand;
    double A[kMaxCand], B[kMaxCand];
    double max_neg_a = 0.0;
#pragma unroll
    for (int c = 0; c < kMaxCand; ++c) {
      A[c] = y_t - cy[c];
      B[c] = cutoff - cl[c];
      if (c < s_eff && -A[c] > max_neg_a) max_neg_a = -A[c];
    }
    // ---- the expectation over x ~ N(0, sigma^2), x > cutoff - l_t
    const double x0 = cutoff - l_t;
    const double lo = fmax(x0, -14.0 * sigma);
    const double hi = 14.0 * sigma + fmin(max_neg_a, 60.0 * sigma);
    double pi_hat = 0.0;
    if (lo < hi) {
      const double w = (hi - lo) / 32.0, mid = lo + ((double)lane + 0.5) * w;
      const double inv_sigma = 1.0 / sigma, r2 = 0.70710678118654752440;
      double acc = 0.0;
#pragma unroll 1
      for (int q = 0; q < kGlOrder; ++q) {
        const double x = mid + 0.5 * w * c_gl_x[q];
        const double xs = x * inv_sigma;
        double f = exp(-0.5 * xs * xs);
#pragma unroll
        for (int c = 0; c < kMaxCand; ++c) {
          if (c < s_eff) {
            const double t = fmax(x + A[c], B[c]) * inv_sigma;
            f *= 0.5 * erfc(-t * r2);
          }
        }
        acc += c_gl_w[q] * f;
      }
      acc *= 0.5 * w * inv_sigma * 0.39894228040143267794;  // 1 / (sigma sqrt(2 pi))
#pragma unroll
      for (int m = 16; m >= 1; m >>= 1) acc += shfl_xor_double(acc, m);
      pi_hat = fmin(fmax(acc, 0.0), 1.0);
    }
    score = log(pi_hat + (double)p.eps);
  }
  if (lane == 0) {
    p.score[row] = (float)score;
    if (p.cutoff) p.cutoff[row] = (float)cutoff;
    if (p.row_status && status_bits) p.row_status[row] |= status_bits;
  }
}


// Token-IPT-DiFR on the filtered distribution (Alg. Token-IPT-DiFR with the generation's top-k / nucleus policy):
// the kept ids are the first ranks of the row's candidate list by logit; the claimed token's CDF interval is
// taken over the kept ids in vocabulary-id order.  One warp per row.
__global__ void __launch_bounds__(kFWarps * 32) ipt_filtered_finalize(const FilterParams p) {
  __shared__ float sm_l[kFWarps][kMaxK];
  __shared__ int sm_id[kFWarps][kMaxK];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row = blockIdx.x * kFWarps + warp;
  if (row >= p.T) return;
  const int tok = p.tokens[row];
  const bool tok_ok = tok >= 0 && tok < p.V;
  const Candidate* list = p.cand_list + (size_t)row * (size_t)p.cand_cap;
  const int n_found = p.cand_count[row];
  const int n = n_found < p.cand_cap ? n_found : p.cand_cap;
  uint32_t status_bits = (n_found > p.cand_cap) ? 4u : 0u;
  const RowPolicy rp = row_policy(p, row);
  if (rp.bad || isnan(p.score[row]) || (rp.none && rp.top_k == 0)) {
    // unusable values: NaN; no filter at all (and a vocabulary too large to resolve here): the first pass's
    // finalize has already written the unfiltered score
    if (lane == 0) {
      if (rp.bad) {
        p.score[row] = CUDART_NAN_F;
        if (p.row_status) p.row_status[row] |= 8u;
      }
      if (p.cutoff) p.cutoff[row] = (rp.bad || !rp.none) ? CUDART_NAN_F : -CUDART_INF_F;
    }
    return;
  }
  const int k_eff = rp.top_k < n ? rp.top_k : n;

  // (a long list is cut down to the entries that reach its k_eff-th largest logit before they are ranked)
  const float need_l = (n > 256 && k_eff > 0) ? warp_kth_largest(list, n, k_eff, false, -1, lane) : -CUDART_INF_F;
  for (int j = 0; j < n; ++j) {
    const Candidate cj = list[j];
    if (n > 256 && !(cj.l >= need_l)) continue;
    int rl = 0;
    for (int i = lane; i < n; i += 32) {
      const Candidate ci = list[i];
      rl += (ci.l > cj.l || (ci.l == cj.l && ci.id < cj.id)) ? 1 : 0;
    }
#pragma unroll
    for (int m = 16; m >= 1; m >>= 1) rl += __shfl_xor_sync(0xffffffffu, rl, m);
    if (lane == 0 && rl < k_eff) { sm_l[warp][rl] = cj.l; sm_id[warp][rl] = cj.id; }
  }
  __syncwarp();

  const uint64_t seed = p.seeds[row];
  const uint32_t pos = p.positions[row];
  uint32_t x[4];
  philox4x32_10(0u, pos, 1u, 0u, (uint32_t)seed, (uint32_t)(seed >> 32), x);
  const double mu = ((double)x[0] + 0.5) * (1.0 / 4294967296.0);
  double score = log((double)p.eps), pt = CUDART_NAN, a = CUDART_NAN, cutoff = -CUDART_INF;
  if (k_eff > 0) {
    double e[kChunks];  // unnormalised masses of ranks 32 c + lane
    RowPolicy rank_policy = rp;
    if (!rp.by_rank) rank_policy.top_p = 1.f;  // no filter by rank: every resolved id stays
    int last = nucleus_last_rank(p, rank_policy, row, lane, sm_l[warp], k_eff, e, status_bits);
    if (rp.by_rank)
      cutoff = warp_dot(p.h + (size_t)row * (size_t)p.d, p.W + (size_t)sm_id[warp][last] * (size_t)p.d, p.d, lane);
    if (rp.min_p > 0.f) {
      // min-p: of the ids kept so far, those that reach the bound; logits within fp32 rounding of the bound
      // are compared in fp64
      const double bound = min_p_bound_exact(p, rp, row, lane, sm_l[warp], sm_id[warp], k_eff);
      const uint16_t* hrow = p.h + (size_t)row * (size_t)p.d;
      int keep = -1;
      for (int r = 0; r <= last; ++r) {  // descending logits: stop at the first id below the bound
        const double lf = (double)sm_l[warp][r];
        const double slack = 1e-4 * fmax(1.0, fabs(bound));
        bool in = lf >= bound + slack;
        if (!in && lf > bound - slack)
          in = warp_dot(hrow, p.W + (size_t)sm_id[warp][r] * (size_t)p.d, p.d, lane) >= bound;
        else if (!in)
          break;
        if (in) keep = r;
      }
      if (keep < 0) keep = 0;  // the largest logit always survives
      if (!rp.by_rank && keep == k_eff - 1 && k_eff < p.V) status_bits |= 16u;  // more survivors than resolved
      last = keep;
      cutoff = fmax(cutoff, bound);
    }
    if (tok_ok) {
      // mass of the kept ids, of those below the claimed id, and whether the claimed id is kept
      double z = 0.0, below = 0.0, mine = 0.0;
#pragma unroll
      for (int c = 0; c < kChunks; ++c) {
        const int rank = 32 * c + lane;
        if (rank <= last) {
          const int id = sm_id[warp][rank];
          z += e[c];
          if (id < tok) below += e[c];
          if (id == tok) mine += e[c];
        }
      }
#pragma unroll
      for (int m = 16; m >= 1; m >>= 1) {
        z += shfl_xor_double(z, m);
        below += shfl_xor_double(below, m);
        mine += shfl_xor_double(mine, m);
      }
      a = below / z;
      pt = mine / z;  // zero when the filter removed the claimed id
      const double sigma = (double)p.sigma;
      const double za = (a - mu) / sigma, zb = (a + pt - mu) / sigma, r2 = 0.70710678118654752440;
      double mass;
      if (za >= 0.0) mass = 0.5 * (erfc(za * r2) - erfc(zb * r2));
      else if (zb <= 0.0) mass = 0.5 * (erfc(-zb * r2) - erfc(-za * r2));
      else mass = 1.0 - 0.5 * erfc(zb * r2) - 0.5 * erfc(-za * r2);
      score = log(mass + (double)p.eps);
    }
  }
  if (lane == 0) {
    p.score[row] = (float)score;
    if (p.p_claimed) p.p_claimed[row] = (float)pt;
    if (p.cdf_lo) p.cdf_lo[row] = (float)a;
    if (p.u) p.u[row] = (float)mu;
    if (p.cutoff) p.cutoff[row] = (float)cutoff;
    if (p.row_status && status_bits) p.row_status[row] |= status_bits;
  }
}

// Token-IPT-DiFR on a filtered distribution of any size: the selection kernel has summed the kept ids' masses
// (all of them, those below the claimed id, the claimed id's own); what is left is the uniform, the interval
// and the score, and the cutoff in fp64.  One warp per row.
__global__ void __launch_bounds__(kFWarps * 32) ipt_select_finalize(const FilterParams p) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row = blockIdx.x * kFWarps + warp;
  if (row >= p.T) return;
  const int tok = p.tokens[row];
  const bool tok_ok = tok >= 0 && tok < p.V;
  const RowPolicy rp = row_policy(p, row);
  if (rp.bad || isnan(p.score[row])) {
    if (lane == 0) {
      if (rp.bad) {
        p.score[row] = CUDART_NAN_F;
        if (p.row_status) p.row_status[row] |= 8u;
      }
      if (p.cutoff) p.cutoff[row] = CUDART_NAN_F;
    }
    return;
  }
  const uint16_t* hrow = p.h + (size_t)row * (size_t)p.d;
  const int cid = p.sel_cut_id[row], top = p.sel_top_id[row];
  const bool by_min_p = p.sel_kept_n[row] < 0;  // the min-p bound, not the rank filter, ended the kept prefix
  double cutoff = -CUDART_INF;
  if (rp.none) {
    // (a row of a per-row call that filters nothing: the selection kept every id)
  } else if (by_min_p && top >= 0 && top < p.V)
    cutoff = warp_dot(hrow, p.W + (size_t)top * (size_t)p.d, p.d, lane) + (double)rp.temperature * log((double)rp.min_p);
  else if (cid >= 0 && cid < p.V)
    cutoff = warp_dot(hrow, p.W + (size_t)cid * (size_t)p.d, p.d, lane);
  if (lane == 0) {
    const uint64_t seed = p.seeds[row];
    uint32_t x[4];
    philox4x32_10(0u, p.positions[row], 1u, 0u, (uint32_t)seed, (uint32_t)(seed >> 32), x);
    const double mu = ((double)x[0] + 0.5) * (1.0 / 4294967296.0);
    double score = log((double)p.eps), pt = CUDART_NAN, a = CUDART_NAN;
    if (tok_ok) {
      const double z = p.sel_z[row];
      a = p.sel_below[row] / z;
      pt = p.sel_mine[row] / z;  // zero when the filter removed the claimed id
      const double sigma = (double)p.sigma;
      const double za = (a - mu) / sigma, zb = (a + pt - mu) / sigma, r2 = 0.70710678118654752440;
      double mass;
      if (za >= 0.0) mass = 0.5 * (erfc(za * r2) - erfc(zb * r2));
      else if (zb <= 0.0) mass = 0.5 * (erfc(-zb * r2) - erfc(-za * r2));
      else mass = 1.0 - 0.5 * erfc(zb * r2) - 0.5 * erfc(-za * r2);
      score = log(mass + (double)p.eps);
    }
    p.score[row] = (float)score;
    if (p.p_claimed) p.p_claimed[row] = (float)pt;
    if (p.cdf_lo) p.cdf_lo[row] = (float)a;
    if (p.u) p.u[row] = (float)mu;
    if (p.cutoff) p.cutoff[row] = (float)cutoff;
  }
}

cudaError_t launch_ipt_select_finalize(const FilterParams& p, cudaStream_t stream) {
  ipt_select_finalize<<<(p.T + kFWarps - 1) / kFWarps, kFWarps * 32, 0, stream>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_ipt_filtered_finalize(const FilterParams& p, cudaStream_t stream) {
  ipt_filtered_finalize<<<(p.T + kFWarps - 1) / kFWarps, kFWarps * 32, 0, stream>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_filter_bounds(const FilterParams& p, cudaStream_t stream) {
  filter_bounds<<<(p.T + kFWarps - 1) / kFWarps, kFWarps * 32, 0, stream>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_filtered_finalize(const FilterParams& p, cudaStream_t stream) {
  filtered_finalize<<<(p.T + kFWarps - 1) / kFWarps, kFWarps * 32, 0, stream>>>(p);
  return cudaGetLastError();
}

}  // namespace difr
