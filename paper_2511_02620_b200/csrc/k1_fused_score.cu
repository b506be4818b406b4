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
// the tile's 256 rows of W, and one elected lane of the pair's first CTA issues
// tcgen05.mma.cta_group::2, which reads both CTAs' shared memory and writes rows
// 0..127 of the accumulator to the first CTA's TMEM and rows 128..255 to the
// second's.  Per 256 x 256 x 64 step each SM therefore fills 32 KB of shared
// memory instead of the 48 KB a lone 128 x 256 tile needs.
//
// Warp roles in each CTA: warp 0 issues the TMA loads, warp 1 (first CTA only)
// issues the MMAs, warp 2 owns the TMEM allocation, warp 3 (first CTA only)
// hands out work units, warps 4..19 are the epilogue: warp 4 + 4 g + q reads TMEM
// lanes 32 q .. 32 q + 31 (rows) and columns 64 g .. 64 g + 63 of the CTA's
// 128 x 256 accumulator.  Two accumulator stages (all 512 TMEM columns) let the
// epilogue of tile n overlap the MMAs of tile n + 1.  A work unit is (256-row
// tile, vocabulary strip); its running statistics stay in registers across the
// strip, the four column groups of a row are merged through shared memory at
// the end of the unit and leave as one 32-byte partial record per (row, strip).
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
constexpr int kEpiWarp0 = 4;
constexpr int kColGroups = 4;                  // 64-column groups of the CTA's accumulator tile
constexpr int kEpiWarps = 4 * kColGroups;
constexpr int kThreads = 32 * (kEpiWarp0 + kEpiWarps);
constexpr int kSub = 16;                       // vocabulary ids per TMEM load
constexpr int kSubsPerTile = (kBN / kColGroups) / kSub;
constexpr int kRoleRegs = 32, kEpiRegs = 112;  // 32 * 128 + 112 * 512 = 96 * 640 registers
constexpr int kTmemCols = 512;
constexpr int kSchedSlots = 2;                 // unit ids handed out ahead of their use
constexpr int kSchedReaders = 2 + 1 + 2 * kEpiWarps;  // per pair, one arrival each: two TMA warps, the MMA warp, the epilogue warps
constexpr int kBarBytes = 512;
constexpr int kXchBytes = (kColGroups - 1) * kBM * 32;  // statistics of column groups 1..3 on their way to group 0
constexpr int kSmemBytes = kStages * kStageBytes + kBarBytes + kXchBytes + 1024;  // + slack for 1024-byte alignment
constexpr float kMasked = -3.0e38f;  // stands in for -inf on padded vocabulary columns (keeps keys finite)
static_assert(kSmemBytes <= 227 * 1024, "shared memory budget of one CTA");
static_assert(kPlanBandCap == kBandCap && kPlanBoundPlanes == kBandPlane + 2, "workspace layout");

// Epilogue variants.  GmRank adds the raw-logit rank of the claimed token; Count1 / Count4 regenerate the
// noise only to count the ids whose y reaches one / four per-row bounds (admissible-set sizes).
// GmFilter is Gm that also keeps each strip's two largest 16-id group maxima of the raw logits (the bound of
// the filter's cutoff comes from them); Collect appends every id whose y' or raw logit reaches the row's
// bounds to the row's candidate list.
// IptFilter / CollectLogit are their counterparts without noise, for the IPT estimator under a filter.
enum : int { kModeGm = 0, kModeIpt = 1, kModeDump = 2, kModeGmRank = 3, kModeCount1 = 4, kModeCount4 = 5,
             kModeGmFilter = 6, kModeCollect = 7, kModeIptFilter = 8, kModeCollectLogit = 9 };

template <int MODE>
struct Mode {
  static constexpr bool gm = MODE == kModeGm || MODE == kModeGmRank || MODE == kModeGmFilter;
  static constexpr bool softmax = gm || MODE == kModeIpt || MODE == kModeIptFilter;
  static constexpr bool rank = MODE == kModeGmRank || MODE == kModeCollect;  // Collect: only when asked for
  static constexpr int rank_slot = MODE == kModeGmRank ? 0 : 2;  // which bound holds the claimed logit
  static constexpr bool groupmax = MODE == kModeGmFilter || MODE == kModeIptFilter;
  static constexpr bool collect = MODE == kModeCollect || MODE == kModeCollectLogit;
  static constexpr int ng = MODE == kModeCount1 ? 1 : (MODE == kModeCount4 ? 4 : 0);  // bounds per row
  static constexpr bool noise = gm || ng > 0 || MODE == kModeCollect;
  static constexpr int ncnt = collect ? 3 : (rank ? 1 : (ng > 0 ? ng : 1));  // bounds loaded per row
  static constexpr bool bounds = rank || collect || ng > 0;
  static constexpr bool band = rank || ng > 0;  // ids within rounding of a bound are listed for an exact decision
  // Gumbel-max modes whose records feed the finalize kernel only: an id whose noise word cannot lift it to the
  // row's second best so far skips the Gumbel transform and the top-2 network
  static constexpr bool skip = MODE == kModeGm || MODE == kModeGmRank;
  static constexpr bool record = !collect && MODE != kModeDump;
};

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
  float m1, m2;  // top-2 keys of y' (low 4 mantissa bits cleared)
  int i1, i2;    // their vocabulary ids
  float lmax;    // running max of z = l * c1
  float lsum;    // sum of 2^(z - lmax)
  float lpre;    // the same restricted to ids below the claimed one
  int cnt[4];    // GmRank: cnt[0] (Collect: cnt[2]) = ids whose logit surely exceeds the claimed one; Count: ids
                 // surely at or above bound g
  float bound[4];  // GmRank: bound[0] = claimed logit + its rounding allowance; Count: the row's bounds on y' plus
                   // theirs; Collect: bounds on y', on l, and the claimed logit as in GmRank (+inf: no rank wanted)
  float bw;      // width of the band below such a bound inside which fp32 cannot decide: those ids are listed
  float gm2;     // GmFilter: the second largest 16-id group maximum of z (lmax is the largest)
  uint32_t tie;  // Gumbel-max modes: nonzero once the two best keys of some 16-id group were equal
  float floor;   // skip modes: a lower bound of the row's second largest key (from other strips' records)
  float thrz;    // skip modes: (max(floor, m2) - allowance) * c1, the key an id must be able to reach; -inf: none
};

__device__ __forceinline__ void stats_init(RowStats& s) {
  s.m1 = s.m2 = -CUDART_INF_F;
  s.i1 = s.i2 = -1;
  s.lmax = -CUDART_INF_F;
  s.lsum = s.lpre = 0.f;
  s.cnt[0] = s.cnt[1] = s.cnt[2] = s.cnt[3] = 0;
  s.bw = 0.f;
  s.gm2 = -CUDART_INF_F;
  s.tie = 0u;
  s.floor = s.thrz = -CUDART_INF_F;
}

// Keys are y' with the low four mantissa bits cleared, so values that differ by less than 2^-19 relative count
// as equal, and equal keys rank by vocabulary id (lowest first): of any number of exactly tied ids the two lowest
// survive to the finalize kernel, which orders them exactly.  (Inside one 16-id group the min/max network ranks
// tied keys by their column bits instead; a record whose strip saw such a tie is marked, and the finalize kernel
// then re-evaluates every id of its candidates' groups.)
//
// (k1, j1), (k2, j2): the best two of the next 16 ids of the same thread, k1 >= k2, all ids above those seen.
__device__ __forceinline__ void top2_merge(RowStats& s, float k1, int j1, float k2, int j2) {
  if (k1 > s.m1) {
    const bool q = k2 > s.m1;
    s.m2 = q ? k2 : s.m1;
    s.i2 = q ? j2 : s.i1;
    s.m1 = k1;
    s.i1 = j1;
  } else if (k1 > s.m2) {
    s.m2 = k1;
    s.i2 = j1;
  }
}

// One candidate of another column group (its ids may lie on either side of this group's): ties by id.
__device__ __forceinline__ void top2_insert_any(RowStats& s, float k, int j) {
  if (k > s.m1 || (k == s.m1 && (unsigned)j < (unsigned)s.i1)) {
    s.m2 = s.m1;
    s.i2 = s.i1;
    s.m1 = k;
    s.i1 = j;
  } else if (k > s.m2 || (k == s.m2 && (unsigned)j < (unsigned)s.i2)) {
    s.m2 = k;
    s.i2 = j;
  }
}

// y' = l - Temp ln2 log2(-log2 u) = l + Temp G + Temp ln(ln 2) from the four noise words x of ids [id0, id0 + 4).
__device__ __forceinline__ void noisy4_from_words(const uint32_t (&x)[4], const float (&l)[4], float neg_tl2,
                                                  float (&y)[4]) {
  const float2 minus1 = make_float2(-0.99999994f, -0.99999994f), ntl2 = make_float2(neg_tl2, neg_tl2);
#pragma unroll
  for (int q = 0; q < 4; q += 2) {
    // u = ((x >> 9) + 1/2) 2^-23, exact;  -log2 u = E / ln 2
    const float2 u = fadd2(make_float2(__uint_as_float(0x3F800000u | (x[q] >> 9)),
                                       __uint_as_float(0x3F800000u | (x[q + 1] >> 9))), minus1);
    const float2 g = make_float2(lg2_approx(-lg2_approx(u.x)), lg2_approx(-lg2_approx(u.y)));
    const float2 yy = ffma2(g, ntl2, make_float2(l[q], l[q + 1]));
    y[q] = yy.x;
    y[q + 1] = yy.y;
  }
  // u within 2^-11 of one: -log2 u loses relative accuracy, redo those with a series for -ln(1 - w)
  const uint32_t xm = max(max(x[0], x[1]), max(x[2], x[3]));
  if (xm >= 0xFFE00000u) {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      if (x[q] >= 0xFFE00000u) {
        const float w = __uint_as_float(0x3F800000u | ((~x[q]) >> 9)) - 0.99999994f;  // 1 - u, exact
        const float E = w * fmaf(w, fmaf(w, 0.33333334f, 0.5f), 1.0f);
        y[q] = fmaf(lg2_approx(E * 1.4426950408889634f), neg_tl2, l[q]);
      }
    }
  }
}

__device__ __forceinline__ void noisy4(const RowNoise& rn, int id0, const float (&l)[4], float neg_tl2,
                                       float (&y)[4]) {
  uint32_t x[4];
  row_noise_block(rn, (uint32_t)id0 >> 2, x);
  noisy4_from_words(x, l, neg_tl2, y);
}

// The key an id must be able to reach to matter to the finalize kernel, times c1: the larger of the row's floor
// and this thread's own second best, less the allowance by which the finalize kernel looks below the second
// best key (twice the keys' error) and a little more.
__device__ __forceinline__ float skip_threshold_z(float floor, float m2, float c1, float neg_tl2) {
  const float m = fmaxf(floor, m2);
  const float temp = neg_tl2 * -1.4426950408889634f;
  const float thr = m - (1e-3f * temp + 4e-4f + 1.6e-5f * fabsf(m));
  return (c1 > 0.f && m > -CUDART_INF_F) ? thr * c1 : -CUDART_INF_F;  // greedy replay (c1 = 0): no noise to skip
}

// One more id of a row whose fp32 value cannot decide an integer: (id, the fp32 value) goes to the row's list.
__device__ __forceinline__ void band_append(BandEntry* list, int* count, int cap, int id, float v) {
  if (count == nullptr) return;
  const int pos = atomicAdd(count, 1);
  if (pos < cap) {
    BandEntry e;
    e.id = id; e.v = v;
    list[pos] = e;
  }
}

// 16 consecutive vocabulary ids [base, base + 16) of one row.  `tok` is the id the row singles out: the
// claimed token (scoring modes) or the id left out of the count (counting modes).
template <int MODE>
__device__ __forceinline__ void process16(const uint32_t (&raw)[kSub], int base, int V, int tok, float c1,
                                          float neg_tl2, const RowNoise& rn, RowStats& s, Candidate* cand_list,
                                          int* cand_count, int cand_cap, BandEntry* band_list, int* band_count,
                                          int band_cap) {
  using M = Mode<MODE>;
  float l[kSub];
#pragma unroll
  for (int j = 0; j < kSub; ++j) l[j] = __uint_as_float(raw[j]);
  if (base + kSub > V) {  // padded columns of the last tile (uniform over the warp)
#pragma unroll
    for (int j = 0; j < kSub; ++j)
      if (base + j >= V) l[j] = kMasked;
  }
  const int tl = tok - base;  // position of the singled-out id relative to this group

  float zmax_group = 0.f;  // largest z = l * c1 of these 16 ids
  // ---- softmax statistics (online log-sum-exp in base 2)
  if (M::softmax) {
    float cm = fmax3(l[0], l[1], l[2]);
#pragma unroll
    for (int j = 3; j + 1 < kSub; j += 2) cm = fmax3(cm, l[j], l[j + 1]);
    cm = fmaxf(cm, l[kSub - 1]);
    const float zmax = cm * c1;
    zmax_group = zmax;
    if (M::groupmax) s.gm2 = fmaxf(s.gm2, fminf(s.lmax, zmax));
    if (zmax > s.lmax) {  // rare after the first few groups of a strip
      const float scale = ex2_approx(s.lmax - zmax);  // 0 on the first group
      s.lsum *= scale;
      s.lpre *= scale;
      s.lmax = zmax;
    }
    const float shift = -s.lmax;
    const float2 c1_2 = make_float2(c1, c1), shift2 = make_float2(shift, shift);
    float2 a01 = make_float2(0.f, 0.f), a23 = make_float2(0.f, 0.f);
#pragma unroll
    for (int j = 0; j < kSub; j += 4) {
      const float2 z01 = ffma2(make_float2(l[j + 0], l[j + 1]), c1_2, shift2);
      const float2 z23 = ffma2(make_float2(l[j + 2], l[j + 3]), c1_2, shift2);
      a01 = fadd2(a01, make_float2(ex2_approx(z01.x), ex2_approx(z01.y)));
      a23 = fadd2(a23, make_float2(ex2_approx(z23.x), ex2_approx(z23.y)));
    }
    const float2 a = fadd2(a01, a23);
    const float cs = a.x + a.y;
    s.lsum += cs;
    // ids below the claimed one: all, none, or the first tl of this group
    if (tl >= kSub) {
      s.lpre += cs;
    } else if (tl >= 0) {  // this group holds the claimed id
      float ps = 0.f, lt = 0.f;
#pragma unroll
      for (int j = 0; j < kSub; ++j) {
        if (j < tl) ps += ex2_approx(fmaf(l[j], c1, shift));
        if (j == tl) lt = l[j];
      }
      s.lpre += ps;
      // the claimed token's own fp32 logit travels in the record's last word (modes that do not count there):
      // the finalize kernel swaps its term of the sum for the fp64 one, so that p[t*] is not off by the tensor
      // cores' rounding of the largest logit
      if (!M::rank && !M::groupmax) s.cnt[0] = __float_as_int(lt);
    }
  }

  // ---- raw-logit rank of the claimed token: ids whose logit is larger (the claimed id itself left out).
  // Counted here: logits above the claimed one by more than the tensor cores' rounding.  Ids inside the band
  // [hi - bw, hi] are listed; the finalize kernel compares their fp64 logits with the claimed token's.
  if (M::rank) {
    const float hi = s.bound[M::rank_slot], w = s.bw;
    int c_hi = 0, c_lo = 0;
#pragma unroll
    for (int j = 0; j < kSub; ++j) {
      c_hi += (l[j] > hi) ? 1 : 0;
      c_lo += (l[j] + w >= hi) ? 1 : 0;
    }
    if (c_lo != c_hi) {  // rare: some id of this group lies in the band (the claimed id itself always does)
#pragma unroll
      for (int j = 0; j < kSub; ++j) {
        if ((l[j] + w >= hi) && !(l[j] > hi) && j != tl && base + j < V) {
          if (MODE == kModeCollect) {
            if (cand_count == nullptr) continue;
            const int pos = atomicAdd(cand_count, 1);
            if (pos < cand_cap) {
              Candidate c;
              c.id = (base + j) | kBandOnly; c.l = l[j]; c.y = 0.f;
              cand_list[pos] = c;
            }
          } else {
            band_append(band_list, band_count, band_cap, base + j, l[j]);
          }
        }
      }
    }
    if (tl >= 0 && tl < kSub) {  // the claimed id never counts, whatever its own rounding
#pragma unroll
      for (int j = 0; j < kSub; ++j)
        if (j == tl && l[j] > hi) --c_hi;
    }
    s.cnt[M::rank_slot] += c_hi;
  }

  // ---- candidates by raw logit only (the IPT estimator under a filter needs no noise)
  if (MODE == kModeCollectLogit) {
#pragma unroll
    for (int j = 0; j < kSub; j += 4) {
      const float lm = fmaxf(fmaxf(l[j], l[j + 1]), fmaxf(l[j + 2], l[j + 3]));
      if (lm >= s.bound[1]) {  // rare
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          if (l[j + q] >= s.bound[1] && base + j + q < V) {
            const int pos = atomicAdd(cand_count, 1);
            if (pos < cand_cap) {
              Candidate c;
              c.id = base + j + q; c.l = l[j + q]; c.y = 0.f;
              cand_list[pos] = c;
            }
          }
        }
      }
    }
  }

  // ---- Gumbel-max replay: top-2 of y' = l - Temp*ln2 * log2(-log2 u), or counts of y' against the row's bounds
  if (M::noise) {
    float c1k = -CUDART_INF_F, c2k = -CUDART_INF_F;
    // Skip modes: y' >= thr needs -ln u <= ln2 2^((l - thr) c1), and 1 - u <= -ln u, so a noise word below
    // x_need (taken with the group's largest logit, rounded to the safe side) cannot lift its id to thr.
    uint32_t x_need = 0u;
    if (M::skip) x_need = ~__float2uint_rz(fmaf(ex2_approx(zmax_group - s.thrz), 2.9799e9f, 1024.f));
#pragma unroll
    for (int j = 0; j < kSub; j += 4) {
      const float l4[4] = {l[j], l[j + 1], l[j + 2], l[j + 3]};
      float y[4];
      bool live = true;
      if (M::skip) {
        uint32_t x[4];
        row_noise_block(rn, (uint32_t)(base + j) >> 2, x);
        live = max(max(x[0], x[1]), max(x[2], x[3])) >= x_need;
        if (live) noisy4_from_words(x, l4, neg_tl2, y);  // rare once the row's second best is known
      } else {
        noisy4(rn, base + j, l4, neg_tl2, y);
      }
      if (M::gm && live) {
        float key[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) key[q] = __uint_as_float((__float_as_uint(y[q]) & ~15u) | (uint32_t)(j + q));
        const float h1 = fmaxf(key[0], key[1]), l1 = fminf(key[0], key[1]);
        const float h2 = fmaxf(key[2], key[3]), l2 = fminf(key[2], key[3]);
        const float t1 = fmaxf(h1, h2);
        const float t2 = fmax3(fminf(h1, h2), l1, l2);
        const float n2 = fmax3(fminf(c1k, t1), c2k, t2);
        c1k = fmaxf(c1k, t1);
        c2k = n2;
      }
      if (MODE == kModeCollect) {
        const float ym = fmaxf(fmaxf(y[0], y[1]), fmaxf(y[2], y[3]));
        const float lm = fmaxf(fmaxf(l4[0], l4[1]), fmaxf(l4[2], l4[3]));
        if (ym >= s.bound[0] || lm >= s.bound[1]) {  // rare
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            if ((y[q] >= s.bound[0] || l4[q] >= s.bound[1]) && base + j + q < V) {
              const int pos = atomicAdd(cand_count, 1);
              if (pos < cand_cap) {
                Candidate c;
                c.id = base + j + q; c.l = l4[q]; c.y = y[q];
                cand_list[pos] = c;
              }
            }
          }
        }
      }
      if (M::ng > 0) {
        if (tl >= j && tl < j + 4) {  // the id left out never counts
#pragma unroll
          for (int q = 0; q < 4; ++q)
            if (j + q == tl) y[q] = kMasked;
        }
        // counted here: y' surely at or above bound g (the bounds carry the fp32 noise allowance); an id whose
        // y' lies in the band below some bound is listed with its y', and the finalize kernel decides it exactly
        int n_hi = 0, n_lo = 0;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const float yw = y[q] + s.bw;
#pragma unroll
          for (int g = 0; g < M::ng; ++g) {
            const int a = (y[q] >= s.bound[g]) ? 1 : 0;
            s.cnt[g] += a;
            n_hi += a;
            n_lo += (yw >= s.bound[g]) ? 1 : 0;
          }
        }
        if (n_lo != n_hi) {  // rare
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            bool in_band = false;
#pragma unroll
            for (int g = 0; g < M::ng; ++g) in_band |= (y[q] + s.bw >= s.bound[g]) && !(y[q] >= s.bound[g]);
            if (in_band && base + j + q < V) band_append(band_list, band_count, band_cap, base + j + q, y[q]);
          }
        }
      }
    }
    // merge the group's top-2 into the running top-2 (column bits cleared: earlier ids win ties)
    if (M::gm) {
      const uint32_t b1 = __float_as_uint(c1k), b2 = __float_as_uint(c2k);
      // Equal keys inside one group were ranked by their column bits (the highest column first), not by id: the
      // record says so, and the finalize kernel then looks at every id of its candidates' groups.
      s.tie |= ((b1 ^ b2) < 16u && c1k > -CUDART_INF_F) ? 1u : 0u;
      const float m2_before = s.m2;
      top2_merge(s, __uint_as_float(b1 & ~15u), base + (int)(b1 & 15u), __uint_as_float(b2 & ~15u),
                 base + (int)(b2 & 15u));
      if (M::skip && s.m2 != m2_before) s.thrz = skip_threshold_z(s.floor, s.m2, c1, neg_tl2);  // rare
    }
  }
}

// Floats as integers that order the same way (for atomicMax on a float kept in global memory).
__device__ __forceinline__ int float_to_ordered(float f) {
  const int b = __float_as_int(f);
  return b >= 0 ? b : b ^ 0x7fffffff;
}
__device__ __forceinline__ float ordered_to_float(int o) { return __int_as_float(o >= 0 ? o : o ^ 0x7fffffff); }

// The 32-byte record of a row: what leaves a column group for shared memory and a unit for the workspace.
//   scoring modes:  {m1, i1, m2, i2, lse2_max, lse2_sum, prefix2, count of larger logits}
//   counting modes: {count at bound 0..3, -, -, -, -}
template <int MODE>
__device__ __forceinline__ void record_pack(const RowStats& st, float4& a, float4& b) {
  if (Mode<MODE>::ng > 0) {
    a = make_float4(__int_as_float(st.cnt[0]), __int_as_float(st.cnt[1]), __int_as_float(st.cnt[2]),
                    __int_as_float(st.cnt[3]));
    b = make_float4(0.f, 0.f, 0.f, 0.f);
  } else {
    a = make_float4(st.m1, __int_as_float(st.i1), st.m2, __int_as_float(st.i2));
    // (the sum is never negative: its sign bit carries the tie mark)
    b = make_float4(st.lmax, (Mode<MODE>::gm && st.tie) ? -st.lsum : st.lsum, st.lpre,
                    Mode<MODE>::groupmax ? st.gm2 : __int_as_float(st.cnt[0]));
  }
}
template <int MODE>
__device__ __forceinline__ void record_merge(RowStats& st, const float4& a, const float4& b) {
  if (Mode<MODE>::ng > 0) {
    st.cnt[0] += __float_as_int(a.x);
    st.cnt[1] += __float_as_int(a.y);
    st.cnt[2] += __float_as_int(a.z);
    st.cnt[3] += __float_as_int(a.w);
  } else {
    top2_insert_any(st, a.x, __float_as_int(a.y));
    top2_insert_any(st, a.z, __float_as_int(a.w));
    if (Mode<MODE>::gm) st.tie |= __float_as_uint(b.y) >> 31;
    if (Mode<MODE>::groupmax) st.gm2 = fmax3(st.gm2, b.w, fminf(st.lmax, b.x));  // (b.x, b.w): its two largest
    if (b.x > -CUDART_INF_F) {  // that group saw columns
      const float m = fmaxf(st.lmax, b.x);
      const float fa = ex2_approx(st.lmax - m), fb = ex2_approx(b.x - m);
      st.lsum = st.lsum * fa + fabsf(b.y) * fb;
      st.lpre = st.lpre * fa + b.z * fb;
      st.lmax = m;
    }
    if (!Mode<MODE>::groupmax) st.cnt[0] += __float_as_int(b.w);
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
  //   full[s]        first CTA's copy is used: 1 arrival (its producer) + the bytes of both CTAs' loads
  //   empty[s]       each CTA's own copy: 1 arrival, the MMA thread's commit delivered to both CTAs
  //   acc_full[a]    each CTA's own copy: 1 arrival, the commit after a tile's last MMA, delivered to both
  //   acc_empty[a]   first CTA's copy is used: one arrival per epilogue warp of both CTAs
  //   sched_full[q]  each CTA's own copy: 1 arrival, the scheduler thread's, after it wrote unit id q
  //   sched_empty[q] first CTA's copy is used: one arrival per reader of the pair
  //   xch_full[r]    own: column groups 1..3 of lane quarter r have written their statistics (3 arrivals)
  //   xch_empty[r]   own: column group 0 of lane quarter r has read them (1 arrival)
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kStages * kStageBytes);
  const uint32_t bar0 = smem_base + kStages * kStageBytes;
  constexpr int kBarAcc = 2 * kStages, kBarSched = kBarAcc + 2 * kAccStages, kBarXch = kBarSched + 2 * kSchedSlots,
                kBarEnd = kBarXch + 8;
  static_assert(kBarEnd * 8 + 16 + 4 * kSchedSlots <= kBarBytes, "barrier block");
  auto full_bar = [&](int s) { return bar0 + 8u * (uint32_t)s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (uint32_t)(kStages + s); };
  auto acc_full_bar = [&](int a) { return bar0 + 8u * (uint32_t)(kBarAcc + a); };
  auto acc_empty_bar = [&](int a) { return bar0 + 8u * (uint32_t)(kBarAcc + kAccStages + a); };
  auto sched_full_bar = [&](int q) { return bar0 + 8u * (uint32_t)(kBarSched + q); };
  auto sched_empty_bar = [&](int q) { return bar0 + 8u * (uint32_t)(kBarSched + kSchedSlots + q); };
  auto xch_full_bar = [&](int r) { return bar0 + 8u * (uint32_t)(kBarXch + r); };
  auto xch_empty_bar = [&](int r) { return bar0 + 8u * (uint32_t)(kBarXch + 4 + r); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + kBarEnd);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  volatile int* sched_unit = reinterpret_cast<volatile int*>(tmem_slot + 2);  // [kSchedSlots]
  float4* xch = reinterpret_cast<float4*>(smem + kStages * kStageBytes + kBarBytes);  // [3][128 rows][2]

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
    for (int q = 0; q < kSchedSlots; ++q) {
      mbar_init(sched_full_bar(q), 1);
      mbar_init(sched_empty_bar(q), kSchedReaders);
    }
    for (int r = 0; r < 4; ++r) {
      mbar_init(xch_full_bar(r), kColGroups - 1);
      mbar_init(xch_empty_bar(r), 1);
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

  // Work units reach every role of the pair through a small ring of unit ids that the
  // scheduler thread (warp 3 of the first CTA) fills in both CTAs.  -1 ends the kernel.
  auto next_unit = [&](int& slot, uint32_t& phase, bool one_lane_arrives) -> int {
    if (!mbar_wait(sched_full_bar(slot), phase, abort_flag)) return -1;
    const int u = sched_unit[slot];
    if (one_lane_arrives) {
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster_nofence(map_to_cta(sched_empty_bar(slot), 0));
    } else {
      mbar_arrive_cluster_nofence(map_to_cta(sched_empty_bar(slot), 0));
    }
    if (++slot == kSchedSlots) { slot = 0; phase ^= 1u; }
    return u;
  };

  // The four role warps need few registers; the rest goes to the epilogue warpgroups.
  if (warp < kEpiWarp0) {
  setmaxnreg_dec<kRoleRegs>();
  if (warp == 3) {
    // --------------------------------------------------------------- scheduler
    // Units are taken from a global counter in raster order, so the pairs that run at
    // the same time work on neighbouring units (the same rows of W at about the same
    // moment) however far their speeds drift apart.  Without a counter: round robin.
    if (cta == 0 && lane == 0) {
      int slot = 0, i = 0;
      uint32_t phase = 0;
      while (true) {
        if (!mbar_wait(sched_empty_bar(slot), phase ^ 1u, abort_flag)) break;
        int u = (p.unit_counter != nullptr) ? atomicAdd(p.unit_counter, 1) : pair + i * n_pairs;
        ++i;
        if (u >= p.n_units) u = -1;
        sched_unit[slot] = u;
        st_shared_cluster_u32(map_to_cta(smem_u32(const_cast<int*>(&sched_unit[slot])), 1), (uint32_t)u);
        mbar_arrive_cluster(map_to_cta(sched_full_bar(slot), 0));
        mbar_arrive_cluster(map_to_cta(sched_full_bar(slot), 1));
        if (u < 0) break;
        if (++slot == kSchedSlots) { slot = 0; phase ^= 1u; }
      }
    }
  } else if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    // (the whole warp walks the loop, one elected lane issues: see the MMA issuer)
    {
      // a CTA re-reads its h tile for every vocabulary tile of the strip, and the other strips of the
      // raster group read it too: ask L2 to keep it.  A W tile is wanted by every pair of its strip within
      // a few tile times and then not for a long while: ordinary priority (marking it evict-first loses it
      // before the last pair of the strip has come by).
      const uint64_t keep = l2_policy_evict_last(), stream = l2_policy_evict_normal();
      const uint32_t full0_base = map_to_cta(full_bar(0), 0);  // the first CTA's full[0] as seen from either CTA
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      int uslot = 0;
      uint32_t uphase = 0;
      while (ok) {
        const int u = next_unit(uslot, uphase, true);
        if (u < 0) break;
        const Unit w = decode_unit(p, u);
        const int row0 = w.m * kPairM + (int)cta * kBM;
        for (int n = w.n0; n < w.n1 && ok; ++n) {
          const int wrow0 = n * kBN + (int)cta * (kBN / 2);
          for (int k = 0; k < p.k_steps; ++k) {
            if (!__all_sync(0xffffffffu, mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag))) { ok = false; break; }
            if (elect_one()) {
              if (cta == 0) mbar_arrive_expect_tx(full_bar(stage), 2u * kStageBytes);
              const uint32_t full0 = full0_base + 8u * (uint32_t)stage;
              const uint32_t a_dst = smem_base + (uint32_t)stage * kStageBytes;
              tma_load_2d_pair(a_dst, &tmap_h, k * kBK, row0, full0, keep);
              tma_load_2d_pair(a_dst + kABytes, &tmap_w, k * kBK, wrow0, full0, stream);
            }
            __syncwarp();
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
          }
        }
      }
    }
  } else if (warp == 1) {
    // -------------------------------------------------------------- MMA issuer
    // The whole warp walks the loop and one elected lane issues: with a warp-uniform loop the descriptors and
    // barrier addresses live in uniform registers, and an MMA costs the issuing warp a fraction of the
    // instructions it costs a lone lane.  (As a single-lane loop this thread was the bottleneck: competing for
    // issue slots with the epilogue warps of its scheduler it needed about 590 clocks per 512-clock step.)
    if (cta == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(kPairM, kBN);
      // The descriptors of a stage differ from those of stage 0 only in the 14-bit address field
      // (units of 16 bytes), which never carries out of the field: shared memory ends below 256 KB.
      const uint64_t desc0 = umma_desc_k_major_sw128(smem_base);
      const uint32_t desc_hi = (uint32_t)(desc0 >> 32), desc_lo0 = (uint32_t)desc0;
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true;
      int uslot = 0;
      uint32_t uphase = 0;
      while (ok) {
        const int u = next_unit(uslot, uphase, true);
        if (u < 0) break;
        const Unit w = decode_unit(p, u);
        for (int n = w.n0; n < w.n1 && ok; ++n) {
          if (!__all_sync(0xffffffffu, mbar_wait(acc_empty_bar(acc), acc_phase ^ 1u, abort_flag))) { ok = false; break; }
          tc_fence_after();
          const uint32_t d_tmem = tmem_base + (uint32_t)(acc * kBN);
          uint32_t accumulate = 0;
          for (int k = 0; k < p.k_steps; ++k) {
            if (!__all_sync(0xffffffffu, mbar_wait(full_bar(stage), phase, abort_flag))) { ok = false; break; }
            tc_fence_after();
            const uint32_t a_lo = desc_lo0 + (uint32_t)stage * (kStageBytes >> 4);
            if (elect_one()) {
#pragma unroll
              for (int kk = 0; kk < kBK / 16; ++kk) {
                const uint64_t a_desc = ((uint64_t)desc_hi << 32) | (a_lo + 2u * kk);
                const uint64_t b_desc = ((uint64_t)desc_hi << 32) | (a_lo + (kABytes >> 4) + 2u * kk);
                umma_bf16_pair(d_tmem, a_desc, b_desc, idesc, (kk == 0) ? accumulate : 1u);
              }
              umma_commit_pair(empty_bar(stage), 3);
            }
            __syncwarp();
            accumulate = 1;
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
          }
          if (ok && elect_one()) umma_commit_pair(acc_full_bar(acc), 3);
          __syncwarp();
          if (++acc == kAccStages) { acc = 0; acc_phase ^= 1u; }
        }
      }
    }
  }
  } else {
    // ---------------------------------------------------------------- epilogue
    setmaxnreg_inc<kEpiRegs>();
    const int ew = warp - kEpiWarp0;
    const int quarter = ew & 3;  // == warp % 4: the TMEM lane quarter this warp may read
    const int colg = ew >> 2;    // which 64 columns of the tile
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    const int row_in_cta = quarter * 32 + lane;
    int acc = 0;
    uint32_t acc_phase = 0, xch_phase = 0;
    bool ok = true;
    int uslot = 0;
    uint32_t uphase = 0;
    while (ok) {
      const int u = next_unit(uslot, uphase, true);
      if (u < 0) break;
      const Unit w = decode_unit(p, u);
      const int row = w.m * kPairM + (int)cta * kBM + row_in_cta;
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
        if (Mode<MODE>::noise) row_noise_init(rn, seed, pos);
        // per-row bounds: the claimed logit (rank) or the bounds on y' (counting); rows beyond T count nothing
        if (Mode<MODE>::bounds) {
#pragma unroll
          for (int g = 0; g < Mode<MODE>::ncnt; ++g)
            st.bound[g] = valid ? p.bounds[(size_t)g * (size_t)p.T_pad + row] : CUDART_INF_F;
          st.bw = valid ? p.bounds[(size_t)kBandPlane * (size_t)p.T_pad + row] : 0.f;
        }
      }
      // the temperature is the call's, or the row's own when the caller passes one per row
      float c1 = p.c1, neg_tl2 = p.neg_tl2;
      if (p.temperatures != nullptr && MODE != kModeDump) {
        const float temp = valid ? p.temperatures[row] : 1.f;
        c1 = temp > 0.f ? 1.4426950408889634f / temp : 0.f;
        neg_tl2 = -temp * 0.6931471805599453f;
      }
      if (Mode<MODE>::skip && valid && p.row_floor != nullptr) {
        // what earlier units of this row (other strips) found as their second best: nothing below it matters
        st.floor = ordered_to_float(__ldcg(p.row_floor + row));
        st.thrz = skip_threshold_z(st.floor, st.m2, c1, neg_tl2);
      }
      Candidate* cand_list = nullptr;
      int* cand_count = nullptr;
      if (Mode<MODE>::collect && valid) {
        cand_list = reinterpret_cast<Candidate*>(p.cand_list) + (size_t)row * (size_t)p.cand_cap;
        cand_count = p.cand_count + row;
      }
      BandEntry* band_list = nullptr;
      int* band_count = nullptr;
      if (Mode<MODE>::band && !Mode<MODE>::collect && valid && p.band_count != nullptr) {
        band_list = p.band_list + (size_t)row * (size_t)p.band_cap;
        band_count = p.band_count + row;
      }
      for (int n = w.n0; n < w.n1; ++n) {
        if (!mbar_wait(acc_full_bar(acc), acc_phase, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const int col0 = n * kBN + colg * (kBN / kColGroups);
        if (col0 < p.V) {  // uniform over the warp
          // two register buffers: the load of the next 16 columns is in flight while these are processed
          const uint32_t t0 = tmem_base + lane_addr + (uint32_t)(acc * kBN + colg * (kBN / kColGroups));
          uint32_t buf0[kSub], buf1[kSub];
          tmem_ld_32x16(t0, buf0);
#pragma unroll
          for (int i = 0; i < kSubsPerTile; ++i) {
            uint32_t (&cur)[kSub] = (i & 1) ? buf1 : buf0;
            uint32_t (&nxt)[kSub] = (i & 1) ? buf0 : buf1;
            tmem_ld_wait(cur);
            const bool more = (i + 1 < kSubsPerTile) && (col0 + (i + 1) * kSub < p.V);
            if (more) tmem_ld_32x16(t0 + (uint32_t)((i + 1) * kSub), nxt);
            const int base = col0 + i * kSub;
            if (MODE == kModeDump || (Mode<MODE>::groupmax && p.logits_out != nullptr)) {
              // (the filters' first pass also writes the logits when a selection over them follows)
              if (valid) {
                float* dst = p.logits_out + (size_t)row * (size_t)p.V + base;
                if ((p.V & 7) == 0 && (reinterpret_cast<unsigned long long>(p.logits_out) & 31ull) == 0ull &&
                    base + kSub <= p.V) {
                  // (rows start on 32-byte boundaries and base is a multiple of 16 ids: two 32-byte stores, whole
                  // sectors, 64 contiguous bytes per thread)
#pragma unroll
                  for (int j = 0; j < kSub; j += 8)
                    st_global_v8(dst + j, cur[j], cur[j + 1], cur[j + 2], cur[j + 3], cur[j + 4], cur[j + 5],
                                 cur[j + 6], cur[j + 7]);
                } else if ((p.V & 3) == 0 && (reinterpret_cast<unsigned long long>(p.logits_out) & 15ull) == 0ull &&
                           base + kSub <= p.V) {
#pragma unroll
                  for (int j = 0; j < kSub; j += 4)
                    *reinterpret_cast<uint4*>(dst + j) = make_uint4(cur[j], cur[j + 1], cur[j + 2], cur[j + 3]);
                } else {
#pragma unroll
                  for (int j = 0; j < kSub; ++j)
                    if (base + j < p.V) dst[j] = __uint_as_float(cur[j]);
                }
              }
            }
            if (MODE != kModeDump) {
              process16<MODE>(cur, base, p.V, tok, c1, neg_tl2, rn, st, cand_list, cand_count, p.cand_cap, band_list,
                              band_count, p.band_cap);
            }
            if (!more) break;
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster_nofence(map_to_cta(acc_empty_bar(acc), 0));
        if (++acc == kAccStages) { acc = 0; acc_phase ^= 1u; }
      }
      if (MODE == kModeCollect && ok && valid && p.rank_out != nullptr && st.cnt[2] != 0)
        atomicAdd(p.rank_out + row, st.cnt[2]);  // this thread's share of the claimed token's raw-logit rank
      if (Mode<MODE>::record && ok) {
        // the four column groups of a row meet in shared memory; group 0 merges and writes the record
        if (colg != 0) {
          if (!mbar_wait(xch_empty_bar(quarter), xch_phase ^ 1u, abort_flag)) { ok = false; break; }
          float4* dst = xch + ((size_t)(colg - 1) * kBM + row_in_cta) * 2;
          record_pack<MODE>(st, dst[0], dst[1]);
          __syncwarp();
          if (lane == 0) mbar_arrive(xch_full_bar(quarter));
        } else {
          if (!mbar_wait(xch_full_bar(quarter), xch_phase, abort_flag)) { ok = false; break; }
#pragma unroll
          for (int g = 0; g < kColGroups - 1; ++g) {
            const float4* src = xch + ((size_t)g * kBM + row_in_cta) * 2;
            record_merge<MODE>(st, src[0], src[1]);
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(xch_empty_bar(quarter));
          if (valid) {
            float4* dst = reinterpret_cast<float4*>(p.partials + (size_t)row * (size_t)p.S + w.strip);
            record_pack<MODE>(st, dst[0], dst[1]);
            // this strip's second best is a lower bound of the row's: later units of the row skip below it
            if (Mode<MODE>::skip && p.row_floor != nullptr && st.m2 > st.floor)
              atomicMax(p.row_floor + row, float_to_ordered(st.m2));
          }
        }
        xch_phase ^= 1u;
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

// ------------------------------------------------- the collecting pass over stored logits
// The filters' second pass without the contraction.  Their first pass left the rows' fp32 logits in memory, bit
// for bit what the tensor cores produce, so the collecting modes' epilogue can run over them directly: one warp
// per row and span of columns, each lane taking 16 consecutive ids at a time (a warp reads 2 KB of the row per
// step), with the same per-row bounds, noise and candidate lists as in the fused kernel.
constexpr int kCflWarps = 8;

template <int MODE>
__global__ void __launch_bounds__(kCflWarps * 32) collect_from_logits(const K1Params p, const float* __restrict__ logits,
                                                                       int span, int spans) {
  static_assert(Mode<MODE>::collect, "collecting modes only");
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long unit = (long long)blockIdx.x * kCflWarps + warp;
  const int row = (int)(unit / spans);
  const int c0 = (int)(unit % spans) * span;
  if (row >= p.T || c0 >= p.V) return;
  const int c_end = min(p.V, c0 + span);
  const int tok = p.tokens[row];
  RowNoise rn;
  RowStats st;
  stats_init(st);
  if (Mode<MODE>::noise) row_noise_init(rn, p.seeds[row], p.positions[row]);
#pragma unroll
  for (int g = 0; g < Mode<MODE>::ncnt; ++g) st.bound[g] = p.bounds[(size_t)g * (size_t)p.T_pad + row];
  st.bw = p.bounds[(size_t)kBandPlane * (size_t)p.T_pad + row];
  float c1 = p.c1, neg_tl2 = p.neg_tl2;
  if (p.temperatures != nullptr) {
    const float temp = p.temperatures[row];
    c1 = temp > 0.f ? 1.4426950408889634f / temp : 0.f;
    neg_tl2 = -temp * 0.6931471805599453f;
  }
  Candidate* cand_list = reinterpret_cast<Candidate*>(p.cand_list) + (size_t)row * (size_t)p.cand_cap;
  int* cand_count = p.cand_count + row;
  const float* lrow = logits + (size_t)row * (size_t)p.V;
  const bool vec = (p.V & 3) == 0 && (reinterpret_cast<unsigned long long>(logits) & 15ull) == 0ull;
  for (int base = c0 + lane * kSub; base < c_end; base += 32 * kSub) {
    uint32_t cur[kSub];
    if (vec && base + kSub <= p.V) {
#pragma unroll
      for (int j = 0; j < kSub; j += 4) {
        const uint4 q = *reinterpret_cast<const uint4*>(lrow + base + j);
        cur[j] = q.x; cur[j + 1] = q.y; cur[j + 2] = q.z; cur[j + 3] = q.w;
      }
    } else {
#pragma unroll
      for (int j = 0; j < kSub; ++j) cur[j] = base + j < p.V ? __float_as_uint(lrow[base + j]) : 0u;
    }
    process16<MODE>(cur, base, p.V, tok, c1, neg_tl2, rn, st, cand_list, cand_count, p.cand_cap, nullptr, nullptr, 0);
  }
  if (MODE == kModeCollect && p.rank_out != nullptr && st.cnt[2] != 0)
    atomicAdd(p.rank_out + row, st.cnt[2]);  // this lane's share of the claimed token's raw-logit rank
}

cudaError_t launch_collect_from_logits(int mode, const K1Params& p, const float* logits, cudaStream_t stream) {
  if (p.T <= 0) return cudaSuccess;
  // spans of a multiple of 512 ids (a warp's step), about eight per row
  int span = ((p.V + 7) / 8 + 511) & ~511;
  if (span < 512) span = 512;
  const int spans = (p.V + span - 1) / span;
  const long long units = (long long)p.T * spans;
  const unsigned grid = (unsigned)((units + kCflWarps - 1) / kCflWarps);
  if (mode == kModeCollect) collect_from_logits<kModeCollect><<<grid, kCflWarps * 32, 0, stream>>>(p, logits, span, spans);
  else if (mode == kModeCollectLogit)
    collect_from_logits<kModeCollectLogit><<<grid, kCflWarps * 32, 0, stream>>>(p, logits, span, spans);
  else return cudaErrorInvalidValue;
  return cudaGetLastError();
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
    case kModeGmRank: return launch_mode<kModeGmRank>(tmap_h, tmap_w, p, grid, stream);
    case kModeCount1: return launch_mode<kModeCount1>(tmap_h, tmap_w, p, grid, stream);
    case kModeCount4: return launch_mode<kModeCount4>(tmap_h, tmap_w, p, grid, stream);
    case kModeGmFilter: return launch_mode<kModeGmFilter>(tmap_h, tmap_w, p, grid, stream);
    case kModeIptFilter: return launch_mode<kModeIptFilter>(tmap_h, tmap_w, p, grid, stream);
  }
  return cudaErrorInvalidValue;
}

}  // namespace difr
