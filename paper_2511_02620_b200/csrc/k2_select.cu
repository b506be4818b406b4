// Sampling filters of any size (a top-k above 128 ids, a nucleus over the whole vocabulary, a min-p set): the
// filter keeps a prefix of the row's ids in the order (logit descending, id ascending), and this kernel finds the
// length N of that prefix and its last id exactly, by radix selection over a block of rows whose fp32 logits the
// fused kernel's main loop has written to memory (difr_logits' mode), one CTA per row:
//
//   top-k   keeps positions [0, K)
//   top-p   keeps the shortest prefix whose softmax(l / Temp) mass reaches top_p of the mass of [0, K)
//   min-p   keeps the ids whose logit reaches l_max + Temp ln(min_p), a prefix as well
//
// N is the smallest of the three.  Masses are summed as 64-bit fixed-point integers (2^-40 of the largest
// term), so sums do not depend on the order of the additions and the result is the same on every run.  One
// walk over the row builds a histogram in bins of 1/64 of (l_max - l); each selection then scans it, gathers
// the ids of one bin and pins the exact value by radix rounds over their key bits.  The row (V floats) is
// walked three times (maximum, histogram, one gather per selection) with 16-byte loads, and once more for the
// sums over the kept ids when the IPT estimator asks for them.
#include <cuda_runtime.h>
#include <math_constants.h>

#include "difr_kernels.h"

namespace difr {

constexpr int kSelThreads = 512;
constexpr int kSelBins = 2048;
constexpr int kSelTieCap = 256;

// keys that ascend as the logit descends
__device__ __forceinline__ uint32_t desc_key(float l) {
  const uint32_t b = __float_as_uint(l);
  return ~(b ^ ((b >> 31) ? 0xFFFFFFFFu : 0x80000000u));
}

constexpr int kSelListCap = 2048;

// f(v, row[v]) for every id of the row, the CTA's threads taking turns; 16-byte loads where the row allows.
template <class F>
__device__ __forceinline__ void walk_row(const float* row, int V, F f) {
  if ((reinterpret_cast<unsigned long long>(row) & 15ull) == 0ull) {
    const int n4 = V >> 2;
    const float4* r4 = reinterpret_cast<const float4*>(row);
    // four loads in flight per thread: the walks wait on memory, not on arithmetic
    for (int i0 = threadIdx.x; i0 < n4; i0 += 4 * kSelThreads) {
      float4 q[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int i = i0 + u * kSelThreads;
        if (i < n4) q[u] = r4[i];
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int i = i0 + u * kSelThreads;
        if (i < n4) { f(4 * i, q[u].x); f(4 * i + 1, q[u].y); f(4 * i + 2, q[u].z); f(4 * i + 3, q[u].w); }
      }
    }
    for (int v = (n4 << 2) + threadIdx.x; v < V; v += kSelThreads) f(v, row[v]);
  } else {
    for (int v = threadIdx.x; v < V; v += kSelThreads) f(v, row[v]);
  }
}

__device__ __forceinline__ float key_to_logit(uint32_t key) {
  const uint32_t o = ~key;
  return __uint_as_float(o ^ ((o >> 31) ? 0x80000000u : 0xFFFFFFFFu));
}

struct SelShared {
  unsigned int cnt0[kSelBins];         // level 0: bins of 1/64 in (l_max - l), all ids of the row
  unsigned long long mass0[kSelBins];
  unsigned int cnt[kSelBins];          // inner rounds: key bits of the ids of one level-0 bin
  unsigned long long mass[kSelBins];
  int list[kSelListCap];               // the ids of that level-0 bin (when they fit)
  unsigned int list_n;
  unsigned int list_bin;               // the level-0 bin whose ids the list holds (0xFFFFFFFF: none / overflowed)
  unsigned int warp_cnt[kSelThreads / 32];
  unsigned long long warp_mass[kSelThreads / 32];
  unsigned int found_bin;
  unsigned int c_before;
  unsigned long long m_before;
  unsigned int bin_cnt;
  unsigned long long bin_mass;
  float red_f[kSelThreads / 32];
  unsigned long long red_u[kSelThreads / 32];
  int tie_ids[kSelTieCap];
  unsigned int tie_n;
};

struct Selected {
  uint32_t key;            // key of the element found
  unsigned int c_gt;       // elements with a larger logit
  unsigned long long m_gt; // their mass
  unsigned int ties;       // elements with exactly this logit
  unsigned long long m_tie;  // mass of all of them
};

__device__ __forceinline__ unsigned long long fixed_mass(float l, float lmax, float c1) {
  // 2^(c1 (l - lmax)) in units of 2^-40; terms below 2^-41 of the largest count as zero.  fp32 arithmetic (a
  // relative error of 1e-7 per term, against the 1e-5 the fp32 logits themselves carry): a pure function of
  // its arguments, so the integer sums stay independent of the order of the additions.
  const float e = exp2f(c1 * (l - lmax));  // in [0, 1]
  return (unsigned long long)__float2ull_rn(e * 1099511627776.0f);
}

// slot += q on a 64-bit shared-memory sum, as two 32-bit atomic adds: the low words wrap, and whoever sees the wrap
// carries one into the high word (integer sums: the result does not depend on the order).  Most terms fit the low
// word and wrap nothing, so this is one atomic where a 64-bit add would be a compare-and-swap loop.
__device__ __forceinline__ void add_mass(unsigned long long* slot, unsigned long long q) {
  unsigned int* w = reinterpret_cast<unsigned int*>(slot);  // (little endian: w[0] low, w[1] high)
  const unsigned int lo = (unsigned int)q;
  unsigned int hi = (unsigned int)(q >> 32);
  if (lo != 0u) {
    const unsigned int old = atomicAdd(w, lo);
    hi += (old + lo < old) ? 1u : 0u;
  }
  if (hi != 0u) atomicAdd(w + 1, hi);
}

// Level-0 bin of a logit: monotone in l (larger logits in lower bins, equal logits in one bin), 1/64 wide, the
// last bin open-ended.
__device__ __forceinline__ unsigned int level0_bin(float l, float lmax) {
  const unsigned int b = __float2uint_rz((lmax - l) * 64.f);
  return b < (unsigned int)(kSelBins - 1) ? b : (unsigned int)(kSelBins - 1);
}

// Scan of a histogram (bins in descending order of the logit) from the carried sums (c_acc, m_acc): the first
// bin in which the position `pos` lies (by_mass == false) or the cumulative mass reaches `target`
// (by_mass == true); a target beyond the total gives the last non-empty bin.  Leaves the bin, the sums before
// it and the bin's own count and mass in shared memory.  Whole CTA.
__device__ void locate(const unsigned int* cnt, const unsigned long long* mass, bool by_mass, unsigned int pos,
                       unsigned long long target, unsigned int c_acc, unsigned long long m_acc, SelShared& sh) {
  if (threadIdx.x == 0) sh.found_bin = 0xFFFFFFFFu;
  const int per = kSelBins / kSelThreads;
  unsigned int tc = 0;
  unsigned long long tm = 0;
  for (int i = 0; i < per; ++i) { tc += cnt[threadIdx.x * per + i]; tm += mass[threadIdx.x * per + i]; }
  unsigned int sc = tc;
  unsigned long long sm = tm;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int m = 1; m < 32; m <<= 1) {
    const unsigned int oc = __shfl_up_sync(0xffffffffu, sc, m);
    const unsigned long long om = __shfl_up_sync(0xffffffffu, sm, m);
    if (lane >= m) { sc += oc; sm += om; }
  }
  if (lane == 31) { sh.warp_cnt[warp] = sc; sh.warp_mass[warp] = sm; }
  __syncthreads();
  unsigned int base_c = c_acc;
  unsigned long long base_m = m_acc;
  for (int w = 0; w < warp; ++w) { base_c += sh.warp_cnt[w]; base_m += sh.warp_mass[w]; }
  base_c += sc - tc;
  base_m += sm - tm;  // sums of everything before this thread's first bin
  const unsigned int start_c = base_c;
  const unsigned long long start_m = base_m;
  for (int i = 0; i < per; ++i) {
    const int b = threadIdx.x * per + i;
    const unsigned int bc = cnt[b];
    const unsigned long long bm = mass[b];
    if (bc != 0 && (by_mass ? (base_m + bm >= target) : (base_c + bc > pos))) atomicMin(&sh.found_bin, (unsigned int)b);
    base_c += bc;
    base_m += bm;
  }
  __syncthreads();
  unsigned int fb = sh.found_bin;
  if (fb == 0xFFFFFFFFu) {
    if (threadIdx.x == 0) {
      unsigned int last = 0;
      for (int b = 0; b < kSelBins; ++b) if (cnt[b] != 0) last = (unsigned int)b;
      sh.found_bin = last;
    }
    __syncthreads();
    fb = sh.found_bin;
  }
  if (threadIdx.x == fb / per) {  // the bin's owner knows what lies before it
    unsigned int c = start_c;
    unsigned long long m = start_m;
    for (unsigned int b = (unsigned int)(threadIdx.x * per); b < fb; ++b) { c += cnt[b]; m += mass[b]; }
    sh.c_before = c; sh.m_before = m; sh.bin_cnt = cnt[fb]; sh.bin_mass = mass[fb];
  }
  __syncthreads();
}

// One selection over the row, from its level-0 histogram (built by the caller).  by_mass == false: the element at
// position `pos` (0-based) of the descending order.  by_mass == true: the first element at which the cumulative
// mass reaches `target`.  The level-0 bin that holds the answer is found by a scan; its ids are gathered into a
// list (one walk over the row) and three radix rounds over their key bits (11 + 11 + 10) pin the exact value.
// Whole CTA.
__device__ Selected radix_select(const float* row, int V, float lmax, float c1, bool by_mass, unsigned int pos,
                                 unsigned long long target, bool need_mass, SelShared& sh) {
  locate(sh.cnt0, sh.mass0, by_mass, pos, target, 0u, 0ull, sh);
  const unsigned int bin0 = sh.found_bin;
  unsigned int c_acc = sh.c_before;
  unsigned long long m_acc = sh.m_before;
  if (threadIdx.x == 0) sh.list_n = 0u;
  __syncthreads();
  walk_row(row, V, [&](int v, float l) {
    if (level0_bin(l, lmax) == bin0) {
      const unsigned int at = atomicAdd(&sh.list_n, 1u);
      if (at < (unsigned int)kSelListCap) sh.list[at] = v;
    }
  });
  __syncthreads();
  const unsigned int n_sub = sh.list_n;
  const bool listed = n_sub <= (unsigned int)kSelListCap;  // else: walk the whole row in every round
  if (threadIdx.x == 0) sh.list_bin = listed ? bin0 : 0xFFFFFFFFu;
  uint32_t prefix = 0;  // the key bits decided so far (high bits)
  int decided = 0;      // how many
  const int shifts[3] = {21, 10, 0};
  const int widths[3] = {11, 11, 10};
  Selected out;
  for (int round = 0; round < 3; ++round) {
    const int shift = shifts[round], width = widths[round];
    for (int b = threadIdx.x; b < kSelBins; b += kSelThreads) { sh.cnt[b] = 0; sh.mass[b] = 0; }
    __syncthreads();
    const int n_walk = listed ? (int)n_sub : V;
    for (int i = threadIdx.x; i < n_walk; i += kSelThreads) {
      const int v = listed ? sh.list[i] : i;
      const float l = row[v];
      if (!listed && level0_bin(l, lmax) != bin0) continue;
      const uint32_t k = desc_key(l);
      if (decided == 0 || (k >> (32 - decided)) == prefix) {
        const uint32_t bin = (k >> shift) & ((1u << width) - 1u);
        atomicAdd(&sh.cnt[bin], 1u);
        if (need_mass) add_mass(&sh.mass[bin], fixed_mass(l, lmax, c1));
      }
    }
    __syncthreads();
    locate(sh.cnt, sh.mass, by_mass, pos, target, c_acc, m_acc, sh);
    c_acc = sh.c_before;
    m_acc = sh.m_before;
    prefix = (prefix << width) | sh.found_bin;
    decided += width;
    out.ties = sh.bin_cnt;
    out.m_tie = sh.bin_mass;
    __syncthreads();
  }
  out.key = prefix;
  out.c_gt = c_acc;
  out.m_gt = m_acc;
  return out;
}

__device__ __forceinline__ float block_max(float v, SelShared& sh) {
  for (int m = 16; m >= 1; m >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, m));
  if ((threadIdx.x & 31) == 0) sh.red_f[threadIdx.x >> 5] = v;
  __syncthreads();
  float r = sh.red_f[0];
  for (int w = 1; w < kSelThreads / 32; ++w) r = fmaxf(r, sh.red_f[w]);
  __syncthreads();
  return r;
}

__device__ __forceinline__ unsigned long long block_sum(unsigned long long v, SelShared& sh) {
  for (int m = 16; m >= 1; m >>= 1) v += __shfl_xor_sync(0xffffffffu, v, m);
  if ((threadIdx.x & 31) == 0) sh.red_u[threadIdx.x >> 5] = v;
  __syncthreads();
  unsigned long long r = 0;
  for (int w = 0; w < kSelThreads / 32; ++w) r += sh.red_u[w];
  __syncthreads();
  return r;
}

__global__ void __launch_bounds__(kSelThreads, 3) select_cutoff(const SelectParams p) {
  extern __shared__ __align__(16) unsigned char sel_smem[];
  SelShared& sh = *reinterpret_cast<SelShared*>(sel_smem);
  const int r_local = blockIdx.x;
  const int row = p.row0 + r_local;
  const float* lrow = p.logits + (size_t)r_local * (size_t)p.V;
  const int V = p.V;
  float temp = p.temperatures != nullptr ? p.temperatures[row] : p.temperature;
  const bool usable = temp > 0.f && !isinf(temp);
  if (!usable) temp = 1.f;  // (the finalize kernels mark such a row; keep the arithmetic finite here)
  const float c1 = 1.4426950408889634f / temp;
  int top_k = p.top_k_rows != nullptr ? p.top_k_rows[row] : p.top_k;
  float top_p = p.top_p_rows != nullptr ? p.top_p_rows[row] : p.top_p;
  float min_p = p.min_p_rows != nullptr ? p.min_p_rows[row] : p.min_p;
  if (top_k < 0) top_k = 0;
  if (!(top_p > 0.f) || !(top_p <= 1.f)) top_p = 1.f;
  if (!(min_p >= 0.f) || !(min_p <= 1.f)) min_p = 0.f;

  // the largest logit and its id (the lowest such id)
  float lm = -CUDART_INF_F;
  int lm_id = 0x7fffffff;
  walk_row(lrow, V, [&](int v, float l) {
    if (l > lm || (l == lm && v < lm_id)) { lm = l; lm_id = v; }
  });
  const float lmax = block_max(lm, sh);
  if (threadIdx.x == 0) { sh.found_bin = 0x7fffffffu; sh.list_bin = 0xFFFFFFFFu; }
  __syncthreads();
  if (lm == lmax && lm_id != 0x7fffffff) atomicMin(&sh.found_bin, (unsigned int)lm_id);
  __syncthreads();
  const int top_id = sh.found_bin == 0x7fffffffu ? -1 : (int)sh.found_bin;
  __syncthreads();

  // level-0 histogram (count and mass per 1/64 of l_max - l), total mass, and how many ids reach the min-p bound
  const float bound = min_p > 0.f ? lmax + temp * logf(min_p) : -CUDART_INF_F;
  for (int b = threadIdx.x; b < kSelBins; b += kSelThreads) { sh.cnt0[b] = 0; sh.mass0[b] = 0; }
  __syncthreads();
  const bool need_mass = top_p < 1.f;  // only the nucleus asks for masses
  unsigned long long tm = 0, tb = 0;
  walk_row(lrow, V, [&](int v, float l) {
    const unsigned int b0 = level0_bin(l, lmax);
    atomicAdd(&sh.cnt0[b0], 1u);
    if (need_mass) {
      const unsigned long long q = fixed_mass(l, lmax, c1);
      add_mass(&sh.mass0[b0], q);
      tm += q;
    }
    tb += (l >= bound) ? 1u : 0u;
  });
  const unsigned long long m_total = block_sum(tm, sh);
  const unsigned int n_minp = (unsigned int)block_sum(tb, sh);

  const unsigned int k_eff = (top_k >= 1 && top_k < V) ? (unsigned int)top_k : (unsigned int)V;
  unsigned int n_keep = k_eff;
  Selected last;       // the selection whose position is N - 1, when one of them is
  bool have_last = false;
  unsigned int last_pos = 0;

  unsigned long long m_topk = m_total;
  if (k_eff < (unsigned int)V) {
    const Selected sk = radix_select(lrow, V, lmax, c1, false, k_eff - 1, 0ull, need_mass, sh);
    const unsigned long long e = sk.ties ? sk.m_tie / sk.ties : 0ull;
    m_topk = sk.m_gt + (unsigned long long)(k_eff - sk.c_gt) * e;
    last = sk; have_last = true; last_pos = k_eff - 1;
  }
  if (top_p < 1.f) {
    // the shortest prefix whose mass reaches top_p of the mass the top-k keeps
    const double want = (double)top_p * (double)m_topk;
    unsigned long long target = (unsigned long long)want;
    if ((double)target < want) ++target;
    if (target < 1ull) target = 1ull;
    const Selected sn = radix_select(lrow, V, lmax, c1, true, 0u, target, true, sh);
    const unsigned long long e = sn.ties ? sn.m_tie / sn.ties : 0ull;
    unsigned int in_tie = sn.ties;
    if (e > 0ull && target > sn.m_gt) {
      const unsigned long long need = target - sn.m_gt;
      const unsigned long long q = (need + e - 1ull) / e;
      if (q < (unsigned long long)in_tie) in_tie = (unsigned int)q;
    }
    if (in_tie < 1u) in_tie = 1u;
    const unsigned int n_nucleus = sn.c_gt + in_tie;
    if (n_nucleus < n_keep) {
      n_keep = n_nucleus;
      last = sn; have_last = true; last_pos = n_nucleus - 1;
    }
  }
  bool by_min_p = false;
  if (n_minp >= 1u && n_minp < n_keep) { n_keep = n_minp; have_last = false; by_min_p = true; }
  if (n_keep < 1u) n_keep = 1u;
  if (n_keep > (unsigned int)V) n_keep = (unsigned int)V;
  if (!have_last || last_pos != n_keep - 1u || !(last.c_gt <= n_keep - 1u && n_keep - 1u < last.c_gt + last.ties)) {
    last = radix_select(lrow, V, lmax, c1, false, n_keep - 1u, 0ull, false, sh);
  }

  // the id at position N - 1: the (N - c_gt)-th lowest id among the elements with that logit
  const unsigned int j = n_keep - 1u - last.c_gt;
  if (threadIdx.x == 0) sh.tie_n = 0u;
  __syncthreads();
  const float l_last = key_to_logit(last.key);
  if (sh.list_bin == level0_bin(l_last, lmax)) {
    // the last selection's list holds every id of the bin the value lies in
    const unsigned int n_list = sh.list_n;
    for (unsigned int i = threadIdx.x; i < n_list; i += kSelThreads) {
      const int v = sh.list[i];
      if (desc_key(lrow[v]) == last.key) {
        const unsigned int at = atomicAdd(&sh.tie_n, 1u);
        if (at < (unsigned int)kSelTieCap) sh.tie_ids[at] = v;
      }
    }
  } else {
    walk_row(lrow, V, [&](int v, float l) {
      if (desc_key(l) == last.key) {
        const unsigned int at = atomicAdd(&sh.tie_n, 1u);
        if (at < (unsigned int)kSelTieCap) sh.tie_ids[at] = v;
      }
    });
  }
  __syncthreads();
  const unsigned int n_tie = sh.tie_n < (unsigned int)kSelTieCap ? sh.tie_n : (unsigned int)kSelTieCap;
  int cut_id = -1;
  if (threadIdx.x == 0) sh.found_bin = n_tie ? (unsigned int)sh.tie_ids[0] : 0u;
  __syncthreads();
  for (unsigned int a = threadIdx.x; a < n_tie; a += kSelThreads) {
    unsigned int before = 0;
    for (unsigned int b = 0; b < n_tie; ++b) before += (sh.tie_ids[b] < sh.tie_ids[a]) ? 1u : 0u;
    if (before == (j < n_tie ? j : n_tie - 1u)) sh.found_bin = (unsigned int)sh.tie_ids[a];
  }
  __syncthreads();
  cut_id = (int)sh.found_bin;
  __syncthreads();

  // sums over the kept ids (Token-IPT-DiFR on the filtered distribution)
  unsigned long long z = 0, below = 0, mine = 0;
  if (p.want_sums) {
    const int tok = p.tokens[row];
    unsigned long long kz = 0, kb = 0, km = 0;
    walk_row(lrow, V, [&](int v, float l) {
      const uint32_t k = desc_key(l);
      if (k < last.key || (k == last.key && v <= cut_id)) {
        const unsigned long long q = fixed_mass(l, lmax, c1);
        kz += q;
        if (v < tok) kb += q;
        if (v == tok) km += q;
      }
    });
    z = block_sum(kz, sh); below = block_sum(kb, sh); mine = block_sum(km, sh);
  }
  if (threadIdx.x == 0) {
    p.cut_id[row] = cut_id;
    p.top_id[row] = top_id;
    p.kept_n[row] = by_min_p ? -(int)n_keep : (int)n_keep;
    p.kept_z[row] = (double)z;
    p.kept_below[row] = (double)below;
    p.kept_mine[row] = (double)mine;
    if (sh.tie_n > (unsigned int)kSelTieCap && p.row_status != nullptr) p.row_status[row] |= 16u;
  }
}

cudaError_t launch_select_cutoff(const SelectParams& p, cudaStream_t stream) {
  if (p.rows <= 0) return cudaSuccess;
  const cudaError_t e =
      cudaFuncSetAttribute(select_cutoff, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(SelShared));
  if (e != cudaSuccess) return e;
  select_cutoff<<<p.rows, kSelThreads, sizeof(SelShared), stream>>>(p);
  return cudaGetLastError();
}

}  // namespace difr
