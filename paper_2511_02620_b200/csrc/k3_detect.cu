// K3: threshold detection and per-sequence pooling.  Pure streaming: a cluster of
// CTAs per sequence (1 to 16, by the average sequence length) splits the
// sequence's rows, walks them with 128-bit loads of scores, margins and ranks and
// 32-bit stores of four flags where alignment allows, and reduces (flag count,
// match count, score sum, score minimum) by warp shuffles, shared memory and, across
// the cluster, the first CTA's shared memory, always in the same order: the
// statistics are the same bits on every run.
#include <cuda_runtime.h>
#include <math_constants.h>
#include <string.h>

#include <atomic>

#include "difr_device.cuh"
#include "difr_kernels.h"

namespace difr {

constexpr int kK3Threads = 512;
constexpr int kK3MaxCluster = 16;      // CTAs per sequence (above 8: the non-portable cluster size B200 offers)
constexpr int kK3RowsPerCta = 4096;    // a sequence gets more CTAs once a CTA would walk more rows than this

struct SeqAcc {
  int n_flag, n_match;
  float sum, mn;
};

__device__ __forceinline__ uint8_t classify_row(const K3Params& p, float s, float m, int rank, SeqAcc& a) {
  const bool flagged = (s < p.threshold) || isnan(s);
  uint8_t f = flagged ? 1 : 0;
  if (flagged && p.ranks != nullptr && rank >= p.rank_cutoff) f = 2;  // not among the R largest raw logits
  a.n_flag += flagged;
  if (p.margins != nullptr) a.n_match += (!isnan(m) && !signbit(m));
  a.sum += s;
  if (s < a.mn) a.mn = s;
  return f;
}

__device__ __forceinline__ void row_scalar(const K3Params& p, int64_t r, SeqAcc& a) {
  const float m = p.margins != nullptr ? p.margins[r] : 0.f;
  const int rank = p.ranks != nullptr ? p.ranks[r] : 0;
  const uint8_t f = classify_row(p, p.scores[r], m, rank, a);
  if (p.flags != nullptr) p.flags[r] = f;
}

__device__ __forceinline__ void acc_merge(SeqAcc& a, const SeqAcc& b) {
  a.n_flag += b.n_flag;
  a.n_match += b.n_match;
  a.sum += b.sum;
  a.mn = fminf(a.mn, b.mn);
}

__global__ void __launch_bounds__(kK3Threads) k3_detect(const K3Params p) {
  __shared__ SeqAcc part[kK3Threads / 32];
  __shared__ SeqAcc from_cta[kK3MaxCluster];  // used in the cluster's first CTA
  uint32_t csize, crank;
  asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(csize));
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(crank));
  const int64_t seq = blockIdx.x / csize;
  const int64_t lo = p.seq_offsets ? (int64_t)p.seq_offsets[seq] : 0;
  const int64_t hi = p.seq_offsets ? (int64_t)p.seq_offsets[seq + 1] : p.T;
  // this CTA's share of the sequence: equal parts, each a multiple of four rows
  const int64_t n = hi > lo ? hi - lo : 0;
  const int64_t per = (((n + csize - 1) / csize) + 3) & ~(int64_t)3;
  const int64_t my_lo = lo + (int64_t)crank * per < hi ? lo + (int64_t)crank * per : hi;
  const int64_t my_hi = my_lo + per < hi ? my_lo + per : hi;

  SeqAcc a = {0, 0, 0.f, CUDART_INF_F};
  // head up to a 16-byte boundary of the scores array, body four rows at a time, tail.  The other arrays use
  // 128-bit (flags: 32-bit) accesses when they share that alignment, scalar ones otherwise.
  const int64_t phase = (int64_t)((reinterpret_cast<uintptr_t>(p.scores) >> 2) & 3u);
  int64_t body = my_lo + ((4 - ((phase + my_lo) & 3)) & 3);
  if (body > my_hi) body = my_hi;
  const int64_t body_end = body + ((my_hi - body) & ~(int64_t)3);
  const bool vec_m = p.margins != nullptr && ((reinterpret_cast<uintptr_t>(p.margins + body) & 15u) == 0);
  const bool vec_r = p.ranks != nullptr && ((reinterpret_cast<uintptr_t>(p.ranks + body) & 15u) == 0);
  const bool vec_f = p.flags != nullptr && ((reinterpret_cast<uintptr_t>(p.flags + body) & 3u) == 0);
  for (int64_t r = my_lo + threadIdx.x; r < body; r += kK3Threads) row_scalar(p, r, a);
  for (int64_t r = body + 4 * (int64_t)threadIdx.x; r < body_end; r += 4 * kK3Threads) {
    const float4 s4 = *reinterpret_cast<const float4*>(p.scores + r);
    float4 m4 = make_float4(0.f, 0.f, 0.f, 0.f);
    int4 k4 = make_int4(0, 0, 0, 0);
    if (vec_m) m4 = *reinterpret_cast<const float4*>(p.margins + r);
    else if (p.margins != nullptr) m4 = make_float4(p.margins[r], p.margins[r + 1], p.margins[r + 2], p.margins[r + 3]);
    if (vec_r) k4 = *reinterpret_cast<const int4*>(p.ranks + r);
    else if (p.ranks != nullptr) k4 = make_int4(p.ranks[r], p.ranks[r + 1], p.ranks[r + 2], p.ranks[r + 3]);
    uchar4 f4;
    f4.x = classify_row(p, s4.x, m4.x, k4.x, a);
    f4.y = classify_row(p, s4.y, m4.y, k4.y, a);
    f4.z = classify_row(p, s4.z, m4.z, k4.z, a);
    f4.w = classify_row(p, s4.w, m4.w, k4.w, a);
    if (vec_f) {
      *reinterpret_cast<uchar4*>(p.flags + r) = f4;
    } else if (p.flags != nullptr) {
      p.flags[r] = f4.x; p.flags[r + 1] = f4.y; p.flags[r + 2] = f4.z; p.flags[r + 3] = f4.w;
    }
  }
  for (int64_t r = body_end + threadIdx.x; r < my_hi; r += kK3Threads) row_scalar(p, r, a);

  if (p.seq_stats == nullptr) return;  // (uniform over the cluster: nobody waits for anybody)
#pragma unroll
  for (int m = 16; m >= 1; m >>= 1) {
    SeqAcc o;
    o.n_flag = __shfl_xor_sync(0xffffffffu, a.n_flag, m);
    o.n_match = __shfl_xor_sync(0xffffffffu, a.n_match, m);
    o.sum = __shfl_xor_sync(0xffffffffu, a.sum, m);
    o.mn = __shfl_xor_sync(0xffffffffu, a.mn, m);
    acc_merge(a, o);
  }
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = a;
  __syncthreads();
  if (threadIdx.x == 0) {
    SeqAcc t = part[0];
    for (int w = 1; w < kK3Threads / 32; ++w) acc_merge(t, part[w]);
    if (csize == 1) {
      from_cta[0] = t;
    } else {
      // hand this CTA's partial to the cluster's first CTA (four 32-bit stores into its shared memory)
      const uint32_t dst = map_to_cta(smem_u32(&from_cta[crank]), 0);
      st_shared_cluster_u32(dst, (uint32_t)t.n_flag);
      st_shared_cluster_u32(dst + 4, (uint32_t)t.n_match);
      st_shared_cluster_u32(dst + 8, __float_as_uint(t.sum));
      st_shared_cluster_u32(dst + 12, __float_as_uint(t.mn));
    }
  }
  if (csize > 1) {
    cluster_arrive();  // release: the partials are visible to the first CTA after its wait
    cluster_wait();
  }
  if (crank == 0 && threadIdx.x == 0) {
    SeqAcc t = from_cta[0];
    for (uint32_t c = 1; c < csize; ++c) acc_merge(t, from_cta[c]);
    struct Out { int32_t n_flagged, n_match; float sum, mn; };
    Out o = {t.n_flag, t.n_match, t.sum, t.mn};
    reinterpret_cast<Out*>(p.seq_stats)[seq] = o;
  }
}

cudaError_t launch_k3(const K3Params& p, cudaStream_t stream) {
  const int64_t n_seq = p.seq_offsets ? p.n_seq : 1;
  if (n_seq <= 0) return cudaSuccess;
  // CTAs per sequence by the average length: a power of two, at most 16
  const int64_t avg = p.T / n_seq;
  int csize = 1;
  while (csize < kK3MaxCluster && (int64_t)csize * kK3RowsPerCta < avg) csize *= 2;
  static std::atomic<int> non_portable_ok{0};  // 0 unknown, 1 allowed, -1 refused
  if (csize > 8) {
    int st = non_portable_ok.load(std::memory_order_relaxed);
    if (st == 0) {
      st = cudaFuncSetAttribute(k3_detect, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess ? 1 : -1;
      if (st < 0) (void)cudaGetLastError();
      non_portable_ok.store(st, std::memory_order_relaxed);
    }
    if (st < 0) csize = 8;
  }
  if (n_seq * csize > 0x7fffffffLL) return cudaErrorInvalidValue;
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof cfg);
  cfg.blockDim = dim3(kK3Threads, 1, 1);
  cfg.stream = stream;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeClusterDimension;
  attr.val.clusterDim.y = 1;
  attr.val.clusterDim.z = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  for (;;) {
    cfg.gridDim = dim3((unsigned)(n_seq * csize), 1, 1);
    attr.val.clusterDim.x = (unsigned)csize;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, k3_detect, p);
    if (e == cudaSuccess || csize <= 8) return e;
    // a cluster of 16 could not be placed on this device: remember it and fall back to the portable size
    (void)cudaGetLastError();
    non_portable_ok.store(-1, std::memory_order_relaxed);
    csize = 8;
  }
}

// ------------------------------------------------ exfiltratable information
// Per token log2 |A_t| (safe), log2 R (suspicious) or log2 V (dangerous); one CTA per sequence sums them.
__global__ void __launch_bounds__(kK3Threads) k3_bits(const BitsParams p) {
  const int64_t seq = blockIdx.x;
  const int64_t lo = p.seq_offsets ? (int64_t)p.seq_offsets[seq] : 0;
  const int64_t hi = p.seq_offsets ? (int64_t)p.seq_offsets[seq + 1] : p.T;
  float sum = 0.f;
  for (int64_t r = lo + threadIdx.x; r < hi; r += kK3Threads) {
    const uint8_t c = p.classes[r];
    float b;
    if (c == 0) {
      const int32_t n = p.counts[r];
      b = n > 0 ? log2f((float)n) : 0.f;
    } else {
      b = (c == 1) ? p.log2_r : p.log2_v;
    }
    if (p.bits) p.bits[r] = b;
    sum += b;
  }
  if (p.seq_bits == nullptr) return;
#pragma unroll
  for (int m = 16; m >= 1; m >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, m);
  __shared__ float part[kK3Threads / 32];
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = sum;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = 0.f;
    for (int w = 0; w < kK3Threads / 32; ++w) t += part[w];
    p.seq_bits[seq] = t;
  }
}

cudaError_t launch_bits(const BitsParams& p, cudaStream_t stream) {
  const int64_t blocks = p.seq_offsets ? p.n_seq : 1;
  if (blocks <= 0) return cudaSuccess;
  k3_bits<<<(unsigned)blocks, kK3Threads, 0, stream>>>(p);
  return cudaGetLastError();
}

}  // namespace difr
