// K3: threshold detection and per-sequence pooling.  Pure streaming: one CTA per
// sequence walks its rows with 128-bit loads where alignment allows, writes the
// flags and reduces (flag count, match count, score sum, score minimum).
#include <cuda_runtime.h>
#include <math_constants.h>

#include "difr_kernels.h"

namespace difr {

constexpr int kK3Threads = 256;

struct SeqAcc {
  int n_flag, n_match;
  float sum, mn;
};

__device__ __forceinline__ void row_update(const K3Params& p, int64_t r, float s, SeqAcc& a) {
  const bool flagged = (s < p.threshold) || isnan(s);
  uint8_t f = flagged ? 1 : 0;
  if (flagged && p.ranks != nullptr && p.ranks[r] >= p.rank_cutoff) f = 2;
  if (p.flags) p.flags[r] = f;
  a.n_flag += flagged;
  if (p.margins) {
    const float m = p.margins[r];
    a.n_match += (!isnan(m) && !signbit(m));
  }
  a.sum += s;
  if (s < a.mn) a.mn = s;
}

__global__ void __launch_bounds__(kK3Threads) k3_detect(const K3Params p) {
  const int64_t seq = blockIdx.x;
  const int64_t lo = p.seq_offsets ? (int64_t)p.seq_offsets[seq] : 0;
  const int64_t hi = p.seq_offsets ? (int64_t)p.seq_offsets[seq + 1] : p.T;
  SeqAcc a = {0, 0, 0.f, CUDART_INF_F};
  // head up to a 16-byte boundary of the scores array, body in float4, tail
  const int64_t phase = (int64_t)((reinterpret_cast<uintptr_t>(p.scores) >> 2) & 3u);
  int64_t body = lo + ((4 - ((phase + lo) & 3)) & 3);
  if (body > hi) body = hi;
  const int64_t body_end = body + ((hi - body) & ~(int64_t)3);
  for (int64_t r = lo + threadIdx.x; r < body; r += kK3Threads) row_update(p, r, p.scores[r], a);
  for (int64_t r = body + 4 * (int64_t)threadIdx.x; r < body_end; r += 4 * kK3Threads) {
    const float4 s4 = *reinterpret_cast<const float4*>(p.scores + r);
    row_update(p, r + 0, s4.x, a);
    row_update(p, r + 1, s4.y, a);
    row_update(p, r + 2, s4.z, a);
    row_update(p, r + 3, s4.w, a);
  }
  for (int64_t r = body_end + threadIdx.x; r < hi; r += kK3Threads) row_update(p, r, p.scores[r], a);

  if (p.seq_stats == nullptr) return;
#pragma unroll
  for (int m = 16; m >= 1; m >>= 1) {
    a.n_flag += __shfl_xor_sync(0xffffffffu, a.n_flag, m);
    a.n_match += __shfl_xor_sync(0xffffffffu, a.n_match, m);
    a.sum += __shfl_xor_sync(0xffffffffu, a.sum, m);
    a.mn = fminf(a.mn, __shfl_xor_sync(0xffffffffu, a.mn, m));
  }
  __shared__ SeqAcc part[kK3Threads / 32];
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = a;
  __syncthreads();
  if (threadIdx.x == 0) {
    SeqAcc t = part[0];
    for (int w = 1; w < kK3Threads / 32; ++w) {
      t.n_flag += part[w].n_flag;
      t.n_match += part[w].n_match;
      t.sum += part[w].sum;
      t.mn = fminf(t.mn, part[w].mn);
    }
    struct Out { int32_t n_flagged, n_match; float sum, mn; };
    Out o = {t.n_flag, t.n_match, t.sum, t.mn};
    reinterpret_cast<Out*>(p.seq_stats)[seq] = o;
  }
}

cudaError_t launch_k3(const K3Params& p, cudaStream_t stream) {
  const int64_t blocks = p.seq_offsets ? p.n_seq : 1;
  if (blocks <= 0) return cudaSuccess;
  k3_detect<<<(unsigned)blocks, kK3Threads, 0, stream>>>(p);
  return cudaGetLastError();
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
