// Sequential randomness expansion RO(seed || i || context): the per-row seeds that make a row's
// noise depend on the prompt and on every claimed token before it (footnote to the definition of
// honest sampling, Sec. "Sampling From Large Language Models"; first further measure of
// Sec. "Message-Sampling Secure Seed Expansion").
//
// One block per sequence walks its rows in chunks: every thread turns its row's token and place
// into a 64-bit element word (one Philox block), a block-wide exclusive prefix sum over those words
// (mod 2^64) plus the running carry gives the row's context, and one more Philox block keyed with
// the row's own seed turns the context into the expanded seed.
#include "difr_device.cuh"
#include "difr_kernels.h"

namespace difr {

namespace {

constexpr int kExpandThreads = 256;
constexpr uint32_t kElementKey0 = 0x243F6A88u, kElementKey1 = 0x85A308D3u;  // first fraction bits of pi

__device__ __forceinline__ uint64_t shfl_up_u64(uint64_t v, int delta) {
  uint32_t lo = (uint32_t)v, hi = (uint32_t)(v >> 32);
  lo = __shfl_up_sync(0xffffffffu, lo, delta);
  hi = __shfl_up_sync(0xffffffffu, hi, delta);
  return ((uint64_t)hi << 32) | lo;
}

__global__ void __launch_bounds__(kExpandThreads)
expand_seeds(const uint64_t* __restrict__ seeds, const int32_t* __restrict__ tokens,
             const int32_t* __restrict__ seq_offsets, const uint64_t* __restrict__ prompt_hashes, long long T,
             uint64_t* __restrict__ expanded) {
  __shared__ uint64_t warp_total[kExpandThreads / 32];
  __shared__ uint64_t carry_s;
  const int q = blockIdx.x;
  long long first = 0, last = T;
  if (seq_offsets != nullptr) {
    first = seq_offsets[q];
    last = seq_offsets[q + 1];
  }
  first = first < 0 ? 0 : first;
  last = last > T ? T : last;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) carry_s = prompt_hashes != nullptr ? prompt_hashes[q] : 0ull;
  __syncthreads();
  for (long long base = first; base < last; base += kExpandThreads) {
    const long long r = base + threadIdx.x;
    const bool live = r < last;
    uint64_t e = 0ull;
    if (live) {
      uint32_t x[4];
      philox4x32_10((uint32_t)(r - first), (uint32_t)tokens[r], 0u, 1u, kElementKey0, kElementKey1, x);
      e = ((uint64_t)x[1] << 32) | x[0];
    }
    // inclusive scan inside the warp, then across the warps
    uint64_t incl = e;
#pragma unroll
    for (int dlt = 1; dlt < 32; dlt <<= 1) {
      const uint64_t up = shfl_up_u64(incl, dlt);
      if (lane >= dlt) incl += up;
    }
    if (lane == 31) warp_total[warp] = incl;
    __syncthreads();
    uint64_t before = carry_s;
    for (int w = 0; w < warp; ++w) before += warp_total[w];
    const uint64_t context = before + incl - e;
    if (live) {
      const uint64_t seed = seeds[r];
      uint32_t x[4];
      philox4x32_10((uint32_t)context, (uint32_t)(context >> 32), 0u, 2u, (uint32_t)seed, (uint32_t)(seed >> 32), x);
      expanded[r] = ((uint64_t)x[1] << 32) | x[0];
    }
    __syncthreads();
    if (threadIdx.x == kExpandThreads - 1) carry_s = before + incl;
    __syncthreads();
  }
}

}  // namespace

cudaError_t launch_expand_seeds(const uint64_t* seeds, const int32_t* tokens, const int32_t* seq_offsets,
                                const uint64_t* prompt_hashes, long long n_seq, long long T, uint64_t* expanded,
                                cudaStream_t stream) {
  const long long blocks = seq_offsets != nullptr ? n_seq : 1;
  if (blocks <= 0) return cudaSuccess;
  expand_seeds<<<(unsigned)blocks, kExpandThreads, 0, stream>>>(seeds, tokens, seq_offsets, prompt_hashes, T, expanded);
  return cudaGetLastError();
}

}  // namespace difr
