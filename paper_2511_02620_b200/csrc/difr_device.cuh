// Device-side building blocks shared by the three kernels: the Philox-4x32-10
// random oracle, mbarrier / TMA / tcgen05 wrappers (sm_100a inline PTX) and the
// layout of the per-(row, vocabulary-slot) partial record.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace difr {

// ------------------------------------------------------------------ partials
// One record per (row, strip): what a strip of the vocabulary contributes to the
// row's statistics.  Log-sum-exp terms live in the base-2 domain of
// z_v = l_v * log2(e) / Temp:  lse2_sum = sum_v 2^(z_v - lse2_max).
struct __align__(16) Partial {
  float m1;        // largest  y' = l + Temp*ln2 * (-log2(-log2 u))   (order-preserving shift of l + Temp*G)
  int32_t i1;      // its vocabulary id, -1 if the strip is empty
  float m2;        // second largest
  int32_t i2;
  float lse2_max;  // max_v z_v, -inf if the strip is empty
  float lse2_sum;
  float prefix2;   // sum over v < claimed id of 2^(z_v - lse2_max)
  int32_t larger;  // ids of the strip (claimed id left out) whose logit exceeds the claimed one; rank mode only
};
static_assert(sizeof(Partial) == 32, "partial record is 32 bytes");

// One entry of a row's candidate list (collecting pass of the full Token-DiFR estimator).
struct Candidate {
  int32_t id;
  float l, y;  // fp32 logit and y' = y + Temp ln ln 2 as the fused kernel computes them
};

// An id whose fp32 value (raw logit in the rank mode, y' in the counting modes) lies within rounding of a bound:
// the finalize kernels re-evaluate it in fp64.  Up to kBandCap per row.
struct BandEntry {
  int32_t id;
  float v;
};
constexpr int kBandCap = 64;
constexpr int kBandOnly = (int)0x80000000u;  // candidate lists: an entry kept only for the rank's exact decision
constexpr int kBandPlane = 4;                // plane of the per-row bounds that holds the band width

// -------------------------------------------------------------------- Philox
constexpr uint32_t kPhiloxM0 = 0xD2511F53u;
constexpr uint32_t kPhiloxM1 = 0xCD9E8D57u;
constexpr uint32_t kPhiloxW0 = 0x9E3779B9u;
constexpr uint32_t kPhiloxW1 = 0xBB67AE85u;

__host__ __device__ __forceinline__ void mulhilo(uint32_t a, uint32_t b, uint32_t& hi, uint32_t& lo) {
  uint64_t p = (uint64_t)a * (uint64_t)b;
  hi = (uint32_t)(p >> 32);
  lo = (uint32_t)p;
}

// Generic ten-round block function.
__host__ __device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                       uint32_t k0, uint32_t k1, uint32_t out[4]) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    uint32_t h0, l0, h1, l1;
    mulhilo(kPhiloxM0, c0, h0, l0);
    mulhilo(kPhiloxM1, c2, h1, l1);
    c0 = h1 ^ c1 ^ k0;
    c1 = l1;
    c2 = h0 ^ c3 ^ k1;
    c3 = l0;
    k0 += kPhiloxW0;
    k1 += kPhiloxW1;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// ------------------------------------------------------------ noise per row
// Philox block for counter (c0, position, 0, 0): with the third and fourth
// counter words zero the first two rounds lose three of their four multiplies,
// and everything that depends only on (seed, position) is computed once per row.
struct RowNoise {
  uint32_t ka[10], kb[10];
  uint32_t q;     // hi(M0 * (position ^ ka[0])) ^ kb[1]
  uint32_t p_lo;  // lo(M0 * (position ^ ka[0]))
};

__device__ __forceinline__ void row_noise_init(RowNoise& rn, uint64_t seed, uint32_t position) {
  uint32_t k0 = (uint32_t)seed, k1 = (uint32_t)(seed >> 32);
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    rn.ka[r] = k0 + (uint32_t)r * kPhiloxW0;
    rn.kb[r] = k1 + (uint32_t)r * kPhiloxW1;
  }
  uint32_t hi, lo;
  mulhilo(kPhiloxM0, position ^ rn.ka[0], hi, lo);
  rn.q = hi ^ rn.kb[1];
  rn.p_lo = lo;
}

__device__ __forceinline__ void row_noise_block(const RowNoise& rn, uint32_t c0, uint32_t x[4]) {
  uint32_t h0, l0, h1, l1;
  mulhilo(kPhiloxM0, c0, h0, l0);           // round 1: x0 = pos ^ ka0 (folded), x1 = 0
  uint32_t x2 = h0 ^ rn.kb[0], x3 = l0;
  mulhilo(kPhiloxM1, x2, h1, l1);           // round 2
  uint32_t x0 = h1 ^ rn.ka[1];
  uint32_t x1 = l1;
  x2 = rn.q ^ x3;
  x3 = rn.p_lo;
#pragma unroll
  for (int r = 2; r < 10; ++r) {
    mulhilo(kPhiloxM0, x0, h0, l0);
    mulhilo(kPhiloxM1, x2, h1, l1);
    x0 = h1 ^ x1 ^ rn.ka[r];
    x1 = l1;
    x2 = h0 ^ x3 ^ rn.kb[r];
    x3 = l0;
  }
  x[0] = x0; x[1] = x1; x[2] = x2; x[3] = x3;
}

// ------------------------------------------------------------ PTX: mbarrier
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// One attempt: the thread sleeps in hardware until the phase completes or about
// `kTryWaitNs` have passed, so a waiting warp issues next to no instructions.
constexpr uint32_t kTryWaitNs = 200000u;
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2, %3;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity), "r"(kTryWaitNs)
      : "memory");
  return ok != 0;
}

// Every wait is bounded: after `kWaitCycles` SM clocks without progress the
// waiter raises the CTA-wide abort flag and returns false; every other waiter
// sees the flag and returns false as well, so the CTA always terminates.
constexpr long long kWaitCycles = 4000000000LL;  // about two seconds

__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          long long limit_cycles = kWaitCycles) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (true) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (clock64() - t0 > limit_cycles) {
      *abort_flag = 1;
      return false;
    }
  }
}

// One 32-byte store (the address must be 32-byte aligned): a whole sector per lane.
__device__ __forceinline__ void st_global_v8(float* dst, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                             uint32_t a4, uint32_t a5, uint32_t a6, uint32_t a7) {
  asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst), "r"(a0), "r"(a1), "r"(a2),
               "r"(a3), "r"(a4), "r"(a5), "r"(a6), "r"(a7)
               : "memory");
}

// ----------------------------------------------------------------- PTX: TMA
__device__ __forceinline__ void tma_load_2d(uint32_t dst_smem, const void* tmap, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst_smem), "l"(tmap), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tma_prefetch_desc(const void* tmap) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(tmap) : "memory");
}

// The same load issued by either CTA of a pair: the data lands in the issuing
// CTA's shared memory, the byte count is credited to `bar`, a shared::cluster
// address that may name the partner's barrier.  Each CTA fetches its own tile;
// no load is delivered to more than one CTA.
// `policy` is an L2 eviction policy made by l2_policy_*().
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst_smem, const void* tmap, int x, int y, uint32_t bar,
                                                 uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint "
      "[%0], [%1, {%2, %3}], [%4], %5;"
      ::"r"(dst_smem), "l"(tmap), "r"(x), "r"(y), "r"(bar), "l"(policy)
      : "memory");
}
// L2 eviction policies.
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ uint64_t l2_policy_evict_normal() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}

// ------------------------------------------------------- PTX: CTA pairs
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// shared::cluster address of the same shared-memory offset in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_arrive() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
}
__device__ __forceinline__ void cluster_wait() {
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// The same without a cluster-wide memory fence: for arrivals that publish no memory
// (a thread that has finished reading TMEM or a unit id says so).
__device__ __forceinline__ void mbar_arrive_cluster_nofence(uint32_t bar_cluster_addr) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster_addr) : "memory");
}
__device__ __forceinline__ void st_shared_cluster_u32(uint32_t cluster_addr, uint32_t v) {
  asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(cluster_addr), "r"(v) : "memory");
}
// arrive on a barrier that may live in the partner CTA (shared::cluster address)
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar_cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster_addr) : "memory");
}

// One lane of a converged warp (always the same one for the same mask).
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "elect.sync _|p, 0xffffffff;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(pred));
  return pred != 0;
}

// ------------------------------------------------------------- PTX: tcgen05
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// Pair forms: one warp of each CTA of the pair executes them, with the same arguments.
__device__ __forceinline__ void tmem_alloc_pair(uint32_t dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
// D[tmem] (+)= A[smem] * B[smem]^T, bf16 x bf16 -> fp32, issued by one thread.
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
      "}\n"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// The pair form: issued by one thread of the pair's first CTA.  A (256 x 16) is read as
// 128 rows from each CTA's shared memory, B (256 x 16) as 128 rows from each; the
// accumulator rows 0..127 live in the first CTA's TMEM, rows 128..255 in the second's.
__device__ __forceinline__ void umma_bf16_pair(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                               uint32_t accumulate) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n"
      "}\n"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Once every MMA issued so far by this thread has completed, arrive on the barrier at
// this shared-memory offset in each CTA named by `cta_mask` (a signal, not a data copy).
__device__ __forceinline__ void umma_commit_pair(uint32_t bar, uint16_t cta_mask) {
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
      ::"r"(bar), "h"(cta_mask)
      : "memory");
}
// Arrive on an mbarrier once every MMA issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 32 lanes x 16 consecutive fp32 columns: thread i of the warp receives lane
// (base lane + i), columns [col, col + 16).  The registers are valid only after
// tmem_ld_wait() on the same array.
__device__ __forceinline__ void tmem_ld_32x16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
// Waits for every tcgen05.ld this thread has issued.  The array goes through the
// statement as an in/out operand so that no use of it can be scheduled above the wait.
__device__ __forceinline__ void tmem_ld_wait(uint32_t (&r)[16]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                 "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]),
                 "+r"(r[15])
               :
               : "memory");
}

// Shared-memory matrix descriptor of a K-major bf16 tile stored as rows of 128
// bytes with the 128-byte swizzle (what a TMA box of 64 bf16 x R rows with
// CU_TENSOR_MAP_SWIZZLE_128B writes): 8-row groups are 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc_k_major_sw128(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);  // start address, 16-byte units
  d |= (uint64_t)1 << 16;                        // leading byte offset: unused for swizzled K-major
  d |= (uint64_t)(1024 >> 4) << 32;              // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                        // descriptor version of sm_100
  d |= (uint64_t)2 << 61;                        // 128-byte swizzle
  return d;
}

// Instruction descriptor: dense, fp32 accumulator, bf16 A and B, both K-major.
__host__ __device__ constexpr uint32_t umma_idesc_bf16(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// Register re-allocation between warpgroups (all four warps of a warpgroup execute it).
template <int N>
__device__ __forceinline__ void setmaxnreg_inc() {
  asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N));
}
template <int N>
__device__ __forceinline__ void setmaxnreg_dec() {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N));
}

// Two fp32 operations in one instruction (sm_100 packed arithmetic on register pairs).
__device__ __forceinline__ float2 ffma2(float2 a, float2 b, float2 c) {
  unsigned long long d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;"
      : "=l"(d)
      : "l"(*reinterpret_cast<unsigned long long*>(&a)), "l"(*reinterpret_cast<unsigned long long*>(&b)),
        "l"(*reinterpret_cast<unsigned long long*>(&c)));
  return *reinterpret_cast<float2*>(&d);
}
__device__ __forceinline__ float2 fadd2(float2 a, float2 b) {
  unsigned long long d;
  asm("add.rn.f32x2 %0, %1, %2;"
      : "=l"(d)
      : "l"(*reinterpret_cast<unsigned long long*>(&a)), "l"(*reinterpret_cast<unsigned long long*>(&b)));
  return *reinterpret_cast<float2*>(&d);
}

__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float lg2_approx(float x) {
  float y;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// ------------------------------------------------- exact (fp64) re-evaluation, shared by the finalize kernels
__device__ __forceinline__ double shfl_xor_double(double v, int mask) {
  int lo = __double2loint(v), hi = __double2hiint(v);
  lo = __shfl_xor_sync(0xffffffffu, lo, mask);
  hi = __shfl_xor_sync(0xffffffffu, hi, mask);
  return __hiloint2double(hi, lo);
}

__device__ __forceinline__ double bf16_to_double(uint32_t bits16) {
  return (double)__uint_as_float(bits16 << 16);
}

// fp64 dot product of two bf16 rows of length d (d % 8 == 0, rows 16-byte aligned), whole warp.
__device__ __forceinline__ double warp_dot(const uint16_t* a, const uint16_t* b, int d, int lane) {
  double acc = 0.0;
  for (int k = lane * 8; k < d; k += 32 * 8) {
    const uint4 va = *reinterpret_cast<const uint4*>(a + k);
    const uint4 vb = *reinterpret_cast<const uint4*>(b + k);
    const uint32_t wa[4] = {va.x, va.y, va.z, va.w};
    const uint32_t wb[4] = {vb.x, vb.y, vb.z, vb.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      acc = fma(bf16_to_double(wa[q] & 0xFFFFu), bf16_to_double(wb[q] & 0xFFFFu), acc);
      acc = fma(bf16_to_double(wa[q] >> 16), bf16_to_double(wb[q] >> 16), acc);
    }
  }
#pragma unroll
  for (int m = 16; m >= 1; m >>= 1) acc += shfl_xor_double(acc, m);
  return acc;
}

// Up to three such dot products against the same row a, their loads in flight together; a null row gives 0.
// Each sum is taken in warp_dot's order, so the values are the same as separate calls.
__device__ __forceinline__ void warp_dot3(const uint16_t* a, const uint16_t* b0, const uint16_t* b1,
                                          const uint16_t* b2, int d, int lane, double out[3]) {
  const uint16_t* b[3] = {b0, b1, b2};
  double acc[3] = {0.0, 0.0, 0.0};
  for (int k = lane * 8; k < d; k += 32 * 8) {
    const uint4 va = *reinterpret_cast<const uint4*>(a + k);
    uint4 vb[3];
#pragma unroll
    for (int j = 0; j < 3; ++j)
      vb[j] = b[j] != nullptr ? *reinterpret_cast<const uint4*>(b[j] + k) : make_uint4(0u, 0u, 0u, 0u);
    const uint32_t wa[4] = {va.x, va.y, va.z, va.w};
#pragma unroll
    for (int j = 0; j < 3; ++j) {
      const uint32_t wb[4] = {vb[j].x, vb[j].y, vb[j].z, vb[j].w};
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        acc[j] = fma(bf16_to_double(wa[q] & 0xFFFFu), bf16_to_double(wb[q] & 0xFFFFu), acc[j]);
        acc[j] = fma(bf16_to_double(wa[q] >> 16), bf16_to_double(wb[q] >> 16), acc[j]);
      }
    }
  }
#pragma unroll
  for (int m = 16; m >= 1; m >>= 1) {
#pragma unroll
    for (int j = 0; j < 3; ++j) acc[j] += shfl_xor_double(acc[j], m);
  }
#pragma unroll
  for (int j = 0; j < 3; ++j) out[j] = acc[j];
}

__device__ __forceinline__ double gumbel_exact(uint64_t seed, uint32_t position, uint32_t id) {
  uint32_t x[4];
  philox4x32_10(id >> 2, position, 0u, 0u, (uint32_t)seed, (uint32_t)(seed >> 32), x);
  const double u = ((double)(x[id & 3u] >> 9) + 0.5) * (1.0 / 8388608.0);
  return -log(-log(u));
}

}  // namespace difr
