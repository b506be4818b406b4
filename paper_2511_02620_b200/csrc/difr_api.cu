// C ABI of libdifr.so: argument validation, work planning, tensor-map encoding
// and kernel launches.  Nothing here computes; every step of the scoring path
// runs in the three kernels.
#include <cuda.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <string.h>

#include <atomic>
#include <mutex>
#include <vector>

#include "../../include/difr.h"
#include "difr_kernels.h"
#include "difr_plan.h"

namespace {

using namespace difr;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(sym);
  }
  return fn;
}

// bf16 [rows, cols] row-major, box = 64 columns (128 bytes, 128-byte swizzle) x box_rows rows.
bool encode_tmap(CUtensorMap* map, const void* base, int64_t rows, int64_t cols, int box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (fn == nullptr) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  const cuuint32_t box[2] = {(cuuint32_t)kBK, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// A tensor map is a host object that depends on the base address and the shape only (never on the contents), and
// callers pass the same W, and often the same h buffers, call after call: the encoded maps are remembered in a
// short most-recently-used list under a mutex.
bool make_tmap(CUtensorMap* map, const void* base, int64_t rows, int64_t cols, int box_rows) {
  struct Entry {
    const void* base;
    int64_t rows, cols;
    int box_rows;
    CUtensorMap map;
  };
  constexpr size_t kEntries = 16;
  static std::mutex mu;
  static std::vector<Entry> cache;  // most recently used first
  {
    std::lock_guard<std::mutex> lock(mu);
    for (size_t i = 0; i < cache.size(); ++i) {
      if (cache[i].base == base && cache[i].rows == rows && cache[i].cols == cols && cache[i].box_rows == box_rows) {
        *map = cache[i].map;
        if (i != 0) {
          const Entry hit = cache[i];
          cache.erase(cache.begin() + (long)i);
          cache.insert(cache.begin(), hit);
        }
        return true;
      }
    }
  }
  if (!encode_tmap(map, base, rows, cols, box_rows)) return false;
  std::lock_guard<std::mutex> lock(mu);
  if (cache.size() >= kEntries) cache.pop_back();
  cache.insert(cache.begin(), Entry{base, rows, cols, box_rows, *map});
  return true;
}

struct DeviceInfo {
  int major;
  int pairs;  // CTA pairs of the fused kernel that are resident at once (0 on other architectures)
};

bool device_info(DeviceInfo* info) {
  constexpr int kMaxDevices = 64;
  // 0: not asked yet; otherwise (major << 16) | pairs + 1 (threads that race here store the same value)
  static std::atomic<int> cached[kMaxDevices];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return false;
  const bool slot = dev >= 0 && dev < kMaxDevices;
  if (slot) {
    const int c = cached[dev].load(std::memory_order_relaxed);
    if (c != 0) {
      info->major = c >> 16;
      info->pairs = (c & 0xffff) - 1;
      return true;
    }
  }
  if (cudaDeviceGetAttribute(&info->major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return false;
  info->pairs = 0;
  if (info->major == 10) {
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return false;
    int pairs = k1_max_resident_pairs();
    if (pairs <= 0) return false;
    if (pairs > sms / 2) pairs = sms / 2;
    info->pairs = pairs;
  }
  if (slot) cached[dev].store((info->major << 16) | (info->pairs + 1), std::memory_order_relaxed);
  return true;
}

// Shape, plan and temperature fields of the fused kernel's parameters; `ws` (nullable) is the workspace that
// holds the partial records and, behind them, the unit counter.
K1Params k1_params(const Plan& pl, int64_t T, int64_t d, int64_t V, float temperature, void* ws) {
  K1Params k1;
  memset(&k1, 0, sizeof k1);
  k1.T = (int)T; k1.d = (int)d; k1.V = (int)V;
  k1.T_pad = pl.T_pad; k1.m_tiles = pl.m_tiles; k1.n_tiles = pl.n_tiles; k1.k_steps = pl.k_steps;
  k1.S = pl.S; k1.Gm = pl.Gm; k1.n_units = pl.n_units;
  k1.c1 = temperature > 0.f ? 1.4426950408889634f / temperature : 0.f;
  k1.neg_tl2 = -temperature * 0.6931471805599453f;
  if (ws != nullptr) {
    k1.partials = reinterpret_cast<Partial*>(ws);
    k1.unit_counter = reinterpret_cast<int*>(static_cast<unsigned char*>(ws) + pl.partial_bytes);
  }
  return k1;
}

int k1_grid(const Plan& pl, int pairs) { return 2 * (pl.n_units < pairs ? pl.n_units : pairs); }

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// kind: 0 Token-DiFR, 1 Token-IPT-DiFR, 2 both.
difr_status score_common(int ipt, const void* h, const void* W, const int32_t* tokens, const uint64_t* seeds,
                         const uint32_t* positions, float temperature, int64_t T, int64_t d, int64_t V,
                         difr_out* out, difr_stream_t stream) {
  if (!h || !W || !tokens || !seeds || !positions || !out || !out->score) return DIFR_ERR_INVALID_ARG;
  if (T < 0 || d <= 0 || V <= 0) return DIFR_ERR_INVALID_ARG;
  if (!(out->sigma > 0.f) || !(out->eps >= 0.f) || !isfinite(out->sigma) || !isfinite(out->eps))
    return DIFR_ERR_INVALID_ARG;
  if (out->temperatures == nullptr &&
      (!(temperature >= 0.f) || !isfinite(temperature) || (ipt && temperature == 0.f)))
    return DIFR_ERR_INVALID_ARG;
  if (out->temperatures != nullptr) temperature = 1.f;  // unused: every row brings its own
  if (ipt == 2 && (!out->score_ipt || !(out->sigma_ipt > 0.f) || !isfinite(out->sigma_ipt))) return DIFR_ERR_INVALID_ARG;
  if ((d % 8) != 0 || V < 2) return DIFR_ERR_SHAPE;
  if (T == 0) return DIFR_OK;
  DeviceInfo info;
  if (!device_info(&info)) return DIFR_ERR_CUDA;
  if (info.major != 10) return DIFR_ERR_ARCH;
  Plan pl;
  if (!make_plan(T, d, V, info.pairs, &pl)) return DIFR_ERR_SHAPE;
  if (!aligned16(h) || !aligned16(W)) return DIFR_ERR_ALIGN;
  if (!out->workspace || out->workspace_bytes < pl.workspace_bytes) return DIFR_ERR_WORKSPACE;
  if (!aligned16(out->workspace)) return DIFR_ERR_ALIGN;

  CUtensorMap tmap_h, tmap_w;
  if (!make_tmap(&tmap_h, h, T, d, kBM) || !make_tmap(&tmap_w, W, V, d, kBN / 2)) return DIFR_ERR_CUDA;

  K1Params k1 = k1_params(pl, T, d, V, temperature, out->workspace);
  k1.tokens = tokens; k1.seeds = seeds; k1.positions = positions;
  k1.device_status = out->device_status;
  k1.temperatures = out->temperatures;
  const int grid = k1_grid(pl, info.pairs);
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  if (cudaMemsetAsync(k1.unit_counter, 0, sizeof(int), s) != cudaSuccess) return DIFR_ERR_CUDA;
  if (ipt != 1) {
    // the rows' running floors (last plane of the bounds): 0x80 in every byte is a float below every key
    k1.row_floor = reinterpret_cast<int*>(static_cast<unsigned char*>(out->workspace) + pl.bounds_offset) +
                   (size_t)(kPlanBoundPlanes - 1) * (size_t)pl.T_pad;
    if (cudaMemsetAsync(k1.row_floor, 0x80, (size_t)pl.T_pad * sizeof(int), s) != cudaSuccess) return DIFR_ERR_CUDA;
  }
  const bool want_rank = (ipt != 1) && out->rank != nullptr;
  if (want_rank) {
    unsigned char* ws = static_cast<unsigned char*>(out->workspace);
    float* bounds = reinterpret_cast<float*>(ws + pl.bounds_offset);
    if (launch_claimed_logits(reinterpret_cast<const uint16_t*>(h), reinterpret_cast<const uint16_t*>(W), tokens,
                              (int)T, (int)d, (int)V, bounds, bounds + (size_t)kBandPlane * (size_t)pl.T_pad, s) !=
        cudaSuccess)
      return DIFR_ERR_CUDA;
    k1.bounds = bounds;
    k1.band_count = reinterpret_cast<int*>(ws + pl.band_count_offset);
    k1.band_list = reinterpret_cast<BandEntry*>(ws + pl.band_list_offset);
    k1.band_cap = kBandCap;
    if (cudaMemsetAsync(k1.band_count, 0, (size_t)pl.T_pad * sizeof(int), s) != cudaSuccess) return DIFR_ERR_CUDA;
  }
  if (out->event_fused_start && cudaEventRecord(reinterpret_cast<cudaEvent_t>(out->event_fused_start), s) != cudaSuccess)
    return DIFR_ERR_CUDA;
  const int k1_mode = (ipt == 1) ? 1 : (want_rank ? 3 : 0);
  if (launch_k1(k1_mode, tmap_h, tmap_w, k1, grid, s) != cudaSuccess) return DIFR_ERR_CUDA;
  if (out->event_fused_stop && cudaEventRecord(reinterpret_cast<cudaEvent_t>(out->event_fused_stop), s) != cudaSuccess)
    return DIFR_ERR_CUDA;

  K2Params k2;
  memset(&k2, 0, sizeof k2);
  k2.h = reinterpret_cast<const uint16_t*>(h); k2.W = reinterpret_cast<const uint16_t*>(W);
  k2.tokens = tokens; k2.seeds = seeds; k2.positions = positions;
  k2.partials = k1.partials; k2.n_slots = pl.n_slots; k2.T_pad = pl.T_pad;
  k2.T = (int)T; k2.d = (int)d; k2.V = (int)V; k2.ipt = ipt;
  k2.temperature = temperature; k2.sigma = out->sigma; k2.eps = out->eps; k2.c1 = k1.c1;
  k2.score = out->score; k2.margin = out->margin; k2.argmax = out->argmax; k2.runner_up = out->runner_up;
  k2.lse = out->lse; k2.p_claimed = out->p_claimed; k2.cdf_lo = out->cdf_lo; k2.u = out->u;
  k2.row_status = out->row_status;
  k2.temperatures = out->temperatures;
  k2.sigma_ipt = out->sigma_ipt; k2.score_ipt = out->score_ipt;
  k2.rank = want_rank ? out->rank : nullptr; k2.y_max = out->y_max; k2.y_second = out->y_second;
  // (the rank mode counts in that word; the Gumbel-max score does not depend on the softmax sum, so the three
  // fp64 transcendentals per row of the exchange are spent only where the IPT outputs are asked for)
  k2.tok_logit_in_records = (want_rank || ipt == 0) ? 0 : 1;
  k2.band_list = k1.band_list; k2.band_count = k1.band_count; k2.band_cap = k1.band_cap;
  if (launch_k2(k2, s) != cudaSuccess) return DIFR_ERR_CUDA;
  return DIFR_OK;
}

}  // namespace

extern "C" {

size_t difr_workspace_bytes(int64_t T, int64_t d, int64_t V) {
  DeviceInfo info;
  if (!device_info(&info)) info.pairs = 0;  // no device: plan for a full B200 (74 pairs)
  Plan pl;
  if (!make_plan(T, d, V, info.pairs, &pl)) return 0;
  return pl.workspace_bytes;
}

difr_status difr_score_gm(const void* h, const void* W, const int32_t* tokens, const uint64_t* seeds,
                          const uint32_t* positions, float temperature, int64_t T, int64_t d, int64_t V,
                          difr_out* out, difr_stream_t stream) {
  return score_common(0, h, W, tokens, seeds, positions, temperature, T, d, V, out, stream);
}

difr_status difr_score_ipt(const void* h, const void* W, const int32_t* tokens, const uint64_t* seeds,
                           const uint32_t* positions, float temperature, int64_t T, int64_t d, int64_t V,
                           difr_out* out, difr_stream_t stream) {
  return score_common(1, h, W, tokens, seeds, positions, temperature, T, d, V, out, stream);
}

difr_status difr_score_both(const void* h, const void* W, const int32_t* tokens, const uint64_t* seeds,
                            const uint32_t* positions, float temperature, int64_t T, int64_t d, int64_t V,
                            difr_out* out, difr_stream_t stream) {
  return score_common(2, h, W, tokens, seeds, positions, temperature, T, d, V, out, stream);
}

// A(tau) = sigma sqrt2 Phi^-1(e^tau - eps): the margin at which the Token-DiFR score equals tau.
static float margin_at_threshold(double tau, double sigma, double eps) {
  const double pr = exp(tau) - eps;
  if (!(pr > 0.0)) return -INFINITY;  // the floor ln(eps) already reaches tau: every id is admissible
  if (pr >= 1.0) return INFINITY;
  double lo = -40.0, hi = 40.0;  // Phi^-1 by bisection on erfc
  for (int i = 0; i < 200; ++i) {
    const double mid = 0.5 * (lo + hi);
    if (0.5 * erfc(-mid / sqrt(2.0)) < pr) lo = mid; else hi = mid;
  }
  return (float)(sigma * sqrt(2.0) * 0.5 * (lo + hi));
}

difr_status difr_admissible(const void* h, const void* W, const uint64_t* seeds, const uint32_t* positions,
                            float temperature, int64_t T, int64_t d, int64_t V, const int32_t* argmax,
                            const int32_t* runner_up, const float* y_max, const float* y_second, float sigma,
                            float eps, const float* taus, int32_t n_tau, int32_t* counts, uint32_t* row_status,
                            void* workspace, size_t workspace_bytes, int32_t* device_status, difr_stream_t stream) {
  if (!h || !W || !seeds || !positions || !argmax || !y_max || !y_second || !taus || !counts)
    return DIFR_ERR_INVALID_ARG;
  if (T < 0 || d <= 0 || V <= 0 || n_tau < 1 || n_tau > 4) return DIFR_ERR_INVALID_ARG;
  if (!(sigma > 0.f) || !(eps >= 0.f) || !isfinite(sigma) || !isfinite(eps)) return DIFR_ERR_INVALID_ARG;
  if (!(temperature >= 0.f) || !isfinite(temperature)) return DIFR_ERR_INVALID_ARG;
  for (int j = 0; j < n_tau; ++j)
    if (isnan(taus[j])) return DIFR_ERR_INVALID_ARG;
  if ((d % 8) != 0 || V < 2) return DIFR_ERR_SHAPE;
  if (T == 0) return DIFR_OK;
  DeviceInfo info;
  if (!device_info(&info)) return DIFR_ERR_CUDA;
  if (info.major != 10) return DIFR_ERR_ARCH;
  Plan pl;
  if (!make_plan(T, d, V, info.pairs, &pl)) return DIFR_ERR_SHAPE;
  if (!aligned16(h) || !aligned16(W)) return DIFR_ERR_ALIGN;
  if (!workspace || workspace_bytes < pl.workspace_bytes) return DIFR_ERR_WORKSPACE;
  if (!aligned16(workspace)) return DIFR_ERR_ALIGN;
  CUtensorMap tmap_h, tmap_w;
  if (!make_tmap(&tmap_h, h, T, d, kBM) || !make_tmap(&tmap_w, W, V, d, kBN / 2)) return DIFR_ERR_CUDA;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  unsigned char* ws = static_cast<unsigned char*>(workspace);

  CountParams cp;
  memset(&cp, 0, sizeof cp);
  cp.h = reinterpret_cast<const uint16_t*>(h); cp.W = reinterpret_cast<const uint16_t*>(W);
  cp.seeds = seeds; cp.positions = positions;
  cp.partials = reinterpret_cast<const Partial*>(ws);
  cp.n_slots = pl.n_slots; cp.T_pad = pl.T_pad; cp.T = (int)T; cp.d = (int)d; cp.V = (int)V; cp.n_tau = n_tau;
  cp.argmax = argmax; cp.runner_up = runner_up; cp.y_max = y_max; cp.y_second = y_second;
  cp.temperature = temperature; cp.sigma = sigma; cp.eps = eps;
  for (int j = 0; j < 4; ++j) {
    cp.a_tau[j] = j < n_tau ? margin_at_threshold(taus[j], sigma, eps) : INFINITY;
    cp.taus[j] = j < n_tau ? taus[j] : INFINITY;
  }
  cp.y_shift = temperature * (float)log(log(2.0));  // the kernel ranks y' = l - Temp ln2 log2(E / ln2) = y + Temp ln ln 2
  cp.bounds = reinterpret_cast<float*>(ws + pl.bounds_offset);
  cp.band_count = reinterpret_cast<int*>(ws + pl.band_count_offset);
  cp.band_list = reinterpret_cast<BandEntry*>(ws + pl.band_list_offset);
  cp.band_cap = kBandCap;
  cp.counts = counts;
  cp.row_status = row_status;
  if (launch_count_bounds(cp, s) != cudaSuccess) return DIFR_ERR_CUDA;

  K1Params k1 = k1_params(pl, T, d, V, temperature, ws);
  k1.tokens = argmax;  // the id the count leaves out
  k1.seeds = seeds; k1.positions = positions;
  k1.bounds = cp.bounds;
  k1.band_count = const_cast<int*>(cp.band_count);
  k1.band_list = const_cast<BandEntry*>(cp.band_list);
  k1.band_cap = kBandCap;
  k1.device_status = device_status;
  if (cudaMemsetAsync(k1.unit_counter, 0, sizeof(int), s) != cudaSuccess) return DIFR_ERR_CUDA;
  if (cudaMemsetAsync(k1.band_count, 0, (size_t)pl.T_pad * sizeof(int), s) != cudaSuccess) return DIFR_ERR_CUDA;
  const int grid = k1_grid(pl, info.pairs);
  if (launch_k1(n_tau == 1 ? 4 : 5, tmap_h, tmap_w, k1, grid, s) != cudaSuccess) return DIFR_ERR_CUDA;
  if (launch_count_finalize(cp, s) != cudaSuccess) return DIFR_ERR_CUDA;
  return DIFR_OK;
}

// ------------------------------------------------- full Token-DiFR estimator
constexpr int kCandCap = 512;      // candidates kept per row when the vocabulary has at least 64 tiles
// Each strip contributes its two largest 16-id group maxima, and the k-th largest of those values bounds the row's
// k-th largest logit from below.  The bound is tight enough to keep the lists short when there are about twice as
// many values as k, i.e. as many strips as k: between 32 and 128 strips, by the largest top_k the call can meet.
constexpr int kFilterFloorStrips = 32;
constexpr int kFilterMinStrips = 64;   // vocabularies with fewer tiles than this list every id instead
constexpr int kFilterMaxStrips = 128;  // the bounds kernel reads at most 128 strips' records per row

// Rows whose logits the filtered calls keep at a time: two gibibytes of fp32 logits (a raster group or so of rows:
// with fewer rows per block the first pass streams W more often and its launches get short).
static int64_t select_block_rows(int64_t V) {
  int64_t rows = (((int64_t)1 << 31) / (4 * V)) & ~(int64_t)255;
  return rows < 256 ? 256 : rows;
}
static int select_chunk_rows(int64_t T_pad, int64_t V) {
  const int64_t rows = select_block_rows(V);
  return (int)(rows > T_pad ? T_pad : rows);
}

// Layout behind the ordinary workspace: per-row candidate counters, the candidate lists, and for filters of any
// size six per-row words of the selection's results and the block of logits it reads.
static bool filtered_layout(int64_t T, int64_t d, int64_t V, int pairs, int min_strips, Plan* pl, int* cap,
                            size_t* count_off, size_t* list_off, size_t* total, size_t* sel_off = nullptr,
                            size_t* logits_off = nullptr) {
  if (!make_plan(T, d, V, pairs, pl, min_strips, kFilterMaxStrips)) return false;
  // with fewer than 64 vocabulary tiles the strips' maxima cannot bound the 128-th largest logit: keep every id
  *cap = (pl->n_tiles < kFilterMinStrips) ? (int)V : kCandCap;
  *count_off = (pl->workspace_bytes + 255) & ~(size_t)255;
  *list_off = *count_off + (((size_t)pl->T_pad * sizeof(int) + 255) & ~(size_t)255);
  const size_t sel = (*list_off + (size_t)T * (size_t)*cap * sizeof(Candidate) + 255) & ~(size_t)255;
  // selection results: three ints and three doubles per padded row, each array 256-byte aligned
  const size_t ints = ((size_t)pl->T_pad * sizeof(int) + 255) & ~(size_t)255;
  const size_t dbls = ((size_t)pl->T_pad * sizeof(double) + 255) & ~(size_t)255;
  const size_t lg = sel + 3 * ints + 3 * dbls;
  if (sel_off) *sel_off = sel;
  if (logits_off) *logits_off = lg;
  *total = lg + (size_t)select_chunk_rows(pl->T_pad, V) * (size_t)V * sizeof(float);
  return true;
}

size_t difr_filtered_workspace_bytes(int64_t T, int64_t d, int64_t V) {
  DeviceInfo info;
  if (!device_info(&info)) info.pairs = 0;
  Plan pl;
  int cap;
  size_t count_off, list_off, total;
  // sized for the most strips a call can ask for
  if (!filtered_layout(T, d, V, info.pairs, kFilterMaxStrips, &pl, &cap, &count_off, &list_off, &total)) return 0;
  // a call that selects over the logits works block by block when T exceeds a block: each block is a call of
  // its own on the same workspace
  const int64_t block = select_block_rows(V);
  if (T > block) {
    size_t t2;
    if (!filtered_layout(block, d, V, info.pairs, kFilterMaxStrips, &pl, &cap, &count_off, &list_off, &t2)) return 0;
    if (t2 > total) total = t2;
    if (T % block != 0) {
      if (!filtered_layout(T % block, d, V, info.pairs, kFilterMaxStrips, &pl, &cap, &count_off, &list_off, &t2))
        return 0;
      if (t2 > total) total = t2;
    }
  }
  return total;
}

// The two filtered estimators share everything but the fused kernel's modes, what the first finalize writes and
// the last kernel: scoring pass (+ the strips' group maxima), ordinary finalize, bounds, collecting pass, finalize
// over the candidate lists.  ipt: 0 Token-DiFR in full, 1 Token-IPT-DiFR on the filtered distribution.
static difr_status filtered_common(int ipt, const void* h, const void* W, const int32_t* tokens,
                                   const uint64_t* seeds, const uint32_t* positions, float temperature, int64_t T,
                                   int64_t d, int64_t V, const difr_filter* filter, difr_out* out,
                                   difr_stream_t stream) {
  if (!h || !W || !tokens || !seeds || !positions || !out || !out->score || !filter) return DIFR_ERR_INVALID_ARG;
  if (T < 0 || d <= 0 || V <= 0) return DIFR_ERR_INVALID_ARG;
  if (!(out->sigma > 0.f) || !(out->eps >= 0.f) || !isfinite(out->sigma) || !isfinite(out->eps))
    return DIFR_ERR_INVALID_ARG;
  // scalars are checked here when they apply to every row; values that come one per row are checked on the
  // device (row_status bit 3).  How top_k and top_p combine is decided per row by the kernels.
  if (out->temperatures == nullptr && (!(temperature > 0.f) || !isfinite(temperature))) return DIFR_ERR_INVALID_ARG;
  if (out->temperatures != nullptr) temperature = 1.f;  // unused
  const int top_k = filter->top_k;
  const float top_p = filter->top_p;
  const int s_comp = ipt ? 0 : filter->s;  // the IPT estimator has no competitors
  if (!ipt && (filter->s < 1 || filter->s > 8)) return DIFR_ERR_INVALID_ARG;
  if (filter->top_k_rows == nullptr && top_k < 0) return DIFR_ERR_INVALID_ARG;
  if (filter->top_p_rows == nullptr && (!(top_p > 0.f) || !(top_p <= 1.f))) return DIFR_ERR_INVALID_ARG;
  const float min_p = filter->min_p;
  if (filter->min_p_rows == nullptr && (!(min_p >= 0.f) || !(min_p <= 1.f))) return DIFR_ERR_INVALID_ARG;
  const bool min_p_on = filter->min_p_rows != nullptr || min_p > 0.f;
  // IPT with one policy for every row that filters nothing: that is difr_score_ipt
  if (ipt && filter->top_k_rows == nullptr && filter->top_p_rows == nullptr && !min_p_on &&
      (top_k < 1 || top_k >= V) && top_p >= 1.f && V > 128)
    return DIFR_ERR_INVALID_ARG;
  if ((d % 8) != 0 || V < 2) return DIFR_ERR_SHAPE;
  if (T == 0) return DIFR_OK;
  DeviceInfo info;
  if (!device_info(&info)) return DIFR_ERR_CUDA;
  if (info.major != 10) return DIFR_ERR_ARCH;
  Plan pl;
  int cap;
  size_t count_off, list_off, total, sel_off, logits_off;
  // One policy for the whole call whose kept set can exceed what the candidate lists resolve (a top-k above
  // 128, a nucleus or a min-p set over the whole vocabulary): the kept prefix is found by selection over the
  // rows' logits, written out a block of rows at a time.  Per-row policies stay within the lists' reach unless
  // the caller asks for the selection (any_size), which then resolves every row.
  const bool scalar_policy = !filter->top_k_rows && !filter->top_p_rows && !filter->min_p_rows;
  const bool whole_vocab = top_k < 1 || top_k >= V;
  const bool select_path =
      V > 128 && (scalar_policy ? ((!whole_vocab && top_k > 128) || (whole_vocab && top_p < 1.f) ||
                                   (ipt && whole_vocab && min_p > 0.f))
                                : filter->any_size != 0);
  if (T > select_block_rows(V)) {
    // block by block, each a call of its own on the same workspace (stream order keeps them apart): a block's
    // logits, written by its first pass, are what its selection and its collecting pass read
    if (!out->workspace || !aligned16(out->workspace) || !aligned16(h) || !aligned16(W)) {
      return !out->workspace ? DIFR_ERR_WORKSPACE : DIFR_ERR_ALIGN;
    }
    if (out->workspace_bytes < difr_filtered_workspace_bytes(T, d, V)) return DIFR_ERR_WORKSPACE;
    const int64_t block = select_block_rows(V);
    for (int64_t r0 = 0; r0 < T; r0 += block) {
      const int64_t rows = T - r0 < block ? T - r0 : block;
      difr_out o = *out;
      difr_filter f = *filter;
      auto shift = [r0](auto*& ptr) { if (ptr != nullptr) ptr += r0; };
      shift(o.score); shift(o.margin); shift(o.argmax); shift(o.runner_up); shift(o.lse); shift(o.p_claimed);
      shift(o.cdf_lo); shift(o.u); shift(o.row_status); shift(o.rank); shift(o.y_max); shift(o.y_second);
      shift(o.score_ipt); shift(o.cutoff); shift(o.temperatures);
      shift(f.top_k_rows); shift(f.top_p_rows); shift(f.min_p_rows);
      const difr_status rc = filtered_common(
          ipt, static_cast<const unsigned char*>(h) + (size_t)r0 * (size_t)d * 2, W, tokens + r0, seeds + r0,
          positions + r0, temperature, rows, d, V, &f, &o, stream);
      if (rc != DIFR_OK) return rc;
    }
    return DIFR_OK;
  }
  // the largest number of ids any row resolves by logit rank (a nucleus without a top-k resolves 128)
  int k_max = 128;
  if (select_path) {
    k_max = (min_p_on && !ipt) ? 1 : 0;
  } else if (filter->top_k_rows == nullptr) {
    if (!whole_vocab) k_max = top_k;
    else if (filter->top_p_rows == nullptr && top_p >= 1.f) k_max = (min_p_on && ipt) ? 128 : 0;
  }
  const int min_strips =
      k_max < kFilterFloorStrips ? kFilterFloorStrips : (k_max > kFilterMaxStrips ? kFilterMaxStrips : k_max);
  if (!filtered_layout(T, d, V, info.pairs, min_strips, &pl, &cap, &count_off, &list_off, &total, &sel_off,
                       &logits_off))
    return DIFR_ERR_SHAPE;
  if (!aligned16(h) || !aligned16(W)) return DIFR_ERR_ALIGN;
  if (!out->workspace || out->workspace_bytes < total) return DIFR_ERR_WORKSPACE;
  if (!aligned16(out->workspace)) return DIFR_ERR_ALIGN;
  CUtensorMap tmap_h, tmap_w;
  if (!make_tmap(&tmap_h, h, T, d, kBM) || !make_tmap(&tmap_w, W, V, d, kBN / 2)) return DIFR_ERR_CUDA;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  unsigned char* ws = static_cast<unsigned char*>(out->workspace);
  const int grid = k1_grid(pl, info.pairs);

  // ---- first pass: the ordinary scoring pass, which also leaves each strip's two largest group maxima
  K1Params k1 = k1_params(pl, T, d, V, temperature, ws);
  k1.tokens = tokens; k1.seeds = seeds; k1.positions = positions;
  k1.device_status = out->device_status;
  k1.temperatures = out->temperatures;
  if (cudaMemsetAsync(k1.unit_counter, 0, sizeof(int), s) != cudaSuccess) return DIFR_ERR_CUDA;
  k1.logits_out = reinterpret_cast<float*>(ws + logits_off);  // for the selection and the collecting pass below
  if (launch_k1(ipt ? 8 : 6, tmap_h, tmap_w, k1, grid, s) != cudaSuccess) return DIFR_ERR_CUDA;
  k1.logits_out = nullptr;

  // ---- the ordinary finalize: the unfiltered outputs (and, for a row without a filter, the IPT score)
  K2Params k2;
  memset(&k2, 0, sizeof k2);
  k2.h = reinterpret_cast<const uint16_t*>(h); k2.W = reinterpret_cast<const uint16_t*>(W);
  k2.tokens = tokens; k2.seeds = seeds; k2.positions = positions;
  k2.partials = k1.partials; k2.n_slots = pl.n_slots; k2.T_pad = pl.T_pad;
  k2.T = (int)T; k2.d = (int)d; k2.V = (int)V; k2.ipt = ipt;
  k2.temperature = temperature; k2.sigma = out->sigma; k2.eps = out->eps; k2.c1 = k1.c1;
  k2.score = out->score; k2.lse = out->lse; k2.row_status = out->row_status;
  k2.temperatures = out->temperatures;
  if (ipt) {
    k2.p_claimed = out->p_claimed; k2.cdf_lo = out->cdf_lo; k2.u = out->u;
  } else {
    k2.margin = out->margin; k2.argmax = out->argmax; k2.runner_up = out->runner_up;
    k2.y_max = out->y_max; k2.y_second = out->y_second;
  }
  if (launch_k2(k2, s) != cudaSuccess) return DIFR_ERR_CUDA;

  // ---- bounds (on y' for the competitors, on the logit for the filter), collecting pass, finalize over the lists
  FilterParams fp;
  memset(&fp, 0, sizeof fp);
  fp.h = k2.h; fp.W = k2.W; fp.tokens = tokens; fp.seeds = seeds; fp.positions = positions;
  fp.partials = k1.partials; fp.n_slots = pl.n_slots; fp.T_pad = pl.T_pad; fp.T = (int)T; fp.d = (int)d; fp.V = (int)V;
  fp.temperature = temperature; fp.sigma = out->sigma; fp.eps = out->eps; fp.c1 = k1.c1;
  fp.top_k = top_k; fp.top_p = top_p; fp.s = s_comp; fp.ipt = ipt;
  fp.top_k_rows = filter->top_k_rows; fp.top_p_rows = filter->top_p_rows; fp.temperatures = out->temperatures;
  fp.min_p = min_p; fp.min_p_rows = filter->min_p_rows;
  fp.bounds = reinterpret_cast<float*>(ws + pl.bounds_offset);
  fp.cand_list = reinterpret_cast<const Candidate*>(ws + list_off);
  fp.cand_count = reinterpret_cast<const int*>(ws + count_off);
  fp.cand_cap = cap;
  fp.score = out->score; fp.cutoff = out->cutoff; fp.row_status = out->row_status;
  if (ipt) {
    fp.p_claimed = out->p_claimed; fp.cdf_lo = out->cdf_lo; fp.u = out->u;
  }
  if (select_path) {
    // ---- the selection over the rows' logits (written by the first pass; T fits one block here)
    const size_t ints = ((size_t)pl.T_pad * sizeof(int) + 255) & ~(size_t)255;
    const size_t dbls = ((size_t)pl.T_pad * sizeof(double) + 255) & ~(size_t)255;
    int* sel_cut = reinterpret_cast<int*>(ws + sel_off);
    int* sel_top = reinterpret_cast<int*>(ws + sel_off + ints);
    int* sel_n = reinterpret_cast<int*>(ws + sel_off + 2 * ints);
    double* sel_z = reinterpret_cast<double*>(ws + sel_off + 3 * ints);
    double* sel_below = reinterpret_cast<double*>(ws + sel_off + 3 * ints + dbls);
    double* sel_mine = reinterpret_cast<double*>(ws + sel_off + 3 * ints + 2 * dbls);
    SelectParams sp;
    memset(&sp, 0, sizeof sp);
    sp.logits = reinterpret_cast<const float*>(ws + logits_off); sp.rows = (int)T; sp.V = (int)V; sp.row0 = 0;
    sp.tokens = tokens; sp.temperatures = out->temperatures; sp.temperature = temperature;
    sp.top_k = top_k; sp.top_p = top_p;
    sp.min_p = ipt ? min_p : 0.f;  // Token-DiFR takes the min-p bound itself as cutoff (exact l_max, below)
    sp.top_k_rows = filter->top_k_rows; sp.top_p_rows = filter->top_p_rows;
    sp.min_p_rows = ipt ? filter->min_p_rows : nullptr;
    sp.cut_id = sel_cut; sp.top_id = sel_top; sp.kept_n = sel_n;
    sp.kept_z = sel_z; sp.kept_below = sel_below; sp.kept_mine = sel_mine;
    sp.want_sums = ipt;
    sp.row_status = out->row_status;
    if (launch_select_cutoff(sp, s) != cudaSuccess) return DIFR_ERR_CUDA;
    fp.sel_cut_id = sel_cut; fp.sel_top_id = sel_top; fp.sel_kept_n = sel_n;
    fp.sel_z = sel_z; fp.sel_below = sel_below; fp.sel_mine = sel_mine;
    if (ipt) {
      // the selection has summed the kept set: no candidate lists are needed
      if (launch_ipt_select_finalize(fp, s) != cudaSuccess) return DIFR_ERR_CUDA;
      return DIFR_OK;
    }
  }
  if (launch_filter_bounds(fp, s) != cudaSuccess) return DIFR_ERR_CUDA;
  if (cudaMemsetAsync(ws + count_off, 0, (size_t)pl.T_pad * sizeof(int), s) != cudaSuccess) return DIFR_ERR_CUDA;
  if (!ipt && out->rank != nullptr) {
    // the raw-logit rank of the claimed token rides on the collecting pass: claimed logits into the third
    // plane of the bounds, the counts added up in out->rank
    if (launch_claimed_logits(k2.h, k2.W, tokens, (int)T, (int)d, (int)V, fp.bounds + 2 * (size_t)pl.T_pad,
                              fp.bounds + (size_t)kBandPlane * (size_t)pl.T_pad, s) != cudaSuccess)
      return DIFR_ERR_CUDA;
    if (cudaMemsetAsync(out->rank, 0, (size_t)T * sizeof(int32_t), s) != cudaSuccess) return DIFR_ERR_CUDA;
    k1.rank_out = out->rank;
    fp.rank = out->rank;
  }
  k1.bounds = fp.bounds;
  k1.cand_list = ws + list_off;
  k1.cand_count = reinterpret_cast<int*>(ws + count_off);
  k1.cand_cap = cap;
  // (the collecting modes' epilogue over the stored logits: no second contraction)
  if (launch_collect_from_logits(ipt ? 9 : 7, k1, reinterpret_cast<const float*>(ws + logits_off), s) != cudaSuccess)
    return DIFR_ERR_CUDA;
  if ((ipt ? launch_ipt_filtered_finalize(fp, s) : launch_filtered_finalize(fp, s)) != cudaSuccess)
    return DIFR_ERR_CUDA;
  return DIFR_OK;
}

difr_status difr_score_gm_filtered(const void* h, const void* W, const int32_t* tokens, const uint64_t* seeds,
                                   const uint32_t* positions, float temperature, int64_t T, int64_t d, int64_t V,
                                   const difr_filter* filter, difr_out* out, difr_stream_t stream) {
  return filtered_common(0, h, W, tokens, seeds, positions, temperature, T, d, V, filter, out, stream);
}

difr_status difr_score_ipt_filtered(const void* h, const void* W, const int32_t* tokens, const uint64_t* seeds,
                                    const uint32_t* positions, float temperature, int64_t T, int64_t d, int64_t V,
                                    const difr_filter* filter, difr_out* out, difr_stream_t stream) {
  return filtered_common(1, h, W, tokens, seeds, positions, temperature, T, d, V, filter, out, stream);
}

difr_status difr_exfiltratable_bits(const uint8_t* classes, const int32_t* counts, int32_t rank_cutoff, int64_t V,
                                    const int32_t* seq_offsets, int64_t n_seq, int64_t T, float* bits,
                                    float* seq_bits, difr_stream_t stream) {
  if (!classes || !counts || T < 0 || n_seq < 0 || V < 1 || rank_cutoff < 1) return DIFR_ERR_INVALID_ARG;
  if (seq_offsets && n_seq == 0) return DIFR_OK;
  BitsParams p;
  memset(&p, 0, sizeof p);
  p.classes = classes; p.counts = counts; p.seq_offsets = seq_offsets; p.n_seq = n_seq; p.T = T;
  p.log2_r = (float)log2((double)rank_cutoff); p.log2_v = (float)log2((double)V);
  p.bits = bits; p.seq_bits = seq_bits;
  if (launch_bits(p, reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess) return DIFR_ERR_CUDA;
  return DIFR_OK;
}

difr_status difr_expand_seeds(const uint64_t* seeds, const int32_t* tokens, const int32_t* seq_offsets,
                              int64_t n_seq, const uint64_t* prompt_hashes, int64_t T, uint64_t* expanded,
                              difr_stream_t stream) {
  if (!seeds || !tokens || !expanded || T < 0 || n_seq < 0 || T >= (1ll << 31) || n_seq >= (1ll << 31))
    return DIFR_ERR_INVALID_ARG;
  if (T == 0 || (seq_offsets && n_seq == 0)) return DIFR_OK;
  if (launch_expand_seeds(seeds, tokens, seq_offsets, prompt_hashes, n_seq, T, expanded,
                          reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess)
    return DIFR_ERR_CUDA;
  return DIFR_OK;
}

difr_status difr_detect(const float* scores, float threshold, const float* margins, const int32_t* ranks,
                        int32_t rank_cutoff, const int32_t* seq_offsets, int64_t n_seq, int64_t T, uint8_t* flags,
                        difr_seq_stats* seq_stats, difr_stream_t stream) {
  if (!scores || T < 0 || n_seq < 0) return DIFR_ERR_INVALID_ARG;
  if (isnan(threshold)) return DIFR_ERR_INVALID_ARG;
  if (seq_offsets && n_seq == 0) return DIFR_OK;
  if (!seq_offsets && T == 0 && !seq_stats) return DIFR_OK;
  K3Params p;
  memset(&p, 0, sizeof p);
  p.scores = scores; p.margins = margins; p.ranks = ranks; p.seq_offsets = seq_offsets;
  p.threshold = threshold; p.rank_cutoff = rank_cutoff; p.n_seq = n_seq; p.T = T;
  p.flags = flags; p.seq_stats = seq_stats;
  if (launch_k3(p, reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess) return DIFR_ERR_CUDA;
  return DIFR_OK;
}

difr_status difr_logits(const void* h, const void* W, int64_t T, int64_t d, int64_t V, float* logits,
                        int32_t* device_status, difr_stream_t stream) {
  if (!h || !W || !logits || T < 0 || d <= 0 || V <= 0) return DIFR_ERR_INVALID_ARG;
  if ((d % 8) != 0 || V < 2) return DIFR_ERR_SHAPE;
  if (T == 0) return DIFR_OK;
  DeviceInfo info;
  if (!device_info(&info)) return DIFR_ERR_CUDA;
  if (info.major != 10) return DIFR_ERR_ARCH;
  Plan pl;
  if (!make_plan(T, d, V, info.pairs, &pl)) return DIFR_ERR_SHAPE;
  if (!aligned16(h) || !aligned16(W)) return DIFR_ERR_ALIGN;
  CUtensorMap tmap_h, tmap_w;
  if (!make_tmap(&tmap_h, h, T, d, kBM) || !make_tmap(&tmap_w, W, V, d, kBN / 2)) return DIFR_ERR_CUDA;
  K1Params k1 = k1_params(pl, T, d, V, 1.f, nullptr);  // no counter: units go round robin
  k1.logits_out = logits; k1.device_status = device_status;
  const int grid = k1_grid(pl, info.pairs);
  if (launch_k1(2, tmap_h, tmap_w, k1, grid, reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess)
    return DIFR_ERR_CUDA;
  return DIFR_OK;
}

difr_status difr_philox(const uint32_t* ctr, const uint32_t* key, int64_t n, uint32_t* out, difr_stream_t stream) {
  if (n < 0 || (n > 0 && (!ctr || !key || !out))) return DIFR_ERR_INVALID_ARG;
  if (launch_philox(ctr, key, n, out, reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess) return DIFR_ERR_CUDA;
  return DIFR_OK;
}

// ------------------------------------------------------- allocation-free entry
// Scratch for difr_score_gm_static: a fixed array inside the library's device
// image, so the caller never has to obtain workspace memory.
constexpr size_t kStaticScratchBytes = (size_t)DIFR_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// In host code `g_static_scratch` only names the symbol; the device address has
// to be asked for, once per device, while that device is current.
static difr_status static_scratch_address(void** ptr) {
  constexpr int kMaxDevices = 64;
  static std::atomic<void*> cached[kMaxDevices];  // host threads may call concurrently
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return DIFR_ERR_CUDA;
  if (dev >= 0 && dev < kMaxDevices) {
    void* known = cached[dev].load(std::memory_order_relaxed);
    if (known != nullptr) {
      *ptr = known;
      return DIFR_OK;
    }
  }
  void* p = nullptr;
  if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return DIFR_ERR_CUDA;
  if (dev >= 0 && dev < kMaxDevices) cached[dev].store(p, std::memory_order_relaxed);  // same value whoever is first
  *ptr = p;
  return DIFR_OK;
}

difr_status difr_score_gm_static(const void* h, const void* W, const int32_t* tokens, const uint64_t* seeds,
                                 const uint32_t* positions, float temperature, int64_t T, int64_t d, int64_t V,
                                 difr_out* out, difr_stream_t stream) {
  if (!out) return DIFR_ERR_INVALID_ARG;
  if (T > 0 && d > 0 && V > 0) {
    DeviceInfo info;
    Plan pl;
    if (device_info(&info) && make_plan(T, d, V, info.pairs, &pl) && pl.workspace_bytes > kStaticScratchBytes)
      return DIFR_ERR_WORKSPACE;  // problem too large for the built-in scratch: use difr_score_gm
  }
  void* scratch = nullptr;
  const difr_status st = static_scratch_address(&scratch);
  if (st != DIFR_OK) return st;
  difr_out local = *out;
  local.workspace = scratch;
  local.workspace_bytes = kStaticScratchBytes;
  return score_common(0, h, W, tokens, seeds, positions, temperature, T, d, V, &local, stream);
}

difr_status difr_debug_plan_override(int32_t strips, int32_t group, int32_t l2_mb) {
  if (strips < 0 || group < 0 || l2_mb < 0) return DIFR_ERR_INVALID_ARG;
  plan_override_word(0).store(strips, std::memory_order_relaxed);
  plan_override_word(1).store(group, std::memory_order_relaxed);
  plan_override_word(2).store(l2_mb, std::memory_order_relaxed);
  return DIFR_OK;
}

difr_status difr_selftest_wait(int32_t* status2, int64_t limit_cycles, difr_stream_t stream) {
  if (!status2 || limit_cycles < 1 || limit_cycles > 1000000000LL) return DIFR_ERR_INVALID_ARG;
  if (launch_wait_selftest(status2, (long long)limit_cycles, reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess)
    return DIFR_ERR_CUDA;
  return DIFR_OK;
}

const char* difr_status_string(difr_status status) {
  switch (status) {
    case DIFR_OK: return "ok";
    case DIFR_ERR_INVALID_ARG: return "invalid argument";
    case DIFR_ERR_SHAPE: return "unsupported shape";
    case DIFR_ERR_ALIGN: return "pointer not 16-byte aligned";
    case DIFR_ERR_WORKSPACE: return "workspace missing or too small";
    case DIFR_ERR_CUDA: return "CUDA call failed";
    case DIFR_ERR_ARCH: return "device is not compute capability 10.x";
    case DIFR_ERR_TIMEOUT: return "a device-side wait ran out";
  }
  return "unknown status";
}

int difr_version(void) { return 221; }

}  // extern "C"
