// Host-side work decomposition of the fused scoring kernel, shared by the
// launcher and the finalize kernel's launcher (both must agree on the number
// of partial slots per row).
#pragma once
#include <stddef.h>
#include <stdint.h>

#include <atomic>
#include <functional>
#include <mutex>
#include <queue>
#include <vector>

namespace difr {

constexpr int kBM = 128;        // rows (tokens) per CTA tile
constexpr int kPairM = 2 * kBM;  // rows per CTA pair: the two CTAs of a pair share one 256 x 256 MMA
constexpr int kBN = 256;        // vocabulary ids per tile
constexpr int kBK = 64;         // hidden-dimension slice per pipeline stage (128 bytes of bf16)
constexpr int kPlanBoundPlanes = 6;  // per-row bounds of the rank / counting / collecting passes (see K1Params);
                                     // the last plane holds the rows' running floors of the scoring pass
constexpr int kPlanBandCap = 64;     // per-row list of ids that fp32 cannot decide (kBandCap)

struct Plan {
  int m_tiles;   // ceil(T / 256): row tiles of a CTA pair
  int n_tiles;   // ceil(V / 256)
  int k_steps;   // ceil(d / 64)
  int S;         // vocabulary strips: a work unit is (m tile, strip)
  int Gm;        // m tiles per raster group (units of a group run back to back)
  int n_units;   // m_tiles * S
  int T_pad;     // m_tiles * 256
  int n_slots;   // partial records per row: one per strip
  size_t partial_bytes;
  size_t bounds_offset;  // [6][T_pad] floats behind the records and the 256-byte tail (unit counter)
  size_t band_count_offset;  // [T_pad] ints: entries in each row's list of undecided ids
  size_t band_list_offset;   // [T_pad][kPlanBandCap] entries of 8 bytes
  size_t workspace_bytes;
};

// Overrides of the planner's choices, for validation sweeps only (difr_debug_plan_override): 0 = the planner's own
// value.  Process-wide; part of the plan cache's key.
struct PlanOverride {
  int strips;    // number of vocabulary strips S
  int group;     // row tiles per raster group Gm
  int l2_mb;     // megabytes of h per raster group that the planner aims at (default 40)
};
inline std::atomic<int>& plan_override_word(int i) {
  static std::atomic<int> words[3];
  return words[i];
}
inline PlanOverride plan_override() {
  PlanOverride o;
  o.strips = plan_override_word(0).load(std::memory_order_relaxed);
  o.group = plan_override_word(1).load(std::memory_order_relaxed);
  o.l2_mb = plan_override_word(2).load(std::memory_order_relaxed);
  return o;
}

// Tile times until the last pair is done when the units (in raster order, each as long as its strip, plus
// a small fixed cost per unit) are taken on demand by `num_pairs` pairs that all start together.
inline double makespan_tiles(int m_tiles, int n_tiles, int S, int gm, int num_pairs) {
  std::priority_queue<double, std::vector<double>, std::greater<double>> free_at;
  for (int i = 0; i < num_pairs; ++i) free_at.push(0.0);
  double last = 0.0;
  for (int m0 = 0; m0 < m_tiles; m0 += gm) {
    const int cnt = (m_tiles - m0 < gm) ? m_tiles - m0 : gm;
    for (int strip = 0; strip < S; ++strip) {
      const int n0 = (int)(((long long)strip * n_tiles) / S), n1 = (int)(((long long)(strip + 1) * n_tiles) / S);
      for (int i = 0; i < cnt; ++i) {
        const double t = free_at.top() + (double)(n1 - n0) + 0.05;
        free_at.pop();
        free_at.push(t);
        if (t > last) last = t;
      }
    }
  }
  return last;
}

// A unit walks its strip tile by tile keeping running statistics in registers and
// leaves one partial record per (row, strip).  Units are handed out in
// raster order: groups of Gm row tiles, inside a group strip by strip, inside a strip
// row tile by row tile.  The pairs that run at the same time therefore share Gm row
// tiles of h (each re-read once per vocabulary tile) and stream the same few strips of
// W.  Pairs on one strip start within about Gm * len / pairs tiles of one another, so a
// W tile has to survive in L2 for that long: the strip length `len` and Gm are sized so
// that the h tiles of a group plus the W tiles in flight stay within a part of L2.
// `num_pairs` is the number of CTA pairs resident at once (one persistent pair per two SMs).
// `min_strips` > 0 asks for at least that many strips (fewer only if there are fewer vocabulary tiles),
// `max_strips` > 0 for at most that many (the strips grow longer instead).
inline bool compute_plan(int64_t T, int64_t d, int64_t V, int num_pairs, Plan* out, int min_strips, int max_strips,
                         const PlanOverride& ov) {
  if (T <= 0 || d <= 0 || V < 2 || (d % 8) != 0) return false;
  // (tile origins n * 256 and row origins m * 256 are 32-bit in the kernels: leave room for the last tile's padding)
  if (T > (int64_t)1 << 30 || V > ((int64_t)1 << 31) - 1024 || d > (int64_t)1 << 20) return false;
  Plan p;
  p.m_tiles = (int)((T + kPairM - 1) / kPairM);
  p.n_tiles = (int)((V + kBN - 1) / kBN);
  p.k_steps = (int)((d + kBK - 1) / kBK);
  if (num_pairs <= 0) num_pairs = 74;
  // Measured on B200 (126 MB of L2): about 40 MB of h per raster group (larger groups push W out of L2 before
  // its strip is done with it), and strips whose W tiles hold about 12288 k-columns between them (two tiles at
  // d = 5120, six at d = 2048).  The pairs that share a strip drift apart by up to one unit, so a shorter strip
  // keeps fewer W tiles waiting in L2 for the last pair (at d = 5120, eight-tile strips re-read W 2.2 times per
  // group, two-tile strips 1.2 times, and the DRAM power saved shows as clock under the power cap: 3 % at
  // T = 65536); below that length the hand-over between units and the extra records cost more than they save.
  const double tile_bytes = 2.0 * kPairM * (double)d;  // one 256-row tile of h or of W
  const double group_bytes = (double)(ov.l2_mb > 0 ? ov.l2_mb : 40) * 1048576.0;
  int gm = (int)(group_bytes / tile_bytes);
  if (gm < 4) gm = 4;
  int len_target = (int)((12288 + d / 2) / d);
  if (len_target < 1) len_target = 1;
  if (len_target > 8) len_target = 8;
  if (len_target > p.n_tiles) len_target = p.n_tiles;
  // strip count: n_tiles / len_target when there are many rounds of units; otherwise the count near it
  // (or, for small problems, up to one unit per pair) whose on-demand schedule finishes first
  int best_S = (p.n_tiles + len_target - 1) / len_target;
  if ((long long)p.m_tiles * best_S < 64LL * num_pairs) {
    int s_lo = (2 * p.n_tiles + 3 * len_target - 1) / (3 * len_target);
    int s_hi = (4 * p.n_tiles + 3 * len_target - 1) / (3 * len_target);
    if (s_hi < num_pairs / p.m_tiles) s_hi = num_pairs / p.m_tiles;
    if (s_hi > p.n_tiles) s_hi = p.n_tiles;
    if (s_lo < 1) s_lo = 1;
    if (s_lo > s_hi) s_lo = s_hi;
    double best_cost = 1e300;
    for (int S = s_lo; S <= s_hi; ++S) {
      const double cost = makespan_tiles(p.m_tiles, p.n_tiles, S, gm, num_pairs) + 0.02 * S;
      if (cost < best_cost - 1e-9) {
        best_cost = cost;
        best_S = S;
      }
    }
  }
  if (best_S < min_strips) best_S = min_strips;
  if (max_strips > 0 && best_S > max_strips) best_S = max_strips;
  p.S = ov.strips > 0 ? ov.strips : best_S;
  if (p.S < 1) p.S = 1;
  if (p.S > p.n_tiles) p.S = p.n_tiles;
  if (ov.group > 0) gm = ov.group;
  if (gm < 1) gm = 1;
  p.Gm = gm < p.m_tiles ? gm : p.m_tiles;
  if ((long long)p.m_tiles * p.S > 0x7fffffffLL) return false;  // unit ids are 32-bit
  p.n_units = p.m_tiles * p.S;
  p.T_pad = p.m_tiles * kPairM;
  p.n_slots = p.S;
  p.partial_bytes = (size_t)p.n_slots * (size_t)p.T_pad * 32;
  p.bounds_offset = p.partial_bytes + 256;
  p.band_count_offset = p.bounds_offset + (size_t)kPlanBoundPlanes * (size_t)p.T_pad * sizeof(float);
  p.band_list_offset = p.band_count_offset + (size_t)p.T_pad * sizeof(int);
  p.workspace_bytes = p.band_list_offset + (size_t)p.T_pad * (size_t)kPlanBandCap * 8;
  *out = p;
  return true;
}

// The plan of a problem, remembered: small problems pick their strip count by simulating the on-demand schedule
// for a few dozen candidates, which costs about a millisecond of host time, and callers score the same shapes
// over and over.  A short most-recently-used list under a mutex (a hit costs a lock and a few compares).
inline bool make_plan(int64_t T, int64_t d, int64_t V, int num_pairs, Plan* out, int min_strips = 0,
                      int max_strips = 0) {
  struct Entry {
    int64_t T, d, V;
    int pairs, min_strips, max_strips;
    PlanOverride ov;
    Plan plan;
  };
  constexpr size_t kEntries = 32;
  static std::mutex mu;
  static std::vector<Entry> cache;  // most recently used first
  const PlanOverride ov = plan_override();
  {
    std::lock_guard<std::mutex> lock(mu);
    for (size_t i = 0; i < cache.size(); ++i) {
      const Entry& e = cache[i];
      if (e.T == T && e.d == d && e.V == V && e.pairs == num_pairs && e.min_strips == min_strips &&
          e.max_strips == max_strips && e.ov.strips == ov.strips && e.ov.group == ov.group &&
          e.ov.l2_mb == ov.l2_mb) {
        *out = e.plan;
        if (i != 0) {
          const Entry hit = e;
          cache.erase(cache.begin() + (long)i);
          cache.insert(cache.begin(), hit);
        }
        return true;
      }
    }
  }
  Plan p;
  if (!compute_plan(T, d, V, num_pairs, &p, min_strips, max_strips, ov)) return false;
  {
    std::lock_guard<std::mutex> lock(mu);
    if (cache.size() >= kEntries) cache.pop_back();
    cache.insert(cache.begin(), Entry{T, d, V, num_pairs, min_strips, max_strips, ov, p});
  }
  *out = p;
  return true;
}

}  // namespace difr
