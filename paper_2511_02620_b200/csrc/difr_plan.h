// Host-side work decomposition of the fused scoring kernel, shared by the
// launcher and the finalize kernel's launcher (both must agree on the number
// of partial slots per row).
#pragma once
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>

namespace difr {

constexpr int kBM = 128;        // rows (tokens) per CTA tile
constexpr int kPairM = 2 * kBM;  // rows per CTA pair: the two CTAs of a pair share one 256 x 256 MMA
constexpr int kBN = 256;        // vocabulary ids per tile
constexpr int kBK = 64;         // hidden-dimension slice per pipeline stage (128 bytes of bf16)

struct Plan {
  int m_tiles;   // ceil(T / 256): row tiles of a CTA pair
  int n_tiles;   // ceil(V / 256)
  int k_steps;   // ceil(d / 64)
  int S;         // vocabulary strips: a work unit is (m tile, strip)
  int Gm;        // m tiles per raster group (units of a group run back to back)
  int n_units;   // m_tiles * S
  int T_pad;     // m_tiles * 256
  int n_slots;   // partial records per row: 2 column halves per strip
  size_t partial_bytes;
  size_t workspace_bytes;
};

inline int env_int(const char* name, int fallback) {
  const char* v = getenv(name);
  return (v && *v) ? atoi(v) : fallback;
}

// A unit walks its strip tile by tile keeping running statistics in registers,
// so more strips mean more partial records but better balance over the SMs.
// Pick the strip count that minimises the number of tiles on the critical path.
// `num_pairs` is the number of CTA pairs resident at once (one persistent pair per two SMs).
inline bool make_plan(int64_t T, int64_t d, int64_t V, int num_pairs, Plan* out) {
  if (T <= 0 || d <= 0 || V < 2 || (d % 8) != 0) return false;
  if (T > (int64_t)1 << 30 || V >= (int64_t)1 << 31 || d > (int64_t)1 << 20) return false;
  Plan p;
  p.m_tiles = (int)((T + kPairM - 1) / kPairM);
  p.n_tiles = (int)((V + kBN - 1) / kBN);
  p.k_steps = (int)((d + kBK - 1) / kBK);
  if (num_pairs <= 0) num_pairs = 74;
  int best_S = 1;
  double best_cost = 1e300;
  int max_S = p.n_tiles < 64 ? p.n_tiles : 64;
  for (int S = 1; S <= max_S; ++S) {
    long long units = (long long)p.m_tiles * S;
    long long waves = (units + num_pairs - 1) / num_pairs;
    long long len = (p.n_tiles + S - 1) / S;
    double cost = (double)waves * (double)len + 0.25 * (double)waves;
    if (cost < best_cost - 1e-9) {
      best_cost = cost;
      best_S = S;
    }
  }
  p.S = env_int("DIFR_DEBUG_STRIPS", best_S);
  if (p.S < 1) p.S = 1;
  if (p.S > p.n_tiles) p.S = p.n_tiles;
  // Units of one raster group share their W tiles through L2 while each keeps
  // its own h tile resident: bound the group's h footprint to a few tens of MB.
  int gm = (d <= 2560) ? 37 : 19;
  gm = env_int("DIFR_DEBUG_GROUP", gm);
  if (gm < 1) gm = 1;
  p.Gm = gm < p.m_tiles ? gm : p.m_tiles;
  p.n_units = p.m_tiles * p.S;
  p.T_pad = p.m_tiles * kPairM;
  p.n_slots = 2 * p.S;
  p.partial_bytes = (size_t)p.n_slots * (size_t)p.T_pad * 32;
  p.workspace_bytes = p.partial_bytes + 256;
  *out = p;
  return true;
}

}  // namespace difr
