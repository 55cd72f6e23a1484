// Host-side pieces of the library: byte model (Eq. (1)), cap policy (Sec. 5), eps^2(b) calibration
// (Eq. (2)), and the Lagrangian dual solved by bisection (Eq. (3), (4)).  No CUDA in this header.
#pragma once
#include <cmath>
#include <cstdint>
#include <limits>
#include <vector>
#include <cuda_fp16.h>
#include "common.cuh"
#include "../../include/jolt.h"

namespace jolt {

inline int64_t cell_bytes(int64_t m, int64_t T, int64_t d, int64_t r_t, int64_t r_f, int64_t bits, bool scales) {
  int64_t s = (m * r_t * r_f + T * r_t + d * r_f) * 2 + (bits * m * T * d) / 8;
  if (bits > 0 && scales) s += 2 * (m * T * d) / kGroup;
  return s;
}

inline int cap_policy(int T, double ratio) {
  const int q_min = ratio <= 4.0 ? 32 : 64;
  int v = (T + 31) / 32;
  if (v < q_min) v = q_min;
  return v > 512 ? 512 : v;
}

// Host restatement of the quantiser for the calibration only (mid-rise, absmax, fp16 step).
inline void host_quant_roundtrip(const double *x, int n, int bits, double *xh) {
  const float half_levels = (float)(1 << (bits - 1));
  for (int g0 = 0; g0 < n; g0 += kGroup) {
    float a = 0.f;
    for (int j = 0; j < kGroup; ++j) a = fmaxf(a, fabsf((float)x[g0 + j]));
    const float delta = __half2float(__float2half_rn(a * (1.0f / half_levels)));
    const float inv = delta == 0.f ? 0.f : 1.0f / delta;
    for (int j = 0; j < kGroup; ++j) {
      float q = floorf((float)x[g0 + j] * inv);
      q = fminf(fmaxf(q, -half_levels), half_levels - 1.0f) + half_levels;
      if (delta == 0.f) q = half_levels;
      xh[g0 + j] = (double)delta * ((double)q - half_levels + 0.5);
    }
  }
}

inline void eps2_calibration(double out[9]) {
  const int n = 1 << 20;
  std::vector<double> g(n), gh(n);
  const uint64_t base = stream_base(0, 0, STREAM_EPS);
  double tot = 0;
  for (int i = 0; i < n; ++i) { g[i] = gaussian_from_u64(mix64(base + (uint64_t)i)); tot += g[i] * g[i]; }
  for (int b = 0; b <= 8; ++b) out[b] = std::numeric_limits<double>::quiet_NaN();
  out[0] = 1.0;
  const int widths[5] = {1, 2, 3, 4, 8};
  for (int b : widths) {
    host_quant_roundtrip(g.data(), n, b, gh.data());
    double e = 0;
    for (int i = 0; i < n; ++i) { const double d = g[i] - gh[i]; e += d * d; }
    out[b] = e / tot;
  }
}

struct CellOptions {
  std::vector<double> err, cost;
  std::vector<jolt_cell_plan> trip;
};

inline size_t argmin_lagrangian(const CellOptions &c, double lam) {
  size_t best = 0;
  double bv = c.err[0] + lam * c.cost[0];
  for (size_t i = 1; i < c.err.size(); ++i) {
    const double v = c.err[i] + lam * c.cost[i];
    if (v < bv || (v == bv && c.cost[i] < c.cost[best])) { best = i; bv = v; }
  }
  return best;
}

// Returns false when even the cheapest allocation exceeds the budget (choice = cheapest).
inline bool dual_allocate(const std::vector<CellOptions> &cells, double budget, std::vector<size_t> &choice,
                          double &total) {
  auto solve = [&](double lam, std::vector<size_t> &ch) {
    double cost = 0;
    ch.resize(cells.size());
    for (size_t c = 0; c < cells.size(); ++c) { ch[c] = argmin_lagrangian(cells[c], lam); cost += cells[c].cost[ch[c]]; }
    return cost;
  };
  total = solve(0.0, choice);
  if (total <= budget) return true;
  double min_cost = 0;
  std::vector<size_t> cheapest(cells.size());
  for (size_t c = 0; c < cells.size(); ++c) {
    size_t b = 0;
    for (size_t i = 1; i < cells[c].cost.size(); ++i)
      if (cells[c].cost[i] < cells[c].cost[b] || (cells[c].cost[i] == cells[c].cost[b] && cells[c].err[i] < cells[c].err[b])) b = i;
    cheapest[c] = b;
    min_cost += cells[c].cost[b];
  }
  if (min_cost > budget) { choice = cheapest; total = min_cost; return false; }
  double lo = 0.0, hi = 1e-12;
  std::vector<size_t> ch_hi, ch_m;
  double cost_hi = solve(hi, ch_hi);
  while (cost_hi > budget) { lo = hi; hi *= 2.0; cost_hi = solve(hi, ch_hi); }
  for (int it = 0; it < 200; ++it) {
    const double mid = 0.5 * (lo + hi);
    if (mid == lo || mid == hi) break;
    const double cm = solve(mid, ch_m);
    if (cm <= budget) { hi = mid; ch_hi = ch_m; cost_hi = cm; } else { lo = mid; }
  }
  choice = ch_hi;
  total = cost_hi;
  return true;
}

}  // namespace jolt
