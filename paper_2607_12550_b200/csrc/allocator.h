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

// Index of a cell's cheapest option (ties: the smaller error).
inline size_t cheapest_option(const CellOptions &c) {
  size_t b = 0;
  for (size_t i = 1; i < c.cost.size(); ++i)
    if (c.cost[i] < c.cost[b] || (c.cost[i] == c.cost[b] && c.err[i] < c.err[b])) b = i;
  return b;
}

// Greedy allocator of the ablations (paper Sec. 6: "spends each marginal byte on whichever group offers the largest
// error reduction per byte", no global multiplier).  Every cell starts at its cheapest option; each step applies, among
// all moves of one cell to a costlier option with a smaller error that still fits the remaining budget, the one with
// the largest error reduction per extra byte (ties: fewer extra bytes, then lower cell, then lower option index).
inline bool greedy_allocate(const std::vector<CellOptions> &cells, double budget, std::vector<size_t> &choice, double &total) {
  choice.resize(cells.size());
  total = 0;
  for (size_t c = 0; c < cells.size(); ++c) { choice[c] = cheapest_option(cells[c]); total += cells[c].cost[choice[c]]; }
  if (total > budget) return false;
  for (;;) {
    bool found = false;
    double best_ratio = 0, best_extra = 0;
    size_t bc = 0, bi = 0;
    for (size_t c = 0; c < cells.size(); ++c) {
      const double e0 = cells[c].err[choice[c]], c0 = cells[c].cost[choice[c]];
      for (size_t i = 0; i < cells[c].cost.size(); ++i) {
        const double extra = cells[c].cost[i] - c0, gain = e0 - cells[c].err[i];
        if (!(extra > 0) || !(gain > 0) || total + extra > budget) continue;
        const double ratio = gain / extra;
        if (!found || ratio > best_ratio || (ratio == best_ratio && extra < best_extra)) {
          found = true; best_ratio = ratio; best_extra = extra; bc = c; bi = i;
        }
      }
    }
    if (!found) break;
    total += best_extra;
    choice[bc] = bi;
  }
  return true;
}

// Uniform allocator of the ablations (ranks shared instead of per group): one option for all cells of class 0 (even
// cell index: keys) and one for all cells of class 1 (odd: values), the pair with the smallest summed error whose
// summed cost fits the budget (ties: the cheaper pair, then the earlier one).  Options are matched across cells by
// their (r_t, r_f, bits) triple; a triple that some cell of the class does not offer is not a candidate.
inline bool uniform_allocate(const std::vector<CellOptions> &cells, double budget, std::vector<size_t> &choice, double &total) {
  struct Cand { jolt_cell_plan t; double err, cost; std::vector<size_t> idx; };
  std::vector<Cand> cand[2];
  for (int cls = 0; cls < 2; ++cls) {
    size_t first = cls;
    if (first >= cells.size()) continue;
    for (size_t i = 0; i < cells[first].trip.size(); ++i) {
      Cand k{cells[first].trip[i], 0, 0, {}};
      bool everywhere = true;
      for (size_t c = first; c < cells.size() && everywhere; c += 2) {
        size_t j = 0;
        for (; j < cells[c].trip.size(); ++j)
          if (cells[c].trip[j].r_t == k.t.r_t && cells[c].trip[j].r_f == k.t.r_f && cells[c].trip[j].bits == k.t.bits) break;
        if (j == cells[c].trip.size()) { everywhere = false; break; }
        k.err += cells[c].err[j]; k.cost += cells[c].cost[j]; k.idx.push_back(j);
      }
      if (everywhere) cand[cls].push_back(k);
    }
  }
  choice.assign(cells.size(), 0);
  if (cells.size() < 2 || cand[0].empty() || cand[1].empty()) {      // a single class: fall back to one shared option
    for (size_t c = 0; c < cells.size(); ++c) choice[c] = cheapest_option(cells[c]);
    total = 0;
    for (size_t c = 0; c < cells.size(); ++c) total += cells[c].cost[choice[c]];
    return total <= budget;
  }
  bool found = false;
  size_t ba = 0, bb = 0;
  double be = 0, bcst = 0;
  size_t ca = 0, cb = 0;                       // cheapest pair, for the infeasible case
  for (size_t a = 0; a < cand[0].size(); ++a) if (cand[0][a].cost < cand[0][ca].cost || (cand[0][a].cost == cand[0][ca].cost && cand[0][a].err < cand[0][ca].err)) ca = a;
  for (size_t b = 0; b < cand[1].size(); ++b) if (cand[1][b].cost < cand[1][cb].cost || (cand[1][b].cost == cand[1][cb].cost && cand[1][b].err < cand[1][cb].err)) cb = b;
  for (size_t a = 0; a < cand[0].size(); ++a)
    for (size_t b = 0; b < cand[1].size(); ++b) {
      const double cst = cand[0][a].cost + cand[1][b].cost, e = cand[0][a].err + cand[1][b].err;
      if (cst > budget) continue;
      if (!found || e < be || (e == be && cst < bcst)) { found = true; ba = a; bb = b; be = e; bcst = cst; }
    }
  if (!found) { ba = ca; bb = cb; bcst = cand[0][ca].cost + cand[1][cb].cost; }
  for (size_t c = 0, n0 = 0, n1 = 0; c < cells.size(); ++c) choice[c] = (c % 2 == 0) ? cand[0][ba].idx[n0++] : cand[1][bb].idx[n1++];
  total = bcst;
  return found;
}

}  // namespace jolt
