// Hooks through which the tcgen05 / TMA kernels replace stages of the portable pipeline.  A cell takes
// the tensor-core kernels when its shape fits them (fp16 data, r_t a multiple of 16 up to 256, r_f a
// multiple of 8); every other cell stays on the portable kernels, in the same call.
#pragma once
#include "tc_backbone.cuh"
#include "tc_decode.cuh"
#include "tc_decode_p.cuh"
#include "tc_gemm.cuh"
#include "tc_orth.cuh"

namespace {

inline bool tc_shape_ok(const CellDesc &c) {
  return c.r_t > 0 && c.r_t % 16 == 0 && c.r_t <= 256 && c.r_f % 8 == 0 && c.r_f >= 8 && c.T % 128 == 0;
}

inline void fast_carve(Bump &, std::vector<CellWork> &, bool) {}

// Tensor maps of the stored factors (constant for the life of a handle).
inline bool encode_store_maps(CellStore &cs) {
  const CellDesc &c = cs.c;
  cs.tc_ok = false;
  if (!tc_shape_ok(c)) return false;
  {
    const uint64_t dims[2] = {(uint64_t)c.r_t, (uint64_t)c.T};
    const uint64_t str[1] = {(uint64_t)c.r_t * 2};
    const uint32_t box[2] = {64, 128};
    if (!make_tmap_f16(&cs.tmUT, cs.UT16, 2, dims, str, box)) return false;
  }
  {  // projected core P[m * r_t][128]: a box is one head's r_t rows by 64 features (one MN-major operand panel)
    if (!cs.P16) return false;
    const uint64_t dims[2] = {(uint64_t)kD, (uint64_t)c.m * c.r_t};
    const uint64_t str[1] = {(uint64_t)kD * 2};
    const uint32_t box[2] = {64, (uint32_t)c.r_t};
    if (!make_tmap_f16(&cs.tmP, cs.P16, 2, dims, str, box)) return false;
  }
  cs.tc_ok = true;
  return true;
}

// Launch with an explicit execution priority (the least one for the kernels that fill the machine: a cell group's
// cache-wide sweeps and its residual pass then yield to the other groups' small latency-bound kernels, whose side
// streams run at a higher priority).  Outside the concurrent cell groups the priority has nothing to compete with.
inline int heavy_kernel_priority() {
  static int lo = 0, hi = 0;
  static bool have = false;
  if (!have) { cudaDeviceGetStreamPriorityRange(&lo, &hi); have = true; }
  return lo;
}
template <typename... KArgs, typename... Args>
inline void launch_heavy(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args... args) {
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof cfg);
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
  cudaLaunchAttribute at;
  memset(&at, 0, sizeof at);
  at.id = cudaLaunchAttributePriority; at.val.priority = heavy_kernel_priority();
  cfg.attrs = &at; cfg.numAttrs = 1;
  cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

inline void bb_split(int total_heads, int n_tiles, int &tiles_per_item, int &items_per_head) {
  int per_head = (888 + total_heads / 2) / std::max(total_heads, 1);
  per_head = std::max(1, std::min(per_head, n_tiles));
  tiles_per_item = (n_tiles + per_head - 1) / per_head;
  items_per_head = (n_tiles + tiles_per_item - 1) / tiles_per_item;
}

template <bool RESIDUAL>
inline void add_backbone_tc(Program &P, int stage, const std::vector<tc::BBCell> &cells, uint64_t seed) {
  if (cells.empty()) return;
  static bool attr_done[2] = {false, false};
  if (!attr_done[RESIDUAL]) {
    cudaFuncSetAttribute(tc::backbone_kernel<RESIDUAL>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::BB_SMEM_BYTES);
    attr_done[RESIDUAL] = true;
  }
  int gx = 0;
  for (auto &c : cells) gx = std::max(gx, c.m * c.items_per_head);
  const size_t off = P.push(cells);
  const int n = (int)cells.size();
  P.add(stage, [=](char *dev_t, cudaStream_t s) {
    launch_heavy(tc::backbone_kernel<RESIDUAL>, dim3(gx, n), dim3(tc::BB_THREADS), (size_t)tc::BB_SMEM_BYTES, s, (const tc::BBCell *)(dev_t + off), seed);
    LAUNCHED();
  });
}

inline void add_decode_tc(Program &P, int stage, std::vector<tc::BBCell> cells, uint64_t seed) {
  if (cells.empty()) return;
  using LY = tc::DecLayout;
  static bool attr_done = false;
  static int n_sm = 0;
  if (!attr_done) {
    cudaFuncSetAttribute(tc::decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, LY::SMEM_BYTES);
    cudaFuncSetAttribute(tc::decode_persistent_kernel<false, 0x11Fu>, cudaFuncAttributeMaxDynamicSharedMemorySize, LY::SMEM_BYTES);
    cudaFuncSetAttribute(tc::decode_persistent_kernel<true, 0x11Fu>, cudaFuncAttributeMaxDynamicSharedMemorySize, LY::SMEM_BYTES);
    cudaFuncSetAttribute(tc::decode_persistent_kernel<true, 0x110u>, cudaFuncAttributeMaxDynamicSharedMemorySize, LY::SMEM_BYTES);
    cudaFuncSetAttribute(tc::decode_persistent_kernel<true, 0x010u>, cudaFuncAttributeMaxDynamicSharedMemorySize, LY::SMEM_BYTES);
    cudaFuncSetAttribute(tc::decode_persistent_kernel<true, 0x100u>, cudaFuncAttributeMaxDynamicSharedMemorySize, LY::SMEM_BYTES);
    cudaFuncSetAttribute(tc::decode_persistent_kernel<true, 0x014u>, cudaFuncAttributeMaxDynamicSharedMemorySize, LY::SMEM_BYTES);
    cudaFuncSetAttribute(tc::decode_persistent_kernel<true, 0x018u>, cudaFuncAttributeMaxDynamicSharedMemorySize, LY::SMEM_BYTES);
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
    attr_done = true;
  }
  // persistent form: every cell with r_t <= 128, the same sequence length and no rotation of keys at decode.  It is
  // instantiated per output mode and per set of bit widths: with at most two tile loops compiled in (and fp16 output
  // through bulk tensor stores only) ptxas keeps the whole epilogue in registers; with three or more it spills 50-60
  // bytes, and a spill reload inside the tile loop costs several per cent of the launch.
  bool persistent = (g_fast.load() & 128) != 0 && n_sm > 0, tma_only = true;
  unsigned bitmask = 0;
  long long total = 0;
  for (auto &c : cells) {
    if (c.r_t > 128 || c.T != cells[0].T) persistent = false;
    if (c.rope) persistent = false;
    if (!(c.tma_out != 0 && c.out_dtype == DT_F16)) tma_only = false;
    bitmask |= 1u << c.bits;
    c.tile_base = (int)total;
    total += (long long)c.m * (c.T / 128);
  }
  if (total >= (1ll << 30)) persistent = false;
  int gx = 0;
  for (auto &c : cells) gx = std::max(gx, c.m * c.items_per_head);
  const int nt = cells[0].T / 128, tot = (int)total;
  const size_t off = P.push(cells);
  const int n = (int)cells.size();
  const int grid_p = (int)std::min<long long>(n_sm, total);
  // The persistent kernel takes a fixed contiguous share per CTA and can hand a tail of the list out in chunks through
  // a counter (zero at every launch: it travels in the argument table).  The tail is empty unless a test asks for one: measured on the
  // benchmark mix, a 5 % tail in 8-tile chunks made the launch slower (0.199 against 0.192 ms), because every chunk
  // reloads its head's projected core into the single P buffer and restarts the unpack -> rotation pipeline.
  const size_t off_cnt = P.push(std::vector<int>(4, 0));
  std::vector<int2> run0(std::max(grid_p, 1), make_int2(tot, tot));
  const int pool = (int)((long long)tot * (100 - g_dec_tail_pct.load()) / 100), chunk = std::max(1, g_dec_tail_chunk.load());
  for (int i = 0; i < grid_p; ++i) run0[i] = make_int2((int)((long long)pool * i / grid_p), (int)((long long)pool * (i + 1) / grid_p));
  const size_t off_run0 = P.push(run0);
  P.add(stage, [=](char *dev_t, cudaStream_t s) {
    if (persistent) {
      tc::DecPArgs a{(const tc::BBCell *)(dev_t + off), n, nt, tot, seed, (const int2 *)(dev_t + off_run0), pool, chunk, (int *)(dev_t + off_cnt)};
      if (tma_only && bitmask == 0x010u) tc::decode_persistent_kernel<true, 0x010u><<<grid_p, LY::THREADS, LY::SMEM_BYTES, s>>>(a);
      else if (tma_only && bitmask == 0x100u) tc::decode_persistent_kernel<true, 0x100u><<<grid_p, LY::THREADS, LY::SMEM_BYTES, s>>>(a);
      else if (tma_only && (bitmask & ~0x110u) == 0) tc::decode_persistent_kernel<true, 0x110u><<<grid_p, LY::THREADS, LY::SMEM_BYTES, s>>>(a);
      else if (tma_only && (bitmask & ~0x014u) == 0) tc::decode_persistent_kernel<true, 0x014u><<<grid_p, LY::THREADS, LY::SMEM_BYTES, s>>>(a);
      else if (tma_only && (bitmask & ~0x018u) == 0) tc::decode_persistent_kernel<true, 0x018u><<<grid_p, LY::THREADS, LY::SMEM_BYTES, s>>>(a);
      else if (tma_only) tc::decode_persistent_kernel<true, 0x11Fu><<<grid_p, LY::THREADS, LY::SMEM_BYTES, s>>>(a);
      else tc::decode_persistent_kernel<false, 0x11Fu><<<grid_p, LY::THREADS, LY::SMEM_BYTES, s>>>(a);
    } else {
      tc::decode_kernel<<<dim3(gx, n), LY::THREADS, LY::SMEM_BYTES, s>>>((const tc::BBCell *)(dev_t + off), seed);
    }
    LAUNCHED();
  });
}

inline void fill_bb_common(tc::BBCell &b, const CellStore &cs, int *status) {
  memset(&b, 0, sizeof b);
  b.tmUT = cs.tmUT; b.tmP = cs.tmP;
  b.words = cs.words; b.scales = cs.scales; b.e = cs.e;
  const CellDesc &c = cs.c;
  b.m = c.m; b.n_heads = c.n_heads; b.T = c.T; b.r_t = c.r_t; b.r_f = c.r_f; b.bits = c.bits; b.cell = c.cell;
  b.status = status;
}


// ------------------------------------------------------------------ tensor-core sweeps of the factor stage

inline bool make_x_map(CUtensorMap *tm, const CellDesc &c, uint32_t box_tok) {
  const uint64_t dims[4] = {(uint64_t)kD, (uint64_t)c.T, (uint64_t)c.n_heads, (uint64_t)(c.m / c.n_heads)};
  const uint64_t str[3] = {(uint64_t)c.st * 2, (uint64_t)c.sh * 2, (uint64_t)c.sl * 2};
  const uint32_t box[4] = {64, box_tok, 1, 1};
  return make_tmap_f16(tm, c.X, 4, dims, str, box);
}

inline bool x_tma_ok(const CellDesc &c) {
  return c.dtype == DT_F16 && c.st % 8 == 0 && c.sh % 8 == 0 && c.sl % 8 == 0 && ((uintptr_t)c.X % 16 == 0) && c.T % 128 == 0;
}

// A cell's factor-stage sweeps can run on tensor cores: fp16 data TMA can address.  One MMA takes N <= 256
// columns; wider sketches are swept in column chunks (one more read of X per chunk).
constexpr int kTcMaxSketch = 768;
inline bool tc_sweep_ok(const CellDesc &c, bool staged_from_host) {
  if (c.dtype != DT_F16 || c.st % 8 || c.sh % 8 || c.sl % 8 || c.T % 128) return false;
  if (!staged_from_host && ((uintptr_t)c.X % 16)) return false;
  return c.k >= 1 && c.k <= kTcMaxSketch;
}

// column chunks of a padded sketch width: equal multiples of 16, each <= 256
inline void sketch_chunks(int kp, std::vector<std::pair<int, int>> &out) {
  const int n = (kp + 255) / 256;
  const int w = (((kp + n - 1) / n) + 15) & ~15;
  out.clear();
  for (int c0 = 0; c0 < kp; c0 += w) out.push_back({c0, std::min(w, kp - c0)});
}

inline int ilog2_floor(long long v) { int e = 0; while ((1ll << (e + 1)) <= v) ++e; return e; }

template <int MODE>
inline void launch_tc_gemm(Program &P, int stage, std::vector<tc::GemmCell> &cells) {
  if (cells.empty()) return;
  uint32_t max_stage = 0;
  int gx = 0;
  for (auto &c : cells) {
    const uint32_t b_bytes = MODE == tc::GM_GRAM ? 0u : (uint32_t)c.kp * 128u;
    const uint32_t b_pitch = (b_bytes + 1023u) & ~1023u;
    max_stage = std::max(max_stage, 16384u + ((c.has_lo && MODE != tc::GM_GRAM) ? 2 * b_pitch : b_pitch));
    gx = std::max(gx, MODE == tc::GM_TOK ? c.T / 128 : c.m);
  }
  int n_stages = std::min(8, (int)((tc::GM_SMEM_LIMIT - 1536) / max_stage));
  const size_t smem = (size_t)n_stages * max_stage + 1024 + 512;
  static size_t attr[3] = {0, 0, 0};
  if (attr[MODE] < smem) {
    cudaFuncSetAttribute(tc::tc_gemm_kernel<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::GM_SMEM_LIMIT);
    attr[MODE] = tc::GM_SMEM_LIMIT;
  }
  const size_t off = P.push(cells);
  const int n = (int)cells.size();
  P.add(stage, [=](char *dev_t, cudaStream_t s) {
    launch_heavy(tc::tc_gemm_kernel<MODE>, dim3(gx, n), dim3(tc::GM_THREADS), smem, s, (const tc::GemmCell *)(dev_t + off), n_stages);
    LAUNCHED();
  });
}

template <int MODE>
inline void launch_tc_gemm2(Program &P, int stage, std::vector<tc::Gemm2Cell> &cells) {
  if (cells.empty()) return;
  uint32_t max_stage = 0;
  int gx = 0;
  for (auto &c : cells) {
    const uint32_t b_pitch = ((uint32_t)c.kp * 128u + 1023u) & ~1023u;
    max_stage = std::max(max_stage, 32768u + (c.has_lo ? 2 * b_pitch : b_pitch));
    gx = std::max(gx, MODE == tc::GM_TOK ? (c.T / 128 + 1) / 2 : c.m / 2);
  }
  const int n_stages = std::min(8, (int)((tc::GM_SMEM_LIMIT - 1536) / max_stage));
  const size_t smem = (size_t)n_stages * max_stage + 1024 + 512;
  static bool attr[3] = {false, false, false};
  if (!attr[MODE]) {
    cudaFuncSetAttribute(tc::tc_gemm2_kernel<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::GM_SMEM_LIMIT);
    attr[MODE] = true;
  }
  const size_t off = P.push(cells);
  const int n = (int)cells.size();
  P.add(stage, [=](char *dev_t, cudaStream_t s) {
    launch_heavy(tc::tc_gemm2_kernel<MODE>, dim3(gx, n), dim3(tc::GM_THREADS), smem, s, (const tc::Gemm2Cell *)(dev_t + off), n_stages);
    LAUNCHED();
  });
}

inline bool make_x_map4(CUtensorMap *tm, const CellDesc &c, uint32_t box_tok, uint32_t box_heads) {
  const uint64_t dims[4] = {(uint64_t)kD, (uint64_t)c.T, (uint64_t)c.n_heads, (uint64_t)(c.m / c.n_heads)};
  const uint64_t str[3] = {(uint64_t)c.st * 2, (uint64_t)c.sh * 2, (uint64_t)c.sl * 2};
  const uint32_t box[4] = {64, box_tok, box_heads, 1};
  return make_tmap_f16(tm, c.X, 4, dims, str, box);
}

inline void launch_split(Program &P, int stage, const std::vector<tc::SplitJob> &jobs) {
  if (jobs.empty()) return;
  const size_t off = P.push(jobs);
  const int n = (int)jobs.size();
  P.add(stage, [=](char *dev_t, cudaStream_t s) {
    tc::split_transpose_kernel<<<dim3(148, 1, n), 256, 0, s>>>((const tc::SplitJob *)(dev_t + off));
    LAUNCHED();
  });
}

// mode-3 Gram of the tensor-core cells: fp32 partial per head, summed in fp64.
inline void add_gram_tc(Program &P, int stage, std::vector<CellWork> &ws) {
  std::vector<tc::GemmCell> gc;
  std::vector<const float *> parts; std::vector<double *> outs; std::vector<int> counts;
  for (auto &w : ws) {
    if (!w.active || !w.tc_gram) continue;
    tc::GemmCell g;
    memset(&g, 0, sizeof g);
    make_x_map(&g.tmX, w.c, 64);
    g.ldc = kD; g.ncols = kD; g.kp = kD; g.has_lo = 0; g.scale_exp = 0;
    g.m = w.c.m; g.n_heads = w.c.n_heads; g.T = w.c.T; g.status = w.status;
    const int nseg = tok_segments(w.c.T);
    for (int sg = 0; sg < nseg; ++sg) {
      g.C = (float *)w.gram_part + (size_t)sg * w.c.m * kD * kD;
      g.t0 = sg * kTokSegment; g.n_tok = std::min(kTokSegment, w.c.T - g.t0);
      gc.push_back(g);
    }
    parts.push_back((const float *)w.gram_part); outs.push_back(w.C); counts.push_back(w.c.m * nseg);
  }
  if (gc.empty()) return;
  launch_tc_gemm<tc::GM_GRAM>(P, stage, gc);
  const size_t o1 = P.push(parts), o2 = P.push(outs), o3 = P.push(counts);
  const int n = (int)parts.size();
  P.add(stage, [=](char *dev_t, cudaStream_t s) {
    tc::reduce_gram_partials_kernel<<<dim3(kD * kD / 256, n), 256, 0, s>>>((const float *const *)(dev_t + o1),
                                                                        (double *const *)(dev_t + o2), (const int *)(dev_t + o3));
    LAUNCHED();
  });
}

// S = sum_h X_h W_h for the tensor-core cells.  src: 0 = fp16 sketch already in Bhi, 1 = split W (fp32,
// [h][128][k]), 2 = split Z (fp32, [h][128][k], orthonormal columns over N rows).
inline bool orth_tc_ok(const CellWork &w);
inline void add_tok_tc(Program &P, int stage, std::vector<CellWork> &ws, const std::vector<int> &src) {
  std::vector<tc::SplitJob> sp;
  std::vector<tc::GemmCell> gc;
  std::vector<tc::Gemm2Cell> gc2;
  for (size_t i = 0; i < ws.size(); ++i) {
    CellWork &w = ws[i];
    if (!w.active || !w.tc) continue;
    const CellDesc &c = w.c;
    int se = 0;
    if (src[i] == 2 && w.ufI && w.split_ready == 2) {
      se = ilog2_floor((long long)c.N) / 2;          // the triangular solve of orth(Z) has written the operand already
      w.split_ready = 0;
    } else if (src[i] != 0) {
      const float *in = w.W;
      if (src[i] == 2) { in = w.ufI ? w.Z : w.W; se = ilog2_floor((long long)c.N) / 2; }
      tc::SplitJob j;
      j.in = in; j.hi = w.Bhi; j.lo = w.Blo; j.batch = c.m; j.rows = kD; j.cols = c.k; j.ld_in = c.k;
      j.kp = w.kp; j.scale_exp = se; j.absmax = nullptr;
      sp.push_back(j);
    }
    std::vector<std::pair<int, int>> ch;
    sketch_chunks(w.kp, ch);
    if (ch.size() == 1 && (g_fast.load() & 64)) {
      // one column chunk: two token tiles per CTA share every operand tile
      tc::Gemm2Cell g;
      memset(&g, 0, sizeof g);
      const uint64_t dims[3] = {(uint64_t)kD, (uint64_t)w.kp, (uint64_t)c.m};
      const uint64_t str[2] = {(uint64_t)kD * 2, (uint64_t)w.kp * kD * 2};
      const uint32_t box[3] = {64, (uint32_t)w.kp, 1};
      bool okm = make_x_map4(&g.tmX, c, 256, 1) && make_tmap_f16(&g.tmBhi, w.Bhi, 3, dims, str, box) &&
                 make_tmap_f16(&g.tmBlo, w.Blo, 3, dims, str, box);
      (void)okm;
      g.C = w.S; g.ldc = c.k; g.ncols = c.k; g.kp = w.kp; g.has_lo = src[i] != 0; g.scale_exp = se;
      g.m = c.m; g.n_heads = c.n_heads; g.T = c.T; g.status = w.status;
      if (orth_tc_ok(w)) { g.absmax = w.orthMax + (w.orthMaxUsed % kOrthMaxSlots); w.absmax_ready = true; }
      gc2.push_back(g);
      continue;
    }
    for (auto &cc : ch) {
      const int c0 = cc.first, kc = cc.second;
      if (c0 >= c.k) break;
      tc::GemmCell g;
      memset(&g, 0, sizeof g);
      const uint64_t dims[3] = {(uint64_t)kD, (uint64_t)kc, (uint64_t)c.m};
      const uint64_t str[2] = {(uint64_t)kD * 2, (uint64_t)w.kp * kD * 2};
      const uint32_t box[3] = {64, (uint32_t)kc, 1};
      bool okm = make_x_map(&g.tmX, c, 128) && make_tmap_f16(&g.tmBhi, w.Bhi + (size_t)c0 * kD, 3, dims, str, box) &&
                 make_tmap_f16(&g.tmBlo, w.Blo + (size_t)c0 * kD, 3, dims, str, box);
      (void)okm;
      g.C = w.S + c0; g.ldc = c.k; g.ncols = std::min(kc, c.k - c0); g.kp = kc; g.has_lo = src[i] != 0; g.scale_exp = se;
      g.m = c.m; g.n_heads = c.n_heads; g.T = c.T; g.status = w.status;
      gc.push_back(g);
    }
  }
  launch_split(P, stage, sp);
  launch_tc_gemm<tc::GM_TOK>(P, stage, gc);
  launch_tc_gemm2<tc::GM_TOK>(P, stage, gc2);
}

// Z'_h = X_h^T Q for the tensor-core cells (Q = w.S, T x k with orthonormal columns).
inline void add_feat_tc(Program &P, int stage, std::vector<CellWork> &ws) {
  std::vector<tc::SplitJob> sp;
  std::vector<tc::GemmCell> gc;
  std::vector<tc::Gemm2Cell> gc2;
  std::vector<tc::SumJob> sums;
  for (auto &w : ws) {
    if (!w.active || !w.tc) continue;
    const CellDesc &c = w.c;
    const int se = ilog2_floor(c.T) / 2;
    if (w.split_ready != 1) {      // else the triangular solve of orth(S) has written the operand already
      tc::SplitJob j;
      j.in = w.S; j.hi = w.Bhi; j.lo = w.Blo; j.batch = 1; j.rows = c.T; j.cols = c.k; j.ld_in = c.k; j.kp = w.kp; j.scale_exp = se; j.absmax = nullptr;
      sp.push_back(j);
    }
    w.split_ready = 0;
    std::vector<std::pair<int, int>> ch;
    sketch_chunks(w.kp, ch);
    if (ch.size() == 1 && c.n_heads % 2 == 0 && (g_fast.load() & 64)) {
      // one column chunk: two heads of a layer per CTA share every tile of Q
      tc::Gemm2Cell g;
      memset(&g, 0, sizeof g);
      const uint64_t dims[2] = {(uint64_t)c.T, (uint64_t)w.kp};
      const uint64_t str[1] = {(uint64_t)c.T * 2};
      const uint32_t box[2] = {64, (uint32_t)w.kp};
      bool okm = make_x_map4(&g.tmX, c, 64, 2) && make_tmap_f16(&g.tmBhi, w.Bhi, 2, dims, str, box) &&
                 make_tmap_f16(&g.tmBlo, w.Blo, 2, dims, str, box);
      (void)okm;
      g.ldc = c.k; g.ncols = c.k; g.kp = w.kp; g.has_lo = 1; g.scale_exp = se;
      g.m = c.m; g.n_heads = c.n_heads; g.T = c.T; g.status = w.status;
      const int nseg = tok_segments(c.T);
      if (nseg == 1 && orth_tc_ok(w)) { g.absmax = w.orthMax + (w.orthMaxUsed % kOrthMaxSlots); w.absmax_ready = true; }
      for (int sg = 0; sg < nseg; ++sg) {
        g.C = nseg > 1 ? w.Zpart + (size_t)sg * c.m * kD * c.k : w.Zp;
        g.t0 = sg * kTokSegment; g.n_tok = std::min(kTokSegment, c.T - g.t0);
        gc2.push_back(g);
      }
      if (nseg > 1) sums.push_back({w.Zpart, w.Zp, (long long)c.m * kD * c.k, (long long)c.m * kD * c.k, nseg});
      continue;
    }
    for (auto &cc : ch) {
      const int c0 = cc.first, kc = cc.second;
      if (c0 >= c.k) break;
      tc::GemmCell g;
      memset(&g, 0, sizeof g);
      const uint64_t dims[2] = {(uint64_t)c.T, (uint64_t)kc};
      const uint64_t str[1] = {(uint64_t)c.T * 2};
      const uint32_t box[2] = {64, (uint32_t)kc};
      bool okm = make_x_map(&g.tmX, c, 64) && make_tmap_f16(&g.tmBhi, w.Bhi + (size_t)c0 * c.T, 2, dims, str, box) &&
                 make_tmap_f16(&g.tmBlo, w.Blo + (size_t)c0 * c.T, 2, dims, str, box);
      (void)okm;
      g.ldc = c.k; g.ncols = std::min(kc, c.k - c0); g.kp = kc; g.has_lo = 1; g.scale_exp = se;
      g.m = c.m; g.n_heads = c.n_heads; g.T = c.T; g.status = w.status;
      const int nseg = tok_segments(c.T);
      for (int sg = 0; sg < nseg; ++sg) {
        g.C = (nseg > 1 ? w.Zpart + (size_t)sg * c.m * kD * c.k : w.Zp) + c0;
        g.t0 = sg * kTokSegment; g.n_tok = std::min(kTokSegment, c.T - g.t0);
        gc.push_back(g);
      }
    }
    if (tok_segments(c.T) > 1) sums.push_back({w.Zpart, w.Zp, (long long)c.m * kD * c.k, (long long)c.m * kD * c.k, tok_segments(c.T)});
  }
  launch_split(P, stage, sp);
  launch_tc_gemm<tc::GM_FEAT>(P, stage, gc);
  launch_tc_gemm2<tc::GM_FEAT>(P, stage, gc2);
  if (!sums.empty()) {
    const size_t off = P.push(sums);
    const int n = (int)sums.size();
    P.add(stage, [=](char *dev_t, cudaStream_t s) {
      tc::sum_partials_f32_kernel<<<dim3(296, n), 256, 0, s>>>((const tc::SumJob *)(dev_t + off));
      LAUNCHED();
    });
  }
}

// fp16 sketch of the r_f = d tensor-core cells, written straight into the TOK operand layout.
inline void add_sketch_gen_tc(Program &P, int stage, std::vector<CellWork> &ws, int stream_id, uint64_t seed) {
  std::vector<tc::SketchJob> jobs;
  for (auto &w : ws)
    if (w.active && w.tc && w.ufI) jobs.push_back({w.Bhi, w.c.m, w.c.k, w.kp, w.c.cell});
  if (jobs.empty()) return;
  const size_t off = P.push(jobs);
  const int n = (int)jobs.size();
  P.add(stage, [=](char *dev_t, cudaStream_t s) {
    launch_heavy(tc::gen_sketch_f16_kernel, dim3(148, n), dim3(256), (size_t)0, s, (const tc::SketchJob *)(dev_t + off), stream_id, seed);
    LAUNCHED();
  });
}

// ------------------------------------------------------------------ CholeskyQR on tensor cores
// Cells whose basis is already kept as the hi + lo operand of the sweeps (tensor-core cells with r_f = d, sketch
// width up to OR_MAX_K) orthonormalise it there: Gram and Q = R L^-T are tcgen05 GEMMs, the Cholesky factor and its
// inverse one fp64 CTA per cell.
inline bool orth_tc_ok(const CellWork &w) {
  return w.active && w.tc && w.ufI && w.c.k <= tc::OR_MAX_K && w.kp <= tc::OR_MAX_KP && w.c.T % 128 == 0 && w.orthPart != nullptr;
}

inline void add_orth_tc(Program &P, int stage, std::vector<CellWork> &ws, const std::vector<int> &idx, bool token_side, int passes,
                        bool want_fp32) {
  if (idx.empty()) return;
  static bool attr_done = false;
  if (!attr_done) {
    cudaFuncSetAttribute(tc::orth_gram_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::OR_SMEM_LIMIT);
    cudaFuncSetAttribute(tc::orth_apply_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::OR_SMEM_LIMIT);
    cudaFuncSetAttribute(tc::cholinv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tc::cholinv_smem_bytes(tc::kCholInvMaxN));
    attr_done = true;
  }
  // the sweep left the raw basis as fp32 rows: measure its magnitude, split it into the operand layout
  std::vector<tc::AbsMaxJob> am;
  std::vector<tc::SplitJob> sp;
  std::vector<tc::OrthCell> oc, oc_last;      // the fp32 rows of Q are only written by the last pass, and only if someone reads them
  std::vector<tc::CholInvTask> ci;
  int max_chunks = 0, max_tiles = 0, max_kp = 0, max_k = 0;
  for (int i : idx) {
    CellWork &w = ws[i];
    const CellDesc &c = w.c;
    const int rpp = token_side ? c.T : kD, panels = token_side ? 1 : c.m;
    float *src = token_side ? w.S : w.Z;
    unsigned *slot = w.orthMax + (w.orthMaxUsed++ % kOrthMaxSlots);
    if (!w.absmax_ready) am.push_back({src, (long long)rpp * panels * c.k, slot});      // else the sweep's epilogue measured it
    w.absmax_ready = false;
    tc::SplitJob j;
    j.in = src; j.hi = w.Bhi; j.lo = w.Blo; j.batch = panels; j.rows = rpp; j.cols = c.k; j.ld_in = c.k; j.kp = w.kp; j.scale_exp = 0;
    j.absmax = slot;
    sp.push_back(j);
    tc::OrthCell o;
    memset(&o, 0, sizeof o);
    {
      const uint64_t dims[3] = {(uint64_t)rpp, (uint64_t)w.kp, (uint64_t)panels};
      const uint64_t str[2] = {(uint64_t)rpp * 2, (uint64_t)w.kp * rpp * 2};
      const uint32_t box[3] = {64, (uint32_t)w.kp, 1};
      make_tmap_f16(&o.tmHi, w.Bhi, 3, dims, str, box);
      make_tmap_f16(&o.tmLo, w.Blo, 3, dims, str, box);
    }
    {
      const uint64_t dims[2] = {(uint64_t)w.kp, (uint64_t)w.kp};
      const uint64_t str[1] = {(uint64_t)w.kp * 2};
      const uint32_t box[2] = {64, (uint32_t)w.kp};
      make_tmap_f16(&o.tmLhi, w.orthLhi, 2, dims, str, box);
      make_tmap_f16(&o.tmLlo, w.orthLlo, 2, dims, str, box);
    }
    const int steps = panels * (rpp / 64);
    o.part = w.orthPart; o.Lhi = w.orthLhi; o.Llo = w.orthLlo; o.l_exp = w.orthExp;
    o.out32 = nullptr; o.ld = c.k; o.k = c.k; o.kp = w.kp; o.rpp = rpp; o.panels = panels;
    o.n_chunks = (steps + tc::OR_STEPS_PER_CTA - 1) / tc::OR_STEPS_PER_CTA;
    o.out_exp = ilog2_floor((long long)rpp * panels) / 2;
    o.status = w.status;
    oc.push_back(o);
    o.out32 = want_fp32 ? src : nullptr;
    oc_last.push_back(o);
    ci.push_back({w.orthPart, o.n_chunks, w.kp, nullptr, c.k, w.orthLhi, w.orthLlo, w.orthExp, nullptr, w.status, 1e-10});
    max_chunks = std::max(max_chunks, o.n_chunks);
    max_tiles = std::max(max_tiles, panels * (rpp / 128));
    max_kp = std::max(max_kp, w.kp); max_k = std::max(max_k, c.k);
    w.split_ready = token_side ? 1 : 2;
  }
  const size_t o_am = P.push(am), o_oc = P.push(oc), o_ocl = P.push(oc_last), o_ci = P.push(ci);
  const int n = (int)idx.size(), n_am = (int)am.size();
  {
    const size_t o_sp = P.push(sp);
    P.add(stage, [=](char *dev_t, cudaStream_t s) {
      if (n_am) { tc::absmax_kernel<<<dim3(32, n_am), 256, 0, s>>>((const tc::AbsMaxJob *)(dev_t + o_am)); LAUNCHED(); }
      tc::split_transpose_kernel<<<dim3(148, 1, n), 256, 0, s>>>((const tc::SplitJob *)(dev_t + o_sp)); LAUNCHED();
    });
  }
  const uint32_t tile = (uint32_t)max_kp * 128u;
  const int g_stages = std::max(2, std::min(6, (int)((tc::OR_SMEM_LIMIT - 16384 - 2048) / (2 * tile))));
  const size_t g_smem = (size_t)g_stages * 2 * tile + 16384 + 1024 + 1024;
  const size_t a_smem = (size_t)(4 + 2 * ((max_kp + 63) / 64)) * tile + 1024 + 1024;
  const size_t c_smem = tc::cholinv_smem_bytes(max_k);
  for (int pass = 0; pass < passes; ++pass) {
    const size_t o_app = pass + 1 == passes ? o_ocl : o_oc;
    P.add(stage, [=](char *dev_t, cudaStream_t s) {
      tc::orth_gram_kernel<<<dim3(max_chunks, n), tc::OR_THREADS, g_smem, s>>>((const tc::OrthCell *)(dev_t + o_oc), g_stages); LAUNCHED();
      tc::cholinv_kernel<<<n, tc::kCholInvThreads, c_smem, s>>>((const tc::CholInvTask *)(dev_t + o_ci)); LAUNCHED();
      tc::orth_apply_kernel<<<dim3(max_tiles, n), tc::OR_THREADS, a_smem, s>>>((const tc::OrthCell *)(dev_t + o_app)); LAUNCHED();
    });
  }
}

}  // namespace
