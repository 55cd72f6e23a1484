// Hooks through which the tcgen05 / TMA kernels replace stages of the portable pipeline.  A cell takes
// the tensor-core kernels when its shape fits them (fp16 data, r_t a multiple of 16 up to 256, r_f a
// multiple of 8); every other cell stays on the portable kernels, in the same call.
#pragma once
#include "tc_backbone.cuh"

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
  {
    const uint64_t dims[2] = {(uint64_t)c.r_f, (uint64_t)kD};
    const uint64_t str[1] = {(uint64_t)c.r_f * 2};
    const uint32_t box[2] = {64, 128};
    if (!make_tmap_f16(&cs.tmUF, cs.UF16, 2, dims, str, box)) return false;
  }
  {
    const uint64_t dims[2] = {(uint64_t)c.r_f, (uint64_t)c.m * c.r_t};
    const uint64_t str[1] = {(uint64_t)c.r_f * 2};
    const uint32_t box[2] = {64, (uint32_t)c.r_t};
    if (!make_tmap_f16(&cs.tmG, cs.G16, 2, dims, str, box)) return false;
  }
  cs.tc_ok = true;
  return true;
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
    tc::backbone_kernel<RESIDUAL><<<dim3(gx, n), tc::BB_THREADS, tc::BB_SMEM_BYTES, s>>>((const tc::BBCell *)(dev_t + off), seed);
    LAUNCHED();
  });
}

inline void fill_bb_common(tc::BBCell &b, const CellStore &cs, int *status) {
  memset(&b, 0, sizeof b);
  b.tmUT = cs.tmUT; b.tmUF = cs.tmUF; b.tmG = cs.tmG;
  b.words = cs.words; b.scales = cs.scales; b.e = cs.e;
  const CellDesc &c = cs.c;
  b.m = c.m; b.n_heads = c.n_heads; b.T = c.T; b.r_t = c.r_t; b.r_f = c.r_f; b.bits = c.bits; b.cell = c.cell;
  b.status = status;
}

}  // namespace
