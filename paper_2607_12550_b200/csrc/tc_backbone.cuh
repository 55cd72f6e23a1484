// Fused backbone pass on tcgen05 tensor cores, in two modes that share everything but the epilogue:
//
//   DECODE  : X^  = 2^e U_T P_h + s . H(dequant(codes)) / sqrt(d)       -> fp16 / fp32 rows
//   RESIDUAL: r   = x - 2^e U_T P_h ; rotate ; quantise ; pack            -> codes + scales
//
// One CTA owns a (cell, head, run of 128-token tiles).  The projected core P_h = fp16(G_h U_F^T) was formed once
// when the cell was compressed and is kept with the handle: the CTA fetches its head's [r_t][128] block by TMA as
// two 64-feature panels (an MN-major B operand) and streams U_T tiles through a TMA ring into  D = U_T[tile] P_h
// with two TMEM accumulators, so the epilogue of one tile overlaps the MMA of the next.  Residual and decode read
// the SAME stored P, so the backbone the residual is taken against is bit for bit the one the decoder adds back.  Two epilogue warpgroups alternate tiles; each thread owns one
// 128-feature row in registers (TMEM lane = token).
#pragma once
#include "rowquant.cuh"
#include "tc_common.cuh"

namespace jolt {
namespace tc {

constexpr int BB_THREADS = 384;
constexpr int BB_P_BYTES = 65536;            // P: two panels of [r_t rows][128 B], r_t <= 256
constexpr int BB_BIG_BYTES = 131072;         // ring (+ X tiles)
constexpr int BB_STAGE_BYTES = 16384;        // one [128 tokens][64 fp16] box of U_T
constexpr int BB_XTILE_BYTES = 32768;        // two [128 tokens][64 fp16] boxes of X
constexpr int BB_SMEM_BYTES = BB_P_BYTES + BB_BIG_BYTES + 1024 /*align*/ + 512 /*barriers*/;
constexpr int BB_TMEM_COLS = 256;

struct alignas(64) BBCell {
  CUtensorMap tmUT;     // fp16 [T][r_t]           dims {r_t, T},       box {64, 128}
  CUtensorMap tmP;      // fp16 [m*r_t][128]       dims {128, m*r_t},   box {64, r_t}
  CUtensorMap tmX;      // fp16 [L][n_h][T][128]   dims {128, T, n_h, L}, box {64, 128, 1, 1}   (RESIDUAL)
  CUtensorMap tmOut;    // same shape over the output tensor (DECODE, fp16 destinations TMA can address)
  CUtensorMap tmOutW;   // the output tensor again with box {64, 32, 1, 1}: the 32 rows one warp stages and stores
  int tma_out;
  long long *dbg;       // optional: cycle stamps of CTA 0 (profiling aid), 8 per tile per warpgroup
  uint32_t *words;      // [m][T][4*bits]
  __half *scales;       // [m][T][4]
  const int *e;         // core exponent
  void *out;            // DECODE destination (first layer of the cell)
  long long osl, osh, ost;
  int out_dtype;
  int m, n_heads, T, r_t, r_f, bits, cell;
  int tiles_per_item, items_per_head;
  int tile_base;        // persistent decode: first tile of this cell in the launch's linear (cell, head, tile) order
  int *status;
  const float2 *rope;   // DECODE of key cells: (cos, sin) of feature pair j at token t in rope[j * T + t]; null = no rotation
};

template <int BITS>
__device__ __forceinline__ void bb_decode_row(const BBCell &c, uint64_t seed, long long row, float (&r)[128]) {
  if constexpr (BITS > 0) {
    uint32_t words[4 * BITS];
    const uint4 *wp = (const uint4 *)(c.words + row * (4 * BITS));
#pragma unroll
    for (int i = 0; i < BITS; ++i) { const uint4 v = __ldg(wp + i); words[4 * i] = v.x; words[4 * i + 1] = v.y; words[4 * i + 2] = v.z; words[4 * i + 3] = v.w; }
    __half sc[4];
    *(uint2 *)sc = __ldg((const uint2 *)(c.scales + row * 4));
    uint32_t sw[4];
    cell_sign_words(seed, c.cell, sw);
    unpack_dequant_row<BITS>(words, sc, sw, r);
  } else {
#pragma unroll
    for (int f = 0; f < 128; ++f) r[f] = 0.f;
  }
}

template <int BITS>
__device__ __forceinline__ void bb_quant_row(const BBCell &c, uint64_t seed, long long row, float (&r)[128]) {
  uint32_t sw[4];
  cell_sign_words(seed, c.cell, sw);
  uint32_t words[4 * BITS];
  __half sc[4];
  int bad = 0;
  quantize_pack_row<BITS>(r, sw, words, sc, &bad);
  if (bad) *c.status = 4;
  uint4 *wo = (uint4 *)(c.words + row * (4 * BITS));
#pragma unroll
  for (int i = 0; i < BITS; ++i) wo[i] = make_uint4(words[4 * i], words[4 * i + 1], words[4 * i + 2], words[4 * i + 3]);
  *(uint2 *)(c.scales + row * 4) = *(const uint2 *)sc;
}

template <bool RESIDUAL>
__global__ void __launch_bounds__(BB_THREADS, 1) backbone_kernel(const BBCell *__restrict__ cells, uint64_t seed) {
  extern __shared__ unsigned char smem_raw[];
  const BBCell &c = cells[blockIdx.y];
  const int items = c.m * c.items_per_head;
  if ((int)blockIdx.x >= items) return;
  const int h = blockIdx.x / c.items_per_head;
  const int item = blockIdx.x - h * c.items_per_head;
  const int n_tiles_total = c.T / 128;
  const int tile0 = item * c.tiles_per_item;
  const int n_tiles = min(c.tiles_per_item, n_tiles_total - tile0);
  if (n_tiles <= 0) return;

  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char *sm = smem_raw + (base - raw);
  const uint32_t sP = base;
  const uint32_t sBig = base + BB_P_BYTES;
  const uint32_t sBar = sBig + BB_BIG_BYTES;
  volatile int *abort_flag = (volatile int *)(sm + BB_P_BYTES + BB_BIG_BYTES + 256);
  uint32_t *tmem_slot = (uint32_t *)(sm + BB_P_BYTES + BB_BIG_BYTES + 264);

  constexpr int NS = RESIDUAL ? 4 : 8;                 // ring stages
  const uint32_t sRing = sBig;
  const uint32_t sX = sBig + 4 * BB_STAGE_BYTES;       // RESIDUAL: two X tiles behind a 4-stage ring
  // barrier slots (8 bytes each)
  const uint32_t bSetup = sBar + 0;
  auto bFull = [=](int s) { return sBar + 24 + 8 * s; };
  auto bEmpty = [=](int s) { return sBar + 24 + 64 + 8 * s; };
  auto bTfull = [=](int b) { return sBar + 152 + 8 * b; };
  auto bTempty = [=](int b) { return sBar + 168 + 8 * b; };
  auto bXfull = [=](int b) { return sBar + 184 + 8 * b; };
  auto bXempty = [=](int b) { return sBar + 200 + 8 * b; };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int wg = warp >> 2;
  const int nkt = (c.r_t + 63) / 64;
  const uint32_t panel = (uint32_t)c.r_t * 128u;       // bytes of one 64-feature panel of P (r_t is a multiple of 16)

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    mbar_init(bSetup, 1);
    for (int s = 0; s < 8; ++s) { mbar_init(bFull(s), 1); mbar_init(bEmpty(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(bTfull(b), 1); mbar_init(bTempty(b), 128); mbar_init(bXfull(b), 1); mbar_init(bXempty(b), 128); }
    fence_barrier_init();
  }
  if (warp == 8) { tmem_alloc(smem_u32(tmem_slot), BB_TMEM_COLS); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (wg == 2) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
    if (warp == 8 && lane == 0) {
      // ---------------- TMA producer
      tma_prefetch_desc(&c.tmUT); tma_prefetch_desc(&c.tmP);
      if (RESIDUAL) tma_prefetch_desc(&c.tmX);
      mbar_expect_tx(bSetup, 2u * panel);
      tma_load_2d(sP, &c.tmP, bSetup, 0, h * c.r_t);
      tma_load_2d(sP + panel, &c.tmP, bSetup, 64, h * c.r_t);
      bool ok = true;
      int cnt = 0;
      const int l = h / c.n_heads, hd = h - l * c.n_heads;
      for (int i = 0; ok && i < n_tiles; ++i) {
        const int tt = tile0 + i, b = i & 1, nb = i >> 1;
        if (RESIDUAL) {
          ok = mbar_wait(bXempty(b), (nb & 1) ^ 1, abort_flag);
          if (!ok) break;
          mbar_expect_tx(bXfull(b), BB_XTILE_BYTES);
          tma_load_4d(sX + b * BB_XTILE_BYTES, &c.tmX, bXfull(b), 0, tt * 128, hd, l);
          tma_load_4d(sX + b * BB_XTILE_BYTES + 16384, &c.tmX, bXfull(b), 64, tt * 128, hd, l);
        }
        for (int kb = 0; kb < nkt; ++kb, ++cnt) {
          const int s = cnt % NS, n = cnt / NS;
          ok = mbar_wait(bEmpty(s), (n & 1) ^ 1, abort_flag);
          if (!ok) break;
          mbar_expect_tx(bFull(s), BB_STAGE_BYTES);
          tma_load_2d(sRing + s * BB_STAGE_BYTES, &c.tmUT, bFull(s), kb * 64, tt * 128);
        }
      }
    } else if (warp == 9 && lane == 0) {
      // ---------------- MMA issuer
      bool ok = mbar_wait(bSetup, 0, abort_flag);      // the head's projected core has landed
      if (ok) {
        tc_fence_after();
        const uint32_t idesc = umma_idesc_f16(128, 128, 0, 1);   // A = U_T tile, K-major; B = P panels, MN-major
        const int ksteps = c.r_t / 16;
        int cnt = 0;
        for (int i = 0; ok && i < n_tiles; ++i) {
          const int b = i & 1, nb = i >> 1;
          ok = mbar_wait(bTempty(b), (nb & 1) ^ 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
          for (int kb = 0; kb < nkt; ++kb, ++cnt) {
            const int s = cnt % NS, n = cnt / NS;
            ok = mbar_wait(bFull(s), n & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            for (int k4 = 0; k4 < 4 && kb * 4 + k4 < ksteps; ++k4) {
              const uint64_t da = umma_desc_sw128(sRing + s * BB_STAGE_BYTES + k4 * 32, 16, 1024);
              // 16 contraction rows of P = 2048 B per step; the second 64 features one panel further
              const uint64_t db = umma_desc_sw128(sP + (kb * 4 + k4) * 2048, panel, 1024);
              umma_f16(tmem_base + b * 128, da, db, idesc, (kb | k4) != 0);
            }
            umma_commit(bEmpty(s));
          }
          if (ok) umma_commit(bTfull(b));
        }
      }
    }
  } else {
    // ---------------- epilogue warpgroups
    asm volatile("setmaxnreg.inc.sync.aligned.u32 216;");
    const int q = warp & 3;
    const int row_in_tile = q * 32 + lane;
    const uint32_t t_lane = tmem_base + ((uint32_t)(q * 32) << 16);
    bool ok = true;
    const float scale = ldexpf(1.0f, *c.e);
    const int l = h / c.n_heads, hd = h - l * c.n_heads;
    for (int i = wg; ok && i < n_tiles; i += 2) {
      const int tt = tile0 + i, nb = i >> 1;
      const int token = tt * 128 + row_in_tile;
      const long long row = (long long)h * c.T + token;
      float r[128];
      if constexpr (RESIDUAL) {
        ok = __all_sync(0xffffffffu, mbar_wait(bXfull(wg), nb & 1, abort_flag));
        if (!ok) break;
        const unsigned char *xb = sm + BB_P_BYTES + 4 * BB_STAGE_BYTES + wg * BB_XTILE_BYTES;
#pragma unroll
        for (int ck = 0; ck < 16; ++ck) {
          const uint4 v = *(const uint4 *)(xb + (ck >> 3) * 16384 + row_in_tile * 128 + (((ck & 7) ^ (row_in_tile & 7)) << 4));
          const __half2 *hp = (const __half2 *)&v;
#pragma unroll
          for (int j = 0; j < 4; ++j) { const float2 f = __half22float2(hp[j]); r[ck * 8 + 2 * j] = f.x; r[ck * 8 + 2 * j + 1] = f.y; }
        }
        mbar_arrive(bXempty(wg));
      } else {
        switch (c.bits) {
          case 0: bb_decode_row<0>(c, seed, row, r); break;
          case 1: bb_decode_row<1>(c, seed, row, r); break;
          case 2: bb_decode_row<2>(c, seed, row, r); break;
          case 3: bb_decode_row<3>(c, seed, row, r); break;
          case 4: bb_decode_row<4>(c, seed, row, r); break;
          default: bb_decode_row<8>(c, seed, row, r); break;
        }
      }
      ok = __all_sync(0xffffffffu, mbar_wait(bTfull(wg), nb & 1, abort_flag));
      if (!ok) break;
      tc_fence_after();
#pragma unroll
      for (int ch = 0; ch < 4; ++ch) {
        float v[32];
        tmem_ld32(t_lane + wg * 128 + ch * 32, v);
        tmem_wait_ld();
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          if constexpr (RESIDUAL) r[ch * 32 + j] -= scale * v[j];
          else r[ch * 32 + j] += scale * v[j];
        }
      }
      tc_fence_before();
      mbar_arrive(bTempty(wg));
      if constexpr (RESIDUAL) {
        switch (c.bits) {
          case 1: bb_quant_row<1>(c, seed, row, r); break;
          case 2: bb_quant_row<2>(c, seed, row, r); break;
          case 3: bb_quant_row<3>(c, seed, row, r); break;
          case 4: bb_quant_row<4>(c, seed, row, r); break;
          case 8: bb_quant_row<8>(c, seed, row, r); break;
          default: break;
        }
      } else {
        const long long off = (long long)l * c.osl + (long long)hd * c.osh + (long long)token * c.ost;
        if (c.out_dtype == DT_F16) {
          uint4 *p = (uint4 *)((__half *)c.out + off);
#pragma unroll
          for (int k8 = 0; k8 < 16; ++k8) {
            uint4 v;
            __half2 *hp = (__half2 *)&v;
#pragma unroll
            for (int j = 0; j < 4; ++j) hp[j] = __floats2half2_rn(r[k8 * 8 + 2 * j], r[k8 * 8 + 2 * j + 1]);
            p[k8] = v;
          }
        } else {
          float4 *p = (float4 *)((float *)c.out + off);
#pragma unroll
          for (int k4 = 0; k4 < 32; ++k4) p[k4] = make_float4(r[4 * k4], r[4 * k4 + 1], r[4 * k4 + 2], r[4 * k4 + 3]);
        }
      }
    }
  }
  // ---------------- common exit: everyone arrives here, aborted or not
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0) atomicOr(c.status, 8);
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000) {}      // let copies still in flight land before the CTA's memory is reused
    __syncthreads();
  }
  if (warp == 8) { tc_fence_after(); tmem_dealloc(tmem_base, BB_TMEM_COLS); }
}

}  // namespace tc
}  // namespace jolt
