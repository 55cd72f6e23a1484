// The three full sweeps over a cell's fp16 data as tcgen05 GEMMs (TMA-fed ring, accumulator in TMEM):
//
//   TOK  : S[tile]   = sum_h X_h[tile] W_h          (128 tokens x k, contraction over heads x features)
//   FEAT : Z'_h      = X_h^T Q                      (128 features x k, contraction over tokens)
//   GRAM : C_h       = X_h^T X_h                    (128 x 128, contraction over tokens; fp32 partial per head)
//
// The cache operand is exact in fp16.  The dense operand (W, Q) is fp32-grade: it arrives split as
// hi + lo fp16 (pre-scaled by a power of two) and costs two MMAs per K step; a sketch whose entries are
// fp16 by definition has no lo part and costs one.
//
// The fp32 accumulation of tcgen05.mma truncates: a same-sign chain loses about 2^-24 per K step, 2e-5 after
// 4096 tokens.  Contractions over tokens (FEAT, GRAM) are therefore cut into segments of at most kTokSegment
// tokens, each its own accumulator, and the partial results are added in fp64.
#pragma once
#include "tc_common.cuh"

namespace jolt {
namespace tc {

enum { GM_TOK = 0, GM_FEAT = 1, GM_GRAM = 2 };

constexpr int GM_THREADS = 192;           // warps 0-3 epilogue, warp 4 TMA, warp 5 MMA
constexpr int GM_TMEM_COLS = 256;
constexpr int GM_SMEM_LIMIT = 220 * 1024;

struct alignas(64) GemmCell {
  CUtensorMap tmX;      // TOK: box {64 f, 128 tok, 1, 1};  FEAT / GRAM: box {64 f, 64 tok, 1, 1}
  CUtensorMap tmBhi;    // TOK: [m][kp][128] box {64, kp, 1};  FEAT: [kp][T] box {64, kp}
  CUtensorMap tmBlo;    // same shape; unused when has_lo == 0
  float *C;             // TOK: S [T][ldc];  FEAT: Z' [m][128][ldc];  GRAM: partials [m][128][128]
  int ldc, ncols;       // row pitch and number of valid columns (k; 128 for GRAM)
  int kp;               // padded N of the MMA (multiple of 16, <= 256)
  int has_lo;
  int scale_exp;        // result is multiplied by 2^-scale_exp
  int m, n_heads, T;
  int t0, n_tok;        // FEAT / GRAM: the token range this launch item contracts over (a multiple of 64)
  int *status;
};

template <int MODE>
__global__ void __launch_bounds__(GM_THREADS, 1) tc_gemm_kernel(const GemmCell *__restrict__ cells, int n_stages) {
  extern __shared__ unsigned char smem_raw[];
  const GemmCell &c = cells[blockIdx.y];
  const int n_items = MODE == GM_TOK ? c.T / 128 : c.m;
  if ((int)blockIdx.x >= n_items) return;
  const int item = blockIdx.x;

  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char *sm = smem_raw + (base - raw);
  const int kp = MODE == GM_GRAM ? 128 : c.kp;
  const uint32_t a_bytes = 16384;
  const uint32_t b_bytes = MODE == GM_GRAM ? 0u : (uint32_t)kp * 128u;
  const uint32_t b_total = (c.has_lo && MODE != GM_GRAM) ? 2 * b_bytes : b_bytes;
  // B sub-tiles start on 1024-byte boundaries (swizzle atom)
  const uint32_t b_pitch = (b_bytes + 1023u) & ~1023u;
  const uint32_t stage_bytes = a_bytes + ((c.has_lo && MODE != GM_GRAM) ? 2 * b_pitch : b_pitch);
  const uint32_t sStages = base;
  const uint32_t sBar = base + (uint32_t)n_stages * stage_bytes;
  volatile int *abort_flag = (volatile int *)(sm + (size_t)n_stages * stage_bytes + 256);
  uint32_t *tmem_slot = (uint32_t *)(sm + (size_t)n_stages * stage_bytes + 264);
  auto bFull = [=](int s) { return sBar + 8 * s; };
  auto bEmpty = [=](int s) { return sBar + 64 + 8 * s; };
  const uint32_t bDone = sBar + 128;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    *abort_flag = 0;
    for (int s = 0; s < 8; ++s) { mbar_init(bFull(s), 1); mbar_init(bEmpty(s), 1); }
    mbar_init(bDone, 1);
    fence_barrier_init();
  }
  if (warp == 4) { tmem_alloc(smem_u32(tmem_slot), GM_TMEM_COLS); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const int n_steps = MODE == GM_TOK ? 2 * c.m : c.n_tok / 64;

  if (warp == 4 && lane == 0) {
    tma_prefetch_desc(&c.tmX);
    if (MODE != GM_GRAM) { tma_prefetch_desc(&c.tmBhi); if (c.has_lo) tma_prefetch_desc(&c.tmBlo); }
    bool ok = true;
    for (int j = 0; ok && j < n_steps; ++j) {
      const int s = j % n_stages, n = j / n_stages;
      ok = mbar_wait(bEmpty(s), (n & 1) ^ 1, abort_flag);
      if (!ok) break;
      const uint32_t st = sStages + s * stage_bytes;
      mbar_expect_tx(bFull(s), a_bytes + b_total);
      if (MODE == GM_TOK) {
        const int h = j >> 1, kf = j & 1;
        const int l = h / c.n_heads, hd = h - l * c.n_heads;
        tma_load_4d(st, &c.tmX, bFull(s), kf * 64, item * 128, hd, l);
        tma_load_3d(st + a_bytes, &c.tmBhi, bFull(s), kf * 64, 0, h);
        if (c.has_lo) tma_load_3d(st + a_bytes + b_pitch, &c.tmBlo, bFull(s), kf * 64, 0, h);
      } else {
        const int h = item;
        const int l = h / c.n_heads, hd = h - l * c.n_heads;
        const int tok = c.t0 + j * 64;
        tma_load_4d(st, &c.tmX, bFull(s), 0, tok, hd, l);
        tma_load_4d(st + 8192, &c.tmX, bFull(s), 64, tok, hd, l);
        if (MODE == GM_FEAT) {
          tma_load_2d(st + a_bytes, &c.tmBhi, bFull(s), tok, 0);
          if (c.has_lo) tma_load_2d(st + a_bytes + b_pitch, &c.tmBlo, bFull(s), tok, 0);
        }
      }
    }
  } else if (warp == 5 && lane == 0) {
    const uint32_t idesc = MODE == GM_TOK ? umma_idesc_f16(128, kp, 0, 0)
                         : MODE == GM_FEAT ? umma_idesc_f16(128, kp, 1, 0)
                                           : umma_idesc_f16(128, 128, 1, 1);
    bool ok = true;
    for (int j = 0; ok && j < n_steps; ++j) {
      const int s = j % n_stages, n = j / n_stages;
      ok = mbar_wait(bFull(s), n & 1, abort_flag);
      if (!ok) break;
      tc_fence_after();
      const uint32_t st = sStages + s * stage_bytes;
#pragma unroll
      for (int k4 = 0; k4 < 4; ++k4) {
        uint64_t da, db, dl = 0;
        if (MODE == GM_TOK) {
          da = umma_desc_sw128(st + k4 * 32, 16, 1024);
          db = umma_desc_sw128(st + a_bytes + k4 * 32, 16, 1024);
          dl = umma_desc_sw128(st + a_bytes + b_pitch + k4 * 32, 16, 1024);
        } else if (MODE == GM_FEAT) {
          da = umma_desc_sw128(st + k4 * 2048, 8192, 1024);        // MN-major: 16 tokens = 2048 B per K step
          db = umma_desc_sw128(st + a_bytes + k4 * 32, 16, 1024);
          dl = umma_desc_sw128(st + a_bytes + b_pitch + k4 * 32, 16, 1024);
        } else {
          da = umma_desc_sw128(st + k4 * 2048, 8192, 1024);
          db = da;
        }
        umma_f16(tmem_base, da, db, idesc, (j | k4) != 0);
        if (MODE != GM_GRAM && c.has_lo) umma_f16(tmem_base, da, dl, idesc, 1);
      }
      umma_commit(bEmpty(s));
    }
    if (ok) umma_commit(bDone);
  } else if (warp < 4) {
    const bool ok = __all_sync(0xffffffffu, mbar_wait(bDone, 0, abort_flag));
    if (ok) {
      tc_fence_after();
      const int row = warp * 32 + lane;
      const uint32_t t_lane = tmem_base + ((uint32_t)(warp * 32) << 16);
      const float scale = ldexpf(1.0f, -c.scale_exp);
      float *crow;
      if (MODE == GM_TOK) crow = c.C + ((size_t)item * 128 + row) * c.ldc;
      else if (MODE == GM_FEAT) crow = c.C + ((size_t)item * 128 + row) * c.ldc;
      else crow = c.C + ((size_t)item * 128 + row) * 128;
      const int ncols = MODE == GM_GRAM ? 128 : c.ncols;
      for (int ch = 0; ch * 32 < ncols; ++ch) {
        float v[32];
        tmem_ld32(t_lane + ch * 32, v);
        tmem_wait_ld();
#pragma unroll
        for (int j = 0; j < 32; ++j)
          if (ch * 32 + j < ncols) crow[ch * 32 + j] = v[j] * scale;
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0) atomicOr(c.status, 8);
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000) {}
    __syncthreads();
  }
  if (warp == 4) { tc_fence_after(); tmem_dealloc(tmem_base, GM_TMEM_COLS); }
}

// ---- two output tiles per CTA ---------------------------------------------------------------------
// The dense operand B (k columns, hi + lo) is 36 KB per K step against 16 KB of cache data, so with one output tile per
// CTA the sweeps are bound by L2 -> shared-memory traffic of B, not by HBM.  Here a CTA owns TWO output tiles that share
// every B tile: two 128-token tiles (TOK) or two heads of one layer (FEAT), two TMEM accumulators.  The finished tiles
// are staged in shared memory in their global layout (the 128 rows of a tile are one contiguous block of S / Z') and
// leave as 16-byte coalesced stores; the largest |value| goes to an optional slot (the next CholeskyQR scales by it).
struct alignas(64) Gemm2Cell {
  CUtensorMap tmX;      // TOK: box {64 f, 256 tok, 1, 1};  FEAT: box {64 f, 64 tok, 2 heads, 1}
  CUtensorMap tmBhi;    // as in GemmCell
  CUtensorMap tmBlo;
  float *C;             // TOK: S [T][ldc];  FEAT: Z' [m][128][ldc]
  int ldc, ncols, kp, has_lo, scale_exp;
  int m, n_heads, T;
  int t0, n_tok;        // FEAT: token range
  unsigned *absmax;     // optional
  int *status;
};

template <int MODE>
__global__ void __launch_bounds__(GM_THREADS, 1) tc_gemm2_kernel(const Gemm2Cell *__restrict__ cells, int n_stages) {
  extern __shared__ unsigned char smem_raw[];
  const Gemm2Cell &c = cells[blockIdx.y];
  const int n_items = MODE == GM_TOK ? (c.T / 128 + 1) / 2 : c.m / 2;
  if ((int)blockIdx.x >= n_items) return;
  const int item = blockIdx.x;
  const int n_sub = MODE == GM_TOK ? min(2, c.T / 128 - 2 * item) : 2;      // a ragged last TOK item has one tile

  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char *sm = smem_raw + (base - raw);
  const int kp = c.kp;
  const uint32_t a_bytes = 32768;
  const uint32_t b_bytes = (uint32_t)kp * 128u;
  const uint32_t b_pitch = (b_bytes + 1023u) & ~1023u;
  const uint32_t stage_bytes = a_bytes + (c.has_lo ? 2 * b_pitch : b_pitch);
  const uint32_t sStages = base;
  const uint32_t sBar = base + (uint32_t)n_stages * stage_bytes;
  volatile int *abort_flag = (volatile int *)(sm + (size_t)n_stages * stage_bytes + 256);
  uint32_t *tmem_slot = (uint32_t *)(sm + (size_t)n_stages * stage_bytes + 264);
  auto bFull = [=](int s) { return sBar + 8 * s; };
  auto bEmpty = [=](int s) { return sBar + 64 + 8 * s; };
  const uint32_t bDone = sBar + 128;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    *abort_flag = 0;
    for (int s = 0; s < 8; ++s) { mbar_init(bFull(s), 1); mbar_init(bEmpty(s), 1); }
    mbar_init(bDone, 1);
    fence_barrier_init();
  }
  if (warp == 4) { tmem_alloc(smem_u32(tmem_slot), 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const int n_steps = MODE == GM_TOK ? 2 * c.m : c.n_tok / 64;

  if (warp == 4 && lane == 0) {
    tma_prefetch_desc(&c.tmX); tma_prefetch_desc(&c.tmBhi);
    if (c.has_lo) tma_prefetch_desc(&c.tmBlo);
    bool ok = true;
    for (int j = 0; ok && j < n_steps; ++j) {
      const int s = j % n_stages, n = j / n_stages;
      ok = mbar_wait(bEmpty(s), (n & 1) ^ 1, abort_flag);
      if (!ok) break;
      const uint32_t st = sStages + s * stage_bytes;
      if (j == 0 && g_test_skip_first_load == 1) continue;       // test switch: this stage never fills, its consumer's wait runs out
      mbar_expect_tx(bFull(s), a_bytes + (c.has_lo ? 2 : 1) * b_bytes);
      if (MODE == GM_TOK) {
        const int h = j >> 1, kf = j & 1;
        const int l = h / c.n_heads, hd = h - l * c.n_heads;
        tma_load_4d(st, &c.tmX, bFull(s), kf * 64, item * 256, hd, l);        // rows past T are zero-filled
        tma_load_3d(st + a_bytes, &c.tmBhi, bFull(s), kf * 64, 0, h);
        if (c.has_lo) tma_load_3d(st + a_bytes + b_pitch, &c.tmBlo, bFull(s), kf * 64, 0, h);
      } else {
        const int h = 2 * item;
        const int l = h / c.n_heads, hd = h - l * c.n_heads;
        const int tok = c.t0 + j * 64;
        tma_load_4d(st, &c.tmX, bFull(s), 0, tok, hd, l);                      // [2 heads][64 tok][features 0..63]
        tma_load_4d(st + 16384, &c.tmX, bFull(s), 64, tok, hd, l);             // [2 heads][64 tok][features 64..127]
        tma_load_2d(st + a_bytes, &c.tmBhi, bFull(s), tok, 0);
        if (c.has_lo) tma_load_2d(st + a_bytes + b_pitch, &c.tmBlo, bFull(s), tok, 0);
      }
    }
  } else if (warp == 5 && lane == 0) {
    const uint32_t idesc = MODE == GM_TOK ? umma_idesc_f16(128, kp, 0, 0) : umma_idesc_f16(128, kp, 1, 0);
    bool ok = true;
    for (int j = 0; ok && j < n_steps; ++j) {
      const int s = j % n_stages, n = j / n_stages;
      ok = mbar_wait(bFull(s), n & 1, abort_flag);
      if (!ok) break;
      tc_fence_after();
      const uint32_t st = sStages + s * stage_bytes;
#pragma unroll
      for (int k4 = 0; k4 < 4; ++k4) {
        const uint64_t db = umma_desc_sw128(st + a_bytes + k4 * 32, 16, 1024);
        const uint64_t dl = umma_desc_sw128(st + a_bytes + b_pitch + k4 * 32, 16, 1024);
#pragma unroll
        for (int sub = 0; sub < 2; ++sub) {
          if (sub >= n_sub) break;
          uint64_t da;
          if (MODE == GM_TOK) da = umma_desc_sw128(st + sub * 16384 + k4 * 32, 16, 1024);          // K-major, tokens sub*128..
          else da = umma_desc_sw128(st + sub * 8192 + k4 * 2048, 16384, 1024);                      // MN-major, head sub
          umma_f16(tmem_base + sub * 256, da, db, idesc, (j | k4) != 0);
          if (c.has_lo) umma_f16(tmem_base + sub * 256, da, dl, idesc, 1);
        }
      }
      umma_commit(bEmpty(s));
    }
    if (ok) umma_commit(bDone);
  } else if (warp < 4) {
    // every epilogue thread walks the same barriers whether or not the wait timed out
    const bool ok = __all_sync(0xffffffffu, mbar_wait(bDone, 0, abort_flag));
    tc_fence_after();
    const int row = warp * 32 + lane;
    const uint32_t t_lane = tmem_base + ((uint32_t)(warp * 32) << 16);
    const float scale = ldexpf(1.0f, -c.scale_exp);
    const int ncols = c.ncols, ldc = c.ldc;
    float *stg = (float *)sm;                        // every stage has been consumed: [128][ldc] staging tile
    float amax = 0.f;
    for (int sub = 0; sub < n_sub; ++sub) {
      if (ok) {
        for (int ch = 0; ch * 32 < ncols; ++ch) {
          float v[32];
          tmem_ld32(t_lane + sub * 256 + ch * 32, v);
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (ch * 32 + j < ncols) { const float x = v[j] * scale; stg[row * ldc + ch * 32 + j] = x; amax = fmaxf(amax, fabsf(x)); }
        }
      }
      named_bar_sync(1, 128);
      if (ok && !*abort_flag) {
        // the tile's 128 rows are one contiguous block of the output (row pitch ldc = ncols)
        float *dst = c.C + (size_t)(2 * item + sub) * 128 * ldc;
        const int total = 128 * ldc;
        if (((((uintptr_t)dst) & 15) == 0) && (total & 3) == 0) {
          const float4 *s4 = (const float4 *)stg;
          float4 *d4 = (float4 *)dst;
          for (int e = threadIdx.x; e < total / 4; e += 128) d4[e] = s4[e];
        } else {
          for (int e = threadIdx.x; e < total; e += 128) dst[e] = stg[e];
        }
      }
      named_bar_sync(1, 128);
    }
    if (ok && c.absmax) {
      for (int o = 16; o; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
      if (lane == 0 && amax > 0.f && isfinite(amax)) atomicMax(c.absmax, __float_as_uint(amax));
    }
  }
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0) atomicOr(c.status, 8);
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000) {}
    __syncthreads();
  }
  if (warp == 4) { tc_fence_after(); tmem_dealloc(tmem_base, 512); }
}

// ---- operand preparation -----------------------------------------------------------------------

// out_hi/lo[b][c][r] = split(in[b][r][c] * 2^se) for r < rows, c < cols; rows c in [cols, kp) are zero.
struct SplitJob {
  const float *in;      // [batch][rows][cols], pitch `ld_in`
  __half *hi, *lo;      // [batch][kp][rows]
  int batch, rows, cols, ld_in, kp, scale_exp;
  const unsigned *absmax;   // optional: bit pattern of max |in| (measured on the device); the scale is then 2^-(exponent + 1)
};

__global__ void __launch_bounds__(256) split_transpose_kernel(const SplitJob *__restrict__ jobs) {
  const SplitJob j = jobs[blockIdx.z];
  __shared__ float tile[32][33];
  const int tiles_r = (j.rows + 31) / 32, tiles_c = (j.kp + 31) / 32;
  const int per_batch = tiles_r * tiles_c;
  float sc = ldexpf(1.0f, j.scale_exp);
  if (j.absmax) { const float mx = __uint_as_float(*j.absmax); sc = (mx > 0.f && isfinite(mx)) ? ldexpf(1.0f, -(ilogbf(mx) + 1)) : 1.0f; }
  for (int w = blockIdx.x; w < per_batch * j.batch; w += gridDim.x) {
    const int b = w / per_batch, t = w - b * per_batch;
    const int r0 = (t / tiles_c) * 32, c0 = (t % tiles_c) * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    __syncthreads();
    for (int i = ty; i < 32; i += 8) {
      const int r = r0 + i, cc = c0 + tx;
      tile[i][tx] = (r < j.rows && cc < j.cols) ? j.in[((size_t)b * j.rows + r) * j.ld_in + cc] * sc : 0.f;
    }
    __syncthreads();
    for (int i = ty; i < 32; i += 8) {
      const int cc = c0 + i, r = r0 + tx;
      if (cc < j.kp && r < j.rows) {
        const float v = tile[tx][i];
        const __half h = __float2half_rn(v);
        const size_t o = ((size_t)b * j.kp + cc) * j.rows + r;
        j.hi[o] = h;
        if (j.lo) j.lo[o] = __float2half_rn(v - __half2float(h));
      }
    }
  }
}

// Gaussian sketch, fp16 by definition, written in the K-major layout the TOK sweep reads: out[h][c][f],
// counter (h*128 + f) * k + c; rows c in [k, kp) are zero.
struct SketchJob { __half *out; int m, k, kp, cell; };
__global__ void gen_sketch_f16_kernel(const SketchJob *__restrict__ jobs, int stream_id, uint64_t seed) {
  const SketchJob j = jobs[blockIdx.y];
  const uint64_t base = stream_base(seed, j.cell, stream_id);
  const long long n = (long long)j.m * j.kp * kD;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
    const int f = (int)(i % kD);
    const long long t = i / kD;
    const int cidx = (int)(t % j.kp), h = (int)(t / j.kp);
    float v = 0.f;
    if (cidx < j.k) v = (float)gaussian_from_u64(mix64(base + (uint64_t)(((long long)h * kD + f) * j.k + cidx)));
    j.out[i] = __float2half_rn(v);
  }
}

// fp32 partial Grams [m][128][128] -> fp64 sum [128][128]
__global__ void reduce_gram_partials_kernel(const float *const *partials, double *const *out, const int *counts) {
  const int ci = blockIdx.y;
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= kD * kD) return;
  const float *p = partials[ci];
  double s = 0;
  for (int h = 0; h < counts[ci]; ++h) s += (double)p[(size_t)h * kD * kD + e];
  out[ci][e] = s;
}

// out[e] = sum of `count` fp32 partials `stride` elements apart, added in fp64 in a fixed order
struct SumJob { const float *part; float *out; long long n, stride; int count; };
__global__ void sum_partials_f32_kernel(const SumJob *__restrict__ jobs) {
  const SumJob j = jobs[blockIdx.y];
  for (long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x; e < j.n; e += (long long)gridDim.x * blockDim.x) {
    double s = 0;
    for (int p = 0; p < j.count; ++p) s += (double)j.part[(size_t)p * j.stride + e];
    j.out[e] = (float)s;
  }
}

}  // namespace tc
}  // namespace jolt
