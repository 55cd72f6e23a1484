// CholeskyQR of the randomized range finder (Sec. 5; Q = orth(S)) on tensor cores.  The basis (T x k on the token
// side, m*128 x k on the feature side) lives as an fp16 hi + lo pair, transposed in panels: [panels][kp][rows per
// panel] (1 x T on the token side, m x 128 on the feature side) -- the layout the sweeps read their dense operand in.
//
//   orth_gram_kernel    G = R^T R             tcgen05, both MMA operands are the same K-major tile; hi hi + hi lo + lo hi
//   cholinv_kernel      G = L L^T, L^-1       fp64, one CTA per cell (shared memory), L^-1 written as fp16 hi + lo
//   orth_apply_kernel   Q = R L^-T            tcgen05 (A = R^T tile, MN-major; B = L^-1, K-major); writes Q as fp32 rows
//                                             and, in place, as the hi + lo operand of the next sweep
//
// Precision: fp16 products are exact in the fp32 accumulator and hi + lo carries 22 bits, so G is fp32-grade.  The
// accumulator of tcgen05.mma truncates (about 2^-24 of the running sum per MMA), so the Gram kernel flushes it after
// every 64 rows into fp32 registers of the epilogue threads (round-to-nearest adds) and the row chunks of a cell are
// added in fp64 by the Cholesky kernel.
#pragma once
#include "small_solvers.cuh"
#include "tc_common.cuh"

namespace jolt {
namespace tc {

constexpr int OR_MAX_KP = 160;            // D0 (128 x kp) and D1 (rows 128.. x kp - 128), double buffered, fit 512 columns
constexpr int OR_MAX_K = 152;             // the fp64 Cholesky work matrix stays in shared memory
constexpr int OR_THREADS = 192;           // warps 0-3 epilogue, warp 4 TMA, warp 5 MMA
constexpr int OR_STEPS_PER_CTA = 8;       // 64-row steps per Gram CTA
constexpr int OR_SMEM_LIMIT = 222 * 1024;

struct alignas(64) OrthCell {
  CUtensorMap tmHi, tmLo;     // basis [panels][kp][rpp] fp16: dims {rpp, kp, panels}, box {64, kp, 1}
  CUtensorMap tmLhi, tmLlo;   // L^-1 [kp][kp] fp16 (row c, column j): dims {kp, kp}, box {64, kp}
  float *part;                // Gram partials [n_chunks][kp][kp] (rows >= 128 hold columns >= 128 only)
  __half *Lhi, *Llo;          // L^-1 as written by cholinv_kernel, scaled by 2^l_exp
  int *l_exp;
  float *out32;               // apply: rows x ld fp32 (row = panel * rpp + row in panel), may be null
  int ld, k, kp;
  int rpp, panels;
  int n_chunks;
  int out_exp;                // the fp16 copy of Q is scaled by 2^out_exp
  int *status;
};

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float *v) {
  uint32_t *u = (uint32_t *)v;
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(u[0]), "=r"(u[1]), "=r"(u[2]), "=r"(u[3]), "=r"(u[4]), "=r"(u[5]), "=r"(u[6]), "=r"(u[7]), "=r"(u[8]),
        "=r"(u[9]), "=r"(u[10]), "=r"(u[11]), "=r"(u[12]), "=r"(u[13]), "=r"(u[14]), "=r"(u[15])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tma_store_3d(const void *tmap, uint32_t src, int c0, int c1, int c2) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];"
               ::"l"(tmap), "r"(src), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
__device__ __forceinline__ void tma_store_commit_wait() {
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
  asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}

// ---------------------------------------------------------------------------------------------- Gram
__global__ void __launch_bounds__(OR_THREADS, 1) orth_gram_kernel(const OrthCell *__restrict__ cells, int n_stages) {
  extern __shared__ unsigned char smem_raw[];
  const OrthCell &c = cells[blockIdx.y];
  if ((int)blockIdx.x >= c.n_chunks) return;
  const int spp = c.rpp / 64;                         // 64-row steps per panel
  const int total = c.panels * spp;
  const int s0 = blockIdx.x * OR_STEPS_PER_CTA, n_steps = min(OR_STEPS_PER_CTA, total - s0);
  const int kp = c.kp, n1 = kp > 128 ? kp - 128 : 0, n0 = kp > 128 ? 128 : kp;     // D0: rows 0..n0-1 (M = 128), D1: rows 128..

  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char *sm = smem_raw + (base - raw);
  const uint32_t tile = (uint32_t)kp * 128u;           // kp is a multiple of 16: a multiple of 2 KB
  const uint32_t stage_bytes = 2 * tile;
  // a 128-row A operand starting at row 128 of the last tile reads up to 16 KB past it: the slack below
  const uint32_t sBar = base + (uint32_t)n_stages * stage_bytes + 16384u;
  volatile int *abort_flag = (volatile int *)(sm + (size_t)n_stages * stage_bytes + 16384 + 256);
  uint32_t *tmem_slot = (uint32_t *)(sm + (size_t)n_stages * stage_bytes + 16384 + 264);
  auto bFull = [=](int s) { return sBar + 8 * s; };
  auto bEmpty = [=](int s) { return sBar + 64 + 8 * s; };
  auto bAfull = [=](int b) { return sBar + 128 + 8 * b; };
  auto bAempty = [=](int b) { return sBar + 144 + 8 * b; };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    *abort_flag = 0;
    for (int s = 0; s < 8; ++s) { mbar_init(bFull(s), 1); mbar_init(bEmpty(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(bAfull(b), 1); mbar_init(bAempty(b), 128); }
    fence_barrier_init();
  }
  if (warp == 4) { tmem_alloc(smem_u32(tmem_slot), 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 4 && lane == 0) {
    tma_prefetch_desc(&c.tmHi); tma_prefetch_desc(&c.tmLo);
    bool ok = true;
    for (int j = 0; ok && j < n_steps; ++j) {
      const int s = j % n_stages, n = j / n_stages;
      ok = mbar_wait(bEmpty(s), (n & 1) ^ 1, abort_flag);
      if (!ok) break;
      const int step = s0 + j, panel = step / spp, r0 = (step - panel * spp) * 64;
      const uint32_t st = base + s * stage_bytes;
      mbar_expect_tx(bFull(s), 2 * tile);
      tma_load_3d(st, &c.tmHi, bFull(s), r0, 0, panel);
      tma_load_3d(st + tile, &c.tmLo, bFull(s), r0, 0, panel);
    }
  } else if (warp == 5 && lane == 0) {
    const uint32_t id0 = umma_idesc_f16(128, kp, 0, 0);
    const uint32_t id1 = umma_idesc_f16(128, n1 > 0 ? n1 : 16, 0, 0);
    bool ok = true;
    for (int j = 0; ok && j < n_steps; ++j) {
      const int s = j % n_stages, n = j / n_stages, b = j & 1, nb = j >> 1;
      ok = mbar_wait(bFull(s), n & 1, abort_flag);
      if (ok) ok = mbar_wait(bAempty(b), (nb & 1) ^ 1, abort_flag);
      if (!ok) break;
      tc_fence_after();
      const uint32_t hi = base + s * stage_bytes, lo = hi + tile;
      const uint32_t d0 = tmem_base + b * 256, d1 = d0 + 160;
#pragma unroll
      for (int k4 = 0; k4 < 4; ++k4) {
        const uint64_t aH = umma_desc_sw128(hi + k4 * 32, 16, 1024), aL = umma_desc_sw128(lo + k4 * 32, 16, 1024);
        umma_f16(d0, aH, aH, id0, k4 != 0);
        umma_f16(d0, aH, aL, id0, 1);
        umma_f16(d0, aL, aH, id0, 1);
        if (n1 > 0) {
          const uint64_t a1H = umma_desc_sw128(hi + 16384 + k4 * 32, 16, 1024), a1L = umma_desc_sw128(lo + 16384 + k4 * 32, 16, 1024);
          umma_f16(d1, a1H, a1H, id1, k4 != 0);
          umma_f16(d1, a1H, a1L, id1, 1);
          umma_f16(d1, a1L, a1H, id1, 1);
        }
      }
      umma_commit(bEmpty(s));
      umma_commit(bAfull(b));
    }
  } else if (warp < 4) {
    float acc0[OR_MAX_KP], acc1[32];
#pragma unroll
    for (int i = 0; i < OR_MAX_KP; ++i) acc0[i] = 0.f;
#pragma unroll
    for (int i = 0; i < 32; ++i) acc1[i] = 0.f;
    const uint32_t t_lane = tmem_base + ((uint32_t)(warp * 32) << 16);
    bool ok = true;
    for (int j = 0; j < n_steps; ++j) {
      const int b = j & 1, nb = j >> 1;
      if (ok) ok = __all_sync(0xffffffffu, mbar_wait(bAfull(b), nb & 1, abort_flag));
      if (!ok) break;
      tc_fence_after();
#pragma unroll
      for (int ch = 0; ch < OR_MAX_KP / 16; ++ch) {
        if (ch * 16 < kp) {
          float v[16];
          tmem_ld16(t_lane + b * 256 + ch * 16, v);
          tmem_wait_ld();
#pragma unroll
          for (int i = 0; i < 16; ++i) acc0[ch * 16 + i] += v[i];
        }
      }
      if (warp == 0) {
#pragma unroll
        for (int ch = 0; ch < 2; ++ch) {
          if (ch * 16 < n1) {
            float v[16];
            tmem_ld16(t_lane + b * 256 + 160 + ch * 16, v);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 16; ++i) acc1[ch * 16 + i] += v[i];
          }
        }
      }
      tc_fence_before();
      mbar_arrive(bAempty(b));
    }
    if (ok) {
      const int row = warp * 32 + lane;
      float *out = c.part + (size_t)blockIdx.x * kp * kp;
      if (row < n0) {
#pragma unroll
        for (int i = 0; i < OR_MAX_KP; ++i)
          if (i < kp) out[(size_t)row * kp + i] = acc0[i];
      }
      if (warp == 0 && lane < n1) {
#pragma unroll
        for (int i = 0; i < 32; ++i)
          if (i < n1) out[(size_t)(128 + lane) * kp + 128 + i] = acc1[i];
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
  if (warp == 4) { tc_fence_after(); tmem_dealloc(tmem_base, 512); }
}

// ---------------------------------------------------------------------------------------------- Cholesky + inverse
// G = L L^T in fp64, one CTA per matrix, right-looking by panels of 8 columns, with X = L^-T formed by the same
// panel operations on the rows of an identity appended below G ([G; I] = [L; X] L^T).  X is upper triangular and the
// Schur complement only needs its lower triangle, so both live in one n x n array (column-major: lower triangle L,
// upper triangle X, the diagonal of X in `invd`).  Per panel: (1) warp 0 factors the 8 x 8 diagonal block in
// registers, (2) one thread per row solves its 8 panel entries against the block (rows above the panel are rows of X,
// rows below are rows of L, the same recurrence), (3) the trailing update W[i][j] -= sum_c P[i][c] P[j][c] for the
// rows of X (i < panel end) and of the Schur complement (i >= j): first the next panel's eight columns, then -- while
// warp 0 already factors the next diagonal block (look-ahead) -- the rest, four columns per warp pass.  Three barriers
// per panel.
// A pivot not above `dead_rel` of its original diagonal entry belongs to a direction that is dependent to working
// accuracy: its column of L and its row / column of L^-1 are zero, status bit 1.
// Input: fp32 row-chunk partials of the Gram kernel (summed here in fp64) or an fp64 matrix.  Output: L^-1 as fp16
// hi + lo (times 2^l_exp) and / or L itself in fp64 for the Jacobi kernel.
struct CholInvTask {
  const float *part; int n_chunks, kp;      // Gram partials [n_chunks][kp][kp] (rows >= 128 hold columns >= 128 only), or
  const double *A64;                        // n x n symmetric fp64
  int k;
  __half *Lhi, *Llo;        // optional: L^-1 [kp][kp], rows / columns >= k zero
  int *l_exp;               // L^-1 is stored times 2^l_exp
  double *L64;              // optional: L column-major n x n, zeros above the diagonal, followed by one double holding
                            // the exponent e with max |L| < 2^e
  int *status;
  double dead_rel;
};
constexpr int kCholInvThreads = 512;
constexpr int kCholInvMaxN = 152;
inline size_t cholinv_smem_bytes(int k) { return ((size_t)k * k + 8 * (size_t)k + 72 + 8 + 2 * (size_t)k + 64) * sizeof(double); }

__global__ void __launch_bounds__(kCholInvThreads, 1) cholinv_kernel(const CholInvTask *__restrict__ tasks) {
  const CholInvTask t = tasks[blockIdx.x];
  const int n = t.k, kp = t.kp;
  if (n <= 0) return;
  extern __shared__ double ci_sh[];
  double *W = ci_sh;                        // element (row i, column j) at W[j * n + i]
  double *pan = W + (size_t)n * n;          // [8][n] the solved panel: X values for rows up to the panel, L values below
  double (*blkd)[9] = (double (*)[9])(pan + 8 * (size_t)n);
  double *ipiv = (double *)(blkd + 8);      // [8]
  double *diag0 = ipiv + 8;                 // [n] original diagonal
  double *invd = diag0 + n;                 // [n] diagonal of X = 1 / L_ii (0 for a dead pivot)
  __shared__ float s_red[32];
  __shared__ int s_exp, s_dead;
  const int tid = threadIdx.x, nt = blockDim.x, warp = tid >> 5, lane = tid & 31, nw = nt >> 5;
  if (tid == 0) s_dead = 0;
  // a warp per column j, lanes over the rows i >= j: both the fp64 input (its upper triangle, (row j, column i): the
  // matrix is symmetric) and the Gram partials are then read along contiguous addresses
  for (int j = warp; j < n; j += nw) {
    for (int i = lane; i < n; i += 32) {
      double v = 0.0;
      if (i >= j) {
        if (t.A64) v = t.A64[(size_t)j * n + i];
        else {
          // entry (i, j), i >= j, is read as (row j, column i) of the partials, which is stored for every such pair
          // (row j < 128 holds all columns; j >= 128 implies i >= 128)
          const float *p = t.part + (size_t)j * kp + i;
          const size_t cs = (size_t)kp * kp;
          int ch = 0;
          for (; ch + 8 <= t.n_chunks; ch += 8) {
            float a[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) a[q] = __ldg(p + (size_t)(ch + q) * cs);
            v += (((double)a[0] + (double)a[1]) + ((double)a[2] + (double)a[3])) + (((double)a[4] + (double)a[5]) + ((double)a[6] + (double)a[7]));
          }
          for (; ch < t.n_chunks; ++ch) v += (double)__ldg(p + (size_t)ch * cs);
        }
      }
      W[(size_t)j * n + i] = v;
    }
  }
  __syncthreads();
  for (int i = tid; i < n; i += nt) diag0[i] = W[(size_t)i * n + i];
  __syncthreads();
  // (1) the 8 x 8 diagonal block at j0: every lane of warp 0 factors it in registers (broadcast loads, no shuffles on
  // the dependent chain), then publishes the block and the reciprocal pivots
  auto factor_block = [&](int j0) {
    const int w = min(8, n - j0);
    double Lb[8][8], piv[8];
    int dead = 0;
#pragma unroll
    for (int r = 0; r < 8; ++r)
#pragma unroll
      for (int cc = 0; cc <= r; ++cc) Lb[r][cc] = (r < w && cc < w) ? W[(size_t)(j0 + cc) * n + j0 + r] : (r == cc ? 1.0 : 0.0);
#pragma unroll
    for (int cc = 0; cc < 8; ++cc) {
      piv[cc] = 0.0;
      if (cc < w) {
        const double d = Lb[cc][cc], dg = diag0[j0 + cc];
        const bool bad = !(d > t.dead_rel * dg) || !(dg > 0);
        const double rs = bad ? 0.0 : rsqrt_pos(d);
        Lb[cc][cc] = bad ? 0.0 : d * rs;
        dead |= bad ? 1 : 0;
        piv[cc] = rs;
#pragma unroll
        for (int r = cc + 1; r < 8; ++r) Lb[r][cc] *= rs;
#pragma unroll
        for (int c2 = cc + 1; c2 < 8; ++c2)
#pragma unroll
          for (int r = c2; r < 8; ++r) Lb[r][c2] = fma(-Lb[r][cc], Lb[c2][cc], Lb[r][c2]);
      }
    }
    if (lane < 8) {
#pragma unroll
      for (int rr = 0; rr < 8; ++rr)
        if (rr == lane) {
#pragma unroll
          for (int cc = 0; cc < 8; ++cc) blkd[rr][cc] = cc <= rr ? Lb[rr][cc] : 0.0;
        }
    }
    if (lane == 0) {
#pragma unroll
      for (int cc = 0; cc < 8; ++cc) ipiv[cc] = piv[cc];
      if (dead) s_dead = 1;
    }
  };
  if (warp == 0) factor_block(0);
  __syncthreads();
  for (int j0 = 0; j0 < n; j0 += 8) {
    const int w = min(8, n - j0);
    // (2) the panel entries of every row: x_c = (p_c - sum_{l<c} x_l L[c][l]) / L[c][c]
    for (int i = tid; i < n; i += nt) {
      const int r = i - j0;                   // row inside the panel when 0 <= r < w
      const bool inside = r >= 0 && r < w;
      double x[8];
#pragma unroll
      for (int cc = 0; cc < 8; ++cc) x[cc] = inside ? (cc == r ? 1.0 : 0.0) : (cc < w ? W[(size_t)(j0 + cc) * n + i] : 0.0);
#pragma unroll
      for (int cc = 0; cc < 8; ++cc) {
        if (cc < w) {
          double a = x[cc];
#pragma unroll
          for (int l = 0; l < cc; ++l) a = fma(-x[l], blkd[cc][l], a);
          x[cc] = a * ipiv[cc];
        }
      }
#pragma unroll
      for (int cc = 0; cc < 8; ++cc) {
        if (cc < w) {
          pan[cc * n + i] = x[cc];
          if (!inside) W[(size_t)(j0 + cc) * n + i] = x[cc];
          else if (cc > r) W[(size_t)(j0 + cc) * n + i] = x[cc];              // row of X
          else W[(size_t)(j0 + cc) * n + i] = blkd[r][cc];                    // row of L (diagonal included)
          if (inside && cc == r) invd[i] = x[cc];
        }
      }
    }
    __syncthreads();
    const int m0 = j0 + w;
    if (m0 >= n) break;
    // (3a) trailing update of the NEXT panel's columns only (one thread per row), so that warp 0 can factor the next
    // diagonal block while the other warps finish the update (look-ahead)
    const int wn = min(8, n - m0);
    for (int i = tid; i < n; i += nt) {
      double pi[8];
#pragma unroll
      for (int cc = 0; cc < 8; ++cc) pi[cc] = pan[cc * n + i];
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        const int j = m0 + q;
        if (q < wn && (i < m0 || i >= j)) {
          double a0 = 0, a1 = 0;
#pragma unroll
          for (int cc = 0; cc < 8; cc += 2) { a0 = fma(pi[cc], pan[cc * n + j], a0); a1 = fma(pi[cc + 1], pan[(cc + 1) * n + j], a1); }
          W[(size_t)j * n + i] -= a0 + a1;
        }
      }
    }
    __syncthreads();
    // (1') next diagonal block on warp 0 || (3b) the other columns on the other warps, four columns per warp pass;
    // rows i < m0 belong to X, rows i >= column to the Schur complement
    if (warp == 0) factor_block(m0);
    else {
      for (int j = m0 + wn + 4 * (warp - 1); j < n; j += 4 * (nw - 1)) {
        double pj[4][8];
#pragma unroll
        for (int q = 0; q < 4; ++q)
#pragma unroll
          for (int cc = 0; cc < 8; ++cc) pj[q][cc] = (j + q < n) ? pan[cc * n + j + q] : 0.0;
        const int nv = m0 + (n - j);
        for (int v = lane; v < nv; v += 32) {
          const int i = v < m0 ? v : j + (v - m0);
          double acc[4] = {0, 0, 0, 0};
#pragma unroll
          for (int cc = 0; cc < 8; ++cc) {
            const double pv = pan[cc * n + i];
#pragma unroll
            for (int q = 0; q < 4; ++q) acc[q] = fma(pv, pj[q][cc], acc[q]);
          }
#pragma unroll
          for (int q = 0; q < 4; ++q)
            if (j + q < n && (i < m0 || i >= j + q)) W[(size_t)(j + q) * n + i] -= acc[q];
        }
      }
    }
    __syncthreads();
  }
  if (tid == 0 && s_dead && t.status) atomicOr(t.status, 2);
  if (t.L64) {
    for (int j = warp; j < n; j += nw)
      for (int i = lane; i < n; i += 32) t.L64[(size_t)j * n + i] = i >= j ? W[(size_t)j * n + i] : 0.0;
    if (tid == 0) {      // max |L_ij|^2 <= max G_ii: exponent for the single-precision Jacobi iteration
      double mxd = 0.0;
      for (int i = 0; i < n; ++i) mxd = fmax(mxd, diag0[i]);
      int e2 = 0;
      if (mxd > 0.0 && mxd < 1e300) frexp(mxd, &e2);
      t.L64[(size_t)n * n] = (double)((e2 + 1) / 2 + 1);
    }
  }
  if (!t.Lhi) return;
  // ---- L^-1: (L^-1)_ic = X[c][i] for c < i, diagonal invd.  Scaled so that the largest entry lies in [2^9, 2^10).
  float mx = 0.f;
  for (int i = warp; i < n; i += nw) {           // column i of W, rows cidx < i hold row i of L^-1
    for (int cidx = lane; cidx < i; cidx += 32) mx = fmaxf(mx, fabsf((float)W[(size_t)i * n + cidx]));
    if (lane == 0) mx = fmaxf(mx, (float)invd[i]);
  }
  for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  if (lane == 0) s_red[warp] = mx;
  __syncthreads();
  if (tid == 0) {
    for (int i = 0; i < nw; ++i) mx = fmaxf(mx, s_red[i]);
    int e = 0;
    if (mx > 0.f && isfinite(mx)) e = 9 - ilogbf(mx);
    s_exp = e;
    *t.l_exp = e;
  }
  __syncthreads();
  const double sc = ldexp(1.0, s_exp);
  for (int i = warp; i < kp; i += nw) {          // row i (output column of Q), a pair of columns cidx (contraction index) per lane
    for (int c2 = 2 * lane; c2 < kp; c2 += 64) {
      float f[2];
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const int cidx = c2 + u;
        double v = 0.0;
        if (i < n && cidx < i) v = W[(size_t)i * n + cidx];
        else if (i < n && cidx == i) v = invd[i];
        f[u] = (float)(v * sc);
      }
      const __half2 h = __floats2half2_rn(f[0], f[1]);
      const float2 hf = __half22float2(h);
      *(__half2 *)(t.Lhi + (size_t)i * kp + c2) = h;
      *(__half2 *)(t.Llo + (size_t)i * kp + c2) = __floats2half2_rn(f[0] - hf.x, f[1] - hf.y);
    }
  }
}

// ---------------------------------------------------------------------------------------------- apply
// One CTA per 128 rows of the basis: D[128 rows][kp] = sum_j R[row][j] Linv[c][j].
__global__ void __launch_bounds__(OR_THREADS, 1) orth_apply_kernel(const OrthCell *__restrict__ cells) {
  extern __shared__ unsigned char smem_raw[];
  const OrthCell &c = cells[blockIdx.y];
  const int tpp = c.rpp / 128;                        // 128-row tiles per panel
  if ((int)blockIdx.x >= c.panels * tpp) return;
  const int panel = blockIdx.x / tpp, r0 = (blockIdx.x - panel * tpp) * 128;
  const int kp = c.kp, nkb = (kp + 63) / 64;

  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char *sm = smem_raw + (base - raw);
  const uint32_t tile = (uint32_t)kp * 128u;           // [kp rows][64 elements]
  const uint32_t sAhi = base, sAlo = base + 2 * tile, sBhi = base + 4 * tile, sBlo = sBhi + nkb * tile;
  const uint32_t sBar = sBlo + nkb * tile;
  const size_t bar_off = (size_t)(4 + 2 * nkb) * tile;
  volatile int *abort_flag = (volatile int *)(sm + bar_off + 64);
  uint32_t *tmem_slot = (uint32_t *)(sm + bar_off + 72);
  const uint32_t bLoad = sBar, bDone = sBar + 8;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    *abort_flag = 0;
    mbar_init(bLoad, 1); mbar_init(bDone, 1);
    fence_barrier_init();
  }
  if (warp == 4) { tmem_alloc(smem_u32(tmem_slot), 256); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 4 && lane == 0) {
    tma_prefetch_desc(&c.tmHi); tma_prefetch_desc(&c.tmLo); tma_prefetch_desc(&c.tmLhi); tma_prefetch_desc(&c.tmLlo);
    mbar_expect_tx(bLoad, (4 + 2 * nkb) * tile);
    for (int hf = 0; hf < 2; ++hf) {
      tma_load_3d(sAhi + hf * tile, &c.tmHi, bLoad, r0 + hf * 64, 0, panel);
      tma_load_3d(sAlo + hf * tile, &c.tmLo, bLoad, r0 + hf * 64, 0, panel);
    }
    for (int kb = 0; kb < nkb; ++kb) {
      tma_load_2d(sBhi + kb * tile, &c.tmLhi, bLoad, kb * 64, 0);
      tma_load_2d(sBlo + kb * tile, &c.tmLlo, bLoad, kb * 64, 0);
    }
  } else if (warp == 5 && lane == 0) {
    if (mbar_wait(bLoad, 0, abort_flag)) {
      tc_fence_after();
      const uint32_t idesc = umma_idesc_f16(128, kp, 1, 0);
      for (int ks = 0; ks < kp / 16; ++ks) {
        // A: MN-major, 16 contraction rows = 2048 B per step, the second 64 rows of the tile `tile` bytes further
        const uint64_t aH = umma_desc_sw128(sAhi + ks * 2048, tile, 1024), aL = umma_desc_sw128(sAlo + ks * 2048, tile, 1024);
        const uint32_t boff = (uint32_t)(ks >> 2) * tile + (uint32_t)(ks & 3) * 32;
        const uint64_t bH = umma_desc_sw128(sBhi + boff, 16, 1024), bL = umma_desc_sw128(sBlo + boff, 16, 1024);
        umma_f16(tmem_base, aH, bH, idesc, ks != 0);
        umma_f16(tmem_base, aH, bL, idesc, 1);
        umma_f16(tmem_base, aL, bH, idesc, 1);
      }
      umma_commit(bDone);
    }
  } else if (warp < 4) {
    const bool ok = __all_sync(0xffffffffu, mbar_wait(bDone, 0, abort_flag));
    if (ok) {
      tc_fence_after();
      const int row = warp * 32 + lane;                       // row of the tile
      const uint32_t t_lane = tmem_base + ((uint32_t)(warp * 32) << 16);
      const float s_in = ldexpf(1.0f, -*c.l_exp), s_out = ldexpf(1.0f, c.out_exp);
      float *orow = c.out32 ? c.out32 + ((size_t)panel * c.rpp + r0 + row) * c.ld : nullptr;
      // the operand tiles are consumed: stage the fp16 result over them in the layout they were loaded in
      unsigned char *hiT = sm + (row >> 6) * tile, *loT = sm + 2 * tile + (row >> 6) * tile;
      const int rr = row & 63;
      for (int ch = 0; ch * 16 < kp; ++ch) {
        float v[16];
        tmem_ld16(t_lane + ch * 16, v);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const int col = ch * 16 + i;
          const float q = v[i] * s_in;
          if (orow && col < c.k) orow[col] = q;
          const float qs = col < c.k ? q * s_out : 0.f;
          const __half h = __float2half_rn(qs);
          const uint32_t off = (uint32_t)col * 128u + ((((uint32_t)rr >> 3) ^ ((uint32_t)col & 7u)) << 4) + ((uint32_t)rr & 7u) * 2u;
          *(__half *)(hiT + off) = h;
          *(__half *)(loT + off) = __float2half_rn(qs - __half2float(h));
        }
      }
      fence_proxy_async();
    }
    named_bar_sync(1, 128);
    if (ok && threadIdx.x == 0) {
      for (int hf = 0; hf < 2; ++hf) {
        tma_store_3d(&c.tmHi, sAhi + hf * tile, r0 + hf * 64, 0, panel);
        tma_store_3d(&c.tmLo, sAlo + hf * tile, r0 + hf * 64, 0, panel);
      }
      tma_store_commit_wait();
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
  if (warp == 4) { tc_fence_after(); tmem_dealloc(tmem_base, 256); }
}

// ---------------------------------------------------------------------------------------------- split with a measured scale
// |x| maximum of fp32 arrays (one slot per job, zeroed by the caller); values are non-negative, so the integer
// maximum of the bit patterns is the floating-point maximum.
struct AbsMaxJob { const float *in; long long n; unsigned *slot; };
__global__ void absmax_kernel(const AbsMaxJob *__restrict__ jobs) {
  const AbsMaxJob j = jobs[blockIdx.y];
  float mx = 0.f;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < j.n; i += (long long)gridDim.x * blockDim.x)
    mx = fmaxf(mx, fabsf(j.in[i]));
  for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  if ((threadIdx.x & 31) == 0 && mx > 0.f && isfinite(mx)) atomicMax(j.slot, __float_as_uint(mx));
}

}  // namespace tc
}  // namespace jolt
