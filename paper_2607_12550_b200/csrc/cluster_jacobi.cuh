// Batched symmetric eigen-solver for the small Gram matrices of the path (the mode-3 Gram, Sec. 4, and B B^T of the
// randomized token factor, Sec. 5): one thread-block CLUSTER of eight CTAs per matrix, all matrices in one launch,
// the whole iteration resident in shared memory.
//
//   M = L L^T (Cholesky in fp64, chol_factor_kernel)   ->   one-sided Jacobi on the columns of L (single precision):
//   L J = U Sigma, so the normalised columns are the eigenvectors of M and the squared column norms its eigenvalues.
//
// Working on the triangular factor instead of M halves the number of sweeps (the iteration sees the singular values,
// not their squares), needs no eigenvector accumulator, and is what makes single precision enough: one-sided Jacobi
// resolves every column relative to its own norm, so the small singular directions keep the relative accuracy of the
// fp64 factor they start from (the paper's own decomposition numerics are float32, Sec. 6 "Setup").  Measured on
// spectra shaped like the benchmark's: eigenvector orthogonality 2e-6, dominant-subspace projectors within 4e-5 of an
// fp64 solve at a relative gap of 1e-2, eigenvalues to 4e-6.
//
// The n columns are cut into 16 blocks of g columns; CTA c holds two blocks.  A block round orthogonalises every
// column of the left block against every column of the right block (g sub-rounds of g disjoint pairs, one warp per
// pair, the left column stays in registers); then the blocks move one place round the tournament ring: the rotated
// columns of the last sub-round are written straight into the destination CTA's shared memory (distributed shared
// memory) and a cluster barrier ends the round.  Fifteen block rounds and one round inside the blocks make a sweep.
// A sub-round is a chain of ~100 dependent instructions (dot products, a five-level shuffle reduction, the angle,
// the update), so the time of a solve is latency, not throughput: the fp64 form of this kernel ran four times longer
// on the same schedule.  Nothing spins: the only waits are __syncthreads and the hardware cluster barrier.
#pragma once
#include <cooperative_groups.h>
#include "small_solvers.cuh"

namespace jolt {

constexpr int kCJCluster = 8;
constexpr int kCJBlocks = 2 * kCJCluster;
constexpr int kCJMaxN = 288;              // 9 rows per lane, 18 columns per block
constexpr int kCJMaxSweeps = 30;
// a sweep whose largest |cos| between two columns stayed below 1e-5 ends the iteration: its own rotations have then
// taken the cosines to about the square of that
constexpr float kCJStopCos2 = 1e-10f;

struct CJTask {
  const double *L;      // n x n, column j at L + j * n (lower triangular factor, zeros above the diagonal); L[n * n] holds
                        // the power-of-two exponent e with max |L| < 2^e
  int n;
  float *U_out;         // optional: n x r_out, column j = eigenvector of the j-th largest eigenvalue
  int ld_out, r_out;
  float *w_out;         // optional: n eigenvalues, descending
  int w_sqrt;           // 1: singular values (square roots) instead
  int *status;          // bit 0 if the sweep limit ran out
  int *sweeps_out;      // optional: number of sweeps run
};

// rows per lane the kernel is instantiated for: 4 (n <= 128), 5 (<= 160), 8 (<= 256), 9 (<= 288)
inline int cj_rows_per_lane(int n) { return n <= 128 ? 4 : (n <= 160 ? 5 : (n <= 256 ? 8 : 9)); }
inline size_t cj_smem_bytes(int n, int nr) {
  const int g = (n + kCJBlocks - 1) / kCJBlocks;
  return ((size_t)4 * g * 32 * nr + (size_t)kCJBlocks * g + 2 * kCJCluster + 64) * sizeof(float);
}
inline int cj_threads(int n) {
  const int g = (n + kCJBlocks - 1) / kCJBlocks;
  return 32 * ((g + 1) & ~1);
}

__device__ __forceinline__ float cj_rsqrt(float x) {
  float y;
  asm("rsqrt.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// a column of 32 NR rows (zero-padded) as NR registers per lane: 16-byte pieces first, single rows for the remainder
template <int NR>
__device__ __forceinline__ void cj_load(const float *col, int lane, float (&v)[NR]) {
#pragma unroll
  for (int q = 0; q < NR / 4; ++q) {
    const float4 x = *(const float4 *)(col + q * 128 + lane * 4);
    v[4 * q] = x.x; v[4 * q + 1] = x.y; v[4 * q + 2] = x.z; v[4 * q + 3] = x.w;
  }
#pragma unroll
  for (int q = 0; q < NR % 4; ++q) v[(NR / 4) * 4 + q] = col[(NR / 4) * 128 + q * 32 + lane];
}
template <int NR>
__device__ __forceinline__ void cj_store(float *col, int lane, const float (&v)[NR]) {
#pragma unroll
  for (int q = 0; q < NR / 4; ++q) *(float4 *)(col + q * 128 + lane * 4) = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
#pragma unroll
  for (int q = 0; q < NR % 4; ++q) col[(NR / 4) * 128 + q * 32 + lane] = v[(NR / 4) * 4 + q];
}

// Makes the columns a, b orthogonal (new a = c a - s b, new b = s a + c b; the rotation with |tan| <= 1);
// mx2 keeps the largest cos^2 between two columns seen before their rotation.
template <int NR>
__device__ __forceinline__ void cj_rotate(float (&a)[NR], float (&b)[NR], float &mx2) {
  float al = 0.f, be = 0.f, ga = 0.f;
#pragma unroll
  for (int i = 0; i < NR; ++i) { al = fmaf(a[i], a[i], al); be = fmaf(b[i], b[i], be); ga = fmaf(a[i], b[i], ga); }
#pragma unroll
  for (int o = 16; o; o >>= 1) {
    const float ta = __shfl_xor_sync(0xffffffffu, al, o), tb = __shfl_xor_sync(0xffffffffu, be, o), tg = __shfl_xor_sync(0xffffffffu, ga, o);
    al += ta; be += tb; ga += tg;
  }
  // the angle depends on the ratios of (al, be, ga) only: bring the larger norm into [1/2, 1) by a power of two first, so
  // that two columns that are both tiny against the rest (the null directions of a rank-deficient factor) do not push
  // the products below into the denormal range, where the approximate reciprocal square root returns infinity
  const float big = fmaxf(al, be);
  const float sc = __uint_as_float(0x7E800000u - (__float_as_uint(big) & 0x7F800000u));
  al *= sc; be *= sc; ga *= sc;
  const float ab = al * be, g2 = ga * ga;
  if (!(ab > 1e-36f)) return;                       // a zero (padding or deflated) column, or one 1e-36 of the other
  mx2 = fmaxf(mx2, g2 * __frcp_rn(ab));
  if (!(g2 > 1e-14f * ab)) return;                   // already orthogonal to single precision
  const float d = 0.5f * (be - al);
  const float rh = cj_rsqrt(fmaf(d, d, g2));
  const float x = fmaf(0.5f * fabsf(d), rh, 0.5f);   // cos^2 of the rotation angle
  const float rc = cj_rsqrt(x);
  float c = x * rc, s = (d >= 0.f ? 0.5f : -0.5f) * ga * rh * rc;
  const float corr = fmaf(fmaf(c, c, fmaf(s, s, -1.0f)), -0.5f, 1.0f);
  c *= corr; s *= corr;
#pragma unroll
  for (int i = 0; i < NR; ++i) {
    const float xx = a[i], yy = b[i];
    a[i] = fmaf(c, xx, -s * yy);
    b[i] = fmaf(s, xx, c * yy);
  }
}

template <int NR>
__global__ void __cluster_dims__(kCJCluster, 1, 1) __launch_bounds__(32 * ((NR * 32 / kCJBlocks + 2) & ~1))
    cj_eig_kernel(const CJTask *__restrict__ tasks) {
  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();
  constexpr int C = kCJCluster, B = kCJBlocks, NP = 32 * NR;     // NP: padded column length
  const int rank = (int)cluster.block_rank();
  const CJTask t = tasks[blockIdx.y];
  const int n = t.n;
  const int g = (n + B - 1) / B, ge = (g + 1) & ~1;
  const int blk = g * NP;
  extern __shared__ __align__(16) float cj_sh[];
  float *buf = cj_sh;                        // [2 parity][2 side][g][NP]
  float *lam_all = cj_sh + 4 * (size_t)blk;  // [B * g] squared column norms by final position
  float *conv = lam_all + B * g;             // [2][C] largest cos^2 per CTA, per sweep parity
  __shared__ float red[32];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, nw = blockDim.x >> 5;

  // columns of the two blocks this CTA starts with: slots rank (left) and B - 1 - rank (right), scaled into [-1, 1]
  const int sexp = (int)t.L[(size_t)n * n];
  const double scale = ldexp(1.0, -sexp);
  for (int side = 0; side < 2; ++side) {
    const int slot = side == 0 ? rank : B - 1 - rank;
    for (int e = tid; e < blk; e += blockDim.x) {
      const int i = e / NP, r = e - i * NP, col = slot * g + i;
      buf[side * blk + e] = (col < n && r < n) ? (float)(t.L[(size_t)col * n + r] * scale) : 0.f;
    }
  }
  __syncthreads();

  int par = 0, sweep = 0;
  bool done = false;
  for (; sweep < kCJMaxSweeps && !done; ++sweep) {
    float mx = 0.f;
    float *cur = buf + par * 2 * blk;
    // ---- pairs inside each of the two blocks (circle method on ge players; left block on the first ge/2 warps)
    for (int s = 0; s < ge - 1; ++s) {
      if (warp < ge) {
        const int side = warp / (ge / 2), i = warp - side * (ge / 2);
        int p, q;
        rr_pair(s, i, ge, p, q);
        if (q < g) {
          float *cp = cur + side * blk + p * NP, *cq = cur + side * blk + q * NP;
          float a[NR], b[NR];
          cj_load<NR>(cp, lane, a); cj_load<NR>(cq, lane, b);
          cj_rotate<NR>(a, b, mx);
          cj_store<NR>(cp, lane, a); cj_store<NR>(cq, lane, b);
        }
      }
      __syncthreads();
    }
    // ---- fifteen block rounds
    for (int r_blk = 0; r_blk < B - 1; ++r_blk) {
      cur = buf + par * 2 * blk;
      const int np = par ^ 1;
      // where the blocks go: left -> next CTA's left (the last CTA's left turns into its own right; CTA 0's stays),
      // right -> previous CTA's right (CTA 0's right becomes CTA 1's left)
      float *dstL, *dstR;
      {
        float *mine = buf + np * 2 * blk;
        if (rank == 0) dstL = mine;
        else if (rank < C - 1) dstL = cluster.map_shared_rank(mine, rank + 1);
        else dstL = mine + blk;
        if (rank > 0) dstR = cluster.map_shared_rank(mine + blk, rank - 1);
        else dstR = cluster.map_shared_rank(mine, 1);
      }
      float a[NR];
      if (warp < g) cj_load<NR>(cur + warp * NP, lane, a);
      for (int s = 0; s < g; ++s) {
        if (warp < g) {
          int j = warp + s;
          if (j >= g) j -= g;
          float *cq = cur + blk + j * NP;
          float b[NR];
          cj_load<NR>(cq, lane, b);
          cj_rotate<NR>(a, b, mx);
          if (s + 1 < g) cj_store<NR>(cq, lane, b);
          else { cj_store<NR>(dstR + j * NP, lane, b); cj_store<NR>(dstL + warp * NP, lane, a); }
        }
        if (s + 1 < g) __syncthreads();
      }
      if (r_blk == B - 2) {
        // end of the sweep: every CTA tells every CTA its largest cos^2
        if (lane == 0) red[warp] = mx;
        __syncthreads();
        if (tid < C) {
          float m = 0.f;
          for (int w = 0; w < nw; ++w) m = fmaxf(m, red[w]);
          cluster.map_shared_rank(conv, tid)[(sweep & 1) * C + rank] = m;
        }
      }
      cluster.sync();
      par = np;
    }
    float m = 0.f;
    for (int c = 0; c < C; ++c) m = fmaxf(m, conv[(sweep & 1) * C + c]);
    done = m <= kCJStopCos2;
  }
  if (!done && tid == 0 && rank == 0 && t.status) atomicOr(t.status, 1);
  if (t.sweeps_out && tid == 0 && rank == 0) *t.sweeps_out = sweep;

  // ---- squared column norms of this CTA's blocks, sent to every CTA under the column's final position
  float *cur = buf + par * 2 * blk;
  for (int ci = warp; ci < 2 * g; ci += nw) {
    const int side = ci / g, i = ci - side * g;
    const float *cp = cur + side * blk + i * NP;
    float s2 = 0.f;
    for (int r = lane; r < NP; r += 32) s2 = fmaf(cp[r], cp[r], s2);
#pragma unroll
    for (int o = 16; o; o >>= 1) s2 += __shfl_xor_sync(0xffffffffu, s2, o);
    const int slot = side == 0 ? rank : B - 1 - rank;
    if (lane < C) cluster.map_shared_rank(lam_all, lane)[slot * g + i] = s2;
  }
  cluster.sync();
  // ---- rank of each column by descending eigenvalue (ties by position), scatter
  const double unscale = ldexp(1.0, 2 * sexp);
  for (int ci = warp; ci < 2 * g; ci += nw) {
    const int side = ci / g, i = ci - side * g;
    const int slot = side == 0 ? rank : B - 1 - rank;
    const int me = slot * g + i;
    const float lam = lam_all[me];
    int rk = 0;
    for (int j = lane; j < B * g; j += 32) { const float lj = lam_all[j]; rk += (lj > lam) || (lj == lam && j < me); }
#pragma unroll
    for (int o = 16; o; o >>= 1) rk += __shfl_xor_sync(0xffffffffu, rk, o);
    if (rk >= n) continue;
    if (t.w_out && lane == 0) { const double v = (double)lam * unscale; t.w_out[rk] = (float)(t.w_sqrt ? sqrt(v) : v); }
    if (t.U_out && rk < t.r_out) {
      const float inv = lam > 0.f ? rsqrtf(lam) : 0.f;
      const float *cp = cur + side * blk + i * NP;
      for (int r = lane; r < n; r += 32) t.U_out[(size_t)r * t.ld_out + rk] = cp[r] * inv;
    }
  }
}

inline void cj_launch(const CJTask *d_tasks, int n_tasks, int max_n, int nr, cudaStream_t st) {
  const size_t shm = cj_smem_bytes(max_n, nr);
  const dim3 grid(kCJCluster, n_tasks);
  const int threads = cj_threads(max_n);
  switch (nr) {
    case 4: cj_eig_kernel<4><<<grid, threads, shm, st>>>(d_tasks); break;
    case 5: cj_eig_kernel<5><<<grid, threads, shm, st>>>(d_tasks); break;
    case 8: cj_eig_kernel<8><<<grid, threads, shm, st>>>(d_tasks); break;
    default: cj_eig_kernel<9><<<grid, threads, shm, st>>>(d_tasks); break;
  }
}
inline void cj_opt_in_smem() {
  const int lim = 200 * 1024;
  cudaFuncSetAttribute(cj_eig_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, lim);
  cudaFuncSetAttribute(cj_eig_kernel<5>, cudaFuncAttributeMaxDynamicSharedMemorySize, lim);
  cudaFuncSetAttribute(cj_eig_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, lim);
  cudaFuncSetAttribute(cj_eig_kernel<9>, cudaFuncAttributeMaxDynamicSharedMemorySize, lim);
}

// ---- M = L L^T in fp64, one CTA per matrix, right-looking by panels of 8 columns; L is written column-major with
// zeros above the diagonal.  The work matrix lives in shared memory when it fits (n <= kCholFactorSmemN), else in the
// output buffer (read back through L1; all threads of the CTA sit on one SM).  A pivot that is not above 1e-13 of its
// original diagonal entry belongs to a numerically dependent direction: its column of L is set to zero (the Jacobi
// iteration above treats a zero column as a zero eigenvalue), status bit 1.
struct CholFactorTask { const double *A; double *L; int n; int *status; };    // L: n * n + 1 doubles
constexpr int kCholFactorSmemN = 152;
constexpr int kCholFactorThreads = 512;
inline size_t chol_factor_smem_bytes(int n) {
  return ((n <= kCholFactorSmemN ? (size_t)n * n : 0) + 8 * (size_t)n + 8 * 9 + 8 + n) * sizeof(double);
}

__global__ void __launch_bounds__(kCholFactorThreads, 1) chol_factor_kernel(const CholFactorTask *__restrict__ tasks) {
  const CholFactorTask t = tasks[blockIdx.x];
  const int n = t.n;
  if (n <= 0) return;
  extern __shared__ double cf_sh[];
  const bool in_smem = n <= kCholFactorSmemN;
  double *W = in_smem ? cf_sh : t.L;                        // column-major n x n
  double *pan = cf_sh + (in_smem ? (size_t)n * n : 0);      // [8][n] the solved panel
  double (*blkd)[9] = (double (*)[9])(pan + 8 * (size_t)n);
  double *ipiv = (double *)(blkd + 8);
  double *diag0 = ipiv + 8;                                 // [n] original diagonal
  const int tid = threadIdx.x, nt = blockDim.x, warp = tid >> 5, lane = tid & 31, nw = nt >> 5;
  for (int e = tid; e < n * n; e += nt) {
    const int j = e / n, i = e - j * n;      // column j, row i
    W[e] = i >= j ? 0.5 * (t.A[(size_t)i * n + j] + t.A[(size_t)j * n + i]) : 0.0;
  }
  for (int i = tid; i < n; i += nt) diag0[i] = t.A[(size_t)i * n + i];
  __syncthreads();
  int any_dead = 0;
  for (int j0 = 0; j0 < n; j0 += 8) {
    const int w = min(8, n - j0);
    // (1) 8 x 8 diagonal block: every lane of warp 0 factors it in registers, lane r writes row r
    if (tid < 32) {
      double Lb[8][8], piv[8];
#pragma unroll
      for (int r = 0; r < 8; ++r)
#pragma unroll
        for (int c = 0; c <= r; ++c) Lb[r][c] = (r < w && c < w) ? W[(size_t)(j0 + c) * n + j0 + r] : (r == c ? 1.0 : 0.0);
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        piv[c] = 0.0;
        if (c < w) {
          const double d = Lb[c][c], dg = diag0[j0 + c];
          const bool bad = !(d > 1e-13 * dg) || !(dg > 0);
          const double rs = bad ? 0.0 : rsqrt_pos(d);
          Lb[c][c] = bad ? 0.0 : d * rs;
          if (bad) any_dead = 1;
          piv[c] = rs;
#pragma unroll
          for (int r = c + 1; r < 8; ++r) Lb[r][c] *= rs;
#pragma unroll
          for (int cc = c + 1; cc < 8; ++cc)
#pragma unroll
            for (int r = cc; r < 8; ++r) Lb[r][cc] = fma(-Lb[r][c], Lb[cc][c], Lb[r][cc]);
        }
      }
      if (tid < 8) {
#pragma unroll
        for (int rr = 0; rr < 8; ++rr)
          if (rr == tid) {
#pragma unroll
            for (int c = 0; c < 8; ++c) blkd[rr][c] = c <= rr ? Lb[rr][c] : 0.0;
          }
      }
      if (tid == 0) {
#pragma unroll
        for (int c = 0; c < 8; ++c) ipiv[c] = piv[c];
      }
    }
    __syncthreads();
    // (2) rows of the panel: x_c = (p_c - sum_{l<c} x_l L[c][l]) / L[c][c]; rows inside the block take the factored values
    for (int i = j0 + tid; i < n; i += nt) {
      double x[8];
      if (i < j0 + w) {
#pragma unroll
        for (int c = 0; c < 8; ++c) x[c] = blkd[i - j0][c];
      } else {
#pragma unroll
        for (int c = 0; c < 8; ++c) x[c] = c < w ? W[(size_t)(j0 + c) * n + i] : 0.0;
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          if (c < w) {
            double acc = x[c];
#pragma unroll
            for (int l = 0; l < c; ++l) acc = fma(-x[l], blkd[c][l], acc);
            x[c] = acc * ipiv[c];
          }
        }
      }
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        if (c < w) { W[(size_t)(j0 + c) * n + i] = x[c]; pan[c * n + i] = x[c]; }
      }
    }
    __syncthreads();
    // (3) trailing update of the lower triangle: W[i][j] -= sum_c P[i][c] P[j][c], a warp per column, lanes along rows
    const int m0 = j0 + w;
    for (int j = m0 + warp; j < n; j += nw) {
      double pj[8];
#pragma unroll
      for (int c = 0; c < 8; ++c) pj[c] = pan[c * n + j];
      for (int i = j + lane; i < n; i += 32) {
        double acc = 0;
#pragma unroll
        for (int c = 0; c < 8; ++c) acc = fma(pan[c * n + i], pj[c], acc);
        W[(size_t)j * n + i] -= acc;
      }
    }
    __syncthreads();
  }
  if (in_smem)
    for (int e = tid; e < n * n; e += nt) t.L[e] = W[e];
  if (tid == 0) {      // max |L_ij|^2 <= max M_ii: exponent for the single-precision iteration
    double mxd = 0.0;
    for (int i = 0; i < n; ++i) mxd = fmax(mxd, diag0[i]);
    int e2 = 0;
    if (mxd > 0.0 && mxd < 1e300) { frexp(mxd, &e2); }
    t.L[(size_t)n * n] = (double)((e2 + 1) / 2 + 1);
  }
  if (tid == 0 && any_dead && t.status) atomicOr(t.status, 2);
}

}  // namespace jolt
