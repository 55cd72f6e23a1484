// Starting basis for the fp64 block Jacobi solver (the mode-3 Gram eigenproblem, Sec. 4).
//
// The block solver needs eight to nine sweeps from the identity, each sweep a chain of launches; from a basis that
// already diagonalises the matrix to single precision it needs one.  Such a basis is cheap: the Cholesky factor of the
// (slightly shifted) matrix, then the cluster-resident single-precision one-sided Jacobi on its columns (~0.45 ms for
// n = 128 against ~1.2 ms of block rounds).  The kernels here do what surrounds that: the shift that keeps the factor
// defined when the matrix is rank deficient, and the congruence A' = U^T A U in fp64, which the block solver then
// diagonalises starting with V = U.  U is orthogonal only to ~4e-6 (single precision); the eigenvectors V = U J
// inherit that, which is below the fp16 resolution of the stored factor by two orders of magnitude.
#pragma once
#include "common.cuh"

namespace jolt {

struct PresolveTask {
  const double *A;   // n x n symmetric, row-major (not modified)
  double *Ash;       // n x n: A + shift I, the input of the Cholesky factorisation; later overwritten by A' = U^T A U
  const float *U;    // n x n, column j = j-th approximate eigenvector (row-major, leading dimension n)
  double *T;         // n x n scratch: A U
  int n;
};

// Ash = A + (1e-12 * trace / n) I: every pivot of the factorisation stays positive, the null directions of a rank
// deficient A become tiny columns of L that the one-sided Jacobi still orthogonalises (it works relative to each
// column's own norm), so U is a complete basis.  The shift never reaches the eigenvalues: A' is formed from A itself.
// grid (slices, matrices): every CTA sums the diagonal itself and shifts its slice of the rows.
__global__ void presolve_shift_kernel(const PresolveTask *__restrict__ tasks) {
  const PresolveTask t = tasks[blockIdx.y];
  const int n = t.n;
  __shared__ double red[32];
  double tr = 0.0;
  for (int i = threadIdx.x; i < n; i += blockDim.x) tr += t.A[(size_t)i * n + i];
  for (int o = 16; o; o >>= 1) tr += __shfl_xor_sync(0xffffffffu, tr, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = tr;
  __syncthreads();
  tr = 0.0;
  for (int w = 0; w < (int)blockDim.x / 32; ++w) tr += red[w];
  const double shift = 1e-12 * fabs(tr) / n;
  const int per = (n * n + gridDim.x - 1) / gridDim.x, e0 = blockIdx.x * per, e1 = min(n * n, e0 + per);
  for (int e = e0 + threadIdx.x; e < e1; e += blockDim.x) {
    const int i = e / n, j = e - i * n;
    t.Ash[e] = t.A[e] + (i == j ? shift : 0.0);
  }
}

// out[r0 .. r0+16)[0 .. n) = Lhs[r0 .. r0+16)[:] * Rhs, fp64.  SECOND = false: Lhs = A, Rhs = U (fp32), out = T;
// SECOND = true: Lhs = U^T, Rhs = T, out = Ash (= A').  grid (ceil(n / 16), matrices), 256 threads; n <= 256.
template <bool SECOND>
__global__ void __launch_bounds__(256) presolve_mul_kernel(const PresolveTask *__restrict__ tasks) {
  const PresolveTask t = tasks[blockIdx.y];
  const int n = t.n, r0 = blockIdx.x * 16;
  if (r0 >= n) return;
  __shared__ double lhs[16][257];
  for (int e = threadIdx.x; e < 16 * n; e += 256) {
    const int ri = e / n, k = e - ri * n;
    double v = 0.0;
    if (r0 + ri < n) v = SECOND ? (double)t.U[(size_t)k * n + r0 + ri] : t.A[(size_t)(r0 + ri) * n + k];
    lhs[ri][k] = v;
  }
  __syncthreads();
  const int ty = threadIdx.x >> 5, tx = threadIdx.x & 31;      // rows 2 ty, 2 ty + 1; columns tx + 32 c
  double *out = SECOND ? t.Ash : t.T;
  for (int c0 = 0; c0 < n; c0 += 128) {
    double acc[2][4] = {{0, 0, 0, 0}, {0, 0, 0, 0}};
    // unrolled: the loads of eight steps are in flight together (one step at a time left the kernel waiting on an L2
    // round trip per step)
#pragma unroll 8
    for (int k = 0; k < n; ++k) {
      const double a0 = lhs[2 * ty][k], a1 = lhs[2 * ty + 1][k];
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const int col = c0 + tx + 32 * c;
        double b = 0.0;
        if (col < n) b = SECOND ? t.T[(size_t)k * n + col] : (double)t.U[(size_t)k * n + col];
        acc[0][c] = fma(a0, b, acc[0][c]);
        acc[1][c] = fma(a1, b, acc[1][c]);
      }
    }
#pragma unroll
    for (int rr = 0; rr < 2; ++rr)
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const int row = r0 + 2 * ty + rr, col = c0 + tx + 32 * c;
        if (row < n && col < n) out[(size_t)row * n + col] = acc[rr][c];
      }
  }
}

}  // namespace jolt
