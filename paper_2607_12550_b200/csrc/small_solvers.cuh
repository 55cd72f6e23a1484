// Batched small dense solvers in fp64, one CTA per problem: symmetric eigen-decomposition by
// parallel two-sided Jacobi (round-robin ordering), Cholesky with dead-pivot deflation and the
// inverse of the triangular factor (the pieces of CholeskyQR2).  Problems live in global memory
// (L2-resident: n <= 522 in the randomized path).
#pragma once
#include "common.cuh"

namespace jolt {

struct EigTask {
  double *A;        // n x n symmetric, row-major; destroyed
  double *Vt;       // n x n scratch; row i holds eigenvector i (unsorted) on exit
  double *w;        // n scratch eigenvalues (unsorted)
  float *U_out;     // optional: n x r_out, column j = eigenvector of the j-th largest eigenvalue
  int ld_out, r_out;
  float *w_out;     // optional: n eigenvalues, descending, clamped at 0
  int w_sqrt;       // 1: write sqrt(max(w,0)) instead (singular values)
  int n;
  int *status;      // set to 1 if not converged
};

constexpr int kEigThreads = 1024;
constexpr int kEigMaxSweeps = 40;

__device__ __forceinline__ void rr_pair(int r, int i, int ne, int &p, int &q) {
  // circle method on ne (even) players: round r in [0, ne-1), slot i in [0, ne/2)
  const int md = ne - 1;
  if (i == 0) { p = md; q = r % md; }
  else { p = (r + i) % md; q = (r - i + md) % md; }
  if (p > q) { const int tmp = p; p = q; q = tmp; }
}

__global__ void __launch_bounds__(kEigThreads) jacobi_eig_kernel(const EigTask *__restrict__ tasks) {
  const EigTask t = tasks[blockIdx.x];
  const int n = t.n;
  if (n <= 0) return;
  double *A = t.A, *Vt = t.Vt;
  const int tid = threadIdx.x, nt = blockDim.x;
  const int ne = (n + 1) & ~1;          // padded to even; index n (if present) is a bye
  const int np = ne / 2;
  extern __shared__ double sh[];        // c[np], s[np], red[32]
  double *cs_c = sh, *cs_s = sh + np, *red = sh + 2 * np;
  __shared__ int pp[1024], qq[1024];    // np <= 1024 (n <= 2048)
  __shared__ int rk[2048];
  __shared__ double s_total, s_off;

  for (int i = tid; i < n * n; i += nt) Vt[i] = ((i / n) == (i % n)) ? 1.0 : 0.0;
  // ||A||_F^2
  double loc = 0;
  for (int i = tid; i < n * n; i += nt) loc += A[i] * A[i];
  for (int o = 16; o; o >>= 1) loc += __shfl_xor_sync(0xffffffffu, loc, o);
  if ((tid & 31) == 0) red[tid >> 5] = loc;
  __syncthreads();
  if (tid == 0) { double s = 0; for (int i = 0; i < nt / 32; ++i) s += red[i]; s_total = s; }
  __syncthreads();
  const double total = s_total;
  bool converged = (total == 0.0);
  int sweep = 0;
  for (; sweep < kEigMaxSweeps && !converged; ++sweep) {
    for (int r = 0; r < ne - 1; ++r) {
      for (int i = tid; i < np; i += nt) {
        int p, q; rr_pair(r, i, ne, p, q);
        double c = 1.0, s = 0.0;
        if (q < n) {
          const double apq = A[(size_t)p * n + q];
          const double app = A[(size_t)p * n + p], aqq = A[(size_t)q * n + q];
          if (fabs(apq) > 1e-300 && fabs(apq) > 1e-17 * sqrt(fabs(app * aqq))) {
            const double tau = (aqq - app) / (2.0 * apq);
            const double tt = (tau >= 0 ? 1.0 : -1.0) / (fabs(tau) + sqrt(1.0 + tau * tau));
            c = 1.0 / sqrt(1.0 + tt * tt);
            s = tt * c;
          }
        } else { q = p; }
        pp[i] = p; qq[i] = q; cs_c[i] = c; cs_s[i] = s;
      }
      __syncthreads();
      // rows of A and of Vt:  row_p' = c row_p - s row_q ; row_q' = s row_p + c row_q
      for (int it = tid; it < np * n; it += nt) {
        const int i = it / n, j = it - i * n;
        const int p = pp[i], q = qq[i];
        if (p == q) continue;
        const double c = cs_c[i], s = cs_s[i];
        if (s == 0.0) continue;
        double ap = A[(size_t)p * n + j], aq = A[(size_t)q * n + j];
        A[(size_t)p * n + j] = c * ap - s * aq;
        A[(size_t)q * n + j] = s * ap + c * aq;
        double vp = Vt[(size_t)p * n + j], vq = Vt[(size_t)q * n + j];
        Vt[(size_t)p * n + j] = c * vp - s * vq;
        Vt[(size_t)q * n + j] = s * vp + c * vq;
      }
      __syncthreads();
      // columns of A
      for (int it = tid; it < np * n; it += nt) {
        const int row = it / np, i = it - row * np;
        const int p = pp[i], q = qq[i];
        if (p == q) continue;
        const double c = cs_c[i], s = cs_s[i];
        if (s == 0.0) continue;
        double ap = A[(size_t)row * n + p], aq = A[(size_t)row * n + q];
        A[(size_t)row * n + p] = c * ap - s * aq;
        A[(size_t)row * n + q] = s * ap + c * aq;
      }
      __syncthreads();
    }
    // off-diagonal mass
    double off = 0;
    for (int i = tid; i < n * n; i += nt) { if ((i / n) != (i % n)) off += A[i] * A[i]; }
    for (int o = 16; o; o >>= 1) off += __shfl_xor_sync(0xffffffffu, off, o);
    if ((tid & 31) == 0) red[tid >> 5] = off;
    __syncthreads();
    if (tid == 0) { double s = 0; for (int i = 0; i < nt / 32; ++i) s += red[i]; s_off = s; }
    __syncthreads();
    converged = (s_off <= 1e-26 * total);
    __syncthreads();
  }
  if (!converged && tid == 0 && t.status) *t.status = 1;
  for (int i = tid; i < n; i += nt) t.w[i] = A[(size_t)i * n + i];
  __syncthreads();
  // rank sort (descending, ties by index) and scatter
  for (int i = tid; i < n; i += nt) {
    const double wi = t.w[i];
    int rank = 0;
    for (int j = 0; j < n; ++j) { const double wj = t.w[j]; rank += (wj > wi) || (wj == wi && j < i); }
    if (t.w_out) { const double v = wi > 0 ? wi : 0.0; t.w_out[rank] = (float)(t.w_sqrt ? sqrt(v) : v); }
    if (n <= 2048) rk[i] = rank;
  }
  __syncthreads();
  if (t.U_out) {
    for (int it = tid; it < n * n; it += nt) {
      const int i = it / n, j = it - i * n;   // eigenvector i, component j
      int rank;
      if (n <= 2048) rank = rk[i];
      else {
        const double wi = t.w[i]; rank = 0;
        for (int jj = 0; jj < n; ++jj) { const double wj = t.w[jj]; rank += (wj > wi) || (wj == wi && jj < i); }
      }
      if (rank < t.r_out) t.U_out[(size_t)j * t.ld_out + rank] = (float)Vt[(size_t)i * n + j];
    }
  }
}

struct CholTask {
  double *G;        // n x n symmetric positive semi-definite (lower part used); overwritten by L
  double *Linv;     // n x n out: inverse of L (lower), rows of dead pivots zero
  float *LinvT32;   // optional n x n out, row-major: (L^-1)^T in fp32 (entry [c][j] = Linv[j][c])
  int n;
  int *status;      // bit 1 set if a pivot was deflated (rank deficiency; not an error)
};

__global__ void __launch_bounds__(1024) cholesky_inv_kernel(const CholTask *__restrict__ tasks) {
  const CholTask t = tasks[blockIdx.x];
  const int n = t.n;
  if (n <= 0) return;
  double *G = t.G;
  const int tid = threadIdx.x, nt = blockDim.x;
  __shared__ int dead[2048];
  __shared__ double s_piv;
  __shared__ double diag0[2048];
  for (int i = tid; i < n; i += nt) { diag0[i] = G[(size_t)i * n + i]; dead[i] = 0; }
  __syncthreads();
  for (int j = 0; j < n; ++j) {
    if (tid == 0) {
      const double a = G[(size_t)j * n + j];
      if (!(a > 1e-10 * diag0[j]) || !(diag0[j] > 0)) { dead[j] = 1; s_piv = 0.0; G[(size_t)j * n + j] = 1.0; }
      else { s_piv = sqrt(a); G[(size_t)j * n + j] = s_piv; }
    }
    __syncthreads();
    const double piv = s_piv;
    for (int i = j + 1 + tid; i < n; i += nt)
      G[(size_t)i * n + j] = (piv > 0) ? G[(size_t)i * n + j] / piv : 0.0;
    __syncthreads();
    if (piv > 0) {
      const int rem = n - j - 1;
      for (int it = tid; it < rem * rem; it += nt) {
        const int i = j + 1 + it / rem, l = j + 1 + it % rem;
        if (l <= i) G[(size_t)i * n + l] -= G[(size_t)i * n + j] * G[(size_t)l * n + j];
      }
    }
    __syncthreads();
  }
  // Linv by forward substitution, one thread per column c: solve L x = e_c
  for (int c = tid; c < n; c += nt) {
    for (int i = 0; i < n; ++i) {
      double v = 0.0;
      if (i >= c && !dead[i] && !dead[c]) {
        double acc = (i == c) ? 1.0 : 0.0;
        for (int l = c; l < i; ++l) acc -= G[(size_t)i * n + l] * t.Linv[(size_t)l * n + c];
        v = acc / G[(size_t)i * n + i];
      }
      t.Linv[(size_t)i * n + c] = v;
    }
  }
  __syncthreads();
  if (t.LinvT32)
    for (int it = tid; it < n * n; it += nt) {
      const int c = it / n, j = it - c * n;
      t.LinvT32[it] = (float)t.Linv[(size_t)j * n + c];
    }
  if (tid == 0 && t.status) { int any = 0; for (int i = 0; i < n; ++i) any |= dead[i]; if (any) atomicOr(t.status, 2); }
}

}  // namespace jolt
