// Batched small dense solvers: symmetric eigen-decomposition by parallel two-sided Jacobi in fp64 (round-robin
// ordering, one CTA per problem; the multi-CTA block version is in block_jacobi.cuh) and the pieces of
// CholeskyQR2: tall Gram (fp64), Cholesky with dead-pivot deflation (fp64), row-wise triangular solve (fp32).
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
  // optional scratch of the multi-launch block solver (null: single-CTA kernels)
  double *bjA, *bjV, *bjJ, *bjOff; int *bjDone;
  // optional scratch of the single-precision pre-solve that gives the block solver its starting basis (null: start
  // from the identity): preL n*n+8 doubles, preU n*n floats, preT and preA n*n doubles each
  double *preL; float *preU; double *preT, *preA;
};

constexpr int kEigThreads = 1024;
constexpr int kEigMaxSweeps = 40;

// Jacobi rotation that annihilates apq, without divisions: with d = (aqq - app)/2 and h = hypot(d, apq),
// cos 2t = |d|/h, so c = sqrt((1 + |d|/h)/2) and s = sgn(d) apq / (2 h c); two reciprocal square roots.
__device__ __forceinline__ void jacobi_cs(double app, double aqq, double apq, double &c, double &s) {
  c = 1.0; s = 0.0;
  const double d = 0.5 * (aqq - app);
  const double u = d * d + apq * apq;
  if (!(fabs(apq) > 1e-17 * sqrt(fabs(app * aqq))) || !(u > 1e-280)) return;
  const double rh = rsqrt(u);
  const double x = 0.5 + 0.5 * fabs(d) * rh;
  const double rc = rsqrt(x);
  c = x * rc;
  s = (d >= 0 ? 0.5 : -0.5) * apq * rh * rc;
}

// Same rotation with the angle evaluated in fp32 (hardware rsqrt) and the pair (c, s) then renormalised
// in fp64: the rotation is orthogonal to 1e-15, its angle is good to ~1e-7, which leaves a residual
// apq' ~ 1e-7 apq for the next sweep instead of an exact zero.
__device__ __forceinline__ void jacobi_cs_fast(double app, double aqq, double apq, double &c, double &s) {
  c = 1.0; s = 0.0;
  const double d = 0.5 * (aqq - app);
  if (!(apq * apq > 1e-34 * fabs(app * aqq))) return;
  const double mx = fmax(fabs(d), fabs(apq));
  if (!(mx > 1e-290) || !(mx < 1e290)) return;
  // scale by a power of two near 1/mx (exponent arithmetic only)
  const int ex = ((__double2hiint(mx) >> 20) & 0x7ff) - 1023;
  const double sc = __hiloint2double((1023 - ex) << 20, 0);
  const float df = (float)(d * sc), af = (float)(apq * sc);
  const float rh = rsqrtf(df * df + af * af);
  const float x = 0.5f + 0.5f * fabsf(df) * rh;
  const float rc = rsqrtf(x);
  double cc = (double)(x * rc), ss = (double)((df >= 0.f ? 0.5f : -0.5f) * af * rh * rc);
  const double e = fma(cc, cc, fma(ss, ss, -1.0));
  const double corr = fma(e, fma(e, 0.375, -0.5), 1.0);
  c = cc * corr; s = ss * corr;
}

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

// Shared-memory variant for n <= kEigSmemMaxN: the symmetric matrix lives as a packed lower triangle in
// fp64, the eigenvector accumulator as fp32 rows.  One round = rotation parameters for n/2 disjoint pairs,
// then ONE fused update: every 2x2 block A[{p_a,q_a}][{p_b,q_b}] (a <= b) becomes J_a^T blk J_b, and rows
// p, q of V^T rotate.  Two barriers per round, no global traffic.
constexpr int kEigSmemMaxN = 168;
constexpr size_t kSmemOptIn = 232448;    // 227 KB of dynamic shared memory per CTA

__host__ __device__ inline size_t eig_smem_bytes(int n, size_t vsize) {
  const int np = (n + 1) / 2;
  size_t b = (size_t)n * (n + 1) / 2 * sizeof(double);       // packed A
  b += (size_t)np * 2 * sizeof(double);                       // c, s
  b += 40 * sizeof(double);                                   // reduction scratch
  b += (size_t)n * n * vsize;                                 // V^T
  b += (size_t)np * 2 * sizeof(int) + (size_t)n * sizeof(int) + 64;
  return b;
}

__device__ __forceinline__ int tri_idx(int i, int j) { return i >= j ? i * (i + 1) / 2 + j : j * (j + 1) / 2 + i; }

template <typename VT>
__global__ void __launch_bounds__(kEigThreads, 1) jacobi_eig_smem_kernel(const EigTask *__restrict__ tasks) {
  const EigTask t = tasks[blockIdx.x];
  const int n = t.n;
  if (n <= 0) return;
  extern __shared__ double shd[];
  const int ne = (n + 1) & ~1, np = ne / 2;
  const int ntri = n * (n + 1) / 2;
  double *A = shd;
  double *cs_c = A + ntri, *cs_s = cs_c + np, *red = cs_s + np;
  VT *Vt = (VT *)(red + 40);
  int *pp = (int *)(Vt + (size_t)n * n), *qq = pp + np, *rk = qq + np;
  __shared__ double s_total, s_off;
  const int tid = threadIdx.x, nt = blockDim.x;

  double loc = 0;
  for (int e = tid; e < n * n; e += nt) {
    const int i = e / n, j = e - i * n;
    const double v = t.A[e];
    loc += v * v;
    if (j <= i) A[i * (i + 1) / 2 + j] = (i == j) ? v : 0.5 * (v + t.A[(size_t)j * n + i]);
    Vt[e] = (i == j) ? VT(1) : VT(0);
  }
  for (int o = 16; o; o >>= 1) loc += __shfl_xor_sync(0xffffffffu, loc, o);
  if ((tid & 31) == 0) red[tid >> 5] = loc;
  __syncthreads();
  if (tid == 0) { double s = 0; for (int i = 0; i < nt / 32; ++i) s += red[i]; s_total = s; }
  __syncthreads();
  const double total = s_total;
  bool converged = (total == 0.0);
  // static work assignment (the same every round): up to 4 pair-blocks (a <= b) per thread, one column of
  // V^T per thread with a fixed stride over the pairs
  const int nblk = np * (np + 1) / 2;
  int blk_ab[4];
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    const int w = tid + u * nt;
    blk_ab[u] = -1;
    if (w < nblk) {
      int b = (int)((sqrtf(8.0f * w + 1.0f) - 1.0f) * 0.5f);
      while ((b + 1) * (b + 2) / 2 <= w) ++b;
      while (b * (b + 1) / 2 > w) --b;
      blk_ab[u] = (b << 16) | (w - b * (b + 1) / 2);
    }
  }
  const int vcols = nt / n;                 // thread groups over the pairs
  const int vj = tid % n, vi0 = tid / n;    // this thread's column and first pair
  for (int sweep = 0; sweep < kEigMaxSweeps && !converged; ++sweep) {
    for (int r = 0; r < ne - 1; ++r) {
      for (int i = tid; i < np; i += nt) {
        int p, q; rr_pair(r, i, ne, p, q);
        double c = 1.0, s = 0.0;
        if (q < n) {
          const double apq = A[q * (q + 1) / 2 + p];
          const double app = A[p * (p + 1) / 2 + p], aqq = A[q * (q + 1) / 2 + q];
          jacobi_cs(app, aqq, apq, c, s);
        } else { q = -1; }
        pp[i] = p; qq[i] = q; cs_c[i] = c; cs_s[i] = s;
      }
      __syncthreads();
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (blk_ab[u] < 0) continue;
        const int b = blk_ab[u] >> 16, a = blk_ab[u] & 0xffff;
        const int pa = pp[a], qa = qq[a], pb = pp[b], qb = qq[b];
        const double ca = cs_c[a], sa = cs_s[a], cb = cs_c[b], sb = cs_s[b];
        if (a == b) {
          if (qa < 0 || sa == 0.0) continue;
          const int ipp = pa * (pa + 1) / 2 + pa, iqq = qa * (qa + 1) / 2 + qa, ipq = qa * (qa + 1) / 2 + pa;
          const double app = A[ipp], aqq = A[iqq], apq = A[ipq];
          A[ipp] = ca * ca * app - 2.0 * ca * sa * apq + sa * sa * aqq;
          A[iqq] = sa * sa * app + 2.0 * ca * sa * apq + ca * ca * aqq;
          A[ipq] = 0.0;
          continue;
        }
        if (sa == 0.0 && sb == 0.0) continue;
        const int i_pp = tri_idx(pa, pb);
        double x_pp = A[i_pp], x_pq = 0, x_qp = 0, x_qq = 0;
        int i_pq = -1, i_qp = -1, i_qq = -1;
        if (qb >= 0) { i_pq = tri_idx(pa, qb); x_pq = A[i_pq]; }
        if (qa >= 0) { i_qp = tri_idx(qa, pb); x_qp = A[i_qp]; }
        if (qa >= 0 && qb >= 0) { i_qq = tri_idx(qa, qb); x_qq = A[i_qq]; }
        const double r_pp = ca * x_pp - sa * x_qp, r_pq = ca * x_pq - sa * x_qq;
        const double r_qp = sa * x_pp + ca * x_qp, r_qq = sa * x_pq + ca * x_qq;
        A[i_pp] = cb * r_pp - sb * r_pq;
        if (i_pq >= 0) A[i_pq] = sb * r_pp + cb * r_pq;
        if (i_qp >= 0) A[i_qp] = cb * r_qp - sb * r_qq;
        if (i_qq >= 0) A[i_qq] = sb * r_qp + cb * r_qq;
      }
      if (vi0 < vcols) {
        for (int i = vi0; i < np; i += vcols) {
          const int q = qq[i];
          const VT s = (VT)cs_s[i];
          if (q < 0 || s == VT(0)) continue;
          const int p = pp[i];
          const VT c = (VT)cs_c[i];
          const VT vp = Vt[p * n + vj], vq = Vt[q * n + vj];
          Vt[p * n + vj] = c * vp - s * vq;
          Vt[q * n + vj] = s * vp + c * vq;
        }
      }
      __syncthreads();
    }
    double off = 0;
    for (int e = tid; e < ntri; e += nt) {
      int i = (int)((sqrtf(8.0f * e + 1.0f) - 1.0f) * 0.5f);
      while ((i + 1) * (i + 2) / 2 <= e) ++i;
      while (i * (i + 1) / 2 > e) --i;
      if (e - i * (i + 1) / 2 != i) { const double v = A[e]; off += v * v; }   // skip the diagonal (no cancellation)
    }
    for (int o = 16; o; o >>= 1) off += __shfl_xor_sync(0xffffffffu, off, o);
    if ((tid & 31) == 0) red[tid >> 5] = off;
    __syncthreads();
    if (tid == 0) { double s = 0; for (int i = 0; i < nt / 32; ++i) s += red[i]; s_off = 2.0 * s; }
    __syncthreads();
    converged = (s_off <= 1e-24 * total);
    __syncthreads();
  }
  if (!converged && tid == 0 && t.status) atomicOr(t.status, 1);
  for (int i = tid; i < n; i += nt) t.w[i] = A[i * (i + 1) / 2 + i];
  __syncthreads();
  for (int i = tid; i < n; i += nt) {
    const double wi = t.w[i];
    int rank = 0;
    for (int j = 0; j < n; ++j) { const double wj = t.w[j]; rank += (wj > wi) || (wj == wi && j < i); }
    if (t.w_out) { const double v = wi > 0 ? wi : 0.0; t.w_out[rank] = (float)(t.w_sqrt ? sqrt(v) : v); }
    rk[i] = rank;
  }
  __syncthreads();
  if (t.U_out)
    for (int it = tid; it < n * n; it += nt) {
      const int j = it / n, i = it - j * n;
      const int rank = rk[i];
      if (rank < t.r_out) t.U_out[(size_t)j * t.ld_out + rank] = (float)Vt[i * n + j];
    }
}

// ---- CholeskyQR pieces ------------------------------------------------------------------------------------
// cholesky_smem_kernel: G = L L^T in fp64.  A pivot that is not above 1e-10 of its original diagonal entry is
// deflated (the column of L is zeroed, the diagonal set to 1, status bit 2): rank-deficient sketches lose the
// dependent directions instead of dividing by rounding noise.  Writes
// LT[l][j] = L[j][l] (fp32, pitch kp = n rounded up to 8, zero above the diagonal of L) and invd[j] = 1 / L[j][j]
// (0 for a dead pivot).  trsm_rows_kernel then solves  dst_row * L^T = src_row  for 128 rows per CTA.
constexpr int kCholSmemMaxN = 168;

// 1 / sqrt(d) for d > 0: single-precision seed and two Newton steps in fp64 (full accuracy), the library routine
// outside the single-precision range
__device__ __forceinline__ double rsqrt_pos(double d) {
  if (!(d > 1e-30 && d < 1e30)) return rsqrt(d);
  const double h = 0.5 * d;
  double y = (double)rsqrtf((float)d);
  y = y * fma(-h * y, y, 1.5);
  y = y * fma(-h * y, y, 1.5);
  return y;
}


struct CholSmemTask { const double *G; float *LT; float *invd; int n; int *status; double *work; };

__global__ void __launch_bounds__(512, 1) cholesky_smem_kernel(const CholSmemTask *__restrict__ tasks, int in_global) {
  // Left-looking Cholesky by panels of 8 columns.  (1) The panel loses the contribution of the finished columns,
  // one dot product per entry on four independent accumulators.  (2) Warp 0 factors the 8 x 8 diagonal block in
  // registers (reciprocal square roots instead of divisions).  (3) The rows below are solved against the
  // block, one thread per row.  Three barriers per panel.
  const CholSmemTask t = tasks[blockIdx.x];
  const int n = t.n;
  if (n <= 0) return;
  extern __shared__ double shd[];
  const int ld = n + 1;
  // the work matrix lives in shared memory when it fits (n <= kCholSmemMaxN), else in a global buffer that the
  // CTA reads through L1 (all its threads sit on one SM, so their writes are seen after a barrier)
  double *A = in_global ? t.work : shd;                         // n x (n+1)
  double *diag0 = in_global ? shd : shd + (size_t)n * ld;       // n
  int *dead = (int *)(diag0 + n);                               // n
  __shared__ double blk[8][9];           // the factored diagonal block
  __shared__ double ipiv[8];
  const int tid = threadIdx.x, nt = blockDim.x;
  for (int e0 = tid; e0 < n * n; e0 += nt * 8) {
    double v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) { const int e = e0 + u * nt; v[u] = e < n * n ? t.G[e] : 0.0; }
#pragma unroll
    for (int u = 0; u < 8; ++u) { const int e = e0 + u * nt; if (e < n * n) { const int i = e / n, j = e - i * n; A[i * ld + j] = v[u]; } }
  }
  __syncthreads();
  for (int i = tid; i < n; i += nt) { diag0[i] = A[i * ld + i]; dead[i] = 0; }
  __syncthreads();
  for (int j0 = 0; j0 < n; j0 += 8) {
    const int w = min(8, n - j0);
    // (1) panel minus the contribution of the finished columns (lower part of the diagonal block included)
    for (int e = tid; e < (n - j0) * 8; e += nt) {
      const int i = j0 + (e >> 3), c = e & 7;
      if (c >= w || j0 + c > i) continue;
      const double *ri = A + i * ld, *rc = A + (j0 + c) * ld;
      double a0 = 0, a1 = 0, a2 = 0, a3 = 0;
      int l = 0;
      for (; l + 4 <= j0; l += 4) {
        a0 = fma(ri[l], rc[l], a0); a1 = fma(ri[l + 1], rc[l + 1], a1);
        a2 = fma(ri[l + 2], rc[l + 2], a2); a3 = fma(ri[l + 3], rc[l + 3], a3);
      }
      for (; l < j0; ++l) a0 = fma(ri[l], rc[l], a0);
      A[i * ld + j0 + c] -= (a0 + a1) + (a2 + a3);
    }
    __syncthreads();
    // (2) the 8 x 8 diagonal block: every lane of warp 0 factors the whole block in its own registers (36 entries,
    // broadcast loads, no shuffles on the dependent chain); lane r then writes row r back
    if (tid < 32) {
      double L[8][8], piv[8];
#pragma unroll
      for (int r = 0; r < 8; ++r)
#pragma unroll
        for (int c = 0; c <= r; ++c) L[r][c] = (r < w) ? A[(j0 + r) * ld + j0 + c] : (r == c ? 1.0 : 0.0);
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        piv[c] = 0.0;
        if (c < w) {
          const double d = L[c][c], dg = diag0[j0 + c];
          const bool bad = !(d > 1e-10 * dg) || !(dg > 0);
          const double rs = bad ? 0.0 : rsqrt_pos(d);
          L[c][c] = bad ? 1.0 : d * rs;
          if (tid == 0 && bad) dead[j0 + c] = 1;
          piv[c] = rs;
#pragma unroll
          for (int r = c + 1; r < 8; ++r) L[r][c] *= rs;
#pragma unroll
          for (int cc = c + 1; cc < 8; ++cc)
#pragma unroll
            for (int r = cc; r < 8; ++r) L[r][cc] = fma(-L[r][c], L[cc][c], L[r][cc]);
        }
      }
      const int r = tid & 7;
      if (tid < w) {
#pragma unroll
        for (int rr = 0; rr < 8; ++rr)
          if (rr == r) {
#pragma unroll
            for (int c = 0; c <= rr; ++c) { A[(j0 + rr) * ld + j0 + c] = L[rr][c]; blk[rr][c] = L[rr][c]; }
          }
      }
      if (tid == 0) {
#pragma unroll
        for (int c = 0; c < 8; ++c) ipiv[c] = piv[c];
      }
    }
    __syncthreads();
    // (3) rows below the block: x_c = (p_c - sum_{l<c} x_l L[c][l]) / L[c][c]
    for (int i = j0 + w + tid; i < n; i += nt) {
      double *ri = A + i * ld + j0;
      double x[8];
#pragma unroll
      for (int c = 0; c < 8; ++c) x[c] = c < w ? ri[c] : 0.0;
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        if (c < w) {
          double acc = x[c];
#pragma unroll
          for (int l = 0; l < c; ++l) acc = fma(-x[l], blk[c][l], acc);
          x[c] = acc * ipiv[c];
          ri[c] = x[c];
        }
      }
    }
    __syncthreads();
  }
  const int kp = (n + 7) & ~7;
  for (int e = tid; e < n * kp; e += nt) {
    const int l = e / kp, j = e - l * kp;
    t.LT[e] = (j < n && j >= l) ? (float)A[j * ld + l] : 0.f;
  }
  for (int j = tid; j < n; j += nt) t.invd[j] = dead[j] ? 0.f : (float)(1.0 / A[j * ld + j]);
  if (tid == 0 && t.status) { int any = 0; for (int i = 0; i < n; ++i) any |= dead[i]; if (any) atomicOr(t.status, 2); }
}

inline size_t chol_smem_bytes(int n, bool in_global = false) {
  return ((in_global ? 0 : (size_t)n * (n + 1)) + n) * sizeof(double) + (size_t)n * sizeof(int) + 64;
}

// Optional second output: the solved rows again as the hi + lo fp16 operand of the next tensor-core sweep (scaled by
// 2^scale_exp, zero-padded to kp16 columns), so that no separate split / transpose pass is needed.
//   split_mode 1: [kp16][rows]           (token-side basis, operand of the projection sweep)
//   split_mode 2: [rows / 128][kp16][128] (feature-side basis, rows = (head, feature), operand of the sketch sweep)
struct TrsmJob {
  const float *src; float *dst; int rows, k; const float *LT; const float *invd;
  __half *hi, *lo; int split_mode, kp16, scale_exp;
};

inline size_t trsm_smem_bytes(int k, int rb, bool lt_global = false) {
  const int kp = (k + 7) & ~7;
  return ((lt_global ? 0 : (size_t)k * kp) + (size_t)kp * (rb + 1) + kp) * sizeof(float) + 64;
}

// RB rows per CTA (256 when the tile fits shared memory, else 128 or 64), RB / 2 threads: a thread solves two rows,
// eight columns at a time, so that one pair of 16-byte loads of L^T feeds 16 FMAs.
template <int RB>
__global__ void __launch_bounds__(RB / 2) trsm_rows_kernel(const TrsmJob *__restrict__ jobs, int lt_global) {
  constexpr int NT = RB / 2;
  const TrsmJob t = jobs[blockIdx.y];
  const int r0 = blockIdx.x * RB;
  if (r0 >= t.rows) return;
  const int k = t.k, kp = (k + 7) & ~7;
  constexpr int PITCH = RB + 1;
  extern __shared__ float shf[];
  // L^T stays in global memory (read through L1, every lane of a warp reads the same entries) when it does not fit
  // beside the row tile
  float *LTs = shf;                                              // k x kp
  float *sp = lt_global ? shf : shf + (size_t)k * kp;            // kp x PITCH  (feature j, row r)
  float *invd = sp + (size_t)kp * PITCH;                         // kp
  const float *__restrict__ LT = lt_global ? t.LT : LTs;
  const int tid = threadIdx.x;
  const int nrows = min(RB, t.rows - r0);
  // staging loops read several elements into registers before the first shared-memory store, so that the global
  // loads of a trip are in flight together
  if (!lt_global) {
    const float4 *g4 = (const float4 *)t.LT;
    float4 *s4 = (float4 *)LTs;
    const int n4 = k * kp / 4;
    for (int e0 = tid; e0 < n4; e0 += NT * 4) {
      float4 v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) { const int e = e0 + u * NT; if (e < n4) v[u] = g4[e]; }
#pragma unroll
      for (int u = 0; u < 4; ++u) { const int e = e0 + u * NT; if (e < n4) s4[e] = v[u]; }
    }
  }
  for (int j = tid; j < kp; j += NT) invd[j] = j < k ? t.invd[j] : 0.f;
  const float *src = t.src + (size_t)r0 * k;
  const int tot = nrows * k;
  if ((((size_t)r0 * k) & 3) == 0) {          // the row block starts on a 16-byte boundary: vector loads
    const float4 *src4 = (const float4 *)src;
    const int tot4 = tot >> 2;
    for (int e0 = tid; e0 < tot4; e0 += NT * 8) {
      float4 v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) { const int e = e0 + u * NT; if (e < tot4) v[u] = src4[e]; }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int e = e0 + u * NT;
        if (e < tot4) {
          int r = (4 * e) / k, j = 4 * e - r * k;
          const float vv[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
          for (int c = 0; c < 4; ++c) { sp[j * PITCH + r] = vv[c]; if (++j == k) { j = 0; ++r; } }
        }
      }
    }
    for (int e = (tot4 << 2) + tid; e < tot; e += NT) { const int r = e / k, j = e - r * k; sp[j * PITCH + r] = src[e]; }
  } else {
    for (int e0 = tid; e0 < tot; e0 += NT * 8) {
      float v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) { const int e = e0 + u * NT; v[u] = e < tot ? src[e] : 0.f; }
#pragma unroll
      for (int u = 0; u < 8; ++u) { const int e = e0 + u * NT; if (e < tot) { const int r = e / k, j = e - r * k; sp[j * PITCH + r] = v[u]; } }
    }
  }
  for (int e = tid; e < (kp - k) * PITCH; e += NT) sp[k * PITCH + e] = 0.f;
  __syncthreads();
  if (tid < nrows) {
    const int ra = tid, rb = tid + NT;            // row rb may lie beyond the ragged end: computed, never written out
    for (int jb = 0; jb < kp; jb += 8) {
      float a[8], b[8];
#pragma unroll
      for (int c = 0; c < 8; ++c) { a[c] = sp[(jb + c) * PITCH + ra]; b[c] = sp[(jb + c) * PITCH + rb]; }
      // jb is a multiple of 8: four finished columns per trip, all loads of a trip issued before its 64 FMAs
      for (int l = 0; l < jb; l += 4) {
        float xa[4], xb[4]; float4 L0[4], L1[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          xa[u] = sp[(l + u) * PITCH + ra]; xb[u] = sp[(l + u) * PITCH + rb];
          L0[u] = *(const float4 *)&LT[(l + u) * kp + jb]; L1[u] = *(const float4 *)&LT[(l + u) * kp + jb + 4];
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const float Lv[8] = {L0[u].x, L0[u].y, L0[u].z, L0[u].w, L1[u].x, L1[u].y, L1[u].z, L1[u].w};
#pragma unroll
          for (int c = 0; c < 8; ++c) { a[c] = fmaf(-xa[u], Lv[c], a[c]); b[c] = fmaf(-xb[u], Lv[c], b[c]); }
        }
      }
      // the 8 x 8 triangle of the block itself
#pragma unroll
      for (int c = 0; c < 8; ++c) {
#pragma unroll
        for (int i = 0; i < c; ++i) { const float Lic = LT[(jb + i) * kp + jb + c]; a[c] = fmaf(-a[i], Lic, a[c]); b[c] = fmaf(-b[i], Lic, b[c]); }
        const float d = invd[jb + c];
        a[c] *= d; b[c] *= d;
      }
#pragma unroll
      for (int c = 0; c < 8; ++c) { sp[(jb + c) * PITCH + ra] = a[c]; sp[(jb + c) * PITCH + rb] = b[c]; }
    }
  }
  __syncthreads();
  float *dst = t.dst + (size_t)r0 * k;
  for (int e = tid; e < nrows * k; e += NT) { const int r = e / k, j = e - r * k; dst[e] = sp[j * PITCH + r]; }
  if (t.split_mode) {
    const float sc = ldexpf(1.0f, t.scale_exp);
    for (int e = tid; e < nrows * t.kp16; e += NT) {
      const int j = e / nrows, r = e - j * nrows;          // r fastest: conflict-free reads, contiguous writes
      const float v = j < k ? sp[j * PITCH + r] * sc : 0.f;
      const __half h = __float2half_rn(v);
      const int row = r0 + r;
      const size_t o = t.split_mode == 1 ? (size_t)j * t.rows + row
                                         : ((size_t)(row >> 7) * t.kp16 + j) * 128 + (row & 127);
      t.hi[o] = h;
      t.lo[o] = __float2half_rn(v - __half2float(h));
    }
  }
}

// sum of fp64 partials with a per-job element count
struct ReduceJob { const double *parts; double *out; int count, n_elems; };
__global__ void reduce_partials_var_kernel(const ReduceJob *__restrict__ jobs) {
  const ReduceJob j = jobs[blockIdx.y];
  for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < j.n_elems; e += gridDim.x * blockDim.x) {
    double s = 0;
    for (int h = 0; h < j.count; ++h) s += j.parts[(size_t)h * j.n_elems + e];
    j.out[e] = s;
  }
}


// ---- G = M^T M for a tall fp32 matrix, fp64 accumulation, one partial per row chunk ---------------------
// Each of the 16 x 16 threads owns a TI x TI register tile of the k x k result (k <= 16 TI), rows stream
// through shared memory 16 at a time (converted to fp64 once, on the way in).
// One job = one block (columns [ca, ca+wa) x [cb, cb+wb)) of the k x k Gram; k <= 16 TI takes a single block,
// wider matrices the lower-triangular blocks, whose results are also written mirrored.
struct TallGramJob { const float *M; int rows, k, chunk; double *part; int ca, wa, cb, wb; };

template <int TI, bool SAME>      // SAME: diagonal block (ca == cb), one staged tile serves both operands
__global__ void __launch_bounds__(256, 1) tall_gram_kernel(const TallGramJob *__restrict__ jobs) {
  const TallGramJob t = jobs[blockIdx.y];
  const int r_begin = blockIdx.x * t.chunk;
  if (r_begin >= t.rows) return;
  const int r_end = min(t.rows, r_begin + t.chunk);
  constexpr int W = 16 * TI;
  __shared__ double Ma[16][W + 2], Mb[SAME ? 1 : 16][W + 2];
  constexpr bool same = SAME;
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  double acc[TI][TI];
#pragma unroll
  for (int i = 0; i < TI; ++i)
#pragma unroll
    for (int j = 0; j < TI; ++j) acc[i][j] = 0.0;
  // the 16 x W tile is TI elements per thread (and per operand); the next tile's elements are fetched into registers
  // while the current one is being multiplied, so the global-load latency hides behind the 16 * TI * TI FMAs
  float pa[TI], pb[TI];
  auto fetch = [&](int r0) {
    const int nr = min(16, r_end - r0);
#pragma unroll
    for (int u = 0; u < TI; ++u) {
      const int e = tid + u * 256, r = e / W, c = e - r * W;
      const float *row = t.M + (size_t)(r0 + r) * t.k;
      pa[u] = (r < nr && c < t.wa) ? row[t.ca + c] : 0.f;
      if (!same) pb[u] = (r < nr && c < t.wb) ? row[t.cb + c] : 0.f;
    }
  };
  if (r_begin < r_end) fetch(r_begin);
  for (int r0 = r_begin; r0 < r_end; r0 += 16) {
#pragma unroll
    for (int u = 0; u < TI; ++u) {
      const int e = tid + u * 256, r = e / W, c = e - r * W;
      Ma[r][c] = (double)pa[u];
      if (!same) Mb[r][c] = (double)pb[u];
    }
    __syncthreads();
    if (r0 + 16 < r_end) fetch(r0 + 16);
#pragma unroll 4
    for (int r = 0; r < 16; ++r) {
      double a[TI], b[TI];
#pragma unroll
      for (int i = 0; i < TI; ++i) { a[i] = Ma[r][ty + 16 * i]; b[i] = same ? Ma[r][tx + 16 * i] : Mb[r][tx + 16 * i]; }
#pragma unroll
      for (int i = 0; i < TI; ++i)
#pragma unroll
        for (int j = 0; j < TI; ++j) acc[i][j] = fma(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
  double *out = t.part + (size_t)blockIdx.x * t.k * t.k;
#pragma unroll
  for (int i = 0; i < TI; ++i) {
    const int row = ty + 16 * i;
    if (row >= t.wa) continue;
#pragma unroll
    for (int j = 0; j < TI; ++j) {
      const int col = tx + 16 * j;
      if (col >= t.wb) continue;
      out[(size_t)(t.ca + row) * t.k + t.cb + col] = acc[i][j];
      if (!same) out[(size_t)(t.cb + col) * t.k + t.ca + row] = acc[i][j];
    }
  }
}

}  // namespace jolt
