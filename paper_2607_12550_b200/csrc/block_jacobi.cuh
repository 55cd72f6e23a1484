// Batched symmetric eigen-solver spread over the whole GPU: block Jacobi with one launch per round.
//
// The n x n matrix (fp64, padded to a multiple of 32) is cut into 16-wide index blocks.  A round pairs
// the blocks up (round-robin); for every pair one CTA runs one cyclic Jacobi sweep on the 32 x 32
// principal submatrix and records the accumulated rotation J (solve kernel); then every 32 x 32 block of
// A becomes J_a^T blk J_b and every row slab of V is multiplied by J_a (apply kernel).  Rounds are separate
// launches, so nothing ever waits inside a kernel; all matrices of a call share the launches.  After each
// sweep a small kernel measures the off-diagonal mass and raises a per-matrix `done` flag that turns the
// remaining launches into no-ops.
#pragma once
#include "small_solvers.cuh"

namespace jolt {

constexpr int kBJBlock = 16;
constexpr int kBJMaxSweeps = 10;

struct BJTask {
  const double *A_in;   // n x n symmetric input (untouched)
  double *A;            // nP x nP work matrix
  double *V;            // nP x nP, column i = eigenvector i on exit
  double *J;            // (nbe/2) x 32 x 32 rotations of the current round
  double *off;          // [4]: off-diagonal mass (accumulator), total mass, last measured off-diagonal mass, sweeps run
  int *done;            // [1]
  unsigned *ticket;     // [1] block counter of the check kernel
  int n, nP, nbe;       // size, padded size (16 * nbe), even number of blocks
  double *w;            // nP scratch (eigenvalues)
  float *U_out; int ld_out, r_out; float *w_out; int w_sqrt;
  int *status;
};

__global__ void bj_init_kernel(const BJTask *__restrict__ tasks) {
  const BJTask t = tasks[blockIdx.y];
  const int nP = t.nP, n = t.n;
  double tot = 0;
  for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < nP * nP; e += gridDim.x * blockDim.x) {
    const int i = e / nP, j = e - i * nP;
    double v = 0;
    if (i < n && j < n) v = 0.5 * (t.A_in[(size_t)i * n + j] + t.A_in[(size_t)j * n + i]);
    t.A[e] = v;
    t.V[e] = (i == j) ? 1.0 : 0.0;
    tot += v * v;
  }
  for (int o = 16; o; o >>= 1) tot += __shfl_xor_sync(0xffffffffu, tot, o);
  if ((threadIdx.x & 31) == 0 && tot != 0.0) atomicAdd(&t.off[1], tot);
}

// One cyclic sweep of 2x2 rotations on the 32 x 32 principal submatrix of block pair `blockIdx.x`.
__global__ void __launch_bounds__(256) bj_solve_kernel(const BJTask *__restrict__ tasks, int round, int cross_only) {
  const BJTask t = tasks[blockIdx.y];
  if (*t.done || (int)blockIdx.x >= t.nbe / 2) return;
  int I, Jb;
  rr_pair(round, blockIdx.x, t.nbe, I, Jb);
  __shared__ double S[32][33], Jm[32][33];
  __shared__ double cs_c[16], cs_s[16];
  __shared__ int pp[16], qq[16];
  const int tid = threadIdx.x, nP = t.nP;
  for (int e = tid; e < 1024; e += 256) {
    const int i = e >> 5, j = e & 31;
    const int gi = (i < 16 ? I * 16 + i : Jb * 16 + i - 16), gj = (j < 16 ? I * 16 + j : Jb * 16 + j - 16);
    S[i][j] = t.A[(size_t)gi * nP + gj];
    Jm[i][j] = (i == j) ? 1.0 : 0.0;
  }
  __syncthreads();
  // The first round of a sweep rotates every pair of the 32 indices (31 inner rounds), which also covers
  // the pairs inside each 16-block once per sweep; the other rounds rotate the 16 x 16 cross pairs only.
  const int n_inner = cross_only ? 16 : 31;
  for (int r = 0; r < n_inner; ++r) {
    if (tid < 16) {
      int p, q;
      if (cross_only) { p = tid; q = 16 + ((tid + r) & 15); } else rr_pair(r, tid, 32, p, q);
      double c = 1.0, s = 0.0;
      const double apq = S[p][q], app = S[p][p], aqq = S[q][q];
      jacobi_cs_fast(app, aqq, apq, c, s);
      pp[tid] = p; qq[tid] = q; cs_c[tid] = c; cs_s[tid] = s;
    }
    __syncthreads();
    {  // 16 x 16 pair-blocks, one per thread
      const int a = tid >> 4, b = tid & 15;
      const int pa = pp[a], qa = qq[a], pb = pp[b], qb = qq[b];
      const double ca = cs_c[a], sa = cs_s[a], cb = cs_c[b], sb = cs_s[b];
      const double x_pp = S[pa][pb], x_pq = S[pa][qb], x_qp = S[qa][pb], x_qq = S[qa][qb];
      const double r_pp = ca * x_pp - sa * x_qp, r_pq = ca * x_pq - sa * x_qq;
      const double r_qp = sa * x_pp + ca * x_qp, r_qq = sa * x_pq + ca * x_qq;
      S[pa][pb] = cb * r_pp - sb * r_pq; S[pa][qb] = sb * r_pp + cb * r_pq;
      S[qa][pb] = cb * r_qp - sb * r_qq; S[qa][qb] = sb * r_qp + cb * r_qq;
      // Jm <- Jm * Jrot : columns p, q of pair (tid >> 5 ... ) two items per thread
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const int it = tid + u * 256, pr = it >> 5, row = it & 31;
        const int p = pp[pr], q = qq[pr];
        const double c = cs_c[pr], s = cs_s[pr];
        const double vp = Jm[row][p], vq = Jm[row][q];
        Jm[row][p] = c * vp - s * vq;
        Jm[row][q] = s * vp + c * vq;
      }
    }
    __syncthreads();
  }
  double *Jo = t.J + (size_t)blockIdx.x * 1024;
  for (int e = tid; e < 1024; e += 256) Jo[e] = Jm[e >> 5][e & 31];
}

// blockIdx.x < np*np : A block (a, b) <- J_a^T blk J_b ;  otherwise V slab (a, row chunk) <- slab J_a
__global__ void __launch_bounds__(256) bj_apply_kernel(const BJTask *__restrict__ tasks, int round) {
  const BJTask t = tasks[blockIdx.y];
  if (*t.done) return;
  const int np = t.nbe / 2, nP = t.nP;
  const int n_ablk = np * (np + 1) / 2, n_vblk = np * (nP / 32);       // A is symmetric: blocks a <= b only
  if ((int)blockIdx.x >= n_ablk + n_vblk) return;
  __shared__ double Ja[32][33], Jb[32][33], X[32][33], Y[32][33];
  __shared__ int ra[32], rb[32];
  const int tid = threadIdx.x;
  const bool is_a = (int)blockIdx.x < n_ablk;
  int a, b;
  if (is_a) {
    const int w = blockIdx.x;
    b = (int)((sqrtf(8.0f * w + 1.0f) - 1.0f) * 0.5f);
    while ((b + 1) * (b + 2) / 2 <= w) ++b;
    while (b * (b + 1) / 2 > w) --b;
    a = w - b * (b + 1) / 2;
  }
  else { const int v = blockIdx.x - n_ablk; a = v / (nP / 32); b = v - a * (nP / 32); }
  if (tid < 32) {
    int I, J2; rr_pair(round, a, t.nbe, I, J2);
    ra[tid] = tid < 16 ? I * 16 + tid : J2 * 16 + tid - 16;
    if (is_a) { rr_pair(round, b, t.nbe, I, J2); rb[tid] = tid < 16 ? I * 16 + tid : J2 * 16 + tid - 16; }
    else rb[tid] = b * 32 + tid;       // V: plain row chunk
  }
  __syncthreads();
  const double *Jga = t.J + (size_t)a * 1024;
  for (int e = tid; e < 1024; e += 256) {
    const int i = e >> 5, j = e & 31;
    Ja[i][j] = Jga[e];
    if (is_a) { Jb[i][j] = t.J[(size_t)b * 1024 + e]; X[i][j] = t.A[(size_t)ra[i] * nP + rb[j]]; }
    else X[i][j] = t.V[(size_t)rb[i] * nP + ra[j]];      // rows = chunk, cols = pair indices
  }
  __syncthreads();
  const int i0 = (tid >> 5) * 4, j = tid & 31;
  if (is_a) {
    // Y = J_a^T X
    double acc[4] = {0, 0, 0, 0};
    for (int k = 0; k < 32; ++k) {
      const double x = X[k][j];
#pragma unroll
      for (int u = 0; u < 4; ++u) acc[u] += Ja[k][i0 + u] * x;
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) Y[i0 + u][j] = acc[u];
    __syncthreads();
    // out = Y J_b
    double o[4] = {0, 0, 0, 0};
    for (int k = 0; k < 32; ++k) {
      const double x = Jb[k][j];
#pragma unroll
      for (int u = 0; u < 4; ++u) o[u] += Y[i0 + u][k] * x;
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      t.A[(size_t)ra[i0 + u] * nP + rb[j]] = o[u];
      if (a != b) t.A[(size_t)rb[j] * nP + ra[i0 + u]] = o[u];      // mirrored block
    }
  } else {
    double o[4] = {0, 0, 0, 0};
    for (int k = 0; k < 32; ++k) {
      const double x = Ja[k][j];
#pragma unroll
      for (int u = 0; u < 4; ++u) o[u] += X[i0 + u][k] * x;
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) t.V[(size_t)rb[i0 + u] * nP + ra[j]] = o[u];
  }
}

// Off-diagonal mass after a sweep; the last block to finish (ticket counter) compares it with the total mass,
// raises `done` and resets the accumulators: one launch per sweep.
__global__ void bj_check_kernel(const BJTask *__restrict__ tasks) {
  const BJTask t = tasks[blockIdx.y];
  if (*t.done) return;
  double off = 0;
  for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < t.nP * t.nP; e += gridDim.x * blockDim.x) {
    const int i = e / t.nP, j = e - i * t.nP;
    if (i != j) { const double v = t.A[e]; off += v * v; }
  }
  for (int o = 16; o; o >>= 1) off += __shfl_xor_sync(0xffffffffu, off, o);
  __shared__ double red[8];
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = off;
  __syncthreads();
  if (threadIdx.x == 0) {
    double s = 0;
    for (int i = 0; i < (int)blockDim.x / 32; ++i) s += red[i];
    if (s != 0.0) atomicAdd(&t.off[0], s);
    __threadfence();
    const unsigned ticket = atomicAdd(t.ticket, 1u);
    if (ticket == gridDim.x - 1) {           // every block's contribution is in
      __threadfence();
      const double total_off = atomicAdd(&t.off[0], 0.0);
      // relative off-diagonal norm 3e-10: above the round-off floor of the 32-term block products on a
      // rank-deficient matrix (measured 5e-11), far below the fp32 grade of what is read out
      if (total_off <= 1e-19 * t.off[1]) *t.done = 1;
      t.off[2] = total_off;
      t.off[3] += 1.0;
      t.off[0] = 0.0;
      *t.ticket = 0u;
    }
  }
}

__global__ void __launch_bounds__(256) bj_finish_kernel(const BJTask *__restrict__ tasks) {
  const BJTask t = tasks[blockIdx.x];
  const int n = t.n, nP = t.nP, tid = threadIdx.x, nt = blockDim.x;
  __shared__ int rk[2048];
  // not converged to the tight threshold after the last sweep: still accepted when the off-diagonal norm is below
  // 1e-7 of the matrix norm (fp32 grade); flagged otherwise
  if (tid == 0 && !*t.done && t.status && !(t.off[2] <= 1e-14 * t.off[1])) atomicOr(t.status, 1);
  for (int i = tid; i < n; i += nt) t.w[i] = t.A[(size_t)i * nP + i];
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
      const int j = it / n, i = it - j * n;        // component j of eigenvector i
      const int rank = rk[i];
      if (rank < t.r_out) t.U_out[(size_t)j * t.ld_out + rank] = (float)t.V[(size_t)j * nP + i];
    }
}

}  // namespace jolt
