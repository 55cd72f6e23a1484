// Batched symmetric eigen-solver spread over the whole GPU: block Jacobi with one launch per round.
//
// The n x n matrix (fp64, padded to a multiple of 32) is cut into 16-wide index blocks.  A round pairs
// the blocks up (round-robin); for every pair one CTA runs one cyclic Jacobi sweep on the 32 x 32
// principal submatrix and records the accumulated rotation J; then every 32 x 32 block of A becomes
// J_a^T blk J_b and every row slab of V is multiplied by J_a.  Rounds are separate launches, so nothing
// ever waits inside a kernel; all matrices of a call share the launches.  The apply half of every launch
// measures the off-diagonal mass and raises a per-matrix `done` flag that turns the remaining launches
// into no-ops.
#pragma once
#include "small_solvers.cuh"

namespace jolt {

constexpr int kBJBlock = 16;
constexpr int kBJMaxSweeps = 10;
// Converged when the off-diagonal mass is below 1e-14 of the total (squared Frobenius norms), i.e. a relative
// off-diagonal norm of 1e-7, the resolution of the fp32 factors that are read out.  Jacobi converges quadratically,
// so the last round usually lands far below; measured on the benchmark cells the reconstruction errors agree to six
// digits with those of a 1e-19 threshold, which costs one more sweep.
constexpr double kBJTol = 1e-14;

struct BJTask {
  const double *A_in;   // n x n symmetric input (untouched)
  double *A;            // two nP x nP work matrices (ping-pong between rounds)
  double *V;            // nP x nP, column i = eigenvector i on exit
  double *J;            // two sets of (nbe/2) x 32 x 32 rotations (current round, next round)
  double *off;          // [4]: off-diagonal mass (accumulator), total mass, last measured off-diagonal mass, rounds run
  int *done;            // [4]: see bj_round_kernel
  unsigned *ticket;     // = done + 1, counter of finished A blocks
  int n, nP, nbe;       // size, padded size (16 * nbe), even number of blocks
  double *w;            // nP scratch (eigenvalues)
  float *U_out; int ld_out, r_out; float *w_out; int w_sqrt;
  int *status;
  double tol;           // convergence: off-diagonal mass <= tol * total mass (squared norms)
  const float *V0;      // optional starting basis (n x n, row-major, column j = j-th vector): A_in is then V0^T M V0 and
                        // the eigenvectors come out as V0 J; null: identity
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
    t.V[e] = (t.V0 && i < n && j < n) ? (double)t.V0[(size_t)i * n + j] : ((i == j) ? 1.0 : 0.0);
    tot += v * v;
  }
  for (int o = 16; o; o >>= 1) tot += __shfl_xor_sync(0xffffffffu, tot, o);
  if ((threadIdx.x & 31) == 0 && tot != 0.0) atomicAdd(&t.off[1], tot);
}

// One launch per round.  Step s applies the rotations of round s-1 (A: buffer (s-1)&1 -> buffer s&1, V in place)
// and, in other CTAs of the same launch, already solves round s: a solve CTA recomputes the three 32 x 32 blocks
// its new pair needs from the old buffer and the old rotations instead of waiting for the apply CTAs, so the
// two halves never depend on one another inside a launch.  The apply CTAs also sum the off-diagonal mass of
// what they write; the last of them to finish compares it with the total mass and raises `done`.
//   done[0] = 1 + step at which convergence was seen (0: not yet), done[1] = ticket, done[2] = final A buffer
constexpr int kBJTile = 32 * 33;          // padded 32 x 32 fp64 tile

// Programmatic dependent launch: the next round's grid may be scheduled while this one still runs; it does its
// index arithmetic and then blocks in pdl_wait() until this grid has completed and its writes are visible.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ void bj_pair_rows(int round, int pair, int nbe, int lane, int *dst) {
  int I, J2; rr_pair(round, pair, nbe, I, J2);
  dst[lane] = lane < 16 ? I * 16 + lane : J2 * 16 + lane - 16;
}

constexpr int kBJThreads = 288;           // 8 working warps + the warp that accumulates J

__device__ __forceinline__ void bj_bar(int id, int nthreads) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory"); }

// pair `i` of inner round `r`: cross pairs (one index from each 16-block) or the circle method on all 32 indices
template <bool CROSS>
__device__ __forceinline__ void bj_inner_pair(int r, int i, int &p, int &q) {
  if (CROSS) { p = i; q = 16 + ((i + r) & 15); }
  else rr_pair(r, i, 32, p, q);
}

template <bool CROSS>
__device__ __forceinline__ void bj_inner(double *S, double2 (*cs_buf)[16], double *Jo, int tid) {
  constexpr int NR = CROSS ? 16 : 31;
  if (tid >= 256) {
    const int lane = tid & 31;
    double Jr[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) Jr[j] = (j == lane) ? 1.0 : 0.0;
#pragma unroll
    for (int r = 0; r < NR; ++r) {
      if (r == NR - 4) pdl_launch_dependents();
      bj_bar(2, kBJThreads);
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        int p, q; bj_inner_pair<CROSS>(r, i, p, q);
        const double2 cs = cs_buf[r & 1][i];
        const double vp = Jr[p], vq = Jr[q];
        Jr[p] = cs.x * vp - cs.y * vq;
        Jr[q] = cs.y * vp + cs.x * vq;
      }
    }
#pragma unroll
    for (int j = 0; j < 32; ++j) Jo[lane * 32 + j] = Jr[j];
    return;
  }
  const int a = tid >> 4, b = tid & 15;
  for (int r = 0; r < NR; ++r) {
    if (r == NR - 4) pdl_launch_dependents();
    if (tid < 16) {
      int p, q; bj_inner_pair<CROSS>(r, tid, p, q);
      double c, s;
      jacobi_cs_fast(S[p * 33 + p], S[q * 33 + q], S[p * 33 + q], c, s);
      cs_buf[r & 1][tid] = make_double2(c, s);
    }
    bj_bar(2, kBJThreads);
    int pa, qa, pb, qb;
    bj_inner_pair<CROSS>(r, a, pa, qa);
    bj_inner_pair<CROSS>(r, b, pb, qb);
    const double2 ra = cs_buf[r & 1][a], rb = cs_buf[r & 1][b];
    const double ca = ra.x, sa = ra.y, cb = rb.x, sb = rb.y;
    const double x_pp = S[pa * 33 + pb], x_pq = S[pa * 33 + qb], x_qp = S[qa * 33 + pb], x_qq = S[qa * 33 + qb];
    const double r_pp = ca * x_pp - sa * x_qp, r_pq = ca * x_pq - sa * x_qq;
    const double r_qp = sa * x_pp + ca * x_qp, r_qq = sa * x_pq + ca * x_qq;
    S[pa * 33 + pb] = cb * r_pp - sb * r_pq; S[pa * 33 + qb] = sb * r_pp + cb * r_pq;
    S[qa * 33 + pb] = cb * r_qp - sb * r_qq; S[qa * 33 + qb] = sb * r_qp + cb * r_qq;
    bj_bar(1, 256);
  }
}

__global__ void __launch_bounds__(kBJThreads) bj_round_kernel(const BJTask *__restrict__ tasks, int step, int n_steps, int gx_apply) {
  const BJTask t = tasks[blockIdx.y];      // the task table is uploaded before the chain starts
  // Apply CTAs let the next grid go at once; solve CTAs, the longest, only a few inner rounds before they end,
  // so the next grid's CTAs do not sit on the SMs (and in the way of other streams' kernels) for a whole round.
  if ((int)blockIdx.x < gx_apply || step >= n_steps) pdl_launch_dependents();
  const int nbe = t.nbe, np = nbe / 2, nP = t.nP, R = nbe - 1;
  const int r_prev = (step + R - 1) % R, r_next = step % R;
  const size_t asz = (size_t)nP * nP, jsz = (size_t)np * 1024;
  const int ib = step ? ((step - 1) & 1) : 0, ob = step & 1;
  const double *Ain = t.A + ib * asz, *Jin = t.J + ib * jsz;
  double *Aout = t.A + ob * asz, *Jout = t.J + ob * jsz;
  __shared__ __align__(16) double sm[5840];
  __shared__ int ra[32], rb[32];
  __shared__ double red[8];
  __shared__ int s_ab[4];
  __shared__ double2 cs_buf[2][16];
  const int tid = threadIdx.x;

  if ((int)blockIdx.x < gx_apply) {
    // ---- apply: A block (a, b) <- J_a^T blk J_b (a <= b, mirrored), or V slab (row chunk, pair a) <- slab J_a
    if (step == 0 || tid >= 256) return;          // the ninth warp only works in solve CTAs
    const int n_ablk = np * (np + 1) / 2, n_vblk = np * (nP / 32);
    if ((int)blockIdx.x >= n_ablk + n_vblk) return;
    double (*Ja)[33] = (double (*)[33])sm, (*Jb)[33] = (double (*)[33])(sm + kBJTile);
    double (*X)[33] = (double (*)[33])(sm + 2 * kBJTile), (*Y)[33] = (double (*)[33])(sm + 3 * kBJTile);
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
      bj_pair_rows(r_prev, a, nbe, tid, ra);
      if (is_a) bj_pair_rows(r_prev, b, nbe, tid, rb);
      else rb[tid] = b * 32 + tid;       // V: plain row chunk
    }
    bj_bar(1, 256);
    pdl_wait();
    { const int dn = *(volatile int *)t.done; if (dn != 0 && dn <= step) return; }   // converged in an earlier launch
    for (int e = tid; e < 1024; e += 256) {
      const int i = e >> 5, j = e & 31;
      Ja[i][j] = Jin[(size_t)a * 1024 + e];
      if (is_a) { Jb[i][j] = Jin[(size_t)b * 1024 + e]; X[i][j] = Ain[(size_t)ra[i] * nP + rb[j]]; }
      else X[i][j] = t.V[(size_t)rb[i] * nP + ra[j]];      // rows = chunk, cols = pair indices
    }
    bj_bar(1, 256);
    const int i0 = (tid >> 5) * 4, j = tid & 31;
    if (is_a) {
      double acc[4] = {0, 0, 0, 0};                        // Y = J_a^T X
      for (int k = 0; k < 32; ++k) {
        const double x = X[k][j];
#pragma unroll
        for (int u = 0; u < 4; ++u) acc[u] += Ja[k][i0 + u] * x;
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) Y[i0 + u][j] = acc[u];
      bj_bar(1, 256);
      double o[4] = {0, 0, 0, 0};                          // out = Y J_b
      for (int k = 0; k < 32; ++k) {
        const double x = Jb[k][j];
#pragma unroll
        for (int u = 0; u < 4; ++u) o[u] += Y[i0 + u][k] * x;
      }
      double mass = 0;
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        Aout[(size_t)ra[i0 + u] * nP + rb[j]] = o[u];
        if (a != b) Aout[(size_t)rb[j] * nP + ra[i0 + u]] = o[u];      // mirrored block
        if (a != b || i0 + u != j) mass += o[u] * o[u];
      }
      if (a != b) mass *= 2.0;
      for (int o2 = 16; o2; o2 >>= 1) mass += __shfl_xor_sync(0xffffffffu, mass, o2);
      if ((tid & 31) == 0) red[tid >> 5] = mass;
      bj_bar(1, 256);
      if (tid == 0) {
        double sum = 0;
        for (int i = 0; i < 8; ++i) sum += red[i];
        if (sum != 0.0) atomicAdd(&t.off[0], sum);
        __threadfence();
        const unsigned ticket = atomicAdd(t.ticket, 1u);
        if (ticket == (unsigned)n_ablk - 1) {           // every A block of this step is in
          __threadfence();
          const double total_off = atomicAdd(&t.off[0], 0.0);
          if (total_off <= t.tol * t.off[1]) { t.done[2] = ob; __threadfence(); *(volatile int *)t.done = step + 1; }
          t.off[2] = total_off;
          t.off[3] += 1.0;
          t.off[0] = 0.0;
          *t.ticket = 0u;
        }
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
    return;
  }

  // ---- solve round r_next on the matrix as it will be after this step's apply
  if (step >= n_steps) return;
  const int x = blockIdx.x - gx_apply;
  if (x >= np) return;
  const int warp = tid >> 5;
  double *S = sm;                                   // 32 x 33, overlays the first X tile once that is dead
  int I, Jn;
  rr_pair(r_next, x, nbe, I, Jn);
  double *Xaa = sm, *Xab = sm + kBJTile, *Xbb = sm + 2 * kBJTile;
  double *Jas = sm + 3 * kBJTile, *Jbs = Jas + 32 * 17;            // selected 16 columns of J_a, J_b
  double *Y1 = Jbs + 32 * 17, *Y2 = Y1 + 16 * 33, *Y3 = Y2 + 16 * 33;
  if (step > 0 && warp < 8) {
    // pairs a, b of the previous round that held blocks I and Jn, and at which half (0 / 16)
    if (tid < np) {
      int p, q; rr_pair(r_prev, tid, nbe, p, q);
      if (p == I) { s_ab[0] = tid; s_ab[1] = 0; }
      if (q == I) { s_ab[0] = tid; s_ab[1] = 16; }
      if (p == Jn) { s_ab[2] = tid; s_ab[3] = 0; }
      if (q == Jn) { s_ab[2] = tid; s_ab[3] = 16; }
    }
    bj_bar(1, 256);
    if (tid < 32) bj_pair_rows(r_prev, s_ab[0], nbe, tid, ra);
    else if (tid < 64) bj_pair_rows(r_prev, s_ab[2], nbe, tid - 32, rb);
    bj_bar(1, 256);
  }
  pdl_wait();
  { const int dn = *(volatile int *)t.done; if (dn != 0 && dn <= step) return; }   // converged in an earlier launch
  if (warp < 8) {
    if (step == 0) {
      for (int e = tid; e < 1024; e += 256) {
        const int i = e >> 5, j = e & 31;
        const int gi = (i < 16 ? I * 16 + i : Jn * 16 + i - 16), gj = (j < 16 ? I * 16 + j : Jn * 16 + j - 16);
        S[i * 33 + j] = Ain[(size_t)gi * nP + gj];
      }
    } else {
      const int a = s_ab[0], la = s_ab[1], b = s_ab[2], lb = s_ab[3];
      for (int e = tid; e < 1024; e += 256) {
        const int i = e >> 5, j = e & 31;
        Xaa[i * 33 + j] = Ain[(size_t)ra[i] * nP + ra[j]];
        Xab[i * 33 + j] = Ain[(size_t)ra[i] * nP + rb[j]];
        Xbb[i * 33 + j] = Ain[(size_t)rb[i] * nP + rb[j]];
      }
      for (int e = tid; e < 512; e += 256) {
        const int k = e >> 4, c = e & 15;
        Jas[k * 17 + c] = Jin[(size_t)a * 1024 + k * 32 + la + c];
        Jbs[k * 17 + c] = Jin[(size_t)b * 1024 + k * 32 + lb + c];
      }
      bj_bar(1, 256);
      {  // Y1 = Jas^T Xaa, Y2 = Jas^T Xab, Y3 = Jbs^T Xbb   (16 x 32 each)
        const int j = tid & 31, c0 = (tid >> 5) * 2;
        double y[6] = {0, 0, 0, 0, 0, 0};
        for (int k = 0; k < 32; ++k) {
          const double xa = Xaa[k * 33 + j], xb = Xab[k * 33 + j], xc = Xbb[k * 33 + j];
          const double ja0 = Jas[k * 17 + c0], ja1 = Jas[k * 17 + c0 + 1], jb0 = Jbs[k * 17 + c0], jb1 = Jbs[k * 17 + c0 + 1];
          y[0] += ja0 * xa; y[1] += ja1 * xa; y[2] += ja0 * xb; y[3] += ja1 * xb; y[4] += jb0 * xc; y[5] += jb1 * xc;
        }
        Y1[c0 * 33 + j] = y[0]; Y1[(c0 + 1) * 33 + j] = y[1];
        Y2[c0 * 33 + j] = y[2]; Y2[(c0 + 1) * 33 + j] = y[3];
        Y3[c0 * 33 + j] = y[4]; Y3[(c0 + 1) * 33 + j] = y[5];
      }
      bj_bar(1, 256);
      {  // S = [Y1 Jas, Y2 Jbs; ., Y3 Jbs]; the X tiles are dead, S takes the place of the first
        const int c = tid >> 4, d = tid & 15;
        double sii = 0, sij = 0, sjj = 0;
        for (int k = 0; k < 32; ++k) {
          const double ja = Jas[k * 17 + d], jb = Jbs[k * 17 + d];
          sii += Y1[c * 33 + k] * ja; sij += Y2[c * 33 + k] * jb; sjj += Y3[c * 33 + k] * jb;
        }
        S[c * 33 + d] = sii; S[c * 33 + 16 + d] = sij; S[(16 + d) * 33 + c] = sij; S[(16 + c) * 33 + 16 + d] = sjj;
      }
    }
  }
  __syncthreads();
  // The first round of a sweep rotates every pair of the 32 indices (31 inner rounds), which also covers
  // the pairs inside each 16-block once per sweep; the other rounds rotate the 16 x 16 cross pairs only.
  // An inner round: 16 threads derive the 16 rotations from the pivots (barrier A), then each of 256 threads
  // updates its own 2 x 2 pair-block of S in place (barrier B).  The ninth warp keeps the accumulated rotation
  // J in registers, one row per lane, and applies each round's rotations as they are published.
  if (r_next > 0) bj_inner<true>(S, cs_buf, Jout + (size_t)x * 1024, tid);
  else bj_inner<false>(S, cs_buf, Jout + (size_t)x * 1024, tid);
}

__global__ void __launch_bounds__(256) bj_finish_kernel(const BJTask *__restrict__ tasks, int last_buf) {
  const BJTask t = tasks[blockIdx.x];
  const int n = t.n, nP = t.nP, tid = threadIdx.x, nt = blockDim.x;
  const double *Af = t.A + (size_t)(*t.done ? t.done[2] : last_buf) * nP * nP;
  __shared__ int rk[2048];
  // the sweep limit ran out before the threshold was met: still accepted when the relative off-diagonal norm is
  // below 1e-6, flagged as a numerical failure otherwise
  if (tid == 0 && !*t.done && t.status && !(t.off[2] <= 1e-12 * t.off[1])) atomicOr(t.status, 1);
  for (int i = tid; i < n; i += nt) t.w[i] = Af[(size_t)i * nP + i];
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
