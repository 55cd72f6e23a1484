// Single-step attention computed on the compressed cache, without materialising keys or values.
//
// The paper names this as the route to decode parity ("a fused kernel that runs attention directly on the
// factors, without materializing the cache", Sec. 7 and the closing discussion) and gives no algorithm.  What is
// computed here, per layer group, merged head h and query i (n_q queries per KV head):
//     s_t = scale <q_i, K^[h, t]>,   p = softmax_t(s),   o_i = sum_t p_t V^[h, t],
// with K^, V^ the decoded (not yet rounded) cells  X^ = 2^e U_T P_h + s . H(r^') / sqrt(d),  P_h = fp16(G_h U_F^T).
// Both contractions move to the small side:
//     <q, K^[h, t]>     = 2^e sum_k U_T[t, k] (P_h q)[k]  +  < H(s . q) / sqrt(d), r^'[h, t] >
//     sum_t p_t V^[h,t] = 2^e (p^T U_T) P_h               +  s . H( sum_t p_t r^'[h, t] ) / sqrt(d)
// so a call streams U_T and the packed codes once each (the compressed bytes) instead of the fp16 cache, and the
// Hadamard rotation is applied to one query / one output row per head instead of every token.
//
// Kernels of a call (the contractions with a tensor-core shape are warp-level fp16 MMAs with fp32 accumulation, an fp32
// operand entering as hi + lo fp16; the rest is CUDA-core fp32):
//   (P_h = fp16(G_h U_F^T), the projected core the decoder also reads, is kept with the handle since compress)
//   attend_prep_kernel     per (group, head, query): rotated scaled query (fp32, and scaled hi + lo fp16), w = P_h q
//   attend_bscore_kernel   backbone scores U_T w of all heads of a cell as one dense product (U_T is shared by the heads)
//   attend_scores_mma_kernel / attend_scores_kernel   per (group, head, 256-token chunk): residual scores added (codes
//                          times rotated query: MMAs for 1-, 2-, 4- and 8-bit codes, CUDA cores for 3-bit codes and for
//                          cells without a residual), chunk maximum, p = exp(s - max), chunk sum
//   attend_values_mma_kernel / attend_values_kernel   per (group, head, chunk): sum_t p_t r^'_t (MMAs with M = features,
//                          K = tokens over an fp16 tile of expanded codes for 1-, 2-, 4- and 8-bit codes; CUDA cores,
//                          codes staged in shared memory and read feature-wise, for 3-bit codes)
//   attend_bvalue_kernel   p^T U_T per chunk for all heads of a cell as one dense product
//   attend_combine_kernel  per (group, head, query): merges the chunks (running-maximum rescaling), applies P_h of the
//                          value cell and the inverse rotation, divides by the softmax denominator
// Keys compressed before a rotary embedding cannot use the first identity (the rotation differs per token).
#pragma once
#include <cuda_fp16.h>

#include "common.cuh"
#include "rowquant.cuh"

namespace jolt {

constexpr int kAttChunk = 256;      // tokens per chunk = threads per CTA of the two streaming kernels
constexpr int kAttMaxQ = 8;         // queries per KV head (padded to 4 or 8 inside)

struct AttendCell {
  const __half *G, *UT, *UF;        // [m * r_t][r_f], [T][r_t], [128][r_f]
  const int *e;
  const uint32_t *words;            // [m][T][4 * bits]
  const __half *scales;             // [m][T][4]
  int r_t, r_f, bits, cell;
};

struct AttendJob {                  // one per layer group
  AttendCell k, v;
  int m, T;
  const float *q;                   // [m][n_q][128]
  float *out;                       // [m][n_q][128]
  __half *kP, *vP;                  // [m * r_t][128]    P_h = fp16(G_h U_F^T) of the key / value cell (scaled units)
  __half *wh, *wl;                  // [m NQP][k.r_t]    P_h q times 2^-E_n per column n = (head, query), as hi + lo fp16
  float *we;                        // [m NQP]           scale 2^e 2^E_n
  float *qt;                        // [m][128][NQP]     scale H(s . q) / sqrt(d)
  __half *qh, *ql;                  // [m][8][128]       the same, times 2^-E per (head, query), as hi + lo fp16 (MMA operand)
  float *qe;                        // [m][8]            2^E
  float *p;                         // [m][T][NQP]       exp(s - chunk maximum)
  float *ml;                        // [m][n_chunks][2][NQP]  chunk maximum, chunk sum
  float *y;                         // [m][n_chunks][v.r_t][NQP]
  float *a;                         // [m][n_chunks][128][NQP]
};

// 128-point Walsh-Hadamard transform of buf[0..127] by 128 threads (thread f owns element f on return).
__device__ __forceinline__ float att_wht_smem(float *buf, int f) {
  float v = buf[f];
#pragma unroll
  for (int len = 1; len < 128; len <<= 1) {
    const float o = buf[f ^ len];
    __syncthreads();
    v = (f & len) ? o - v : v + o;
    buf[f] = v;
    __syncthreads();
  }
  return v;
}

__device__ __forceinline__ float att_sign(uint64_t seed, int cell, int f) {
  uint32_t sw[4];
  cell_sign_words(seed, cell, sw);
  return ((sw[f >> 5] >> (f & 31)) & 1u) ? -1.f : 1.f;
}

// grid (m, groups, NQP), 128 threads (thread = feature), 128 floats of dynamic shared memory.  CTA z rotates query z
// and forms every NQP-th group of four rows of w.
__global__ void __launch_bounds__(128) attend_prep_kernel(const AttendJob *__restrict__ jobs, int n_q, int NQP, float scale,
                                                          uint64_t seed) {
  const AttendJob &jb = jobs[blockIdx.y];
  const int h = blockIdx.x, f = threadIdx.x, i = blockIdx.z;
  if (h >= jb.m) return;
  extern __shared__ unsigned char att_smem[];
  float *buf = (float *)att_smem;
  if (jb.k.bits > 0) {
    buf[f] = i < n_q ? att_sign(seed, jb.k.cell, f) * jb.q[((size_t)h * n_q + i) * 128 + f] : 0.f;
    __syncthreads();
    const float v = att_wht_smem(buf, f) * kInvSqrtD * scale;
    jb.qt[((size_t)h * 128 + f) * NQP + i] = v;
    // the tensor-core form of the same row: scaled by a power of two so that hi + lo fp16 hold it (|entry| < 2^13)
    __shared__ float wmax[4];
    float mx = fabsf(v);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    if ((f & 31) == 0) wmax[f >> 5] = mx;
    __syncthreads();
    mx = fmaxf(fmaxf(wmax[0], wmax[1]), fmaxf(wmax[2], wmax[3]));
    int ex = 0;
    if (mx > 0.f && mx < INFINITY) frexpf(mx, &ex);                  // mx < 2^ex
    const float sv = ldexpf(v, 13 - ex);
    const __half hi = __float2half_rn(sv);
    jb.qh[((size_t)h * kAttMaxQ + i) * 128 + f] = hi;
    jb.ql[((size_t)h * kAttMaxQ + i) * 128 + f] = __float2half_rn(sv - __half2float(hi));
    if (f == 0) jb.qe[h * kAttMaxQ + i] = ldexpf(1.f, ex - 13);
  }
  if (jb.k.r_t > 0) {
    // w[n][k] = sum_f P_h[k][f] q[f] for column n = (head, query): a warp per row k, a lane per four features.  Stored as
    // hi + lo fp16 times 2^-E_n with 2^E_n > |q|_2: a row of P_h has norm below 2^14.52 (|G| 2^-e < 2^11, r_f <= 128, U_F
    // orthonormal, fp16 rounding), so every scaled entry is below 2^14.52 in magnitude and fits fp16.
    const float se = scale * ldexpf(1.f, *jb.k.e);
    const int warp = f >> 5, lane = f & 31;
    float q[kAttMaxQ][4];
    int ex[kAttMaxQ];
    float inv[kAttMaxQ];
#pragma unroll
    for (int c = 0; c < kAttMaxQ; ++c) {
      const float4 v = c < n_q ? *(const float4 *)(jb.q + ((size_t)h * n_q + c) * 128 + lane * 4) : make_float4(0.f, 0.f, 0.f, 0.f);
      q[c][0] = v.x; q[c][1] = v.y; q[c][2] = v.z; q[c][3] = v.w;
      float sq = fmaf(v.x, v.x, fmaf(v.y, v.y, fmaf(v.z, v.z, v.w * v.w)));
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
      const float nrm = sqrtf(sq);
      ex[c] = 0;
      if (nrm > 0.f && nrm < INFINITY) frexpf(nrm, &ex[c]);              // |q|_2 < 2^ex
      ++ex[c];                                                          // headroom for the rounding of the norm itself
      inv[c] = ldexpf(1.f, -ex[c]);
    }
    if (blockIdx.z == 0 && f < NQP) {
      int e_f = 0;
#pragma unroll
      for (int c = 0; c < kAttMaxQ; ++c)
        if (c == f) e_f = ex[c];
      jb.we[h * NQP + f] = se * ldexpf(1.f, e_f);
    }
    for (int k = warp + 4 * blockIdx.z; k < jb.k.r_t; k += 4 * gridDim.z) {
      const uint2 p4 = __ldg((const uint2 *)(jb.kP + ((size_t)h * jb.k.r_t + k) * 128 + lane * 4));
      const __half *ph = (const __half *)&p4;
      const float p0 = __half2float(ph[0]), p1 = __half2float(ph[1]), p2 = __half2float(ph[2]), p3 = __half2float(ph[3]);
      float v[kAttMaxQ];
#pragma unroll
      for (int c = 0; c < kAttMaxQ; ++c) v[c] = fmaf(p0, q[c][0], fmaf(p1, q[c][1], fmaf(p2, q[c][2], p3 * q[c][3])));
#pragma unroll
      for (int o = 16; o > 0; o >>= 1)
#pragma unroll
        for (int c = 0; c < kAttMaxQ; ++c) v[c] += __shfl_xor_sync(0xffffffffu, v[c], o);
      // lane c stores column c (every lane holds all the sums)
      float sv = 0.f;
#pragma unroll
      for (int c = 0; c < kAttMaxQ; ++c)
        if (c == lane) sv = v[c] * inv[c];
      if (lane < NQP) {
        const __half hi = __float2half_rn(sv);
        jb.wh[((size_t)h * NQP + lane) * jb.k.r_t + k] = hi;
        jb.wl[((size_t)h * NQP + lane) * jb.k.r_t + k] = __float2half_rn(sv - __half2float(hi));
      }
    }
  }
}

// Code j of 32-feature group g of a packed row (little-endian bit string per group, BITS words per group).
template <int BITS>
__device__ __forceinline__ uint32_t att_code(const uint32_t *row, int g, int j) {
  const int bit = j * BITS, wi = g * BITS + (bit >> 5), sh = bit & 31;
  uint32_t u = row[wi] >> sh;
  if (sh + BITS > 32) u |= row[wi + 1] << (32 - sh);
  return u & ((1u << BITS) - 1u);
}

// grid (n_chunks, m, groups), kAttChunk threads (thread = token).  Dynamic shared memory: (128 + r_t) * NQP floats.
template <int BITS>
__global__ void __launch_bounds__(kAttChunk, 3) attend_scores_kernel(const AttendJob *__restrict__ jobs, int NQP) {
  const AttendJob &jb = jobs[blockIdx.z];
  if (jb.k.bits != BITS) return;
  const int h = blockIdx.y, chunk = blockIdx.x;
  if (h >= jb.m || chunk * kAttChunk >= jb.T) return;
  extern __shared__ unsigned char att_smem[];
  float *qts = (float *)att_smem;                   // [128][NQP]
  __shared__ float red[2][kAttChunk / 32][kAttMaxQ];
  __shared__ float qsum[4 * kAttMaxQ];              // per 32-feature group: sum of the rotated query's entries
  const int tid = threadIdx.x, r_t = jb.k.r_t;
  if (BITS > 0)
    for (int i = tid; i < 128 * NQP; i += kAttChunk) qts[i] = jb.qt[(size_t)h * 128 * NQP + i];
  __syncthreads();
  if (BITS > 0 && tid < 4 * kAttMaxQ) {
    const int g = tid / kAttMaxQ, i = tid % kAttMaxQ;
    float a = 0.f;
    if (i < NQP)
      for (int j = 0; j < 32; ++j) a += qts[(g * 32 + j) * NQP + i];
    qsum[tid] = a;
  }
  __syncthreads();
  const int t = chunk * kAttChunk + tid;
  const bool live = t < jb.T;
  float s[kAttMaxQ];
#pragma unroll
  for (int i = 0; i < kAttMaxQ; ++i) s[i] = 0.f;
  if (live) {
    if constexpr (BITS > 0) {
      uint32_t row[4 * BITS];
      const uint4 *wp = (const uint4 *)(jb.k.words + ((size_t)h * jb.T + t) * (4 * BITS));
#pragma unroll
      for (int i = 0; i < BITS; ++i) { const uint4 v = __ldg(wp + i); row[4 * i] = v.x; row[4 * i + 1] = v.y; row[4 * i + 2] = v.z; row[4 * i + 3] = v.w; }
      __half sc[4];
      *(uint2 *)sc = __ldg((const uint2 *)(jb.k.scales + ((size_t)h * jb.T + t) * 4));
      // integer code to float without a conversion instruction: 2^23 + u, minus (2^23 + 2^(b-1))
      // (the half-step offset is applied per group through the sum of the group's query entries, qsum)
      constexpr float off = 8388608.0f + (float)(1 << (BITS - 1));
      const bool q8 = NQP == 8;
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        float g0 = 0.f, g1 = 0.f, g2 = 0.f, g3 = 0.f, g4 = 0.f, g5 = 0.f, g6 = 0.f, g7 = 0.f;
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const float val = __uint_as_float(0x4B000000u | att_code<BITS>(row, g, j)) - off;
          const float *qp = qts + (g * 32 + j) * NQP;
          const float4 qv = *(const float4 *)qp;
          g0 = fmaf(val, qv.x, g0); g1 = fmaf(val, qv.y, g1); g2 = fmaf(val, qv.z, g2); g3 = fmaf(val, qv.w, g3);
          if (q8) {
            const float4 qw = *(const float4 *)(qp + 4);
            g4 = fmaf(val, qw.x, g4); g5 = fmaf(val, qw.y, g5); g6 = fmaf(val, qw.z, g6); g7 = fmaf(val, qw.w, g7);
          }
        }
        const float delta = __half2float(sc[g]);
        const float *qh = qsum + g * kAttMaxQ;
        g0 = fmaf(0.5f, qh[0], g0); g1 = fmaf(0.5f, qh[1], g1); g2 = fmaf(0.5f, qh[2], g2); g3 = fmaf(0.5f, qh[3], g3);
        g4 = fmaf(0.5f, qh[4], g4); g5 = fmaf(0.5f, qh[5], g5); g6 = fmaf(0.5f, qh[6], g6); g7 = fmaf(0.5f, qh[7], g7);
        s[0] = fmaf(delta, g0, s[0]); s[1] = fmaf(delta, g1, s[1]); s[2] = fmaf(delta, g2, s[2]); s[3] = fmaf(delta, g3, s[3]);
        s[4] = fmaf(delta, g4, s[4]); s[5] = fmaf(delta, g5, s[5]); s[6] = fmaf(delta, g6, s[6]); s[7] = fmaf(delta, g7, s[7]);
      }
    }
    if (r_t > 0) {
      // backbone scores of this token: written to the weight buffer by attend_bscore_kernel, replaced by the weights below
      const float *sb = jb.p + ((size_t)h * jb.T + t) * NQP;
      const float4 b0 = *(const float4 *)sb;
      s[0] += b0.x; s[1] += b0.y; s[2] += b0.z; s[3] += b0.w;
      if (NQP == 8) {
        const float4 b1 = *(const float4 *)(sb + 4);
        s[4] += b1.x; s[5] += b1.y; s[6] += b1.z; s[7] += b1.w;
      }
    }
  }
  // chunk maximum and sum of exp(s - maximum), per query
  const int warp = tid >> 5, lane = tid & 31;
  float mx[kAttMaxQ];
#pragma unroll
  for (int i = 0; i < kAttMaxQ; ++i) {
    float v = live ? s[i] : -INFINITY;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    if (lane == 0) red[0][warp][i] = v;
  }
  __syncthreads();
#pragma unroll
  for (int i = 0; i < kAttMaxQ; ++i) {
    float v = red[0][0][i];
#pragma unroll
    for (int wq = 1; wq < kAttChunk / 32; ++wq) v = fmaxf(v, red[0][wq][i]);
    mx[i] = v;
  }
  float pr[kAttMaxQ];
#pragma unroll
  for (int i = 0; i < kAttMaxQ; ++i) {
    pr[i] = live ? expf(s[i] - mx[i]) : 0.f;
    float v = pr[i];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if (lane == 0) red[1][warp][i] = v;
  }
  __syncthreads();
  if (live) {
    float *pp = jb.p + ((size_t)h * jb.T + t) * NQP;
    *(float4 *)pp = make_float4(pr[0], pr[1], pr[2], pr[3]);
    if (NQP == 8) *(float4 *)(pp + 4) = make_float4(pr[4], pr[5], pr[6], pr[7]);
  }
  if (tid < NQP) {
    float l = 0.f;
    for (int wq = 0; wq < kAttChunk / 32; ++wq) l += red[1][wq][tid];
    const int n_chunks = gridDim.x;
    float *ml = jb.ml + ((size_t)h * n_chunks + chunk) * 2 * NQP;
    float m_i = red[0][0][tid];
    for (int wq = 1; wq < kAttChunk / 32; ++wq) m_i = fmaxf(m_i, red[0][wq][tid]);
    ml[tid] = m_i;
    ml[NQP + tid] = l;
  }
}

// warp-level m16n8k16 MMA, fp16 operands, fp32 accumulation
__device__ __forceinline__ void att_mma_f16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// The score kernel for 1-, 2-, 4- and 8-bit codes with the code-times-query contraction on the tensor cores.
// grid (ceil(n_chunks / 2), m, groups), kAttChunk threads = 8 warps; a CTA walks every gridDim.x-th chunk of its head, a
// warp owns 32 tokens of the chunk = two 16-row MMA tiles.  The chunk's
// packed rows and scales are loaded coalesced and staged in shared memory; the m16n8k16 A fragments are built from
// words read there (odd row pitch: the eight rows of a fragment column fall into eight banks), a pair of codes expanding to the exact fp16
// integers 2u + 1 - 2^b (so the mid-rise half step is part of the operand and the product is twice the wanted sum).
// B = the rotated query as hi + lo fp16, 8 query columns, staged once per CTA in shared memory (4 conflict-free word
// reads per MMA pair).  Per 32-feature group the 16 x 8 partial product is scaled by Delta / 2 of its row.  Registers are
// capped for three CTAs per SM: the kernel is bound by the latency of its row loads, not by any pipe.
__device__ __forceinline__ uint32_t att_pair_f16(uint32_t x, int bits) {
  const uint32_t mask = (1u << bits) - 1u;
  const uint32_t v = ((x & mask) << 1) | (((x >> bits) & mask) << 17) | 0x64016401u;        // half2(1024 + 2u + 1)
  const __half2 off = __float2half2_rn(1024.f + (float)(1 << bits));
  const __half2 r = __hsub2(*(const __half2 *)&v, off);
  return *(const uint32_t *)&r;
}

template <int BITS>
__global__ void __launch_bounds__(kAttChunk, BITS >= 4 ? 2 : 3) attend_scores_mma_kernel(const AttendJob *__restrict__ jobs, int NQP, int n_chunks) {
  static_assert(BITS == 1 || BITS == 2 || BITS == 4 || BITS == 8, "codes that do not straddle words");
  const AttendJob &jb = jobs[blockIdx.z];
  if (jb.k.bits != BITS) return;
  const int h = blockIdx.y;
  if (h >= jb.m || (int)blockIdx.x * kAttChunk >= jb.T) return;
  __shared__ float red[2][kAttChunk / 32][kAttMaxQ];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, c = lane & 3;
  // the chunk's packed rows and scales, requested one chunk ahead: consecutive threads take consecutive 16-byte pieces
  // (coalesced), and put them into shared memory with an odd row pitch, from where the fragment builders read words
  constexpr int RP = 4 * BITS + 1;                 // words per staged row: rows g = 0..7 of one word fall into 8 banks
  __shared__ uint32_t rows[kAttChunk][RP];
  __shared__ uint2 scs[kAttChunk];
  uint4 npc[BITS];                                 // pieces tid, tid + 256, ... of the chunk's kAttChunk * BITS
  uint2 nsc = make_uint2(0u, 0u);
  float2 nsb[4];                   // backbone scores of this lane's four (row, query pair) results
  const bool qok = 2 * c < NQP;
  auto fetch = [&](int chunk) {
#pragma unroll
    for (int r = 0; r < 4; ++r) nsb[r] = make_float2(0.f, 0.f);
    if (chunk >= n_chunks) return;
    const int t0 = chunk * kAttChunk, nt = min(kAttChunk, jb.T - t0);
    if (qok && jb.k.r_t > 0 && warp * 32 < nt) {
#pragma unroll
      for (int r = 0; r < 4; ++r)
        nsb[r] = *(const float2 *)(jb.p + ((size_t)h * jb.T + t0 + warp * 32 + (r >> 1) * 16 + (r & 1) * 8 + g) * NQP + 2 * c);
    }
    const uint4 *wp = (const uint4 *)(jb.k.words + ((size_t)h * jb.T + t0) * (4 * BITS));
#pragma unroll
    for (int i = 0; i < BITS; ++i) {
      const int idx = tid + i * kAttChunk;
      npc[i] = idx < nt * BITS ? __ldg(wp + idx) : make_uint4(0u, 0u, 0u, 0u);
    }
    nsc = tid < nt ? __ldg((const uint2 *)(jb.k.scales + ((size_t)h * jb.T + t0) * 4) + tid) : make_uint2(0u, 0u);
  };
  fetch(blockIdx.x);
  // B operand (rotated query, hi and lo) of the head in shared memory: [query][feature pair], 68 words per row so that
  // the fragment reads (query g, pair 8 s + c) touch 32 different banks
  __shared__ uint32_t Bq[2][kAttMaxQ][68];
  for (int i = tid; i < 2 * kAttMaxQ * 64; i += kAttChunk) {
    const int hl = i >> 9, q = (i >> 6) & 7, w = i & 63;
    const uint32_t *src = (const uint32_t *)((hl ? jb.ql : jb.qh) + ((size_t)h * kAttMaxQ + q) * 128);
    Bq[hl][q][w] = q < NQP ? __ldg(src + w) : 0u;
  }
  __syncthreads();
  for (int chunk = blockIdx.x; chunk < n_chunks; chunk += gridDim.x) {
  const bool live = chunk * kAttChunk + warp * 32 < jb.T;      // T is a multiple of 128: a warp is all in or all out
  __syncthreads();                                       // the previous chunk's rows have been read
#pragma unroll
  for (int i = 0; i < BITS; ++i) {
    const int idx = tid + i * kAttChunk, r = idx / BITS, w4 = (idx % BITS) * 4;
    rows[r][w4] = npc[i].x; rows[r][w4 + 1] = npc[i].y; rows[r][w4 + 2] = npc[i].z; rows[r][w4 + 3] = npc[i].w;
  }
  scs[tid] = nsc;
  float2 sb[4];
#pragma unroll
  for (int r = 0; r < 4; ++r) sb[r] = nsb[r];
  __syncthreads();
  fetch(chunk + gridDim.x);                              // in flight during this chunk's MMAs
  float sc[2][4];          // [tile][row g: queries 2c, 2c+1; row g + 8: queries 2c, 2c+1]
#pragma unroll
  for (int tl = 0; tl < 2; ++tl)
#pragma unroll
    for (int j = 0; j < 4; ++j) sc[tl][j] = 0.f;
#pragma unroll
  for (int tl = 0; tl < 2; ++tl) {
    const uint32_t *ra = rows[warp * 32 + tl * 16 + g], *rb = rows[warp * 32 + tl * 16 + g + 8];      // rows g and g + 8 of this tile
    const uint2 sa = scs[warp * 32 + tl * 16 + g], sbw = scs[warp * 32 + tl * 16 + g + 8];
    const uint32_t sxa = sa.x, sya = sa.y, sxb = sbw.x, syb = sbw.y;
#pragma unroll
    for (int gq = 0; gq < 4; ++gq) {
      float d[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int s2 = 0; s2 < 2; ++s2) {
        const int s8 = gq * 2 + s2;
        uint32_t a[4];
        if constexpr (BITS == 8) {            // 16 bits at bit 128 s2 + 16 c: word 4 s2 + (c >> 1), half c & 1; + 8 columns: two words on
          const int w0 = gq * 8 + s2 * 4 + (c >> 1), sh = 16 * (c & 1);
          a[0] = att_pair_f16(ra[w0] >> sh, 8); a[1] = att_pair_f16(rb[w0] >> sh, 8);
          a[2] = att_pair_f16(ra[w0 + 2] >> sh, 8); a[3] = att_pair_f16(rb[w0 + 2] >> sh, 8);
        } else if constexpr (BITS == 4) {     // 8 bits at bit 64 s2 + 8 c: word 2 s2, byte c; + 8 columns: the next word
          const int w0 = gq * 4 + s2 * 2;
          a[0] = att_pair_f16(ra[w0] >> (8 * c), 4); a[1] = att_pair_f16(rb[w0] >> (8 * c), 4);
          a[2] = att_pair_f16(ra[w0 + 1] >> (8 * c), 4); a[3] = att_pair_f16(rb[w0 + 1] >> (8 * c), 4);
        } else if constexpr (BITS == 2) {     // 4 bits at bit 32 s2 + 4 c: word s2, nibble c; + 8 columns: 16 bits on
          const uint32_t a0 = ra[gq * 2 + s2], b0 = rb[gq * 2 + s2];
          a[0] = att_pair_f16(a0 >> (4 * c), 2); a[1] = att_pair_f16(b0 >> (4 * c), 2);
          a[2] = att_pair_f16(a0 >> (4 * c + 16), 2); a[3] = att_pair_f16(b0 >> (4 * c + 16), 2);
        } else {                              // 2 bits at bit 16 s2 + 2 c of the group's single word; + 8 columns: 8 bits on
          const uint32_t a0 = ra[gq], b0 = rb[gq];
          a[0] = att_pair_f16(a0 >> (16 * s2 + 2 * c), 1); a[1] = att_pair_f16(b0 >> (16 * s2 + 2 * c), 1);
          a[2] = att_pair_f16(a0 >> (16 * s2 + 2 * c + 8), 1); a[3] = att_pair_f16(b0 >> (16 * s2 + 2 * c + 8), 1);
        }
        att_mma_f16(d, a, Bq[0][g][s8 * 8 + c], Bq[0][g][s8 * 8 + c + 4]);
        att_mma_f16(d, a, Bq[1][g][s8 * 8 + c], Bq[1][g][s8 * 8 + c + 4]);
      }
      // Delta / 2 of rows g and g + 8 for this group: half (gq & 1) of scale word gq >> 1
      const uint32_t wa = (gq & 2) ? sya : sxa, wb = (gq & 2) ? syb : sxb;
      const float da = 0.5f * __half2float(__ushort_as_half((unsigned short)((gq & 1) ? (wa >> 16) : (wa & 0xFFFFu))));
      const float db = 0.5f * __half2float(__ushort_as_half((unsigned short)((gq & 1) ? (wb >> 16) : (wb & 0xFFFFu))));
      sc[tl][0] = fmaf(da, d[0], sc[tl][0]); sc[tl][1] = fmaf(da, d[1], sc[tl][1]);
      sc[tl][2] = fmaf(db, d[2], sc[tl][2]); sc[tl][3] = fmaf(db, d[3], sc[tl][3]);
    }
  }
  // undo the query scaling, add the backbone scores; this lane: queries 2c, 2c + 1 of rows g, g + 8, 16 + g, 24 + g
  const float e0 = qok ? jb.qe[h * kAttMaxQ + 2 * c] : 0.f, e1 = qok ? jb.qe[h * kAttMaxQ + 2 * c + 1] : 0.f;
  const int tw = chunk * kAttChunk + warp * 32;
  float *prow[4];
#pragma unroll
  for (int r = 0; r < 4; ++r) prow[r] = jb.p + ((size_t)h * jb.T + tw + (r >> 1) * 16 + (r & 1) * 8 + g) * NQP + 2 * c;
  float sv[4][2];
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    sv[r][0] = sc[r >> 1][(r & 1) * 2] * e0;
    sv[r][1] = sc[r >> 1][(r & 1) * 2 + 1] * e1;
    sv[r][0] += sb[r].x; sv[r][1] += sb[r].y;
  }
  // chunk maximum and sum of exp(s - maximum), per query: over this lane's rows, the lanes of equal c, the warps
  float m0 = -INFINITY, m1 = -INFINITY;
  if (live) {
#pragma unroll
    for (int r = 0; r < 4; ++r) { m0 = fmaxf(m0, sv[r][0]); m1 = fmaxf(m1, sv[r][1]); }
  }
#pragma unroll
  for (int o = 4; o < 32; o <<= 1) { m0 = fmaxf(m0, __shfl_xor_sync(0xffffffffu, m0, o)); m1 = fmaxf(m1, __shfl_xor_sync(0xffffffffu, m1, o)); }
  if (g == 0) { red[0][warp][2 * c] = m0; red[0][warp][2 * c + 1] = m1; }
  __syncthreads();
  m0 = red[0][0][2 * c]; m1 = red[0][0][2 * c + 1];
#pragma unroll
  for (int wq = 1; wq < kAttChunk / 32; ++wq) { m0 = fmaxf(m0, red[0][wq][2 * c]); m1 = fmaxf(m1, red[0][wq][2 * c + 1]); }
  float l0 = 0.f, l1 = 0.f;
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const float p0 = live ? expf(sv[r][0] - m0) : 0.f, p1 = live ? expf(sv[r][1] - m1) : 0.f;
    l0 += p0; l1 += p1;
    if (live && qok) *(float2 *)prow[r] = make_float2(p0, p1);
  }
#pragma unroll
  for (int o = 4; o < 32; o <<= 1) { l0 += __shfl_xor_sync(0xffffffffu, l0, o); l1 += __shfl_xor_sync(0xffffffffu, l1, o); }
  if (g == 0) { red[1][warp][2 * c] = l0; red[1][warp][2 * c + 1] = l1; }
  __syncthreads();
  if (tid < NQP) {
    float l = 0.f, m_i = red[0][0][tid];
    for (int wq = 0; wq < kAttChunk / 32; ++wq) l += red[1][wq][tid];
    for (int wq = 1; wq < kAttChunk / 32; ++wq) m_i = fmaxf(m_i, red[0][wq][tid]);
    float *ml = jb.ml + ((size_t)h * n_chunks + chunk) * 2 * NQP;
    ml[tid] = m_i;
    ml[NQP + tid] = l;
  }
  __syncthreads();            // red is rewritten by the next chunk
  }
}

// grid (n_chunks, m, groups), kAttChunk threads.  The chunk is staged in two halves of 128 tokens (codes, scales and
// weights, coalesced), so that six CTAs fit an SM: the kernel lives on the number of warps that hide its staging
// latency.  NQ = 4 or 8 query slots (compile time: the accumulators are the register budget).  Dynamic shared memory:
// 128 * (NQ floats + 4 BITS words + 4 halves) + 4 * 128 * NQ floats.
constexpr int kAttHalf = kAttChunk / 2;
template <int BITS, int NQ>
__global__ void __launch_bounds__(kAttChunk, NQ == 4 ? 6 : 4) attend_values_kernel(const AttendJob *__restrict__ jobs) {
  const AttendJob &jb = jobs[blockIdx.z];
  if (jb.v.bits != BITS || BITS == 0) return;
  const int h = blockIdx.y, chunk = blockIdx.x, n_chunks = gridDim.x;
  if (h >= jb.m || chunk * kAttChunk >= jb.T) return;
  constexpr int NB = BITS > 0 ? BITS : 1;
  extern __shared__ unsigned char att_smem[];
  float *ps = (float *)att_smem;                                        // [128][NQ]
  uint32_t *cw = (uint32_t *)(ps + kAttHalf * NQ);                      // [128][4 * BITS]
  __half *cs = (__half *)(cw + kAttHalf * 4 * NB);                      // [128][4]
  float *part = (float *)(cs + kAttHalf * 4);                           // [4][128][NQ] slice sums
  const int tid = threadIdx.x;
  // residual: thread = (four neighbouring features, one of eight 16-token slices of the staged half): one word, one scale
  // and one weight load serve four codes; sum_t p_t Delta_t (u_tf - 2^(b-1) + 1/2)
  const int fq = tid & 31, sl = tid >> 5;
  const int f0 = fq * 4, g = f0 >> 5, bit = (f0 & 31) * NB, wi = g * NB + (bit >> 5), sh = bit & 31;
  const bool straddle = NB == 3 && sh + 4 * NB > 32;           // only 3-bit codes cross a word inside a quad
  constexpr uint32_t mask = (1u << NB) - 1u;
  constexpr float off = 8388608.0f + (float)(1 << (NB - 1));
  float acc[4][NQ];
#pragma unroll
  for (int c = 0; c < 4; ++c)
#pragma unroll
    for (int i = 0; i < NQ; ++i) acc[c][i] = 0.f;
  for (int hf = 0; hf < 2; ++hf) {
    const int t0 = chunk * kAttChunk + hf * kAttHalf;
    if (t0 >= jb.T) break;                              // T is a multiple of 128: a half is all in or all out
    if (hf) __syncthreads();                            // the first half has been read
    {
      const float4 *src = (const float4 *)(jb.p + ((size_t)h * jb.T + t0) * NQ);
      for (int i = tid; i < kAttHalf * NQ / 4; i += kAttChunk) ((float4 *)ps)[i] = src[i];
      const uint4 *wsrc = (const uint4 *)(jb.v.words + ((size_t)h * jb.T + t0) * (4 * NB));
      for (int i = tid; i < kAttHalf * NB; i += kAttChunk) ((uint4 *)cw)[i] = __ldg(wsrc + i);
      const uint2 *ssrc = (const uint2 *)(jb.v.scales + ((size_t)h * jb.T + t0) * 4);
      for (int i = tid; i < kAttHalf; i += kAttChunk) ((uint2 *)cs)[i] = __ldg(ssrc + i);
    }
    __syncthreads();
    const int tb = sl * 16;
#pragma unroll 4
    for (int t = tb; t < tb + 16; ++t) {
      const uint32_t *row = cw + t * (4 * NB);
      uint32_t u4 = row[wi] >> sh;
      if (straddle) u4 |= row[wi + 1] << (32 - sh);
      const float delta = __half2float(cs[t * 4 + g]), hd = 0.5f * delta;
      float pv[NQ];
#pragma unroll
      for (int q4 = 0; q4 < NQ; q4 += 4) {
        const float4 p4 = *(const float4 *)(ps + t * NQ + q4);
        pv[q4] = p4.x; pv[q4 + 1] = p4.y; pv[q4 + 2] = p4.z; pv[q4 + 3] = p4.w;
      }
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        // integer code to float without a conversion instruction: 2^23 + u, minus (2^23 + 2^(b-1)); then Delta (u - 2^(b-1) + 1/2)
        const float val = fmaf(__uint_as_float(0x4B000000u | ((u4 >> (c * NB)) & mask)) - off, delta, hd);
#pragma unroll
        for (int i = 0; i < NQ; ++i) acc[c][i] = fmaf(pv[i], val, acc[c][i]);
      }
    }
  }
  // sum over the eight slices: 7..4 -> 3..0, 3..2 -> 1..0, 1 -> 0 through part[4][128][NQ]
#pragma unroll
  for (int stride = 4; stride >= 1; stride >>= 1) {
    if (sl >= stride && sl < 2 * stride) {
#pragma unroll
      for (int c = 0; c < 4; ++c)
#pragma unroll
        for (int i = 0; i < NQ; ++i) part[((sl - stride) * 128 + f0 + c) * NQ + i] = acc[c][i];
    }
    __syncthreads();
    if (sl < stride) {
#pragma unroll
      for (int c = 0; c < 4; ++c)
#pragma unroll
        for (int i = 0; i < NQ; ++i) acc[c][i] += part[(sl * 128 + f0 + c) * NQ + i];
    }
    __syncthreads();
  }
  if (sl == 0) {
    float *ap = jb.a + (((size_t)h * n_chunks + chunk) * 128 + f0) * NQ;
#pragma unroll
    for (int c = 0; c < 4; ++c)
#pragma unroll
      for (int i = 0; i < NQ; ++i) ap[c * NQ + i] = acc[c][i];
  }
}

// The value-side code stream on the tensor cores, for 1-, 2-, 4- and 8-bit codes:
//     a[f][i] = sum_t (2 u_tf + 1 - 2^b) * (Delta_t,g(f) p_t,i / 2)
// is a product with M = features, N = queries, K = tokens.  Per 128-token half of the chunk the CTA expands the packed
// codes to an fp16 tile E[t][f] in shared memory (exact integers; 16-byte pieces swizzled by the token index so that both
// the row-wise writes and the transposed 8 x 8 fragment loads are conflict-free), writes the weights times the steps,
// scaled by one power of two per half so that fp16 holds them, as hi + lo fp16 W[g][i][t], and then every warp owns 16
// features: one transposed ldmatrix.x4 and two MMAs per 16 tokens.  No reduction between warps.
// grid (n_chunks, m, groups), kAttChunk threads.  Dynamic shared memory: 32 KB + 4 * 2 * NQ * 136 halves.
__device__ __forceinline__ void att_ldmatrix_x4_trans(uint32_t (&r)[4], const void *smem_row) {
  const uint32_t addr = (uint32_t)__cvta_generic_to_shared(smem_row);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}

template <int BITS, int NQ>
__global__ void __launch_bounds__(kAttChunk, 4) attend_values_mma_kernel(const AttendJob *__restrict__ jobs) {
  static_assert(BITS == 1 || BITS == 2 || BITS == 4 || BITS == 8, "codes that do not straddle words");
  const AttendJob &jb = jobs[blockIdx.z];
  if (jb.v.bits != BITS) return;
  const int h = blockIdx.y, chunk = blockIdx.x, n_chunks = gridDim.x;
  if (h >= jb.m || chunk * kAttChunk >= jb.T) return;
  extern __shared__ unsigned char att_smem[];
  typedef __half ERow[128];
  typedef __half WBlk[2][NQ][kAttHalf + 8];
  ERow *E = (ERow *)att_smem;                                   // [128 tokens][128 f], swizzled: piece j of row t sits at j ^ (t & 7)
  WBlk *W = (WBlk *)(att_smem + sizeof(ERow) * kAttHalf);       // [group][hi | lo][query][token]
  __shared__ float dmax[kAttChunk / 32];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, c = lane & 3;
  const int row = tid >> 1, hh = tid & 1;              // staging: token row of the half, feature half (groups 2 hh, 2 hh + 1)
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  for (int hf = 0; hf < 2; ++hf) {
    const int t0 = chunk * kAttChunk + hf * kAttHalf;
    if (t0 >= jb.T) break;                             // T is a multiple of 128: a half is all in or all out
    const size_t grow = (size_t)h * jb.T + t0 + row;
    // packed codes of the half: 128 * BITS pieces of 16 bytes, consecutive threads take consecutive pieces (coalesced)
    constexpr int NIT = (kAttHalf * BITS + kAttChunk - 1) / kAttChunk;
    uint4 cw[NIT];
    {
      const uint4 *src = (const uint4 *)(jb.v.words + ((size_t)h * jb.T + t0) * (4 * BITS));
#pragma unroll
      for (int it = 0; it < NIT; ++it) {
        const int idx = tid + it * kAttChunk;
        cw[it] = idx < kAttHalf * BITS ? __ldg(src + idx) : make_uint4(0u, 0u, 0u, 0u);
      }
    }
    const uint32_t sc2 = __ldg((const uint32_t *)(jb.v.scales + grow * 4) + hh);       // steps of groups 2 hh, 2 hh + 1
    const float d0 = __half2float(__ushort_as_half((unsigned short)(sc2 & 0xFFFFu))), d1 = __half2float(__ushort_as_half((unsigned short)(sc2 >> 16)));
    float pv[NQ];
#pragma unroll
    for (int q4 = 0; q4 < NQ; q4 += 4) {
      const float4 p4 = *(const float4 *)(jb.p + grow * NQ + q4);
      pv[q4] = p4.x; pv[q4 + 1] = p4.y; pv[q4 + 2] = p4.z; pv[q4 + 3] = p4.w;
    }
    // one power of two per half so that step * weight / 2 fits fp16: largest step of the half -> below 2^14
    float mx = fmaxf(d0, d1);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    if (hf) __syncthreads();                           // the previous half's tiles have been read
    if (lane == 0) dmax[warp] = mx;
    // codes -> E: a 16-byte piece of a packed row holds 128 / BITS codes = 16 / BITS output pieces of eight fp16 values
#pragma unroll
    for (int it = 0; it < NIT; ++it) {
      const int idx = tid + it * kAttChunk;
      if (idx < kAttHalf * BITS) {
        const int er = idx / BITS, seg = idx % BITS;
        const uint32_t w4[4] = {cw[it].x, cw[it].y, cw[it].z, cw[it].w};
#pragma unroll
        for (int pc = 0; pc < 16 / BITS; ++pc) {
          uint32_t o[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int bit = 2 * (pc * 4 + j) * BITS;                  // pair pc * 4 + j of this piece of the row's bit string
            o[j] = att_pair_f16(w4[bit >> 5] >> (bit & 31), BITS);
          }
          const int piece = seg * (16 / BITS) + pc;
          *(uint4 *)&E[er][((piece ^ (er & 7)) << 3)] = make_uint4(o[0], o[1], o[2], o[3]);
        }
      }
    }
    __syncthreads();
    mx = dmax[0];
#pragma unroll
    for (int wq = 1; wq < kAttChunk / 32; ++wq) mx = fmaxf(mx, dmax[wq]);
    int ex = 0;
    if (mx > 0.f && mx < INFINITY) frexpf(mx, &ex);                    // mx < 2^ex
    const float up = ldexpf(0.5f, 14 - ex), down = ldexpf(1.f, ex - 14);
#pragma unroll
    for (int gl = 0; gl < 2; ++gl) {
      const float ds = (gl ? d1 : d0) * up;
#pragma unroll
      for (int i = 0; i < NQ; ++i) {
        const float x = ds * pv[i];
        const __half hi = __float2half_rn(x);
        W[hh * 2 + gl][0][i][row] = hi;
        W[hh * 2 + gl][1][i][row] = __float2half_rn(x - __half2float(hi));
      }
    }
    __syncthreads();
    // warp = features 16 warp .. +15 (group warp >> 1); 8 steps of 16 tokens
    float d[4] = {0.f, 0.f, 0.f, 0.f};
    const int mi = lane >> 3, r8 = lane & 7, tb8 = mi >> 1, fb = mi & 1;
    const bool have = g < NQ;                           // query columns beyond NQ are zero
    const uint32_t *wh = (const uint32_t *)&W[warp >> 1][0][have ? g : 0][0], *wl = (const uint32_t *)&W[warp >> 1][1][have ? g : 0][0];
#pragma unroll
    for (int s16 = 0; s16 < kAttHalf / 16; ++s16) {
      uint32_t a[4];
      const int tr = s16 * 16 + tb8 * 8 + r8;
      att_ldmatrix_x4_trans(a, &E[tr][(((2 * warp + fb) ^ (tr & 7)) << 3)]);
      // ldmatrix order: (tokens 0-7, f 0-7), (tokens 0-7, f 8-15), (tokens 8-15, f 0-7), (tokens 8-15, f 8-15) = a0, a1, a2, a3
      att_mma_f16(d, a, have ? wh[s16 * 8 + c] : 0u, have ? wh[s16 * 8 + c + 4] : 0u);
      att_mma_f16(d, a, have ? wl[s16 * 8 + c] : 0u, have ? wl[s16 * 8 + c + 4] : 0u);
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[j] = fmaf(d[j], down, acc[j]);
  }
  if (2 * c < NQ) {
    float *ap = jb.a + (((size_t)h * n_chunks + chunk) * 128 + warp * 16 + g) * NQ + 2 * c;
    *(float2 *)ap = make_float2(acc[0], acc[1]);
    *(float2 *)(ap + 8 * NQ) = make_float2(acc[2], acc[3]);
  }
}

// The backbone terms are shared by all heads of a cell (one U_T per cell), so they are two small dense products over the
// whole cell instead of a loop per head:  with n = (head, query),
//   attend_bscore_kernel   S_b[t][n] = sum_k U_T[t][k] w[n][k]            written to the weight buffer p[h][t][i]
//   attend_bvalue_kernel   y[chunk][n][k] = sum_{t in chunk} p[n][t] U_T[t][k]
// Both run on the tensor cores as warp-level m16n8k16 fp16 MMAs with fp32 accumulation: U_T is fp16 as stored, the
// fp32 operand enters as hi + lo fp16 (22 bits) -- p lies in [0, 1]; w is scaled per column by a power of two bounded
// through |q|_2 (see attend_prep_kernel).  0.13 GFLOP per cell each with N = 128: too small to set up TMEM-resident
// tcgen05 tiles for.  (A TF32 m16n8k8 form of the first product ran at the CUDA-core FMA rate and was replaced.)
constexpr int kAttBPitch = 136;     // floats per staged operand row: 8 c + g addresses all 32 banks

// grid (ceil(T / 64), ceil(m NQP / 128), groups), 256 threads: warp w owns 16 tokens (w & 3) x 64 columns n (w >> 2).
// m16n8k16 fp16 MMAs: A = U_T as stored, B = the scaled w as hi + lo.  The operands of the next 32-wide k chunk are
// requested into registers before the MMAs of the current one.
__global__ void __launch_bounds__(256, 2) attend_bscore_kernel(const AttendJob *__restrict__ jobs, int NQP) {
  const AttendJob &jb = jobs[blockIdx.z];
  const int r_t = jb.k.r_t, N = jb.m * NQP, n0 = blockIdx.y * 128, t0 = blockIdx.x * 64;
  if (r_t == 0 || n0 >= N || t0 >= jb.T) return;
  __shared__ __align__(16) uint32_t Bh[16][kAttBPitch], Bl[16][kAttBPitch];       // w chunk as k pairs, hi and lo, [k / 2][n]
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, c = lane & 3;
  const int wt = warp & 3, wn = warp >> 2;
  float acc[8][4];
#pragma unroll
  for (int nt = 0; nt < 8; ++nt)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[nt][j] = 0.f;
  const int ta = min(t0 + wt * 16 + g, jb.T - 1), tb = min(t0 + wt * 16 + g + 8, jb.T - 1);   // rows past the end repeat the last
  const __half *rowa = jb.k.UT + (size_t)ta * r_t, *rowb = jb.k.UT + (size_t)tb * r_t;
  // staging items of a chunk: (hi | lo, column n, block of eight k) -> 2 * 128 * 4 = 1024, four per thread
  uint4 breg[4];
  uint4 areg[4][2];
  auto load_chunk = [&](int k0) {
#pragma unroll
    for (int it = 0; it < 4; ++it) {
      const int idx = tid + it * 256, hl = idx >> 9, nn = (idx >> 2) & 127, kb8 = (idx & 3) * 8, n = n0 + nn;
      breg[it] = make_uint4(0u, 0u, 0u, 0u);
      if (n < N && k0 + kb8 < r_t) breg[it] = *(const uint4 *)((hl ? jb.wl : jb.wh) + (size_t)n * r_t + k0 + kb8);
    }
#pragma unroll
    for (int k8 = 0; k8 < 4; ++k8) {
      areg[k8][0] = make_uint4(0u, 0u, 0u, 0u); areg[k8][1] = areg[k8][0];
      if (k0 + k8 * 8 < r_t) {
        areg[k8][0] = __ldg((const uint4 *)(rowa + k0 + k8 * 8));
        areg[k8][1] = __ldg((const uint4 *)(rowb + k0 + k8 * 8));
      }
    }
  };
  auto word_of = [](const uint4 &u, int w) { return (w & 2) ? ((w & 1) ? u.w : u.z) : ((w & 1) ? u.y : u.x); };
  load_chunk(0);
  for (int k0 = 0; k0 < r_t; k0 += 32) {
    __syncthreads();
#pragma unroll
    for (int it = 0; it < 4; ++it) {
      const int idx = tid + it * 256, hl = idx >> 9, nn = (idx >> 2) & 127, kp0 = (idx & 3) * 4;
      uint32_t (*dst)[kAttBPitch] = hl ? Bl : Bh;
      dst[kp0][nn] = breg[it].x; dst[kp0 + 1][nn] = breg[it].y; dst[kp0 + 2][nn] = breg[it].z; dst[kp0 + 3][nn] = breg[it].w;
    }
    uint4 acur[4][2];
#pragma unroll
    for (int k8 = 0; k8 < 4; ++k8) { acur[k8][0] = areg[k8][0]; acur[k8][1] = areg[k8][1]; }
    __syncthreads();
    if (k0 + 32 < r_t) load_chunk(k0 + 32);
#pragma unroll
    for (int s16 = 0; s16 < 2; ++s16) {
      // A: rows g, g + 8; k = 16 s16 + 2c, +1 (word c of the first eight halves) and + 8 (word c of the next eight)
      const uint32_t a[4] = {word_of(acur[2 * s16][0], c), word_of(acur[2 * s16][1], c), word_of(acur[2 * s16 + 1][0], c), word_of(acur[2 * s16 + 1][1], c)};
#pragma unroll
      for (int nt = 0; nt < 8; ++nt) {
        const int col = wn * 64 + nt * 8 + g;
        att_mma_f16(acc[nt], a, Bh[s16 * 8 + c][col], Bh[s16 * 8 + c + 4][col]);
        att_mma_f16(acc[nt], a, Bl[s16 * 8 + c][col], Bl[s16 * 8 + c + 4][col]);
      }
    }
  }
  const int t_lo = t0 + wt * 16 + g, t_hi = t_lo + 8;
#pragma unroll
  for (int nt = 0; nt < 8; ++nt) {
    const int n = n0 + wn * 64 + nt * 8 + 2 * c;
    if (n >= N) continue;
    const float2 we = *(const float2 *)(jb.we + n);
    const size_t col = (size_t)(n / NQP) * jb.T * NQP + n % NQP;
    if (t_lo < jb.T) *(float2 *)(jb.p + col + (size_t)t_lo * NQP) = make_float2(acc[nt][0] * we.x, acc[nt][1] * we.y);
    if (t_hi < jb.T) *(float2 *)(jb.p + col + (size_t)t_hi * NQP) = make_float2(acc[nt][2] * we.x, acc[nt][3] * we.y);
  }
}

// grid (n_chunks * KT, ceil(m NQP / 128), groups) with KT = ceil(max r_t / 64), 256 threads: 128 columns n x 64 columns k
// of one 256-token chunk; warp w owns 16 n x 64 k.  m16n8k16 fp16 MMAs: U_T is fp16 as stored, a weight p in [0, 1]
// enters as hi + lo fp16 (22 bits; the lo part of a tiny weight may be subnormal, an absolute error below 2^-25).  The
// next 32 tokens' operands are requested into registers before the MMAs of the current 32.
__global__ void __launch_bounds__(256) attend_bvalue_kernel(const AttendJob *__restrict__ jobs, int NQP, int n_chunks, int KT) {
  const AttendJob &jb = jobs[blockIdx.z];
  const int r_t = jb.v.r_t, N = jb.m * NQP, n0 = blockIdx.y * 128;
  const int chunk = blockIdx.x / KT, kb = (blockIdx.x % KT) * 64, t0 = chunk * kAttChunk;
  if (r_t == 0 || n0 >= N || kb >= r_t || t0 >= jb.T) return;
  // token pairs (2 tp, 2 tp + 1) packed as half2, low half = the even token
  __shared__ __align__(16) uint32_t Ph[16][kAttBPitch], Pl[16][kAttBPitch];     // weights hi / lo, [tp][n]
  __shared__ __align__(16) uint32_t Us[16][64 + 8];                             // U_T, [tp][k]
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, c = lane & 3;
  float acc[8][4];
#pragma unroll
  for (int nt = 0; nt < 8; ++nt)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[nt][j] = 0.f;
  const int nt_tok = min(kAttChunk, jb.T - t0);          // a multiple of 128
  float4 preg[2][2];
  uint4 ureg[2];
  const int u_tp = (tid & 127) >> 3, u_k8 = (tid & 7) * 8;
  auto load_step = [&](int tt0) {
#pragma unroll
    for (int it = 0; it < 2; ++it) {
      const int idx = tid + it * 256, tp = idx >> 5, q4 = idx & 31, n = n0 + q4 * 4;
      preg[it][0] = make_float4(0.f, 0.f, 0.f, 0.f); preg[it][1] = preg[it][0];
      if (n < N) {
        const float *src = jb.p + ((size_t)(n / NQP) * jb.T + t0 + tt0 + 2 * tp) * NQP + n % NQP;
        preg[it][0] = *(const float4 *)src;
        preg[it][1] = *(const float4 *)(src + NQP);
      }
    }
    ureg[0] = make_uint4(0u, 0u, 0u, 0u); ureg[1] = ureg[0];
    if (tid < 128 && kb + u_k8 < r_t) {
      const __half *src = jb.v.UT + (size_t)(t0 + tt0 + 2 * u_tp) * r_t + kb + u_k8;
      ureg[0] = __ldg((const uint4 *)src);
      ureg[1] = __ldg((const uint4 *)(src + r_t));
    }
  };
  load_step(0);
  for (int tt0 = 0; tt0 < nt_tok; tt0 += 32) {
    __syncthreads();
#pragma unroll
    for (int it = 0; it < 2; ++it) {
      const int idx = tid + it * 256, tp = idx >> 5, q4 = idx & 31;
      const float4 v0 = preg[it][0], v1 = preg[it][1];
      const float x0[4] = {v0.x, v0.y, v0.z, v0.w}, x1[4] = {v1.x, v1.y, v1.z, v1.w};
      uint32_t hi[4], lo[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const __half2 h2 = __floats2half2_rn(x0[j], x1[j]);
        const float2 hf = __half22float2(h2);
        const __half2 l2 = __floats2half2_rn(x0[j] - hf.x, x1[j] - hf.y);
        hi[j] = *(const uint32_t *)&h2; lo[j] = *(const uint32_t *)&l2;
      }
      *(uint4 *)&Ph[tp][q4 * 4] = make_uint4(hi[0], hi[1], hi[2], hi[3]);
      *(uint4 *)&Pl[tp][q4 * 4] = make_uint4(lo[0], lo[1], lo[2], lo[3]);
    }
    if (tid < 128) {
      const uint32_t w0[4] = {ureg[0].x, ureg[0].y, ureg[0].z, ureg[0].w}, w1[4] = {ureg[1].x, ureg[1].y, ureg[1].z, ureg[1].w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        Us[u_tp][u_k8 + 2 * j] = (w0[j] & 0xFFFFu) | (w1[j] << 16);
        Us[u_tp][u_k8 + 2 * j + 1] = (w0[j] >> 16) | (w1[j] & 0xFFFF0000u);
      }
    }
    __syncthreads();
    if (tt0 + 32 < nt_tok) load_step(tt0 + 32);
#pragma unroll
    for (int s16 = 0; s16 < 2; ++s16) {
      const int nr = warp * 16 + g;
      const uint32_t ah[4] = {Ph[s16 * 8 + c][nr], Ph[s16 * 8 + c][nr + 8], Ph[s16 * 8 + c + 4][nr], Ph[s16 * 8 + c + 4][nr + 8]};
      const uint32_t al[4] = {Pl[s16 * 8 + c][nr], Pl[s16 * 8 + c][nr + 8], Pl[s16 * 8 + c + 4][nr], Pl[s16 * 8 + c + 4][nr + 8]};
#pragma unroll
      for (int nt = 0; nt < 8; ++nt) {
        const uint32_t b0 = Us[s16 * 8 + c][nt * 8 + g], b1 = Us[s16 * 8 + c + 4][nt * 8 + g];
        att_mma_f16(acc[nt], ah, b0, b1);
        att_mma_f16(acc[nt], al, b0, b1);
      }
    }
  }
#pragma unroll
  for (int half = 0; half < 2; ++half) {
    const int n = n0 + warp * 16 + g + half * 8;
    if (n >= N) continue;
    float *yr = jb.y + ((size_t)(n / NQP) * n_chunks + chunk) * r_t * NQP + n % NQP;
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
      const int k = kb + nt * 8 + 2 * c;
      if (k < r_t) yr[(size_t)k * NQP] = acc[nt][half * 2];
      if (k + 1 < r_t) yr[(size_t)(k + 1) * NQP] = acc[nt][half * 2 + 1];
    }
  }
}

// grid (m, groups, n_q), 128 threads (thread = feature); CTA z finishes query z.  Dynamic shared memory:
// (n_chunks + v.r_t + 128 + 1) floats.
__global__ void __launch_bounds__(128) attend_combine_kernel(const AttendJob *__restrict__ jobs, int n_q, int NQP, int n_chunks,
                                                             uint64_t seed) {
  const AttendJob &jb = jobs[blockIdx.y];
  const int h = blockIdx.x, f = threadIdx.x, i = blockIdx.z;
  if (h >= jb.m) return;
  extern __shared__ unsigned char att_smem[];
  const int r_t = jb.v.r_t;
  float *coef = (float *)att_smem;                                   // [n_chunks]
  float *ys = coef + n_chunks;                                       // [r_t]
  float *buf = ys + r_t;                                             // [128]
  float *Ls = buf + 128;                                             // [1]
  const float *ml = jb.ml + (size_t)h * n_chunks * 2 * NQP;
  // running-maximum merge of the chunks: warp 0 finds the maximum and the rescaled sum
  if (f < 32) {
    float M = -INFINITY;
    for (int c = f; c < n_chunks; c += 32) M = fmaxf(M, ml[c * 2 * NQP + i]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
    float L = 0.f;
    for (int c = f; c < n_chunks; c += 32) {
      const float cf = expf(ml[c * 2 * NQP + i] - M);
      coef[c] = cf;
      L = fmaf(cf, ml[c * 2 * NQP + NQP + i], L);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) L += __shfl_xor_sync(0xffffffffu, L, o);
    if (f == 0) Ls[0] = L;
  }
  __syncthreads();
  for (int k = f; k < r_t; k += 128) {
    const float *yp = jb.y + ((size_t)h * n_chunks * r_t + k) * NQP + i;
    float acc = 0.f;
#pragma unroll 8
    for (int c = 0; c < n_chunks; ++c) acc = fmaf(coef[c], __ldg(yp + (size_t)c * r_t * NQP), acc);
    ys[k] = acc;
  }
  float res = 0.f;
  if (jb.v.bits > 0) {
    const float *ap = jb.a + ((size_t)h * n_chunks * 128 + f) * NQP + i;
    float acc = 0.f;
#pragma unroll 8
    for (int c = 0; c < n_chunks; ++c) acc = fmaf(coef[c], __ldg(ap + (size_t)c * 128 * NQP), acc);
    buf[f] = acc;
  }
  __syncthreads();
  if (jb.v.bits > 0) res = att_wht_smem(buf, f) * kInvSqrtD * att_sign(seed, jb.v.cell, f);
  float ob = 0.f;
  if (r_t > 0) {
    const __half *P = jb.vP + (size_t)h * r_t * 128 + f;
    float o0 = 0.f, o1 = 0.f, o2 = 0.f, o3 = 0.f;
    for (int k = 0; k < r_t; k += 4) {       // r_t is a multiple of 8
      o0 = fmaf(ys[k], __half2float(P[(size_t)k * 128]), o0);
      o1 = fmaf(ys[k + 1], __half2float(P[(size_t)(k + 1) * 128]), o1);
      o2 = fmaf(ys[k + 2], __half2float(P[(size_t)(k + 2) * 128]), o2);
      o3 = fmaf(ys[k + 3], __half2float(P[(size_t)(k + 3) * 128]), o3);
    }
    ob = ((o0 + o1) + (o2 + o3)) * ldexpf(1.f, *jb.v.e);
  }
  jb.out[((size_t)h * n_q + i) * 128 + f] = (ob + res) / Ls[0];
}

}  // namespace jolt
