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
// Four kernels, all CUDA-core (the work is a stream of 1..8-bit codes against a handful of query vectors):
//   attend_prep_kernel     per (group, head): rotated scaled queries and w = scale 2^e P_h q
//   attend_scores_kernel   per (group, head, 256-token chunk): scores, chunk maximum, p = exp(s - max), chunk sum
//   attend_values_kernel   per (group, head, chunk): p^T U_T and sum_t p_t r^'_t (codes staged in shared memory and
//                          read feature-wise, so the token reduction stays inside a thread)
//   attend_combine_kernel  per (group, head): merges the chunks (running-maximum rescaling), applies P_h of the
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
  float *w;                         // [m][k.r_t][NQP]   scale 2^e P_h q
  float *qt;                        // [m][128][NQP]     scale H(s . q) / sqrt(d)
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

// U_F of a cell transposed into shared memory: ufs[s * 128 + f]
__device__ __forceinline__ void att_stage_uf(const AttendCell &c, __half *ufs, int tid, int nthr) {
  for (int i = tid; i < 128 * c.r_f; i += nthr) {
    const int f = i / c.r_f, s = i - f * c.r_f;
    ufs[s * 128 + f] = c.UF[i];
  }
}

// P_h[k][f] = fp16( sum_s G_h[k][s] U_F[f][s] ), the decoder's projected core in scaled units
__device__ __forceinline__ float att_p16(const __half *__restrict__ grow, const __half *ufs, int r_f, int f) {
  float acc = 0.f;
  for (int s = 0; s < r_f; s += 8) {
    const uint4 g8 = __ldg((const uint4 *)(grow + s));
    const __half *gh = (const __half *)&g8;
#pragma unroll
    for (int j = 0; j < 8; ++j) acc = fmaf(__half2float(gh[j]), __half2float(ufs[(s + j) * 128 + f]), acc);
  }
  return __half2float(__float2half_rn(acc));
}

// grid (m, groups), 128 threads (thread = feature), dynamic shared memory: 128 * r_f halves + 128 floats + 32 floats
__global__ void __launch_bounds__(128) attend_prep_kernel(const AttendJob *__restrict__ jobs, int n_q, int NQP, float scale,
                                                          uint64_t seed) {
  const AttendJob &jb = jobs[blockIdx.y];
  const int h = blockIdx.x, f = threadIdx.x;
  if (h >= jb.m) return;
  extern __shared__ unsigned char att_smem[];
  __half *ufs = (__half *)att_smem;
  float *buf = (float *)(att_smem + (size_t)128 * jb.k.r_f * sizeof(__half));
  float *red = buf + 128;
  float q[kAttMaxQ];
#pragma unroll
  for (int i = 0; i < kAttMaxQ; ++i) q[i] = i < n_q ? jb.q[((size_t)h * n_q + i) * 128 + f] : 0.f;
  if (jb.k.bits > 0) {
    const float sg = att_sign(seed, jb.k.cell, f);
    for (int i = 0; i < NQP; ++i) {
      buf[f] = sg * q[i];
      __syncthreads();
      const float v = att_wht_smem(buf, f);
      jb.qt[((size_t)h * 128 + f) * NQP + i] = v * kInvSqrtD * scale;
      __syncthreads();
    }
  }
  if (jb.k.r_t > 0) {
    att_stage_uf(jb.k, ufs, f, 128);
    __syncthreads();
    const float se = scale * ldexpf(1.f, *jb.k.e);
    const int warp = f >> 5, lane = f & 31;
    for (int k = 0; k < jb.k.r_t; ++k) {
      const float pk = att_p16(jb.k.G + ((size_t)h * jb.k.r_t + k) * jb.k.r_f, ufs, jb.k.r_f, f);
      for (int i = 0; i < NQP; ++i) {
        float v = pk * q[i];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (lane == 0) red[warp * kAttMaxQ + i] = v;
      }
      __syncthreads();
      if (f < NQP) jb.w[((size_t)h * jb.k.r_t + k) * NQP + f] = se * (red[f] + red[kAttMaxQ + f] + red[2 * kAttMaxQ + f] + red[3 * kAttMaxQ + f]);
      __syncthreads();
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
__global__ void __launch_bounds__(kAttChunk) attend_scores_kernel(const AttendJob *__restrict__ jobs, int NQP) {
  const AttendJob &jb = jobs[blockIdx.z];
  if (jb.k.bits != BITS) return;
  const int h = blockIdx.y, chunk = blockIdx.x;
  if (h >= jb.m || chunk * kAttChunk >= jb.T) return;
  extern __shared__ unsigned char att_smem[];
  float *qts = (float *)att_smem;                   // [128][NQP]
  float *ws = qts + 128 * NQP;                      // [r_t][NQP]
  __shared__ float red[2][kAttChunk / 32][kAttMaxQ];
  const int tid = threadIdx.x, r_t = jb.k.r_t;
  if (BITS > 0)
    for (int i = tid; i < 128 * NQP; i += kAttChunk) qts[i] = jb.qt[(size_t)h * 128 * NQP + i];
  for (int i = tid; i < r_t * NQP; i += kAttChunk) ws[i] = jb.w[(size_t)h * r_t * NQP + i];
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
      constexpr float off = 0.5f - (float)(1 << (BITS - 1));
      for (int qq = 0; qq < NQP; qq += 4) {
        float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
        for (int g = 0; g < 4; ++g) {
          const float delta = __half2float(sc[g]);
          float g0 = 0.f, g1 = 0.f, g2 = 0.f, g3 = 0.f;
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            // integer code to float without a conversion instruction: 2^23 + u, minus 2^23
            const float val = __uint_as_float(0x4B000000u | att_code<BITS>(row, g, j)) - 8388608.0f + off;
            const float4 qv = *(const float4 *)(qts + (g * 32 + j) * NQP + qq);
            g0 = fmaf(val, qv.x, g0); g1 = fmaf(val, qv.y, g1); g2 = fmaf(val, qv.z, g2); g3 = fmaf(val, qv.w, g3);
          }
          a0 = fmaf(delta, g0, a0); a1 = fmaf(delta, g1, a1); a2 = fmaf(delta, g2, a2); a3 = fmaf(delta, g3, a3);
        }
        if (qq == 0) { s[0] = a0; s[1] = a1; s[2] = a2; s[3] = a3; } else { s[4] = a0; s[5] = a1; s[6] = a2; s[7] = a3; }
      }
    }
    if (r_t > 0) {
      const __half *ut = jb.k.UT + (size_t)t * r_t;
      for (int qq = 0; qq < NQP; qq += 4) {
        float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
        for (int k = 0; k < r_t; k += 8) {
          const uint4 u8 = __ldg((const uint4 *)(ut + k));
          const __half *uh = (const __half *)&u8;
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const float u = __half2float(uh[j]);
            const float4 wv = *(const float4 *)(ws + (k + j) * NQP + qq);
            a0 = fmaf(u, wv.x, a0); a1 = fmaf(u, wv.y, a1); a2 = fmaf(u, wv.z, a2); a3 = fmaf(u, wv.w, a3);
          }
        }
        if (qq == 0) { s[0] += a0; s[1] += a1; s[2] += a2; s[3] += a3; } else { s[4] += a0; s[5] += a1; s[6] += a2; s[7] += a3; }
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

// grid (n_chunks, m, groups), kAttChunk threads.  Dynamic shared memory: kAttChunk * (NQP floats + 4 BITS words + 4 halves)
// + 128 * NQP floats.
template <int BITS>
__global__ void __launch_bounds__(kAttChunk) attend_values_kernel(const AttendJob *__restrict__ jobs, int NQP) {
  const AttendJob &jb = jobs[blockIdx.z];
  if (jb.v.bits != BITS) return;
  const int h = blockIdx.y, chunk = blockIdx.x, n_chunks = gridDim.x;
  if (h >= jb.m || chunk * kAttChunk >= jb.T) return;
  extern __shared__ unsigned char att_smem[];
  float *ps = (float *)att_smem;                                        // [kAttChunk][NQP]
  uint32_t *cw = (uint32_t *)(ps + kAttChunk * NQP);                    // [kAttChunk][4 * BITS]
  __half *cs = (__half *)(cw + kAttChunk * 4 * (BITS > 0 ? BITS : 1));  // [kAttChunk][4]
  float *part = (float *)(cs + kAttChunk * 4);                          // [128][NQP] second token half's sums
  const int tid = threadIdx.x, t0 = chunk * kAttChunk;
  const int nt = min(kAttChunk, jb.T - t0);
  {
    const float4 *src = (const float4 *)(jb.p + ((size_t)h * jb.T + t0) * NQP);
    for (int i = tid; i < nt * NQP / 4; i += kAttChunk) ((float4 *)ps)[i] = src[i];
    for (int i = nt * NQP / 4 + tid; i < kAttChunk * NQP / 4; i += kAttChunk) ((float4 *)ps)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    if constexpr (BITS > 0) {
      const uint4 *wsrc = (const uint4 *)(jb.v.words + ((size_t)h * jb.T + t0) * (4 * BITS));
      for (int i = tid; i < nt * BITS; i += kAttChunk) ((uint4 *)cw)[i] = __ldg(wsrc + i);
      const uint2 *ssrc = (const uint2 *)(jb.v.scales + ((size_t)h * jb.T + t0) * 4);
      for (int i = tid; i < nt; i += kAttChunk) ((uint2 *)cs)[i] = __ldg(ssrc + i);
    }
  }
  __syncthreads();
  // residual: thread = (feature f, token half); sum_t p_t Delta_t (u_tf - 2^(b-1) + 1/2)
  if constexpr (BITS > 0) {
    const int f = tid & 127, half = tid >> 7, g = f >> 5, j = f & 31;
    const int bit = j * BITS, wi = g * BITS + (bit >> 5), sh = bit & 31;
    constexpr uint32_t mask = (1u << BITS) - 1u;
    constexpr float off = 0.5f - (float)(1 << (BITS - 1));
    float acc[kAttMaxQ];
#pragma unroll
    for (int i = 0; i < kAttMaxQ; ++i) acc[i] = 0.f;
    const int tb = half * (kAttChunk / 2), te = min(tb + kAttChunk / 2, nt);
    for (int t = tb; t < te; ++t) {
      const uint32_t *row = cw + t * (4 * BITS);
      uint32_t u = row[wi] >> sh;
      if (sh + BITS > 32) u |= row[wi + 1] << (32 - sh);
      const float val = (__uint_as_float(0x4B000000u | (u & mask)) - 8388608.0f + off) * __half2float(cs[t * 4 + g]);
      const float4 p0 = *(const float4 *)(ps + t * NQP);
      acc[0] = fmaf(p0.x, val, acc[0]); acc[1] = fmaf(p0.y, val, acc[1]); acc[2] = fmaf(p0.z, val, acc[2]); acc[3] = fmaf(p0.w, val, acc[3]);
      if (NQP == 8) {
        const float4 p1 = *(const float4 *)(ps + t * NQP + 4);
        acc[4] = fmaf(p1.x, val, acc[4]); acc[5] = fmaf(p1.y, val, acc[5]); acc[6] = fmaf(p1.z, val, acc[6]); acc[7] = fmaf(p1.w, val, acc[7]);
      }
    }
    if (half == 1)
      for (int i = 0; i < NQP; ++i) part[f * NQP + i] = acc[i];
    __syncthreads();
    if (half == 0) {
      float *ap = jb.a + (((size_t)h * n_chunks + chunk) * 128 + f) * NQP;
      for (int i = 0; i < NQP; ++i) ap[i] = acc[i] + part[f * NQP + i];
    }
  }
  // backbone: thread = column k of U_T; y_k = sum_t p_t U_T[t, k]
  const int r_t = jb.v.r_t;
  for (int k = tid; k < r_t; k += kAttChunk) {
    float acc[kAttMaxQ];
#pragma unroll
    for (int i = 0; i < kAttMaxQ; ++i) acc[i] = 0.f;
    const __half *ut = jb.v.UT + (size_t)t0 * r_t + k;
    for (int t = 0; t < nt; ++t) {
      const float u = __half2float(ut[(size_t)t * r_t]);
      const float4 p0 = *(const float4 *)(ps + t * NQP);
      acc[0] = fmaf(p0.x, u, acc[0]); acc[1] = fmaf(p0.y, u, acc[1]); acc[2] = fmaf(p0.z, u, acc[2]); acc[3] = fmaf(p0.w, u, acc[3]);
      if (NQP == 8) {
        const float4 p1 = *(const float4 *)(ps + t * NQP + 4);
        acc[4] = fmaf(p1.x, u, acc[4]); acc[5] = fmaf(p1.y, u, acc[5]); acc[6] = fmaf(p1.z, u, acc[6]); acc[7] = fmaf(p1.w, u, acc[7]);
      }
    }
    float *yp = jb.y + (((size_t)h * n_chunks + chunk) * r_t + k) * NQP;
    for (int i = 0; i < NQP; ++i) yp[i] = acc[i];
  }
}

// grid (m, groups), 128 threads (thread = feature).  Dynamic shared memory: 128 * v.r_f halves + (n_chunks + v.r_t) * NQP
// floats + 128 floats + 2 * kAttMaxQ floats.
__global__ void __launch_bounds__(128) attend_combine_kernel(const AttendJob *__restrict__ jobs, int n_q, int NQP, int n_chunks,
                                                             uint64_t seed) {
  const AttendJob &jb = jobs[blockIdx.y];
  const int h = blockIdx.x, f = threadIdx.x;
  if (h >= jb.m) return;
  extern __shared__ unsigned char att_smem[];
  const int r_t = jb.v.r_t, r_f = jb.v.r_f;
  __half *ufs = (__half *)att_smem;                                  // [r_f][128]
  float *coef = (float *)(att_smem + (size_t)128 * r_f * sizeof(__half));   // [n_chunks][NQP]
  float *ys = coef + n_chunks * NQP;                                 // [r_t][NQP]
  float *buf = ys + r_t * NQP;                                       // [128]
  float *Ls = buf + 128;                                             // [kAttMaxQ]
  if (f < NQP) {
    const float *ml = jb.ml + (size_t)h * n_chunks * 2 * NQP;
    float M = -INFINITY;
    for (int c = 0; c < n_chunks; ++c) M = fmaxf(M, ml[c * 2 * NQP + f]);
    float L = 0.f;
    for (int c = 0; c < n_chunks; ++c) {
      const float cf = expf(ml[c * 2 * NQP + f] - M);
      coef[c * NQP + f] = cf;
      L = fmaf(cf, ml[c * 2 * NQP + NQP + f], L);
    }
    Ls[f] = L;
  }
  if (r_t > 0) att_stage_uf(jb.v, ufs, f, 128);
  __syncthreads();
  for (int i = f; i < r_t * NQP; i += 128) {
    const int q = i % NQP;
    float acc = 0.f;
    for (int c = 0; c < n_chunks; ++c) acc = fmaf(coef[c * NQP + q], jb.y[((size_t)h * n_chunks + c) * r_t * NQP + i], acc);
    ys[i] = acc;
  }
  float ob[kAttMaxQ];
#pragma unroll
  for (int i = 0; i < kAttMaxQ; ++i) ob[i] = 0.f;
  __syncthreads();
  if (r_t > 0) {
    for (int k = 0; k < r_t; ++k) {
      const float pk = att_p16(jb.v.G + ((size_t)h * r_t + k) * r_f, ufs, r_f, f);
#pragma unroll
      for (int i = 0; i < kAttMaxQ; ++i)
        if (i < NQP) ob[i] = fmaf(ys[k * NQP + i], pk, ob[i]);
    }
    const float se = ldexpf(1.f, *jb.v.e);
#pragma unroll
    for (int i = 0; i < kAttMaxQ; ++i) ob[i] *= se;
  }
  const float sg = jb.v.bits > 0 ? att_sign(seed, jb.v.cell, f) : 0.f;
  for (int i = 0; i < n_q; ++i) {
    float res = 0.f;
    if (jb.v.bits > 0) {
      float acc = 0.f;
      for (int c = 0; c < n_chunks; ++c) acc = fmaf(coef[c * NQP + i], jb.a[(((size_t)h * n_chunks + c) * 128 + f) * NQP + i], acc);
      __syncthreads();
      buf[f] = acc;
      __syncthreads();
      res = att_wht_smem(buf, f) * kInvSqrtD * sg;
    }
    float o = 0.f;
#pragma unroll
    for (int q = 0; q < kAttMaxQ; ++q)
      if (q == i) o = ob[q];
    jb.out[((size_t)h * n_q + i) * 128 + f] = (o + res) / Ls[i];
  }
}

}  // namespace jolt
