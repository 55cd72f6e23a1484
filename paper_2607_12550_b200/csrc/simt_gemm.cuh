// Portable batched GEMM on CUDA cores: C = alpha * A B (+ C), arbitrary strides, a K axis that may be
// split into strided segments (the merged layer/head index of a cell), f16 / f32 inputs, fp32 or fp64
// accumulation.  It is the reference kernel family of the library: every tensor-core kernel is checked
// against it, and it serves fp32 caches and shapes the tensor-core kernels do not take.
#pragma once
#include "common.cuh"

namespace jolt {

struct GemmTask {
  const void *A, *B;
  void *C;
  int M, N, K;            // K: length of one segment
  int nseg, seg_inner;    // segment s -> (so, si) = (s / seg_inner, s % seg_inner)
  long long a_rs, a_cs, a_so, a_si;   // A(i, k, s) at i*a_rs + k*a_cs + so*a_so + si*a_si
  long long b_rs, b_cs, b_so, b_si;   // B(k, j, s) at k*b_rs + j*b_cs + so*b_so + si*b_si
  long long c_rs, c_cs;
  int ta, tb, tc;         // DType tags
  float alpha;
  const int *alpha_exp;   // optional: alpha *= 2^(*alpha_exp)
  int accumulate;         // 1: C += result
};

__device__ __forceinline__ float load_elem(const void *p, int t, long long i) {
  if (t == DT_F16) return __half2float(((const __half *)p)[i]);
  if (t == DT_F32) return ((const float *)p)[i];
  return (float)((const double *)p)[i];
}

template <typename Acc>
__global__ void __launch_bounds__(256) simt_gemm_kernel(const GemmTask *__restrict__ tasks) {
  constexpr int BM = 64, BN = 64, BK = 16;
  const GemmTask t = tasks[blockIdx.z];
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  if (m0 >= t.M || n0 >= t.N) return;
  __shared__ float As[BK][BM + 4];
  __shared__ float Bs[BK][BN + 4];
  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;
  Acc acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = Acc(0);
  const bool a_kfast = (t.a_cs == 1);
  const bool b_kfast = (t.b_rs == 1);
  for (int s = 0; s < t.nseg; ++s) {
    const int so = s / t.seg_inner, si = s - so * t.seg_inner;
    const long long abase = so * t.a_so + si * t.a_si;
    const long long bbase = so * t.b_so + si * t.b_si;
    for (int k0 = 0; k0 < t.K; k0 += BK) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int idx = tid + e * 256;
        int i, kk;
        if (a_kfast) { i = idx >> 4; kk = idx & 15; } else { kk = idx >> 6; i = idx & 63; }
        float v = 0.f;
        if (m0 + i < t.M && k0 + kk < t.K)
          v = load_elem(t.A, t.ta, abase + (long long)(m0 + i) * t.a_rs + (long long)(k0 + kk) * t.a_cs);
        As[kk][i] = v;
        int j, kb;
        if (b_kfast) { j = idx >> 4; kb = idx & 15; } else { kb = idx >> 6; j = idx & 63; }
        float w = 0.f;
        if (n0 + j < t.N && k0 + kb < t.K)
          w = load_elem(t.B, t.tb, bbase + (long long)(k0 + kb) * t.b_rs + (long long)(n0 + j) * t.b_cs);
        Bs[kb][j] = w;
      }
      __syncthreads();
#pragma unroll
      for (int kk = 0; kk < BK; ++kk) {
        float a[4], b[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
        for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx * 4 + j];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 4; ++j) acc[i][j] += (Acc)a[i] * (Acc)b[j];
      }
      __syncthreads();
    }
  }
  float alpha = t.alpha;
  if (t.alpha_exp) alpha = ldexpf(alpha, *t.alpha_exp);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = m0 + ty * 4 + i;
    if (r >= t.M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int c = n0 + tx * 4 + j;
      if (c >= t.N) continue;
      const long long o = (long long)r * t.c_rs + (long long)c * t.c_cs;
      Acc v = acc[i][j] * (Acc)alpha;
      if (t.tc == DT_F32) {
        float *C = (float *)t.C;
        C[o] = t.accumulate ? C[o] + (float)v : (float)v;
      } else if (t.tc == DT_F64) {
        double *C = (double *)t.C;
        C[o] = t.accumulate ? C[o] + (double)v : (double)v;
      } else {
        ((__half *)t.C)[o] = __float2half_rn((float)v);
      }
    }
  }
}

// fp32 in, fp32 out, one K segment, no accumulate: 128 x 64 tiles, 8 x 4 results per thread read from shared memory
// as 16-byte vectors, the next K slab fetched into registers while the current one is multiplied.
inline bool sgemm_fast_ok(const GemmTask &t) {
  return t.ta == DT_F32 && t.tb == DT_F32 && t.tc == DT_F32 && t.nseg == 1 && !t.accumulate && !t.alpha_exp;
}

__global__ void __launch_bounds__(256, 2) simt_sgemm_kernel(const GemmTask *__restrict__ tasks) {
  constexpr int BM = 128, BN = 64, BK = 16;
  const GemmTask t = tasks[blockIdx.z];
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  if (m0 >= t.M || n0 >= t.N) return;
  __shared__ __align__(16) float As[BK][BM + 4];
  __shared__ __align__(16) float Bs[BK][BN + 4];
  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;
  const float *A = (const float *)t.A, *B = (const float *)t.B;
  const bool a_kfast = (t.a_cs == 1), b_kfast = (t.b_rs == 1);
  float acc[8][4];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
  float pa[8], pb[4];
  auto fetch = [&](int k0) {
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const int idx = tid + e * 256;
      int i, kk;
      if (a_kfast) { i = idx >> 4; kk = idx & 15; } else { kk = idx >> 7; i = idx & 127; }
      pa[e] = (m0 + i < t.M && k0 + kk < t.K) ? A[(long long)(m0 + i) * t.a_rs + (long long)(k0 + kk) * t.a_cs] : 0.f;
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int idx = tid + e * 256;
      int j, kb;
      if (b_kfast) { j = idx >> 4; kb = idx & 15; } else { kb = idx >> 6; j = idx & 63; }
      pb[e] = (n0 + j < t.N && k0 + kb < t.K) ? B[(long long)(k0 + kb) * t.b_rs + (long long)(n0 + j) * t.b_cs] : 0.f;
    }
  };
  fetch(0);
  for (int k0 = 0; k0 < t.K; k0 += BK) {
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const int idx = tid + e * 256;
      int i, kk;
      if (a_kfast) { i = idx >> 4; kk = idx & 15; } else { kk = idx >> 7; i = idx & 127; }
      As[kk][i] = pa[e];
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int idx = tid + e * 256;
      int j, kb;
      if (b_kfast) { j = idx >> 4; kb = idx & 15; } else { kb = idx >> 6; j = idx & 63; }
      Bs[kb][j] = pb[e];
    }
    __syncthreads();
    if (k0 + BK < t.K) fetch(k0 + BK);
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      const float4 a0 = *(const float4 *)&As[kk][ty * 8], a1 = *(const float4 *)&As[kk][ty * 8 + 4];
      const float4 b4 = *(const float4 *)&Bs[kk][tx * 4];
      const float a[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
      const float b[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
  float *C = (float *)t.C;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int r = m0 + ty * 8 + i;
    if (r >= t.M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int c = n0 + tx * 4 + j;
      if (c < t.N) C[(long long)r * t.c_rs + (long long)c * t.c_cs] = acc[i][j] * t.alpha;
    }
  }
}

}  // namespace jolt
