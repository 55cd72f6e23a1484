// Rotary position embedding re-applied to decoded keys (paper App. "RoPE pre vs. post on K": keys are
// decomposed BEFORE the rotation, which is applied again when the cache is decoded).
//
// The paper names the operation and gives no formula.  This is the common rotate-half form: feature j < 64
// of token position p pairs with feature j + 64 and the pair turns by the angle p * base^(-j/64),
//     y_j = x_j cos - x_{j+64} sin,     y_{j+64} = x_{j+64} cos + x_j sin,        p = pos0 + t.
//
// Two forms.  Key cells whose decode runs on the tensor-core kernel with r_t <= 128 are rotated inside that kernel, on
// the accumulator row in registers, from a (cos, sin) table that rope_table_kernel writes once per call.  All other key
// cells take rope_rows_kernel afterwards:
// one pass over the key tensor in place, bound by HBM (one read and one write of every key).  A thread owns
// one token and eight features of each half; its eight (cos, sin) pairs are computed once in fp64 (the angle
// reaches pos0 + T radians, far past what an fp32 argument resolves) and reused for every (layer, head) row the
// thread visits, so the transcendental work is T * 64 * gridDim.y evaluations per call however many heads
// there are.  The rotation itself is fp32.
#pragma once
#include <cuda_fp16.h>

#include "common.cuh"

namespace jolt {

struct RopeJob {
  void *K;                 // first key element, in the caller's layout
  int dtype;               // DT_F16 | DT_F32
  int n_rows;              // n_layers * n_kv_heads
  int n_heads;
  int T;
  long long sl, sh, st;    // element strides: layer, head, token (features are contiguous)
  double base;
  long long pos0;
};

constexpr int kRopeTokensPerCta = 32;

__device__ __forceinline__ void rope_pair(float &a, float &b, float c, float s) {
  const float ya = __fmaf_rn(a, c, -__fmul_rn(b, s));
  const float yb = __fmaf_rn(b, c, __fmul_rn(a, s));
  a = ya; b = yb;
}

// (cos, sin) of every (feature pair, token) of a call, for the decode kernel's fused rotation: tab[j * T + t].
__global__ void __launch_bounds__(256) rope_table_kernel(float2 *tab, int T, double base, long long pos0) {
  const int t = blockIdx.x * 256 + threadIdx.x, j = blockIdx.y;
  __shared__ double inv_freq;
  if (threadIdx.x == 0) inv_freq = pow(base, -(double)j / (double)(kD / 2));
  __syncthreads();
  if (t >= T) return;
  double s, c;
  sincos((double)(pos0 + t) * inv_freq, &s, &c);
  tab[(size_t)j * T + t] = make_float2((float)c, (float)s);
}

__global__ void __launch_bounds__(256) rope_rows_kernel(RopeJob j) {
  const int tok = blockIdx.x * kRopeTokensPerCta + (threadIdx.x >> 3);
  const int slice = threadIdx.x & 7;                 // features slice*8 .. slice*8+7 and the same + 64
  if (tok >= j.T) return;
  float cs[8], sn[8];
  const double pos = (double)(j.pos0 + tok);
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const double inv_freq = pow(j.base, -(double)(slice * 8 + k) / (double)(kD / 2));
    double s, c;
    sincos(pos * inv_freq, &s, &c);
    cs[k] = (float)c; sn[k] = (float)s;
  }
  const long long tok_off = (long long)tok * j.st + slice * 8;
  for (int r = blockIdx.y; r < j.n_rows; r += gridDim.y) {
    const long long off = (long long)(r / j.n_heads) * j.sl + (long long)(r % j.n_heads) * j.sh + tok_off;
    if (j.dtype == DT_F16) {
      __half *p = (__half *)j.K + off;
      uint4 ua = *(const uint4 *)p, ub = *(const uint4 *)(p + kD / 2);
      __half2 *ha = (__half2 *)&ua, *hb = (__half2 *)&ub;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        float2 a = __half22float2(ha[k]), b = __half22float2(hb[k]);
        rope_pair(a.x, b.x, cs[2 * k], sn[2 * k]);
        rope_pair(a.y, b.y, cs[2 * k + 1], sn[2 * k + 1]);
        ha[k] = __floats2half2_rn(a.x, a.y);
        hb[k] = __floats2half2_rn(b.x, b.y);
      }
      *(uint4 *)p = ua;
      *(uint4 *)(p + kD / 2) = ub;
    } else {
      float *p = (float *)j.K + off;
      float4 a0 = *(const float4 *)p, a1 = *(const float4 *)(p + 4);
      float4 b0 = *(const float4 *)(p + kD / 2), b1 = *(const float4 *)(p + kD / 2 + 4);
      rope_pair(a0.x, b0.x, cs[0], sn[0]); rope_pair(a0.y, b0.y, cs[1], sn[1]);
      rope_pair(a0.z, b0.z, cs[2], sn[2]); rope_pair(a0.w, b0.w, cs[3], sn[3]);
      rope_pair(a1.x, b1.x, cs[4], sn[4]); rope_pair(a1.y, b1.y, cs[5], sn[5]);
      rope_pair(a1.z, b1.z, cs[6], sn[6]); rope_pair(a1.w, b1.w, cs[7], sn[7]);
      *(float4 *)p = a0; *(float4 *)(p + 4) = a1;
      *(float4 *)(p + kD / 2) = b0; *(float4 *)(p + kD / 2 + 4) = b1;
    }
  }
}

}  // namespace jolt
