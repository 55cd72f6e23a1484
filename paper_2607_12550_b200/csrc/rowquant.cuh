// Per-row pieces of the rotated residual code: sign flip + 128-point Walsh-Hadamard transform in
// registers, per-32-feature absmax mid-rise quantiser with an fp16 step, little-endian bit packing,
// and the exact inverse.  One thread owns one 128-feature row.
#pragma once
#include "common.cuh"

namespace jolt {

constexpr float kInvSqrtD = 0.088388347648318440550f;  // 1 / sqrt(128)

// In-place unnormalised Sylvester-ordered WHT of 128 values: y_i = sum_j (-1)^popcount(i & j) x_j.
__device__ __forceinline__ void wht128(float (&v)[128]) {
#pragma unroll
  for (int len = 1; len < 128; len <<= 1) {
#pragma unroll
    for (int i = 0; i < 128; ++i) {
      if ((i & len) == 0) {
        const float a = v[i], b = v[i | len];
        v[i] = a + b;
        v[i | len] = a - b;
      }
    }
  }
}

// sign word w (4 x 32 bits): bit f set -> feature f is negated
__device__ __forceinline__ void apply_signs(float (&v)[128], const uint32_t (&sw)[4]) {
#pragma unroll
  for (int f = 0; f < 128; ++f)
    v[f] = __uint_as_float(__float_as_uint(v[f]) ^ (((sw[f >> 5] >> (f & 31)) & 1u) << 31));
}

// Rotate, quantise and pack one residual row.  words: 4*BITS uint32, scales: 4 halves.
template <int BITS>
__device__ __forceinline__ void quantize_pack_row(float (&r)[128], const uint32_t (&sw)[4],
                                                  uint32_t *__restrict__ words, __half *__restrict__ scales,
                                                  int *bad_scale) {
  apply_signs(r, sw);
  wht128(r);
  constexpr float half_levels = (float)(1 << (BITS - 1));
#pragma unroll
  for (int g = 0; g < 4; ++g) {
    float a = 0.f;
#pragma unroll
    for (int j = 0; j < 32; ++j) { r[g * 32 + j] *= kInvSqrtD; a = fmaxf(a, fabsf(r[g * 32 + j])); }
    const __half dh = __float2half_rn(a * (1.0f / half_levels));
    const float delta = __half2float(dh);
    if (isinf(delta) || isnan(delta)) *bad_scale = 1;
    const float inv = (delta == 0.f) ? 0.f : 1.0f / delta;
    scales[g] = dh;
    uint64_t accw = 0;
    int nb = 0, wi = 0;
#pragma unroll
    for (int j = 0; j < 32; ++j) {
      // clamp(floor(v), -L, L-1) + L without a rounding or conversion instruction (both run on the quarter-rate
      // pipe and bound this pass): clamp v to [-L, L - 1/2] first (same result: floor is monotone), then one
      // round-toward-zero add of 2^23 + L leaves floor(v + L) in the low mantissa bits of a positive float
      const float v = fminf(fmaxf(__fmul_rn(r[g * 32 + j], inv), -half_levels), half_levels - 0.5f);
      const uint32_t code = __float_as_uint(__fadd_rz(v, 8388608.0f + half_levels)) & 0x1FFu;
      const uint32_t u = (delta == 0.f) ? (uint32_t)half_levels : code;
      accw |= (uint64_t)u << nb;
      nb += BITS;
      if (nb >= 32) { words[g * BITS + wi] = (uint32_t)accw; accw >>= 32; nb -= 32; ++wi; }
    }
  }
}

// Unpack, dequantise and rotate back one row: r = s . H(delta * (u - 2^(b-1) + 1/2)) / sqrt(d).
template <int BITS>
__device__ __forceinline__ void unpack_dequant_row(const uint32_t *__restrict__ words,
                                                   const __half *__restrict__ scales, const uint32_t (&sw)[4],
                                                   float (&r)[128]) {
  constexpr float off = 0.5f - (float)(1 << (BITS - 1));
  constexpr uint32_t mask = (1u << BITS) - 1u;
#pragma unroll
  for (int g = 0; g < 4; ++g) {
    const float delta = __half2float(scales[g]);
    uint64_t accw = 0;
    int nb = 0, wi = 0;
#pragma unroll
    for (int j = 0; j < 32; ++j) {
      if (nb < BITS) { accw |= (uint64_t)words[g * BITS + wi] << nb; nb += 32; ++wi; }
      const uint32_t u = (uint32_t)accw & mask;
      accw >>= BITS; nb -= BITS;
      r[g * 32 + j] = ((float)u + off) * delta;
    }
  }
  wht128(r);
#pragma unroll
  for (int f = 0; f < 128; ++f) r[f] *= kInvSqrtD;
  apply_signs(r, sw);
}

__device__ __forceinline__ void cell_sign_words(uint64_t seed, int cell, uint32_t (&sw)[4]) {
  const uint64_t base = stream_base(seed, cell, STREAM_SIGNS);
  const uint64_t w0 = mix64(base + 0), w1 = mix64(base + 1);
  sw[0] = (uint32_t)w0; sw[1] = (uint32_t)(w0 >> 32); sw[2] = (uint32_t)w1; sw[3] = (uint32_t)(w1 >> 32);
}

// ---- unfused kernels: residual against a materialised backbone / plain reconstruction add ----

struct RowJob {          // one per cell
  CellDesc c;
  const float *Xt;       // [m][T][128] fp32 backbone (nullptr when r_t == 0)
  uint32_t *words;       // [m][T][4*bits]
  __half *scales;        // [m][T][4]
  int *status;
  // decompress side
  void *out; int out_dtype; long long osl, osh, ost;
  long long row0;        // first global row index of this cell in the launch (prefix sum of m*T)
};

template <int BITS>
__device__ __forceinline__ void residual_quant_row(const RowJob &jb, uint64_t seed, int h, int t) {
  float r[128];
  const long long off = cell_row_offset(jb.c, h, t);
  if (jb.c.dtype == DT_F16) {
    const uint4 *p = (const uint4 *)((const __half *)jb.c.X + off);
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const uint4 v = p[i];
      const __half2 *hp = (const __half2 *)&v;
#pragma unroll
      for (int j = 0; j < 4; ++j) { const float2 f = __half22float2(hp[j]); r[i * 8 + 2 * j] = f.x; r[i * 8 + 2 * j + 1] = f.y; }
    }
  } else {
    const float4 *p = (const float4 *)((const float *)jb.c.X + off);
#pragma unroll
    for (int i = 0; i < 32; ++i) { const float4 v = p[i]; r[4 * i] = v.x; r[4 * i + 1] = v.y; r[4 * i + 2] = v.z; r[4 * i + 3] = v.w; }
  }
  const long long row = (long long)h * jb.c.T + t;
  if (jb.Xt) {
    const float4 *p = (const float4 *)(jb.Xt + row * 128);
#pragma unroll
    for (int i = 0; i < 32; ++i) { const float4 v = p[i]; r[4 * i] -= v.x; r[4 * i + 1] -= v.y; r[4 * i + 2] -= v.z; r[4 * i + 3] -= v.w; }
  }
  uint32_t sw[4];
  cell_sign_words(seed, jb.c.cell, sw);
  uint32_t words[4 * BITS];
  __half sc[4];
  int bad = 0;
  quantize_pack_row<BITS>(r, sw, words, sc, &bad);
  if (bad) *jb.status = 4;
  uint32_t *wo = jb.words + row * (4 * BITS);
  if constexpr ((4 * BITS) % 4 == 0) {
#pragma unroll
    for (int i = 0; i < BITS; ++i) ((uint4 *)wo)[i] = make_uint4(words[4 * i], words[4 * i + 1], words[4 * i + 2], words[4 * i + 3]);
  }
  *(uint2 *)(jb.scales + row * 4) = *(const uint2 *)sc;
}

__global__ void __launch_bounds__(128) residual_quant_kernel(const RowJob *__restrict__ jobs, int njobs,
                                                            long long total_rows, uint64_t seed) {
  const long long gr = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (gr >= total_rows) return;
  int ji = 0;
  while (ji + 1 < njobs && jobs[ji + 1].row0 <= gr) ++ji;
  const RowJob &jb = jobs[ji];
  if (jb.c.bits == 0) return;
  const long long lr = gr - jb.row0;
  const int h = (int)(lr / jb.c.T), t = (int)(lr - (long long)h * jb.c.T);
  switch (jb.c.bits) {
    case 1: residual_quant_row<1>(jb, seed, h, t); break;
    case 2: residual_quant_row<2>(jb, seed, h, t); break;
    case 3: residual_quant_row<3>(jb, seed, h, t); break;
    case 4: residual_quant_row<4>(jb, seed, h, t); break;
    case 8: residual_quant_row<8>(jb, seed, h, t); break;
    default: break;
  }
}

template <int BITS>
__device__ __forceinline__ void dequant_add_row(const RowJob &jb, uint64_t seed, int h, int t) {
  float r[128];
  const long long row = (long long)h * jb.c.T + t;
  if constexpr (BITS > 0) {
    uint32_t words[4 * BITS];
    const uint4 *wp = (const uint4 *)(jb.words + row * (4 * BITS));
#pragma unroll
    for (int i = 0; i < BITS; ++i) { const uint4 v = wp[i]; words[4 * i] = v.x; words[4 * i + 1] = v.y; words[4 * i + 2] = v.z; words[4 * i + 3] = v.w; }
    __half sc[4];
    *(uint2 *)sc = *(const uint2 *)(jb.scales + row * 4);
    uint32_t sw[4];
    cell_sign_words(seed, jb.c.cell, sw);
    unpack_dequant_row<BITS>(words, sc, sw, r);
  } else {
#pragma unroll
    for (int f = 0; f < 128; ++f) r[f] = 0.f;
  }
  if (jb.Xt) {
    const float4 *p = (const float4 *)(jb.Xt + row * 128);
#pragma unroll
    for (int i = 0; i < 32; ++i) { const float4 v = p[i]; r[4 * i] += v.x; r[4 * i + 1] += v.y; r[4 * i + 2] += v.z; r[4 * i + 3] += v.w; }
  }
  const int l = h / jb.c.n_heads, hd = h - l * jb.c.n_heads;
  const long long off = (long long)l * jb.osl + (long long)hd * jb.osh + (long long)t * jb.ost;
  if (jb.out_dtype == DT_F16) {
    uint4 *p = (uint4 *)((__half *)jb.out + off);
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      uint4 v;
      __half2 *hp = (__half2 *)&v;
#pragma unroll
      for (int j = 0; j < 4; ++j) hp[j] = __floats2half2_rn(r[i * 8 + 2 * j], r[i * 8 + 2 * j + 1]);
      p[i] = v;
    }
  } else {
    float4 *p = (float4 *)((float *)jb.out + off);
#pragma unroll
    for (int i = 0; i < 32; ++i) p[i] = make_float4(r[4 * i], r[4 * i + 1], r[4 * i + 2], r[4 * i + 3]);
  }
}

__global__ void __launch_bounds__(128) dequant_add_kernel(const RowJob *__restrict__ jobs, int njobs,
                                                         long long total_rows, uint64_t seed) {
  const long long gr = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (gr >= total_rows) return;
  int ji = 0;
  while (ji + 1 < njobs && jobs[ji + 1].row0 <= gr) ++ji;
  const RowJob &jb = jobs[ji];
  const long long lr = gr - jb.row0;
  const int h = (int)(lr / jb.c.T), t = (int)(lr - (long long)h * jb.c.T);
  switch (jb.c.bits) {
    case 0: dequant_add_row<0>(jb, seed, h, t); break;
    case 1: dequant_add_row<1>(jb, seed, h, t); break;
    case 2: dequant_add_row<2>(jb, seed, h, t); break;
    case 3: dequant_add_row<3>(jb, seed, h, t); break;
    case 4: dequant_add_row<4>(jb, seed, h, t); break;
    case 8: dequant_add_row<8>(jb, seed, h, t); break;
    default: break;
  }
}

}  // namespace jolt
