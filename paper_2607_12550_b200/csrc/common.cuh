// Shared definitions of the JoLT CUDA library: status plumbing, the counter-based random
// streams, and the per-cell descriptor every kernel reads.
#pragma once
#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <stdint.h>
#include <math.h>

#define JOLT_HD __host__ __device__ __forceinline__

namespace jolt {

constexpr int kD = 128;            // head_dim the kernels are written for
constexpr int kGroup = 32;         // quantisation group along the feature axis
constexpr int kCoreTargetExp = 10; // stored core is scaled so that max|G| lies in [2^10, 2^11)

enum DType : int { DT_F16 = 0, DT_F32 = 1, DT_F64 = 2 };

enum RngStream : int { STREAM_SKETCH = 0, STREAM_SIGNS = 1, STREAM_PROBE = 2, STREAM_EPS = 3 };

// SplitMix64 finaliser of (z + golden increment).
JOLT_HD uint64_t mix64(uint64_t z) {
  z += 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}
JOLT_HD uint64_t stream_base(uint64_t seed, int cell, int stream) {
  return mix64(mix64(seed) ^ (uint64_t)(4 * (int64_t)cell + stream));
}
// Box-Muller (cosine branch), one normal per 64-bit word, evaluated in fp64.
JOLT_HD double gaussian_from_u64(uint64_t r) {
  const double u1 = ((double)(uint32_t)(r >> 32) + 0.5) * (1.0 / 4294967296.0);
  const double u2 = ((double)(uint32_t)(r & 0xFFFFFFFFull) + 0.5) * (1.0 / 4294967296.0);
  return sqrt(-2.0 * log(u1)) * cos(6.283185307179586476925286766559 * u2);
}

// One (layer group, K|V) cell as the kernels see it.
struct CellDesc {
  const void *X;       // first element of the cell's first layer
  int dtype;           // DT_F16 | DT_F32
  int m, n_heads, T;   // merged heads, heads per layer, tokens
  long long sl, sh, st;  // strides in elements (layer, head, token)
  int r_t, r_f, bits, k; // ranks, residual bits, sketch width
  int N;                 // m * r_f
  int cell;              // 2*g + (K:0, V:1), keys the random streams
};

__device__ __forceinline__ long long cell_row_offset(const CellDesc &c, int h, int t) {
  const int l = h / c.n_heads, hd = h - l * c.n_heads;
  return (long long)l * c.sl + (long long)hd * c.sh + (long long)t * c.st;
}

// Longest token range one tensor-core accumulator contracts over (see tc_gemm.cuh); longer sequences are cut
// into segments whose partial results are added in fp64.
constexpr int kTokSegment = 4096;
inline int tok_segments(int T) { return (T + kTokSegment - 1) / kTokSegment; }

}  // namespace jolt
