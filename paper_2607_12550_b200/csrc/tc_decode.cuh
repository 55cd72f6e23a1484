// Fused decompress pass (paper Sec. 4 "decoding simply inverts the rotation", Sec. 7): for a (cell, head,
// run of 128-token tiles)
//
//     X^[tile] = 2^e ( U_T[tile] P_h  +  R^[tile] (H S) )
//
// as ONE tcgen05 accumulation per tile: the backbone (K = r_t) and the inverse rotation of the dequantised
// residual (K = 128, B operand = the +-1 Hadamard matrix with the sign flips folded in, exact in fp16) go into
// the same TMEM accumulator.  The epilogue threads only unpack codes into a half-precision operand tile
// (pre-scaled by Delta / sqrt(128) * 2^-e) and, after the MMA, scale, convert and store their row: no
// Hadamard butterflies on the CUDA cores.  P_h = fp16(G_h U_F^T) is the block stored with the handle at compress
// time, fetched by TMA as an MN-major operand exactly as in the residual kernel.  Rounding the dequantised residual to fp16 before the rotation costs 2^-11 of the residual, i.e.
// ~1e-5 of the cache entries, far below the fp16 rounding of the output itself.
#pragma once
#include "tc_backbone.cuh"

// cycle stamps of CTA 0 (a profiling aid) exist only in builds with -DJOLT_DEBUG
#ifdef JOLT_DEBUG
#define JOLT_DBG(x) x
#else
#define JOLT_DBG(x)
#endif

namespace jolt {
namespace tc {

// Two epilogue warpgroups, a producer warpgroup (TMA thread, MMA thread), 224 KB of shared memory, one CTA per SM.
// Any r_t <= 256: P region 64 KB, 4-stage U_T ring, one operand tile and one accumulator per warpgroup.  For
// r_t <= 128 half of the P region is free and extends the ring to six stages (three U_T tiles in flight), and each
// warpgroup owns TWO accumulators: the MMA thread issues the backbone of a tile two tiles before its rotation, so
// backbones wait in TMEM instead of U_T tiles waiting in shared memory, and a warpgroup only waits for the eight
// rotation MMAs of its tile.
constexpr int DEC_H_BYTES = 32768;
constexpr int DEC_NWG = 2;
struct DecLayout {
  static constexpr int THREADS = (DEC_NWG + 1) * 128;
  static constexpr int P_BYTES = 65536;
  static constexpr int NS = 4;                                          // ring stages in the ring region proper
  static constexpr int BIG_BYTES = NS * 16384 + DEC_NWG * 32768;        // ring + operand tiles (set-up operands first)
  static constexpr int SMEM_BYTES = P_BYTES + DEC_H_BYTES + BIG_BYTES + 1024 /*align*/ + 512 /*barriers*/ + 1024 /*cell descriptor*/;
  static_assert(sizeof(BBCell) <= 1024, "the cell descriptor is staged in 1 KB of shared memory");
  static constexpr int TMEM_COLS = 512;     // two accumulators per warpgroup when r_t <= 128
  // registers move from the producer warpgroup to the epilogue ones (12 warps: the register file has the slack a
  // blocking re-partition needs)
  static constexpr int EPI_REGS = 216;
  static constexpr int PROD_REGS = 56;
};

template <int BITS>
struct DecCodesRow { uint32_t words[BITS > 0 ? 4 * BITS : 1]; uint2 sc; };

template <int BITS>
__device__ __forceinline__ void dec_load_codes_row(const BBCell &c, long long row, DecCodesRow<BITS> &d) {
  if constexpr (BITS > 0) {
    const uint4 *wp = (const uint4 *)(c.words + row * (4 * BITS));
#pragma unroll
    for (int i = 0; i < BITS; ++i) { const uint4 v = __ldg(wp + i); d.words[4 * i] = v.x; d.words[4 * i + 1] = v.y; d.words[4 * i + 2] = v.z; d.words[4 * i + 3] = v.w; }
    d.sc = __ldg((const uint2 *)(c.scales + row * 4));
  }
}

// Code j of a 32-code group as the bit pattern of the float 2^23 + code (the code dropped into the low mantissa
// byte of 0x4B000000 by one byte permute): adding -(2^23 + 2^(BITS-1)) gives code - 2^(BITS-1) exactly, without an
// integer conversion, and one FMA with dq and dq/2 the dequantised value (code - 2^(BITS-1) + 1/2) dq, rounded once.  W = the group's BITS words, code j at bits [j*BITS, j*BITS + BITS).
template <int BITS>
struct DecGroupBytes {      // per-group byte lanes from which every code is one PRMT away
  uint32_t t[BITS == 8 ? 8 : (BITS == 4 ? 8 : (BITS == 2 ? 8 : (BITS == 1 ? 8 : 1)))];
  __device__ __forceinline__ void load(const uint32_t *W) {
    if constexpr (BITS == 8) {
#pragma unroll
      for (int w = 0; w < 8; ++w) t[w] = W[w];
    } else if constexpr (BITS == 4) {       // t[2w] even nibbles, t[2w+1] odd nibbles of word w
#pragma unroll
      for (int w = 0; w < 4; ++w) { t[2 * w] = W[w] & 0x0F0F0F0Fu; t[2 * w + 1] = (W[w] >> 4) & 0x0F0F0F0Fu; }
    } else if constexpr (BITS == 2) {       // t[4w + k]: fields k, k+4, k+8, k+12 of word w
#pragma unroll
      for (int w = 0; w < 2; ++w)
#pragma unroll
        for (int k = 0; k < 4; ++k) t[4 * w + k] = (W[w] >> (2 * k)) & 0x03030303u;
    } else if constexpr (BITS == 1) {       // t[k]: bits k, k+8, k+16, k+24
#pragma unroll
      for (int k = 0; k < 8; ++k) t[k] = (W[0] >> k) & 0x01010101u;
    }
  }
  __device__ __forceinline__ float value(int j) const {     // j is a compile-time constant after unrolling
    uint32_t src; int byte;
    if constexpr (BITS == 8) { src = t[j >> 2]; byte = j & 3; }
    else if constexpr (BITS == 4) { src = t[2 * (j >> 3) + (j & 1)]; byte = (j & 7) >> 1; }
    else if constexpr (BITS == 2) { src = t[4 * (j >> 4) + (j & 3)]; byte = (j & 15) >> 2; }
    else { src = t[j & 7]; byte = j >> 3; }
    return __uint_as_float(__byte_perm(src, 0x4B000000u, 0x7650u + (uint32_t)byte));
  }
};

// codes -> fp16 operand row (pre-scaled), written into the warpgroup's swizzled K-major tile
template <int BITS>
__device__ __forceinline__ void dec_unpack_row_row(const DecCodesRow<BITS> &d, float pre, unsigned char *rbuf, int rit) {
  constexpr float off = 0.5f - (float)(1 << (BITS > 0 ? BITS - 1 : 0));
  constexpr uint32_t mask = (1u << BITS) - 1u;
  constexpr bool kFast = BITS == 8 || BITS == 4 || BITS == 2 || BITS == 1;
  constexpr float c0 = -(8388608.0f + (float)(1 << (BITS > 0 ? BITS - 1 : 0)));
  const __half *sc = (const __half *)&d.sc;
#pragma unroll
  for (int g = 0; g < 4; ++g) {
    const float dq = __half2float(sc[g]) * pre, hdq = 0.5f * dq;
    unsigned char *rowp = rbuf + (g >> 1) * 16384 + rit * 128;
    DecGroupBytes<kFast ? BITS : 8> gb;
    if constexpr (kFast) gb.load(&d.words[g * BITS]);
#pragma unroll
    for (int ck = 0; ck < 4; ++ck) {
      uint4 pk;
      __half2 *hp = (__half2 *)&pk;
#pragma unroll
      for (int e2 = 0; e2 < 4; ++e2) {
        float v2[2];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          const int j = ck * 8 + e2 * 2 + u;
          if constexpr (kFast) {
            v2[u] = fmaf(gb.value(j) + c0, dq, hdq);
          } else {
            // code j of the group sits at bits [j*BITS, j*BITS + BITS) of its BITS little-endian words
            const int bit = j * BITS, w = bit >> 5, sh = bit & 31;
            uint32_t q = d.words[g * BITS + w] >> sh;
            if (sh + BITS > 32) q |= d.words[g * BITS + w + 1] << (32 - sh);
            v2[u] = ((float)(q & mask) + off) * dq;
          }
        }
        hp[e2] = __floats2half2_rn(v2[0], v2[1]);
      }
      const int chunk = (g & 1) * 4 + ck;
      *(uint4 *)(rowp + ((chunk ^ (rit & 7)) << 4)) = pk;
    }
  }
}

// ---- warp-cooperative code path (BITS in {1, 2, 4, 8}) --------------------------------------------------------
// A row of codes is BITS 16-byte chunks.  Instead of every thread fetching its own row (32 rows, 32 half-used
// sectors per load instruction), BITS neighbouring lanes fetch the BITS chunks of one row: a warp instruction then
// reads 512 contiguous bytes, and after BITS instructions the warp holds the codes of its 32 rows.  Each lane
// dequantises the 128 / BITS features of the chunks it holds and writes them into the operand tile itself.
// Which chunk of which of the instruction's rows a lane fetches.  Any assignment covers the same 512 contiguous
// bytes per load instruction; this one is chosen for the 16-byte shared-memory stores of the dequantised values,
// which the hardware serves a quarter-warp (8 lanes) at a time: the 8 lanes of a quarter must hit 8 different
// 16-byte columns of the swizzled operand tile, i.e. (column ^ row) & 7 all different.
//   8-bit: a quarter takes 4 chunks (one 64-feature panel) of 2 rows;  4-bit: 2 chunks of 4 rows;
//   2-bit: 1 chunk of 8 rows;  1-bit: the single chunk of 8 rows.
template <int BITS>
__device__ __forceinline__ void dec_lane_map(int lane, int &chunk, int &rsub) {
  const int q = lane >> 3, i = lane & 7;
  if constexpr (BITS == 8) { chunk = (q & 1) * 4 + (i & 3); rsub = (q >> 1) * 2 + (i >> 2); }
  else if constexpr (BITS == 4) { chunk = (q >> 1) * 2 + (i >> 2); rsub = (q & 1) * 4 + (i & 3); }
  else if constexpr (BITS == 2) { chunk = q & 1; rsub = (q >> 1) * 8 + i; }
  else { chunk = 0; rsub = lane; }
}

template <int BITS>
struct DecCodes {
  static constexpr bool kCoop = BITS == 8 || BITS == 4 || BITS == 2 || BITS == 1;
  uint32_t words[BITS > 0 ? 4 * BITS : 1];     // coop: chunk of iteration `it` at words[4 it ..]; else the thread's row
  alignas(8) __half sc[8];                     // coop: the scales those chunks need; else sc[0..3] = the row's scales
};

// Read-only global loads that stay where they are written: the codes of the NEXT tile are requested a whole tile
// ahead of their use, and a plain load may be moved by the compiler down to its first use (it did, where registers
// were short: the unpack then waited a full memory round trip per tile).  A volatile asm keeps its place among the
// other volatile statements (barrier arrivals and waits).
__device__ __forceinline__ uint4 dec_ldg_v4(const void *p) {
  uint4 v;
  asm volatile("ld.global.nc.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ uint2 dec_ldg_v2(const void *p) {
  uint2 v;
  asm volatile("ld.global.nc.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
  return v;
}
__device__ __forceinline__ uint32_t dec_ldg_u32(const void *p) {
  uint32_t v;
  asm volatile("ld.global.nc.u32 %0, [%1];" : "=r"(v) : "l"(p));
  return v;
}
__device__ __forceinline__ __half dec_ldg_h(const void *p) {
  unsigned short v;
  asm volatile("ld.global.nc.u16 %0, [%1];" : "=h"(v) : "l"(p));
  return __ushort_as_half(v);
}

template <int BITS>
__device__ __forceinline__ void dec_load_codes(const BBCell &c, long long row, DecCodes<BITS> &d) {
  if constexpr (BITS == 0) return;
  else if constexpr (!DecCodes<BITS>::kCoop) {
    const uint4 *wp = (const uint4 *)(c.words + row * (4 * BITS));
#pragma unroll
    for (int i = 0; i < BITS; ++i) { const uint4 v = dec_ldg_v4(wp + i); d.words[4 * i] = v.x; d.words[4 * i + 1] = v.y; d.words[4 * i + 2] = v.z; d.words[4 * i + 3] = v.w; }
    *(uint2 *)d.sc = dec_ldg_v2(c.scales + row * 4);
  } else {
    constexpr int RPI = 32 / BITS;                            // rows per load instruction
    const int lane = threadIdx.x & 31;
    const long long wrow = row - lane;                        // first row of this warp's 32-row slab
    int chunk, rsub;
    dec_lane_map<BITS>(lane, chunk, rsub);
#pragma unroll
    for (int it = 0; it < BITS; ++it) {
      const long long r = wrow + it * RPI + rsub;
      const uint4 v = dec_ldg_v4((const uint4 *)(c.words + r * (4 * BITS)) + chunk);
      d.words[4 * it] = v.x; d.words[4 * it + 1] = v.y; d.words[4 * it + 2] = v.z; d.words[4 * it + 3] = v.w;
      const __half *sp = c.scales + r * 4;
      if constexpr (BITS == 8) d.sc[it] = dec_ldg_h(sp + (chunk >> 1));
      else if constexpr (BITS == 4) d.sc[it] = dec_ldg_h(sp + chunk);
      else if constexpr (BITS == 2) *(uint32_t *)&d.sc[2 * it] = dec_ldg_u32(sp + 2 * chunk);
      else *(uint2 *)&d.sc[0] = dec_ldg_v2(sp);
    }
  }
}

// codes -> fp16 operand values (pre-scaled), written into the warpgroup's swizzled K-major tile.  (code - 2^(BITS-1)
// + 1/2) dq is formed as in dec_unpack_row_row: byte permute into 2^23 + code, one add, one FMA, rounded once.
template <int BITS>
__device__ __forceinline__ void dec_unpack_row(const DecCodes<BITS> &d, float pre, unsigned char *rbuf, int rit) {
  if constexpr (BITS == 0) return;
  else if constexpr (!DecCodes<BITS>::kCoop) {
    DecCodesRow<BITS> r;
#pragma unroll
    for (int i = 0; i < 4 * BITS; ++i) r.words[i] = d.words[i];
    r.sc = *(const uint2 *)d.sc;
    dec_unpack_row_row<BITS>(r, pre, rbuf, rit);
  } else {
    constexpr int RPI = 32 / BITS, NV = 128 / BITS;           // rows per instruction, values per chunk
    constexpr float c0 = -(8388608.0f + (float)(1 << (BITS - 1)));
    const int lane = rit & 31, wrow0 = rit & ~31;
    int chunk, rsub;
    dec_lane_map<BITS>(lane, chunk, rsub);
#pragma unroll
    for (int it = 0; it < BITS; ++it) {
      const int row = wrow0 + it * RPI + rsub;                // row of the tile this chunk belongs to
      const uint32_t *W = &d.words[4 * it];
      unsigned char *rowp = rbuf + row * 128;
#pragma unroll
      for (int v = 0; v < NV; v += 8) {
        uint4 pk;
        __half2 *hp = (__half2 *)&pk;
#pragma unroll
        for (int e2 = 0; e2 < 4; ++e2) {
          float v2[2];
#pragma unroll
          for (int u = 0; u < 2; ++u) {
            const int j = v + e2 * 2 + u;                     // value index within the chunk (compile-time)
            uint32_t src; int byte, gi;
            if constexpr (BITS == 8) { src = W[j >> 2]; byte = j & 3; gi = it; }
            else if constexpr (BITS == 4) { src = (j & 1) ? ((W[j >> 3] >> 4) & 0x0F0F0F0Fu) : (W[j >> 3] & 0x0F0F0F0Fu); byte = (j & 7) >> 1; gi = it; }
            else if constexpr (BITS == 2) { const int gg = j >> 5, jj = j & 31; src = (W[2 * gg + (jj >> 4)] >> (2 * (jj & 3))) & 0x03030303u; byte = (jj & 15) >> 2; gi = 2 * it + gg; }
            else { const int gg = j >> 5, jj = j & 31; src = (W[gg] >> (jj & 7)) & 0x01010101u; byte = jj >> 3; gi = gg; }
            const float dq = __half2float(d.sc[gi]) * pre;
            v2[u] = fmaf(__uint_as_float(__byte_perm(src, 0x4B000000u, 0x7650u + (uint32_t)byte)) + c0, dq, 0.5f * dq);
          }
          hp[e2] = __floats2half2_rn(v2[0], v2[1]);
        }
        const int oc = chunk * (NV / 8) + (v >> 3);           // 16-byte chunk of the 256-byte operand row
        *(uint4 *)(rowp + (oc >> 3) * 16384 + (((oc & 7) ^ (row & 7)) << 4)) = pk;
      }
    }
  }
}

__device__ __forceinline__ void tma_store_4d(const void *tmap, uint32_t src, int c0, int c1, int c2, int c3) {
  asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
               ::"l"(tmap), "r"(src), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// B operand of the inverse rotation: Hs[f][f'] = s_f * (-1)^popcount(f & f'), fp16, K-major, swizzled; built by the
// 256 epilogue threads (et = thread index among them), then announced on bHready.  Thread et owns 16-byte chunk
// et & 15 (features f' = 8 chunk .. 8 chunk + 7) of rows f = (et >> 4) + 16 k: popcount(f & f') splits into the part
// from f's low three bits, the same for all of the thread's rows (f & 7 is), and popcount(f & 8 chunk), one sign per row.
__device__ __forceinline__ void dec_build_rotation(unsigned char *smH, uint64_t seed, int cell, int et, uint32_t bHready) {
  uint32_t sw[4];
  cell_sign_words(seed, cell, sw);
  const int chunk = et & 15, f0 = et >> 4;
  uint32_t basew[4];
#pragma unroll
  for (int e2 = 0; e2 < 4; ++e2) {
    const uint32_t n0 = __popc(f0 & 7 & (2 * e2)) & 1u, n1 = __popc(f0 & 7 & (2 * e2 + 1)) & 1u;
    basew[e2] = (0x3C00u | (n0 << 15)) | ((0x3C00u | (n1 << 15)) << 16);      // +-1.0 in fp16
  }
  unsigned char *colp = smH + (chunk >> 3) * 16384;
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const int f = f0 + 16 * k;
    const uint32_t flip = ((__popc(f & (chunk << 3)) & 1u) ^ ((sw[f >> 5] >> (f & 31)) & 1u)) * 0x80008000u;
    *(uint4 *)(colp + f * 128 + (((chunk & 7) ^ (f & 7)) << 4)) = make_uint4(basew[0] ^ flip, basew[1] ^ flip, basew[2] ^ flip, basew[3] ^ flip);
  }
  fence_proxy_async();
  mbar_arrive(bHready);
}

struct DecCtx {
  uint32_t bTfull, bTempty, bRready, bHready, t_acc, s_obuf;
  unsigned char *rbuf, *obuf, *smH;
  const BBCell *cg;       // the descriptor in global memory: tensor maps are addressed there
  volatile int *abort_flag;
  int wg, nwg, rit, h, tile0, n_tiles, l, hd;
  int ex;                 // core exponent: loaded at kernel start, first USED after the rotation operand is built
  uint64_t seed;
};
// output scale 2^e and the residual operand's pre-scale (the operand is kept in the accumulator's units)
struct DecScales { float scale, pre; };
__device__ __forceinline__ DecScales dec_scales(int ex) { return {ldexpf(1.0f, ex), ldexpf(kInvSqrtD, -ex)}; }

// The per-tile loop of one epilogue warpgroup (tiles wg, wg+2, ...) with one accumulator per warpgroup (r_t > 128).
template <int BITS>
__device__ __forceinline__ bool dec_tile_loop(const BBCell &c, const DecCtx &x) {
  DecCodes<BITS> cur, nxt;
  bool ok = true;
  const bool tma_out = c.tma_out != 0;
  if (x.wg < x.n_tiles) dec_load_codes<BITS>(c, (long long)x.h * c.T + (x.tile0 + x.wg) * 128 + x.rit, cur);
  dec_build_rotation(x.smH, x.seed, c.cell, x.wg * 128 + x.rit, x.bHready);     // the first codes are in flight meanwhile
  const DecScales sc = dec_scales(x.ex);
  JOLT_DBG(const bool stamp = c.dbg && blockIdx.x == 0 && blockIdx.y == gridDim.y / 2 && x.rit == 0;)
  for (int i = x.wg; i < x.n_tiles; i += x.nwg) {
    const int tt = x.tile0 + i, nb = i / x.nwg;
    const int token = tt * 128 + x.rit;
    JOLT_DBG(long long *dbg = stamp ? c.dbg + (size_t)i * 8 : nullptr;)
    JOLT_DBG(if (dbg) dbg[0] = clock64();)
    if (tma_out) {   // the operand tile doubles as staging buffer: the previous store must have read it first
      if (x.rit == 0) tma_store_wait_read();
      named_bar_sync(1 + x.wg, 128);
    }
    JOLT_DBG(if (dbg) dbg[1] = clock64();)
    if constexpr (BITS > 0) {
      if (ok) dec_unpack_row<BITS>(cur, sc.pre, x.rbuf, x.rit);
      fence_proxy_async();
      mbar_arrive(x.bRready);
      JOLT_DBG(if (dbg) dbg[2] = clock64();)
      if (i + x.nwg < x.n_tiles) dec_load_codes<BITS>(c, (long long)x.h * c.T + (tt + x.nwg) * 128 + x.rit, nxt);   // in flight during the MMA
    }
    // after a timed-out wait the warp keeps walking the loop (so the warpgroup's named barriers stay in
    // lockstep) but touches neither TMEM nor the barriers' data again
    if (ok) ok = __all_sync(0xffffffffu, mbar_wait(x.bTfull, nb & 1, x.abort_flag));
    JOLT_DBG(if (dbg) dbg[3] = clock64();)
    tc_fence_after();
    const long long off = (long long)x.l * c.osl + (long long)x.hd * c.osh + (long long)token * c.ost;
    float va[2][32];
    if (ok) tmem_ld32(x.t_acc, va[0]);
#pragma unroll
    for (int ch = 0; ch < 4; ++ch) {
      if (!ok) break;
      tmem_wait_ld();
      if (ch + 1 < 4) tmem_ld32(x.t_acc + (ch + 1) * 32, va[(ch + 1) & 1]);     // next chunk in flight during the conversion
      else { tc_fence_before(); mbar_arrive(x.bTempty); JOLT_DBG(if (dbg) dbg[4] = clock64();) }
      const float *v = va[ch & 1];
      if (c.out_dtype == DT_F16) {
        uint4 o[4];
#pragma unroll
        for (int k8 = 0; k8 < 4; ++k8) {
          __half2 *hp = (__half2 *)&o[k8];
#pragma unroll
          for (int j = 0; j < 4; ++j) hp[j] = __floats2half2_rn(v[k8 * 8 + 2 * j] * sc.scale, v[k8 * 8 + 2 * j + 1] * sc.scale);
        }
        if (tma_out) {      // stage the row, same swizzled layout as a loaded X tile
          unsigned char *rowp = x.obuf + (ch >> 1) * 16384 + x.rit * 128;
#pragma unroll
          for (int k8 = 0; k8 < 4; ++k8) *(uint4 *)(rowp + ((((ch & 1) * 4 + k8) ^ (x.rit & 7)) << 4)) = o[k8];
        } else {
          uint4 *p = (uint4 *)((__half *)c.out + off + ch * 32);
#pragma unroll
          for (int k8 = 0; k8 < 4; ++k8) p[k8] = o[k8];
        }
      } else {
        float4 *p = (float4 *)((float *)c.out + off + ch * 32);
#pragma unroll
        for (int k4 = 0; k4 < 8; ++k4)
          p[k4] = make_float4(v[4 * k4] * sc.scale, v[4 * k4 + 1] * sc.scale, v[4 * k4 + 2] * sc.scale, v[4 * k4 + 3] * sc.scale);
      }
    }
    JOLT_DBG(if (dbg) dbg[5] = clock64();)
    if (tma_out) {
      fence_proxy_async();
      named_bar_sync(1 + x.wg, 128);
      JOLT_DBG(if (dbg) dbg[6] = clock64();)
      if (x.rit == 0 && ok) {
        tma_store_4d(&x.cg->tmOut, x.s_obuf, 0, tt * 128, x.hd, x.l);
        tma_store_4d(&x.cg->tmOut, x.s_obuf + 16384, 64, tt * 128, x.hd, x.l);
        tma_store_commit();
      }
    }
    JOLT_DBG(if (dbg) dbg[7] = clock64();)
    if constexpr (BITS > 0) cur = nxt;
  }
  if (tma_out && x.rit == 0) tma_store_wait_all();
  return ok;
}

// Per-tile loop of one of TWO epilogue warpgroups with two accumulators each (tiles wg, wg+2, ...; local index n,
// accumulator n & 1; barriers and TMEM columns of accumulator 1 sit 16 bytes / 256 columns after accumulator 0).
//   unpack the tile's codes into the warpgroup's operand tile, wait for the tile's MMAs, read the accumulator,
//   convert; the fp16 rows go through the warp's OWN 32 rows of the operand tile (which the MMA has just consumed)
//   and leave as fully coalesced 16-byte stores, two 256-byte rows per warp instruction.  A warp only ever touches
//   its own rows outside the MMA, so the loop needs no barrier between warps and no asynchronous store to wait for.
template <int BITS>
__device__ __forceinline__ bool dec_tile_loop_acc4(const BBCell &c, const DecCtx &x) {
  DecCodes<BITS> cur;
  bool ok = true;
  const long long row0 = (long long)x.h * c.T + x.tile0 * 128 + x.rit;
  if (x.wg < x.n_tiles) dec_load_codes<BITS>(c, row0 + x.wg * 128, cur);
  dec_build_rotation(x.smH, x.seed, c.cell, x.wg * 128 + x.rit, x.bHready);     // the first codes are in flight meanwhile
  const DecScales sc = dec_scales(x.ex);
  const int lane = x.rit & 31, wrow0 = x.rit & ~31;       // this warp's rows of the tile: wrow0 .. wrow0 + 31
  unsigned char *obuf = x.rbuf;
  const bool tma_out = c.tma_out != 0 && c.out_dtype == DT_F16;
  const uint32_t s_wrows = x.s_obuf + (uint32_t)wrow0 * 128u;      // this warp's 32 staging rows (first 64 features)
  int n = 0;
  JOLT_DBG(const bool stamp = c.dbg && blockIdx.x == 0 && blockIdx.y == gridDim.y / 2 && x.rit == 0;)
  for (int i = x.wg; i < x.n_tiles; i += 2, ++n) {
    const int acc = n & 1, ph = n >> 1;
    const int tt = x.tile0 + i, token = tt * 128 + x.rit;
    JOLT_DBG(long long *dbg = stamp ? c.dbg + (size_t)i * 8 : nullptr;)
    JOLT_DBG(if (dbg) dbg[0] = clock64();)
    if (tma_out && n > 0) {      // the previous tile's store must have read this warp's staging rows
      if (lane == 0) tma_store_wait_read();
      __syncwarp();
    }
    JOLT_DBG(if (dbg) dbg[1] = clock64();)
    if constexpr (BITS > 0) {
      if (ok) dec_unpack_row<BITS>(cur, sc.pre, obuf, x.rit);
      fence_proxy_async();
      mbar_arrive(x.bRready + 16 * acc);
      if (i + 2 < x.n_tiles) dec_load_codes<BITS>(c, row0 + (i + 2) * 128, cur);      // in flight during the MMA and the epilogue
    }
    JOLT_DBG(if (dbg) dbg[2] = clock64();)
    // after a timed-out wait the warp keeps walking the loop but touches neither TMEM nor the barriers' data again
    if (ok) ok = __all_sync(0xffffffffu, mbar_wait(x.bTfull + 16 * acc, ph & 1, x.abort_flag));
    JOLT_DBG(if (dbg) dbg[3] = clock64();)
    tc_fence_after();
    const long long off = (long long)x.l * c.osl + (long long)x.hd * c.osh + (long long)token * c.ost;
    const uint32_t t_acc = x.t_acc + acc * 256;
    // the whole accumulator row in one go: four loads in flight, one wait
    float va[4][32];
    if (ok) {
#pragma unroll
      for (int ch = 0; ch < 4; ++ch) tmem_ld32(t_acc + ch * 32, va[ch]);
      tmem_wait_ld();
      tc_fence_before();
      mbar_arrive(x.bTempty + 16 * acc);
    }
    JOLT_DBG(if (dbg) dbg[4] = clock64();)
    if (ok) {
      if (c.out_dtype == DT_F16) {
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) {
          const float *v = va[ch];
          unsigned char *rowp = obuf + (ch >> 1) * 16384 + x.rit * 128;
#pragma unroll
          for (int k8 = 0; k8 < 4; ++k8) {
            uint4 o;
            __half2 *hp = (__half2 *)&o;
#pragma unroll
            for (int j = 0; j < 4; ++j) hp[j] = __floats2half2_rn(v[k8 * 8 + 2 * j] * sc.scale, v[k8 * 8 + 2 * j + 1] * sc.scale);
            *(uint4 *)(rowp + ((((ch & 1) * 4 + k8) ^ (x.rit & 7)) << 4)) = o;
          }
        }
        if (tma_out) {
          // the warp's 32 staged rows leave as two bulk tensor stores (64 features each) issued by one lane: no thread
          // waits for the global writes, only (before the rows are overwritten) for the copy engine to have read them
          fence_proxy_async();
          __syncwarp();
          JOLT_DBG(if (dbg) dbg[5] = clock64();)
          if (lane == 0) {
            tma_store_4d(&x.cg->tmOutW, s_wrows, 0, tt * 128 + wrow0, x.hd, x.l);
            tma_store_4d(&x.cg->tmOutW, s_wrows + 16384, 64, tt * 128 + wrow0, x.hd, x.l);
            tma_store_commit();
          }
        } else {
          __syncwarp();
          JOLT_DBG(if (dbg) dbg[5] = clock64();)
          // read back: lane l takes 16-byte chunk l & 15 of rows 2 it + (l >> 4); a row is 256 contiguous bytes of output
          const int q16 = lane & 15;
          __half *obase = (__half *)c.out + (long long)x.l * c.osl + (long long)x.hd * c.osh;
#pragma unroll 4
          for (int it = 0; it < 16; ++it) {
            const int r = wrow0 + 2 * it + (lane >> 4);
            const uint4 o = *(const uint4 *)(obuf + (q16 >> 3) * 16384 + r * 128 + (((q16 & 7) ^ (r & 7)) << 4));
            *(uint4 *)(obase + (long long)(tt * 128 + r) * c.ost + q16 * 8) = o;
          }
          __syncwarp();
        }
      } else {
        float4 *p = (float4 *)((float *)c.out + off);
#pragma unroll
        for (int ch = 0; ch < 4; ++ch)
#pragma unroll
          for (int k4 = 0; k4 < 8; ++k4)
            p[ch * 8 + k4] = make_float4(va[ch][4 * k4] * sc.scale, va[ch][4 * k4 + 1] * sc.scale, va[ch][4 * k4 + 2] * sc.scale,
                                         va[ch][4 * k4 + 3] * sc.scale);
      }
    }
    JOLT_DBG(if (dbg) dbg[7] = clock64();)
  }
  if (tma_out && lane == 0) tma_store_wait_all();
  return ok;
}

// The loop above for key cells of a decode that re-applies the rotary embedding: feature j pairs with j + 64 and the pair turns by
//   the angle whose (cos, sin) sit in c.rope[j * T + token] (32 consecutive tokens per warp instruction, 256 contiguous
//   bytes, L2-resident across heads).  The accumulator row is then read in two halves, features {0..31, 64..95} and
//   {32..63, 96..127}; the table entries of the first half are requested BEFORE the wait for the tile's MMAs and those of
//   the second half while the first is converted and staged, so no table latency is exposed.
template <int BITS>
__device__ __forceinline__ bool dec_tile_loop_acc4_rope(const BBCell &c, const DecCtx &x) {
  DecCodes<BITS> cur;
  bool ok = true;
  const long long row0 = (long long)x.h * c.T + x.tile0 * 128 + x.rit;
  if (x.wg < x.n_tiles) dec_load_codes<BITS>(c, row0 + x.wg * 128, cur);
  dec_build_rotation(x.smH, x.seed, c.cell, x.wg * 128 + x.rit, x.bHready);     // the first codes are in flight meanwhile
  const DecScales sc = dec_scales(x.ex);
  const int lane = x.rit & 31, wrow0 = x.rit & ~31;       // this warp's rows of the tile: wrow0 .. wrow0 + 31
  unsigned char *obuf = x.rbuf;
  const bool tma_out = c.tma_out != 0 && c.out_dtype == DT_F16;
  const uint32_t s_wrows = x.s_obuf + (uint32_t)wrow0 * 128u;      // this warp's 32 staging rows (first 64 features)
  int n = 0;
  JOLT_DBG(const bool stamp = c.dbg && blockIdx.x == 0 && blockIdx.y == gridDim.y / 2 && x.rit == 0;)
  for (int i = x.wg; i < x.n_tiles; i += 2, ++n) {
    const int acc = n & 1, ph = n >> 1;
    const int tt = x.tile0 + i, token = tt * 128 + x.rit;
    JOLT_DBG(long long *dbg = stamp ? c.dbg + (size_t)i * 8 : nullptr;)
    JOLT_DBG(if (dbg) dbg[0] = clock64();)
    if (tma_out && n > 0) {      // the previous tile's store must have read this warp's staging rows
      if (lane == 0) tma_store_wait_read();
      __syncwarp();
    }
    JOLT_DBG(if (dbg) dbg[1] = clock64();)
    if constexpr (BITS > 0) {
      if (ok) dec_unpack_row<BITS>(cur, sc.pre, obuf, x.rit);
      fence_proxy_async();
      mbar_arrive(x.bRready + 16 * acc);
      if (i + 2 < x.n_tiles) dec_load_codes<BITS>(c, row0 + (i + 2) * 128, cur);      // in flight during the MMA and the epilogue
    }
    JOLT_DBG(if (dbg) dbg[2] = clock64();)
    float2 tb[32];
    const float2 *tp = nullptr;
    {
      tp = c.rope + token;
#pragma unroll
      for (int k = 0; k < 32; ++k) tb[k] = __ldg(tp + (size_t)k * c.T);
    }
    // after a timed-out wait the warp keeps walking the loop but touches neither TMEM nor the barriers' data again
    if (ok) ok = __all_sync(0xffffffffu, mbar_wait(x.bTfull + 16 * acc, ph & 1, x.abort_flag));
    JOLT_DBG(if (dbg) dbg[3] = clock64();)
    tc_fence_after();
    const long long off = (long long)x.l * c.osl + (long long)x.hd * c.osh + (long long)token * c.ost;
    const uint32_t t_acc = x.t_acc + acc * 256;
    // one 32-feature chunk of the row: scaled, rounded and put into the warp's staging rows (fp16) or stored (fp32)
    auto emit = [&](const float *v, int ch) {
      if (c.out_dtype == DT_F16) {
        unsigned char *rowp = obuf + (ch >> 1) * 16384 + x.rit * 128;
#pragma unroll
        for (int k8 = 0; k8 < 4; ++k8) {
          uint4 o;
          __half2 *hp = (__half2 *)&o;
#pragma unroll
          for (int j = 0; j < 4; ++j) hp[j] = __floats2half2_rn(v[k8 * 8 + 2 * j] * sc.scale, v[k8 * 8 + 2 * j + 1] * sc.scale);
          *(uint4 *)(rowp + ((((ch & 1) * 4 + k8) ^ (x.rit & 7)) << 4)) = o;
        }
      } else {
        float4 *p = (float4 *)((float *)c.out + off);
#pragma unroll
        for (int k4 = 0; k4 < 8; ++k4)
          p[ch * 8 + k4] = make_float4(v[4 * k4] * sc.scale, v[4 * k4 + 1] * sc.scale, v[4 * k4 + 2] * sc.scale, v[4 * k4 + 3] * sc.scale);
      }
    };
    {
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        float lo[32], hi[32];
        if (ok) {
          tmem_ld32(t_acc + half * 32, lo);
          tmem_ld32(t_acc + 64 + half * 32, hi);
          tmem_wait_ld();
          if (half == 1) { tc_fence_before(); mbar_arrive(x.bTempty + 16 * acc); }
#pragma unroll
          for (int k = 0; k < 32; ++k) {
            const float a = lo[k], b = hi[k];
            lo[k] = __fmaf_rn(a, tb[k].x, -__fmul_rn(b, tb[k].y));
            hi[k] = __fmaf_rn(b, tb[k].x, __fmul_rn(a, tb[k].y));
          }
        }
        if (half == 0) {
#pragma unroll
          for (int k = 0; k < 32; ++k) tb[k] = __ldg(tp + (size_t)(32 + k) * c.T);
        }
        if (ok) { emit(lo, half); emit(hi, 2 + half); }
      }
      JOLT_DBG(if (dbg) dbg[4] = clock64();)
    }
    if (ok && tma_out) {
      fence_proxy_async();
      __syncwarp();
      JOLT_DBG(if (dbg) dbg[5] = clock64();)
      if (lane == 0) {
        tma_store_4d(&x.cg->tmOutW, s_wrows, 0, tt * 128 + wrow0, x.hd, x.l);
        tma_store_4d(&x.cg->tmOutW, s_wrows + 16384, 64, tt * 128 + wrow0, x.hd, x.l);
        tma_store_commit();
      }
    } else if (ok && c.out_dtype == DT_F16) {
      __syncwarp();
      JOLT_DBG(if (dbg) dbg[5] = clock64();)
      // read back: lane l takes 16-byte chunk l & 15 of rows 2 it + (l >> 4); a row is 256 contiguous bytes of output
      const int q16 = lane & 15;
      __half *obase = (__half *)c.out + (long long)x.l * c.osl + (long long)x.hd * c.osh;
#pragma unroll 4
      for (int it = 0; it < 16; ++it) {
        const int r = wrow0 + 2 * it + (lane >> 4);
        const uint4 o = *(const uint4 *)(obuf + (q16 >> 3) * 16384 + r * 128 + (((q16 & 7) ^ (r & 7)) << 4));
        *(uint4 *)(obase + (long long)(tt * 128 + r) * c.ost + q16 * 8) = o;
      }
      __syncwarp();
    }
    JOLT_DBG(if (dbg) dbg[7] = clock64();)
  }
  if (tma_out && lane == 0) tma_store_wait_all();
  return ok;
}

__global__ void __launch_bounds__(DecLayout::THREADS, 1) decode_kernel(const BBCell *__restrict__ cells, uint64_t seed) {
  using LY = DecLayout;
  constexpr int NWG = DEC_NWG;
  constexpr int DEC_P_BYTES = LY::P_BYTES, DEC_BIG_BYTES = LY::BIG_BYTES, DEC_NS = LY::NS;
  extern __shared__ unsigned char smem_raw[];
  // The cell's descriptor is read from global memory ONCE, cooperatively, into shared memory: the scalar fields are
  // used all over the kernel and each first touch from global would be a dependent L2 round trip on the critical
  // path of the CTA's start.  Only the tensor maps are addressed in global memory (the copy engine requires that).
  const BBCell &cg = cells[blockIdx.y];
  const int items_per_head = cg.items_per_head, tiles_per_item = cg.tiles_per_item, n_tok_tiles = cg.T / 128;
  if ((int)blockIdx.x >= cg.m * items_per_head) return;
  const int h = blockIdx.x / items_per_head;
  const int item = blockIdx.x - h * items_per_head;
  const int tile0 = item * tiles_per_item;
  const int n_tiles = min(tiles_per_item, n_tok_tiles - tile0);
  if (n_tiles <= 0) return;

  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char *sm = smem_raw + (base - raw);
  const uint32_t sP = base, sH = base + DEC_P_BYTES, sBig = sH + DEC_H_BYTES;
  const uint32_t sRing = sBig, sR = sBig + DEC_NS * BB_STAGE_BYTES;
  const uint32_t sBar = sBig + DEC_BIG_BYTES;
  unsigned char *smH = sm + DEC_P_BYTES, *smR = sm + DEC_P_BYTES + DEC_H_BYTES + DEC_NS * BB_STAGE_BYTES;
  volatile int *abort_flag = (volatile int *)(sm + DEC_P_BYTES + DEC_H_BYTES + DEC_BIG_BYTES + 256);
  uint32_t *tmem_slot = (uint32_t *)(sm + DEC_P_BYTES + DEC_H_BYTES + DEC_BIG_BYTES + 264);
  const uint32_t bSetup = sBar + 0, bHready = sBar + 16;
  auto bFull = [=](int s) { return sBar + 24 + 8 * s; };          // up to 6 ring stages
  auto bEmpty = [=](int s) { return sBar + 72 + 8 * s; };
  auto bTfull = [=](int b) { return sBar + 120 + 8 * b; };        // up to 4 accumulators
  auto bTempty = [=](int b) { return sBar + 152 + 8 * b; };
  auto bRready = [=](int b) { return sBar + 184 + 8 * b; };
  auto bBB = [=](int b) { return sBar + 216 + 8 * b; };           // backbone of the accumulator's tile complete

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int wg = warp >> 2;
  JOLT_DBG(long long *kdbg = (cg.dbg && blockIdx.x == 0 && blockIdx.y == gridDim.y / 2 && threadIdx.x == 0) ? cg.dbg + 16 * 8 : nullptr;)
  JOLT_DBG(if (kdbg) { kdbg[0] = clock64(); long long gt; asm volatile("mov.u64 %0, %globaltimer;" : "=l"(gt)); kdbg[6] = gt; })
  BBCell *sc_cell = (BBCell *)(sm + DEC_P_BYTES + DEC_H_BYTES + DEC_BIG_BYTES + 512);
  for (int i = threadIdx.x; i < (int)(sizeof(BBCell) / 16); i += LY::THREADS) ((uint4 *)sc_cell)[i] = __ldg((const uint4 *)&cg + i);

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    mbar_init(bSetup, 1); mbar_init(bHready, NWG * 128);
    for (int s = 0; s < 6; ++s) { mbar_init(bFull(s), 1); mbar_init(bEmpty(s), 1); }
    for (int b = 0; b < 4; ++b) { mbar_init(bTfull(b), 1); mbar_init(bTempty(b), 128); mbar_init(bRready(b), 128); mbar_init(bBB(b), 1); }
    fence_barrier_init();
  }
  if (warp == NWG * 4) { tmem_alloc(smem_u32(tmem_slot), LY::TMEM_COLS); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  JOLT_DBG(if (kdbg) kdbg[1] = clock64();)
  const BBCell &c = *sc_cell;            // scalar fields from here on; tensor maps through cg
  const int nkt = (c.r_t + 63) / 64;
  const uint32_t panel = (uint32_t)c.r_t * 128u;       // bytes of one 64-feature panel of P (r_t is a multiple of 16)
  const bool has_res = c.bits > 0;
  // r_t <= 128 leaves half of the P region free: it extends the ring to six stages, and each warpgroup owns two
  // accumulators (see the top of the file)
  const bool acc4 = nkt <= 2;
  const int ns = acc4 ? 6 : DEC_NS;
  auto sStage = [=](int s) { return s < 4 ? sRing + (uint32_t)s * BB_STAGE_BYTES : sP + 32768u + (uint32_t)(s - 4) * BB_STAGE_BYTES; };

  if (wg == NWG) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(LY::PROD_REGS));
    if (warp == NWG * 4 && lane == 0) {
      // ---------------- TMA producer
      mbar_expect_tx(bSetup, 2u * panel);
      tma_load_2d(sP, &cg.tmP, bSetup, 0, h * c.r_t);
      tma_load_2d(sP + panel, &cg.tmP, bSetup, 64, h * c.r_t);
      bool ok = true;
      int cnt = 0;
      for (int i = 0; ok && i < n_tiles; ++i) {
        const int tt = tile0 + i;
        for (int kb = 0; kb < nkt; ++kb, ++cnt) {
          const int s = cnt % ns, n = cnt / ns;
          ok = mbar_wait(bEmpty(s), (n & 1) ^ 1, abort_flag);
          if (!ok) break;
          mbar_expect_tx(bFull(s), BB_STAGE_BYTES);
          tma_load_2d(sStage(s), &cg.tmUT, bFull(s), kb * 64, tt * 128);
        }
      }
    } else if (warp == NWG * 4 + 1 && lane == 0) {
      // ---------------- backbone MMA issuer.  Issuing an MMA costs its thread tens of cycles of dependent
      // instructions, and a tile needs sixteen of them: the two halves of a tile's accumulation (backbone, rotation)
      // are issued by two threads on different schedulers, ordered per accumulator through bBB.  The backbone thread
      // runs ahead as far as free accumulators and landed U_T stages allow (two accumulators per warpgroup when
      // r_t <= 128), so backbones wait in TMEM instead of U_T tiles in shared memory, and a late U_T stage never
      // holds back a rotation whose operands are complete.
      bool ok = mbar_wait(bSetup, 0, abort_flag);        // the head's projected core has landed
      if (ok) {
        tc_fence_after();
        const uint32_t idescB = umma_idesc_f16(128, 128, 0, 1);     // A = U_T tile, K-major; B = P panels, MN-major
        const int ksteps = c.r_t / 16;
        // P: 16 contraction rows = 2048 B per step, the second 64 features one panel further
        const uint64_t dP0 = umma_desc_sw128(sP, panel, 1024);
        const uint64_t dS0 = umma_desc_sw128(sRing, 16, 1024), dS4 = umma_desc_sw128(sP + 32768, 16, 1024);
        constexpr uint64_t kStep16K = 16384 >> 4;      // address-field step
        int cnt = 0;
        for (int j = 0; ok && j < n_tiles; ++j) {
          // accumulator / barrier index b of tile j and how often it was used before (nb)
          const int wgi = j % NWG, ni = j / NWG;
          const int b = acc4 ? wgi + 2 * (ni & 1) : wgi, nb = acc4 ? ni >> 1 : ni;
          ok = mbar_wait(bTempty(b), (nb & 1) ^ 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
          const uint32_t tacc = tmem_base + b * 128;
          for (int kb = 0; kb < nkt; ++kb, ++cnt) {
            const int s = cnt % ns, n = cnt / ns;
            ok = mbar_wait(bFull(s), n & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            const uint64_t da = s < 4 ? dS0 + (uint64_t)s * kStep16K : dS4 + (uint64_t)(s - 4) * kStep16K;
            const uint64_t db = dP0 + (uint64_t)kb * (8192 >> 4);
#pragma unroll
            for (int k4 = 0; k4 < 4; ++k4)
              if (kb * 4 + k4 < ksteps) umma_f16(tacc, umma_desc_kslice(da, k4), db + (uint64_t)k4 * (2048 >> 4), idescB, (kb | k4) != 0);
            umma_commit(bEmpty(s));
          }
          if (ok) umma_commit(bBB(b));
        }
      }
    } else if (warp == NWG * 4 + 2 && lane == 0) {
      // ---------------- rotation MMA issuer: A = the warpgroup's dequantised residual tile, B = H
      bool ok = mbar_wait(bHready, 0, abort_flag);    // the rotation operand is built
      if (ok) {
        tc_fence_after();
        const uint32_t idesc = umma_idesc_f16(128, 128, 0, 0);      // both operands K-major
        const uint64_t dH0 = umma_desc_sw128(sH, 16, 1024), dR0 = umma_desc_sw128(sR, 16, 1024);
        constexpr uint64_t kStep16K = 16384 >> 4, kStep32K = 32768 >> 4;      // address-field steps
        uint64_t dH[8];
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) dH[ks] = umma_desc_kslice(dH0 + (uint64_t)(ks >> 2) * kStep16K, ks & 3);
        for (int j = 0; ok && j < n_tiles; ++j) {
          const int wgi = j % NWG, ni = j / NWG;
          const int b = acc4 ? wgi + 2 * (ni & 1) : wgi, nb = acc4 ? ni >> 1 : ni;
          ok = mbar_wait(bBB(b), nb & 1, abort_flag);                 // the tile's backbone is in the accumulator
          if (ok && has_res) ok = mbar_wait(bRready(b), nb & 1, abort_flag);
          if (!ok) break;
          if (has_res) {
            tc_fence_after();
            const uint32_t tacc = tmem_base + b * 128;
            const uint64_t dR = dR0 + (uint64_t)wgi * kStep32K;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks)
              umma_f16(tacc, umma_desc_kslice(dR + (uint64_t)(ks >> 2) * kStep16K, ks & 3), dH[ks], idesc, 1);
          }
          umma_commit(bTfull(b));
        }
      }
    }
  } else {
    // ---------------- epilogue warpgroups
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(LY::EPI_REGS));
    JOLT_DBG(if (kdbg) kdbg[2] = clock64();)
    const int q = warp & 3;
    const int rit = q * 32 + lane;                 // row in tile
    const uint32_t t_lane = tmem_base + ((uint32_t)(q * 32) << 16);
    {
      DecCtx x;
      x.cg = &cg;
      x.ex = *c.e;             // requested now, first used after the rotation operand is built
      x.bTfull = bTfull(wg); x.bTempty = bTempty(wg); x.bRready = bRready(wg); x.bHready = bHready;
      x.t_acc = t_lane + wg * 128; x.rbuf = smR + wg * 32768; x.smH = smH; x.seed = seed;
      x.s_obuf = sR + wg * 32768; x.obuf = x.rbuf;
      x.abort_flag = abort_flag; x.wg = wg; x.nwg = NWG; x.rit = rit; x.h = h; x.tile0 = tile0; x.n_tiles = n_tiles;
      x.l = h / c.n_heads; x.hd = h - x.l * c.n_heads;
      if (acc4 && c.rope) {
        switch (c.bits) {
          case 0: dec_tile_loop_acc4_rope<0>(c, x); break;
          case 1: dec_tile_loop_acc4_rope<1>(c, x); break;
          case 2: dec_tile_loop_acc4_rope<2>(c, x); break;
          case 3: dec_tile_loop_acc4_rope<3>(c, x); break;
          case 4: dec_tile_loop_acc4_rope<4>(c, x); break;
          default: dec_tile_loop_acc4_rope<8>(c, x); break;
        }
      } else if (acc4) {
        switch (c.bits) {
          case 0: dec_tile_loop_acc4<0>(c, x); break;
          case 1: dec_tile_loop_acc4<1>(c, x); break;
          case 2: dec_tile_loop_acc4<2>(c, x); break;
          case 3: dec_tile_loop_acc4<3>(c, x); break;
          case 4: dec_tile_loop_acc4<4>(c, x); break;
          default: dec_tile_loop_acc4<8>(c, x); break;
        }
      } else {
        switch (c.bits) {
          case 0: dec_tile_loop<0>(c, x); break;
          case 1: dec_tile_loop<1>(c, x); break;
          case 2: dec_tile_loop<2>(c, x); break;
          case 3: dec_tile_loop<3>(c, x); break;
          case 4: dec_tile_loop<4>(c, x); break;
          default: dec_tile_loop<8>(c, x); break;
        }
      }
    }
  }
  JOLT_DBG(if (kdbg) kdbg[4] = clock64();)
  tc_fence_before();
  __syncthreads();
  JOLT_DBG(if (kdbg) { kdbg[5] = clock64(); long long gt; asm volatile("mov.u64 %0, %globaltimer;" : "=l"(gt)); kdbg[7] = gt; })
  if (*abort_flag) {
    if (threadIdx.x == 0) atomicOr(c.status, 8);
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000) {}
    __syncthreads();
  }
  if (warp == NWG * 4) { tc_fence_after(); tmem_dealloc(tmem_base, LY::TMEM_COLS); }
}

}  // namespace tc
}  // namespace jolt
