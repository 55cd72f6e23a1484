// Persistent form of the fused decompress pass (tc_decode.cuh): one CTA per SM walks a contiguous share of the
// launch's tile list -- (cell, head, 128-token tile) in that order -- instead of one CTA per 16-tile item.
//
// Why: a CTA of the per-item kernel spends the equivalent of five tiles before its first tile is out (descriptor,
// barriers, tensor-memory allocation, the rotation operand, the first codes' trip from HBM, then unpack -> MMA ->
// read), and an item is only sixteen tiles.  Here that is paid once per ~110 tiles: the TMA ring, the two MMA-issuing
// threads and the two epilogue warpgroups run on across head boundaries without draining.  A CTA's work is a sequence
// of runs of consecutive tiles: run 0 is its fixed share; further runs are chunks of a tail that the CTAs take from
// a counter in global memory (the host may leave the tail empty).
//
// The second difference is the order of a warpgroup's work.  In the per-item kernel the dequantised operand tile of a
// warpgroup doubles as the staging area of its output rows, so a warpgroup's cycle is unpack(i) -> rotation MMAs(i)
// -> read and stage(i) -> bulk store reads the rows -> unpack(i + 2): longer than the tensor pipe needs for two
// tiles, and the pipe idles.  Here the output is staged in a region of its own (half a tile per warpgroup, one
// 64-feature box per warp at a time), so the operand tile is free as soon as the rotation MMAs of tile i complete:
// the warpgroup stores the first 64 features of tile i, unpacks tile i + 2 (while that store reads the staging rows),
// then converts and stores the second 64 features of tile i while the rotation of i + 2 runs.
//
// What changes at a boundary:
//   head   the projected core P_h (one 32 KB buffer; the 32 KB next to it is the staging region): a thread of its own
//          requests the next head's block once the backbone thread has released the buffer (a commit barrier) and
//          asks for the block after that to be brought into L2.  The backbone thread runs up to two tiles ahead of the
//          rotation, which absorbs most of the reload; the U_T ring (four stages) is indifferent to heads.
//   cell   bit width, exponent, rotation signs, tensor maps: the epilogue warpgroups meet at a named barrier (all
//          rotation MMAs of the old cell are complete by then: each warpgroup has read its last accumulator), copy
//          the new descriptor, rebuild the rotation operand and re-enter the tile loop compiled for the new bit
//          width.  A CTA's share touches two cells at most once in a while; cells are never interleaved.
// Launches with a cell of r_t > 128 (its P block needs the whole P region), with keys rotated at decode, or with
// mixed sequence lengths take the per-item kernel.
#pragma once
#include "tc_decode.cuh"

namespace jolt {
namespace tc {

struct DecPArgs {
  const BBCell *cells;
  int n_cells;
  int nt;              // 128-token tiles per head (all cells of a launch share T)
  int total;           // tiles of the launch
  uint64_t seed;
  const int2 *run0;    // per CTA: [first, end) of its fixed share
  int pool;            // tiles from here on are handed out in chunks ...
  int chunk;           // ... of this many tiles
  int *counter;        // chunks handed out so far (zero at launch)
};

// linear tile p of the launch -> (cell, head, tile in head); cells[].tile_base is the first linear tile of a cell
struct DecPos { int ci, h, tile; };
__device__ __forceinline__ DecPos dec_locate(const BBCell *cells, int n_cells, int nt, int p, int ci_from = 0) {
  DecPos q;
  q.ci = ci_from;
  while (q.ci + 1 < n_cells && cells[q.ci + 1].tile_base <= p) ++q.ci;
  const int rel = p - cells[q.ci].tile_base;
  q.h = rel / nt;
  q.tile = rel - q.h * nt;
  return q;
}

// accumulator / barrier index of the CTA's j-th tile and how often it was used before: warpgroup j & 1, its
// accumulators alternate
__device__ __forceinline__ void dec_acc_of(int j, int &b, int &nb) {
  const int wgi = j & 1, ni = j >> 1;
  b = wgi + 2 * (ni & 1);
  nb = ni >> 1;
}

struct DecPCtx {
  uint32_t bTfull, bTempty, bRready;      // of accumulator 0 of this warpgroup; accumulator 1 sixteen bytes further
  uint32_t t_acc, s_stg;
  unsigned char *rbuf, *stg;              // the warpgroup's operand tile; the warp's 32 staging rows (128 bytes each)
  const BBCell *cg;                       // the cell's descriptor in global memory (tensor maps)
  volatile int *abort_flag;
  int wg, rit;
  int nt, base;                           // tiles per head; first linear tile of the cell
  int joff;                               // tile p of the current run is the CTA's tile number j = p + joff
  int ex;
};

// brings one box of a tiled tensor into L2 (no shared-memory destination, nothing to wait for)
__device__ __forceinline__ void tma_prefetch_l2_2d(const void *tmap, int c0, int c1) {
  asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];" ::"l"(tmap), "r"(c0), "r"(c1) : "memory");
}

// This warpgroup's tiles p = p0, p0 + 2, ... < p_end of ONE cell.  Per tile: wait for its accumulator (backbone and
// rotation complete, hence the operand tile free), unpack the tile after it into the operand tile and release it to the
// rotation thread, request the codes of the tile after that, then read the accumulator in two halves of 64 features:
// scale, round to fp16, stage the warp's 32 rows and hand them to one bulk tensor store per half.  `pending` says
// whether a bulk store of this warp may still be reading its staging rows.
// returns bit 0: no wait ran out, bit 1: a bulk store of this warp is still pending
template <int BITS, bool TMA_ONLY>
__device__ __forceinline__ int dec_tile_loop_p(const BBCell &c, const DecPCtx &x, int p0, int p_end, bool pending) {
  DecCodes<BITS> cur;
  bool ok = true;
  const DecScales sc = dec_scales(x.ex);
  const int lane = x.rit & 31, wrow0 = x.rit & ~31;
  const bool f16 = TMA_ONLY || c.out_dtype == DT_F16;
  const bool tma_out = TMA_ONLY || (c.tma_out != 0 && f16);
  unsigned char *rowp = x.stg + lane * 128;
  // (head, tile in head) of the tile being finished and of the next tile whose codes are to be requested
  int h = (p0 - x.base) / x.nt, tt = (p0 - x.base) - h * x.nt;
  int hl = h, tl = tt;
  auto advance = [&](int &hh, int &t_) { t_ += 2; while (t_ >= x.nt) { t_ -= x.nt; ++hh; } };
  if (p0 < p_end) {
    // the operand tile is free: this warpgroup has read the accumulator of its last tile of the previous cell
    if constexpr (BITS > 0) {
      dec_load_codes<BITS>(c, (long long)hl * c.T + tl * 128 + x.rit, cur);
      advance(hl, tl);
      dec_unpack_row<BITS>(cur, sc.pre, x.rbuf, x.rit);
      fence_proxy_async();
    }
    // (a cell without residual arrives all the same: the barrier's phases then count tiles, whatever the cells hold)
    mbar_arrive(x.bRready + 16 * (((p0 + x.joff) >> 1) & 1));
    if constexpr (BITS > 0) {
      if (p0 + 2 < p_end) { dec_load_codes<BITS>(c, (long long)hl * c.T + tl * 128 + x.rit, cur); advance(hl, tl); }
    }
  }
  for (int p = p0; p < p_end; p += 2) {
    const int j = p + x.joff, n = j >> 1, acc = n & 1, ph = n >> 1;
    JOLT_DBG(long long *dbg = (c.dbg && blockIdx.x == gridDim.x / 2 && x.rit == 0 && j >= 40 && j < 56) ? c.dbg + (size_t)(j - 40) * 8 : nullptr;)
    JOLT_DBG(if (dbg) dbg[0] = clock64();)
    ok = __all_sync(0xffffffffu, mbar_wait(x.bTfull + 16 * acc, ph & 1, x.abort_flag));
    if (!ok) break;
    tc_fence_after();
    JOLT_DBG(if (dbg) dbg[1] = clock64();)
    const int l = h / c.n_heads, hd = h - l * c.n_heads;
    const uint32_t t_acc = x.t_acc + acc * 256;
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      float va[2][32];
      tmem_ld32(t_acc + half * 64, va[0]);
      tmem_ld32(t_acc + half * 64 + 32, va[1]);
      tmem_wait_ld();
      if (half == 1) { tc_fence_before(); mbar_arrive(x.bTempty + 16 * acc); }
      if (!f16) {
        float4 *pf = (float4 *)((float *)c.out + (long long)l * c.osl + (long long)hd * c.osh + (long long)(tt * 128 + x.rit) * c.ost) + half * 16;
#pragma unroll
        for (int q = 0; q < 2; ++q)
#pragma unroll
          for (int k4 = 0; k4 < 8; ++k4)
            pf[q * 8 + k4] = make_float4(va[q][4 * k4] * sc.scale, va[q][4 * k4 + 1] * sc.scale, va[q][4 * k4 + 2] * sc.scale, va[q][4 * k4 + 3] * sc.scale);
      } else {
      uint4 o[8];
#pragma unroll
      for (int k8 = 0; k8 < 8; ++k8) {
        __half2 *hp = (__half2 *)&o[k8];
#pragma unroll
        for (int q = 0; q < 4; ++q)
          hp[q] = __floats2half2_rn(va[k8 >> 2][(k8 & 3) * 8 + 2 * q] * sc.scale, va[k8 >> 2][(k8 & 3) * 8 + 2 * q + 1] * sc.scale);
      }
      if (pending) {               // the previous bulk store must have read this warp's staging rows
        if (lane == 0) tma_store_wait_read();
        __syncwarp();
        pending = false;
      }
#pragma unroll
      for (int k8 = 0; k8 < 8; ++k8) *(uint4 *)(rowp + ((k8 ^ (lane & 7)) << 4)) = o[k8];
      if (tma_out) {
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) {
          tma_store_4d(&x.cg->tmOutW, x.s_stg, half * 64, tt * 128 + wrow0, hd, l);
          tma_store_commit();
        }
        pending = true;
      } else {
        __syncwarp();
        // read back: lane takes 16-byte chunk lane & 7 of rows 4 it + (lane >> 3); half a row is 128 contiguous bytes
        const int q16 = lane & 7;
        __half *obase = (__half *)c.out + (long long)l * c.osl + (long long)hd * c.osh + half * 64 + q16 * 8;
#pragma unroll 4
        for (int it = 0; it < 8; ++it) {
          const int r = 4 * it + (lane >> 3);
          const uint4 v = *(const uint4 *)(x.stg + r * 128 + ((q16 ^ (r & 7)) << 4));
          *(uint4 *)(obase + (long long)(tt * 128 + wrow0 + r) * c.ost) = v;
        }
        __syncwarp();
      }
      }
      if (half == 0) {
        JOLT_DBG(if (dbg) dbg[2] = clock64();)
        // between the two halves (the first half's bulk store reads the staging rows meanwhile):
        if (p + 2 < p_end) {         // the rotation of tile p is complete: its operand tile takes tile p + 2
          if constexpr (BITS > 0) {
            dec_unpack_row<BITS>(cur, sc.pre, x.rbuf, x.rit);
            fence_proxy_async();
          }
          mbar_arrive(x.bRready + 16 * (acc ^ 1));
          if constexpr (BITS > 0) {
            if (p + 4 < p_end) { dec_load_codes<BITS>(c, (long long)hl * c.T + tl * 128 + x.rit, cur); advance(hl, tl); }
          }
        }
        JOLT_DBG(if (dbg) dbg[3] = clock64();)
      }
    }
    JOLT_DBG(if (dbg) dbg[7] = clock64();)
    advance(h, tt);
  }
  return (ok ? 1 : 0) | (pending ? 2 : 0);
}

// The CTA's work is a sequence of runs of consecutive tiles: run 0 is its fixed share, every later run a chunk taken
// from a counter in global memory (the tail of the list, so that CTAs that fall behind take fewer).  The U_T producer
// thread takes the chunks -- one ahead, so the atomic's trip is hidden behind a run -- and publishes them in a
// shared-memory queue of eight slots {first, end, run number}; the other roles read run k from slot k & 7.  No role
// is more than two runs behind the producer (the ring holds two tiles, an accumulator is reused after four), so a
// slot is never overwritten while somebody still needs it.  A run that starts at `total` ends every role.
struct DecRunQ {
  volatile int *q;
  int total;
  volatile int *abort_flag;
  __device__ __forceinline__ void publish(int k, int first, int end) const {
    volatile int *e = q + (k & 7) * 4;
    e[0] = first; e[1] = end;
    __threadfence_block();
    e[2] = k;
  }
  // run k >= 1 of this CTA; false when a wait ran out
  __device__ __forceinline__ bool get(int k, int &first, int &end) const {
    volatile int *e = q + (k & 7) * 4;
    if (e[2] != k) {
      const long long t0 = clock64(), limit = 2 * g_spin_limit;      // outlasts the producer's own bounded waits
      while (e[2] != k) {
        if (clock64() - t0 > limit) { *abort_flag = 1; return false; }
      }
    }
    first = e[0]; end = e[1];
    return true;
  }
};

// TMA_ONLY: every cell of the launch writes fp16 through bulk tensor stores (the common case gets a tile loop without
// the fp32 and read-back paths)
// BITMASK: bit b set = the tile loop for b-bit cells is compiled in (a launch takes the smallest instantiated superset
// of its cells' bit widths: fewer tile loops, a smaller instruction footprint)
template <bool TMA_ONLY, unsigned BITMASK>
__global__ void __launch_bounds__(DecLayout::THREADS, 1) decode_persistent_kernel(const DecPArgs a) {
  using LY = DecLayout;
  constexpr int NWG = DEC_NWG, NS = LY::NS;
  extern __shared__ unsigned char smem_raw[];
  const BBCell *cells = a.cells;
  const int nt = a.nt, total = a.total;
  const int2 my_run0 = a.run0[blockIdx.x];
  const int run0_first = my_run0.x, run0_end = my_run0.y;
  const int pool = a.pool;
  JOLT_DBG(long long *cta_dbg = cells[0].dbg ? cells[0].dbg + 128 + blockIdx.x * 4 : nullptr;)
  JOLT_DBG(if (cta_dbg && threadIdx.x == 0) { long long g; unsigned sm; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(g)); asm volatile("mov.u32 %0, %%smid;" : "=r"(sm)); cta_dbg[0] = g; cta_dbg[2] = sm; })

  // shared memory: P block (32 KB) | output staging (2 x 16 KB) | rotation operand H | U_T ring | operand tiles | barriers
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char *sm = smem_raw + (base - raw);
  const uint32_t sP = base, sStg = base + 32768u, sH = base + LY::P_BYTES, sBig = sH + DEC_H_BYTES;
  const uint32_t sRing = sBig, sR = sBig + NS * BB_STAGE_BYTES;
  const uint32_t sBar = sBig + LY::BIG_BYTES;
  unsigned char *smStg = sm + 32768, *smH = sm + LY::P_BYTES, *smR = sm + LY::P_BYTES + DEC_H_BYTES + NS * BB_STAGE_BYTES;
  unsigned char *smBar = sm + LY::P_BYTES + DEC_H_BYTES + LY::BIG_BYTES;
  volatile int *abort_flag = (volatile int *)(smBar + 256);
  uint32_t *tmem_slot = (uint32_t *)(smBar + 264);
  DecRunQ runq{(volatile int *)(smBar + 272), total, abort_flag};      // 8 slots of 16 bytes
  const uint32_t bSetup = sBar + 0;          // the P block of a head segment has landed
  const uint32_t bPfree = sBar + 8;          // all backbone MMAs of a head segment are complete
  const uint32_t bHready = sBar + 16;
  auto bFull = [=](int s) { return sBar + 24 + 8 * s; };          // four ring stages
  auto bEmpty = [=](int s) { return sBar + 72 + 8 * s; };
  auto bTfull = [=](int b) { return sBar + 120 + 8 * b; };        // four accumulators
  auto bTempty = [=](int b) { return sBar + 152 + 8 * b; };
  auto bRready = [=](int b) { return sBar + 184 + 8 * b; };
  auto bBB = [=](int b) { return sBar + 216 + 8 * b; };           // backbone of the accumulator's tile complete

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int wg = warp >> 2;
  BBCell *sc_cell = (BBCell *)(smBar + 512);      // the epilogue's copy of the current cell's descriptor

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    for (int k = 0; k < 8; ++k) runq.q[4 * k + 2] = -1;
    mbar_init(bSetup, 1); mbar_init(bPfree, 1);
    mbar_init(bHready, NWG * 128);
    for (int s = 0; s < NS; ++s) { mbar_init(bFull(s), 1); mbar_init(bEmpty(s), 1); }
    for (int b = 0; b < 4; ++b) { mbar_init(bTfull(b), 1); mbar_init(bTempty(b), 128); mbar_init(bRready(b), 128); mbar_init(bBB(b), 1); }
    fence_barrier_init();
  }
  if (warp == NWG * 4) { tmem_alloc(smem_u32(tmem_slot), LY::TMEM_COLS); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (wg == NWG) {
    // The CTA is launched with 168 registers per thread; raising the 256 epilogue threads to 224 takes 14 336 registers,
    // which the 128 threads of this warpgroup must release first: 48 each releases 15 360.  (Releasing fewer than the
    // increase needs makes the blocking increase wait for ever; releasing exactly as many leaves it no slack.)
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(48));
    if (warp == NWG * 4 && lane == 0) {
      // ---------------- U_T producer and scheduler: the ring stages of every tile, in the CTA's order
      int cnt = 0, ci = 0;
      bool ok = true;
      int first = run0_first, end = run0_end;
      int next_chunk = atomicAdd(a.counter, 1);      // asked for one run ahead; read when the run starts
      int k = 0;
      for (;; ++k) {
        if (k >= 1) {
          first = min((long long)total, (long long)pool + (long long)next_chunk * a.chunk);
          end = min(total, first + a.chunk);
          runq.publish(k, first, end);
          if (first >= total) break;
          next_chunk = atomicAdd(a.counter, 1);
        }
        int left = end - first;
        if (left <= 0) continue;
        DecPos w = dec_locate(cells, a.n_cells, nt, first, ci);
        while (ok && left > 0) {
          const BBCell &cg = cells[w.ci];
          const int r_t = cg.r_t, nkt = (r_t + 63) / 64, m = cg.m;
          const int len = min(nt - w.tile, left);
          for (int i = 0; ok && i < len; ++i) {
            const int tt = w.tile + i;
            for (int kb = 0; kb < nkt; ++kb, ++cnt) {
              const int s = cnt % NS, n = cnt / NS;
              ok = mbar_wait(bEmpty(s), (n & 1) ^ 1, abort_flag);
              if (!ok) break;
              if (cnt == 0 && g_test_skip_first_load == 2) continue;      // test switch: the backbone thread's wait runs out
              mbar_expect_tx(bFull(s), BB_STAGE_BYTES);
              tma_load_2d(sRing + s * BB_STAGE_BYTES, &cg.tmUT, bFull(s), kb * 64, tt * 128);
            }
          }
          left -= len;
          w.tile = 0;
          if (++w.h >= m) { w.h = 0; ++w.ci; }
        }
        ci = min(w.ci, a.n_cells - 1);
        if (!ok) { runq.publish(k + 1, total, total); break; }      // the other roles end at the next run
      }
    } else if (warp == NWG * 4 + 3 && lane == 0) {
      // ---------------- P loader: per head segment the projected core, once the backbone thread has released the buffer
      int seg = 0, ci = 0;
      bool ok = true;
      for (int k = 0; ok; ++k) {
        int first = run0_first, end = run0_end;
        if (k >= 1) { ok = runq.get(k, first, end); if (!ok || first >= total) break; }
        int left = end - first;
        if (left <= 0) continue;
        DecPos w = dec_locate(cells, a.n_cells, nt, first, ci);
        while (ok && left > 0) {
          const BBCell &cg = cells[w.ci];
          const int r_t = cg.r_t, m = cg.m;
          const uint32_t panel = (uint32_t)r_t * 128u;
          if (seg >= 1) { ok = mbar_wait(bPfree, (seg - 1) & 1, abort_flag); if (!ok) break; }
          mbar_expect_tx(bSetup, 2u * panel);
          tma_load_2d(sP, &cg.tmP, bSetup, 0, w.h * r_t);
          tma_load_2d(sP + panel, &cg.tmP, bSetup, 64, w.h * r_t);
          const int len = min(nt - w.tile, left);
          left -= len; ++seg;
          w.tile = 0;
          if (++w.h >= m) { w.h = 0; ++w.ci; }
          if (left > 0) {            // the block after this one: into L2 while this head is being decoded
            const BBCell &cn = cells[w.ci];
            tma_prefetch_l2_2d(&cn.tmP, 0, w.h * cn.r_t);
            tma_prefetch_l2_2d(&cn.tmP, 64, w.h * cn.r_t);
          }
        }
        ci = min(w.ci, a.n_cells - 1);
      }
    } else if (warp == NWG * 4 + 1 && lane == 0) {
      // ---------------- backbone MMA issuer
      const uint32_t idescB = umma_idesc_f16(128, 128, 0, 1);     // A = U_T tile, K-major; B = P panels, MN-major
      const uint64_t dS0 = umma_desc_sw128(sRing, 16, 1024);
      constexpr uint64_t kStep16K = 16384 >> 4;
      int seg = 0, cnt = 0, j = 0, ci = 0;
      bool ok = true;
      for (int k = 0; ok; ++k) {
        int first = run0_first, end = run0_end;
        if (k >= 1) { ok = runq.get(k, first, end); if (!ok || first >= total) break; }
        int left = end - first;
        if (left <= 0) continue;
        DecPos w = dec_locate(cells, a.n_cells, nt, first, ci);
        while (ok && left > 0) {
          const BBCell &cg = cells[w.ci];
          const int r_t = cg.r_t, nkt = (r_t + 63) / 64, ksteps = r_t / 16, m = cg.m;
          const uint32_t panel = (uint32_t)r_t * 128u;
          ok = mbar_wait(bSetup, seg & 1, abort_flag);      // the head's projected core has landed
          if (!ok) break;
          tc_fence_after();
          const uint64_t dP0 = umma_desc_sw128(sP, panel, 1024);
          const int len = min(nt - w.tile, left);
          for (int i = 0; ok && i < len; ++i, ++j) {
            int b, nb;
            dec_acc_of(j, b, nb);
            ok = mbar_wait(bTempty(b), (nb & 1) ^ 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            const uint32_t tacc = tmem_base + b * 128;
            for (int kb = 0; kb < nkt; ++kb, ++cnt) {
              const int s = cnt % NS, n = cnt / NS;
              ok = mbar_wait(bFull(s), n & 1, abort_flag);
              if (!ok) break;
              tc_fence_after();
              const uint64_t da = dS0 + (uint64_t)s * kStep16K;
              const uint64_t db = dP0 + (uint64_t)kb * (8192 >> 4);
#pragma unroll
              for (int k4 = 0; k4 < 4; ++k4)
                if (kb * 4 + k4 < ksteps) umma_f16(tacc, umma_desc_kslice(da, k4), db + (uint64_t)k4 * (2048 >> 4), idescB, (kb | k4) != 0);
              umma_commit(bEmpty(s));
            }
            if (ok) umma_commit(bBB(b));
          }
          if (ok) umma_commit(bPfree);
          left -= len; ++seg;
          w.tile = 0;
          if (++w.h >= m) { w.h = 0; ++w.ci; }
        }
        ci = min(w.ci, a.n_cells - 1);
      }
    } else if (warp == NWG * 4 + 2 && lane == 0) {
      // ---------------- rotation MMA issuer: A = the warpgroup's dequantised residual tile, B = H of the current cell
      const uint32_t idesc = umma_idesc_f16(128, 128, 0, 0);
      const uint64_t dH0 = umma_desc_sw128(sH, 16, 1024), dR0 = umma_desc_sw128(sR, 16, 1024);
      constexpr uint64_t kStep16K = 16384 >> 4, kStep32K = 32768 >> 4;
      uint64_t dH[8];
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) dH[ks] = umma_desc_kslice(dH0 + (uint64_t)(ks >> 2) * kStep16K, ks & 3);
      int j = 0, ci = 0, cur_ci = -1, n_built = 0;
      bool ok = true;
      for (int k = 0; ok; ++k) {
        int p = run0_first, end = run0_end;
        if (k >= 1) { ok = runq.get(k, p, end); if (!ok || p >= total) break; }
        if (p >= end) continue;
        ci = dec_locate(cells, a.n_cells, nt, p, ci).ci;
        while (ok && p < end) {
          const BBCell &cg = cells[ci];
          const bool has_res = cg.bits > 0;
          const int cell_end = min(end, cg.tile_base + cg.m * nt);
          if (ci != cur_ci) {
            ok = mbar_wait(bHready, n_built & 1, abort_flag);      // the cell's rotation operand is built
            if (!ok) break;
            tc_fence_after();
            cur_ci = ci; ++n_built;
          }
          for (; ok && p < cell_end; ++p, ++j) {
            int b, nb;
            dec_acc_of(j, b, nb);
            ok = mbar_wait(bBB(b), nb & 1, abort_flag);          // the tile's backbone is in the accumulator
            if (ok) ok = mbar_wait(bRready(b), nb & 1, abort_flag);      // ... and its residual operand is unpacked
            if (!ok) break;
            if (has_res) {
              tc_fence_after();
              const uint32_t tacc = tmem_base + b * 128;
              const uint64_t dR = dR0 + (uint64_t)(j & 1) * kStep32K;
#pragma unroll
              for (int ks = 0; ks < 8; ++ks)
                umma_f16(tacc, umma_desc_kslice(dR + (uint64_t)(ks >> 2) * kStep16K, ks & 3), dH[ks], idesc, 1);
            }
            umma_commit(bTfull(b));
          }
          if (p >= cg.tile_base + cg.m * nt) ++ci;
        }
        ci = min(ci, a.n_cells - 1);
      }
    }
  } else {
    // ---------------- epilogue warpgroups: run by run, cell by cell (both warpgroups walk the same tiles' cells, each
    // its own tiles: the CTA's even-numbered tiles belong to warpgroup 0)
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(224));
    const int qd = warp & 3;
    const int rit = qd * 32 + lane;
    const int et = wg * 128 + rit;                 // thread index among the epilogue threads
    const uint32_t t_lane = tmem_base + ((uint32_t)(qd * 32) << 16);
    bool ok = true, pending = false;
    int j = 0, ci = 0, cur_ci = -1;
    for (int k = 0;; ++k) {
      int p = run0_first, end = run0_end;
      if (k >= 1 && (!runq.get(k, p, end) || p >= total)) break;
      if (p >= end) continue;
      ci = dec_locate(cells, a.n_cells, nt, p, ci).ci;
      while (p < end) {
        const BBCell &cg = cells[ci];
        if (ci != cur_ci) {
          // every rotation MMA that reads the old operand is complete (each warpgroup has read its last accumulator
          // of the old cell) and nobody reads the old descriptor any more
          named_bar_sync(1, NWG * 128);
          for (int i = et; i < (int)(sizeof(BBCell) / 16); i += NWG * 128) ((uint4 *)sc_cell)[i] = __ldg((const uint4 *)&cg + i);
          named_bar_sync(1, NWG * 128);
          dec_build_rotation(smH, a.seed, sc_cell->cell, et, bHready);
          cur_ci = ci;
        }
        const BBCell &c = *sc_cell;
        const int cell_last = c.tile_base + c.m * nt;
        const int cell_end = min(end, cell_last);
        if (ok) {
          DecPCtx x;
          x.cg = &cg;
          x.ex = *c.e;
          x.bTfull = bTfull(wg); x.bTempty = bTempty(wg); x.bRready = bRready(wg);
          x.t_acc = t_lane + wg * 128; x.rbuf = smR + wg * 32768;
          x.s_stg = sStg + (uint32_t)(wg * 16384 + qd * 4096); x.stg = smStg + wg * 16384 + qd * 4096;
          x.abort_flag = abort_flag; x.wg = wg; x.rit = rit; x.nt = nt; x.base = c.tile_base; x.joff = j - p;
          const int p0 = p + (((j & 1) == wg) ? 0 : 1);      // this warpgroup's first tile of the piece
          int rcode = pending ? 2 : 0;      // a bit width that is not compiled in: reported as a failed launch
          const int bits = c.bits;
          if ((BITMASK & 1u) && bits == 0) rcode = dec_tile_loop_p<0, TMA_ONLY>(c, x, p0, cell_end, pending);
          if ((BITMASK & 2u) && bits == 1) rcode = dec_tile_loop_p<1, TMA_ONLY>(c, x, p0, cell_end, pending);
          if ((BITMASK & 4u) && bits == 2) rcode = dec_tile_loop_p<2, TMA_ONLY>(c, x, p0, cell_end, pending);
          if ((BITMASK & 8u) && bits == 3) rcode = dec_tile_loop_p<3, TMA_ONLY>(c, x, p0, cell_end, pending);
          if ((BITMASK & 16u) && bits == 4) rcode = dec_tile_loop_p<4, TMA_ONLY>(c, x, p0, cell_end, pending);
          if ((BITMASK & 256u) && bits == 8) rcode = dec_tile_loop_p<8, TMA_ONLY>(c, x, p0, cell_end, pending);
          ok = (rcode & 1) != 0; pending = (rcode & 2) != 0;
        }
        j += cell_end - p;
        p = cell_end;
        if (p >= cell_last) ++ci;
      }
      ci = min(ci, a.n_cells - 1);
    }
    if (pending && lane == 0) tma_store_wait_all();
  }
  tc_fence_before();
  __syncthreads();
  JOLT_DBG(if (cta_dbg && threadIdx.x == 0) { long long g; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(g)); cta_dbg[1] = g; cta_dbg[3] = 0; })
  if (*abort_flag) {
    if (threadIdx.x == 0) atomicOr(cells[0].status, 8);
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000) {}      // let copies still in flight land before the CTA's memory is reused
    __syncthreads();
  }
  if (warp == NWG * 4) { tc_fence_after(); tmem_dealloc(tmem_base, LY::TMEM_COLS); }
}

}  // namespace tc
}  // namespace jolt
