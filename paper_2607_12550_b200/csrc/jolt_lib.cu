// C-ABI entry points and host orchestration of the JoLT compressor.  Every stage of the path is a
// kernel launched from here; nothing is computed on the host except the allocator (Eq. (3)/(4)),
// argument checks and task tables.
#include <algorithm>
#include <atomic>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <chrono>
#include <functional>
#include <memory>
#include <mutex>
#include <string>
#include <vector>

#include <cuda.h>
#include "allocator.h"
#include "common.cuh"
#include "rowquant.cuh"
#include "simt_gemm.cuh"
#include "small_solvers.cuh"
#include "block_jacobi.cuh"
#include "cluster_jacobi.cuh"
#include "eig_presolve.cuh"
#include "tc_orth.cuh"
#include "rope.cuh"
#include "attend.cuh"

using namespace jolt;

namespace jolt {
thread_local std::string g_err;
std::atomic<long long> g_launches{0};
std::atomic<int> g_eig_smem{1};
#ifdef JOLT_DEBUG
long long *g_dbg_stamps = nullptr;   // device buffer for kernel cycle stamps (profiling aid)
#endif
std::atomic<int> g_n_cell_groups{4};        // concurrent cell groups of jolt_compress (jolt_set_stream_groups)
std::atomic<int> g_dec_tail_pct{0}, g_dec_tail_chunk{8};   // test switch: chunked tail of the persistent decode (off)
std::atomic<int> g_fast{255};  // bit 0: fused backbone kernels, bit 1: factor sweeps, bit 2: Gram on tensor cores,
                              // bit 3: rotary embedding inside the decode kernel, bit 4: cluster-resident eigen-solver,
                              // bit 5: CholeskyQR on tensor cores, bit 6: two output tiles per CTA in the factor sweeps,
                              // bit 7: persistent decode kernel

int fail(int code, const char *fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  g_err = buf;
  return code;
}

// ------------------------------------------------------------------ stage timing
static const char *kStageNames[] = {"stage_in", "sketch_gen", "gram", "eig_feat", "sketch", "orth", "power", "project",
                                    "small_svd", "factors", "store", "backbone", "residual_quant", "decode_backbone",
                                    "decode_rows", "rope", "attend", "stage_out"};
constexpr int kNumStages = sizeof(kStageNames) / sizeof(kStageNames[0]);
struct StageTimer {
  cudaEvent_t ev[kNumStages + 1];
  bool have = false;
  int order[kNumStages + 1];
  int n = 0;
  float ms[kNumStages];
  void init() {
    if (have) return;
    for (auto &e : ev) cudaEventCreate(&e);
    have = true;
  }
  void begin(cudaStream_t s) { init(); n = 0; for (auto &m : ms) m = 0.f; cudaEventRecord(ev[0], s); }
  void mark(int stage, cudaStream_t s) { if (n < kNumStages) { order[n] = stage; ++n; cudaEventRecord(ev[n], s); } }
  void finish() {
    for (auto &m : ms) m = 0.f;
    for (int i = 0; i < n; ++i) { float t = 0; if (cudaEventElapsedTime(&t, ev[i], ev[i + 1]) == cudaSuccess) ms[order[i]] += t; }
  }
};
thread_local StageTimer g_timer;
enum { ST_IN = 0, ST_SKGEN, ST_GRAM, ST_EIGF, ST_SKETCH, ST_ORTH, ST_POWER, ST_PROJ, ST_SVD, ST_FACT, ST_STORE, ST_BACK,
       ST_RQ, ST_DBACK, ST_DROWS, ST_ROPE, ST_ATT, ST_OUT };

// ------------------------------------------------------------------ workspace cache (per device)
struct Workspace { void *base = nullptr; size_t cap = 0; };
static std::mutex g_ws_mu;
static Workspace g_ws[64];

static int ws_reserve(int dev, size_t bytes, void **out) {
  std::lock_guard<std::mutex> lk(g_ws_mu);
  Workspace &w = g_ws[dev];
  if (w.cap < bytes) {
    if (w.base) { cudaDeviceSynchronize(); cudaFree(w.base); w.base = nullptr; w.cap = 0; }
    const size_t want = bytes + (bytes >> 3);
    if (cudaMalloc(&w.base, want) != cudaSuccess) {
      cudaGetLastError();
      if (cudaMalloc(&w.base, bytes) != cudaSuccess) { cudaGetLastError(); w.base = nullptr; return fail(JOLT_ENOMEM, "workspace of %zu bytes", bytes); }
      w.cap = bytes;
    } else w.cap = want;
  }
  *out = w.base;
  return JOLT_OK;
}

// The workspace and the argument-table arena are shared by every call on a device.  A call makes its stream wait for
// the last launch of the previous call that used them (whatever stream that ran on) and leaves an event behind.
static cudaEvent_t g_arena_ev[64] = {};
static int arena_acquire(int dev, cudaStream_t st) {
  std::lock_guard<std::mutex> lk(g_ws_mu);
  if (!g_arena_ev[dev]) {
    if (cudaEventCreateWithFlags(&g_arena_ev[dev], cudaEventDisableTiming) != cudaSuccess) { cudaGetLastError(); g_arena_ev[dev] = nullptr; return fail(JOLT_ECUDA, "event"); }
    return JOLT_OK;        // first use: nothing to wait for
  }
  if (cudaStreamWaitEvent(st, g_arena_ev[dev], 0) != cudaSuccess) { cudaGetLastError(); return fail(JOLT_ECUDA, "cudaStreamWaitEvent"); }
  return JOLT_OK;
}
static void arena_release(int dev, cudaStream_t st) {
  std::lock_guard<std::mutex> lk(g_ws_mu);
  if (g_arena_ev[dev]) { if (cudaEventRecord(g_arena_ev[dev], st) != cudaSuccess) cudaGetLastError(); }
}

struct Bump {
  char *base = nullptr;
  size_t off = 0;
  template <typename T> T *take(size_t n) {
    off = (off + 255) & ~(size_t)255;
    T *p = base ? (T *)(base + off) : nullptr;
    off += n * sizeof(T);
    return p;
  }
};

// ------------------------------------------------------------------ small kernels
__global__ void gen_sketch_kernel(const CellDesc *cells, float *const *omega, const long long *counts, int stream_id,
                                  uint64_t seed) {
  const int ci = blockIdx.y;
  const long long n = counts[ci];
  const uint64_t base = stream_base(seed, cells[ci].cell, stream_id);
  float *o = omega[ci];
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
    o[i] = __half2float(__double2half(gaussian_from_u64(mix64(base + (uint64_t)i))));
}

__global__ void reduce_partials_kernel(const double *const *partials, double *const *out, const int *counts, int n_elems) {
  const int ci = blockIdx.y;
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= n_elems) return;
  const double *p = partials[ci];
  double s = 0;
  for (int h = 0; h < counts[ci]; ++h) s += p[(size_t)h * n_elems + e];
  out[ci][e] = s;
}

__global__ void set_identity_kernel(float *const *U, const int *ld) {
  const int ci = blockIdx.y;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < kD * ld[ci]) U[ci][i] = ((i / ld[ci]) == (i % ld[ci])) ? 1.f : 0.f;
}

struct StoreJob {
  const float *G32; const float *UT32; const float *UF32;
  __half *G16, *UT16, *UF16;
  int *e;
  float *pmax;        // kCoreMaxParts partial maxima of |G| (scratch)
  long long nG, nUT, nUF;
  int round_inputs;   // 1: UT32/UF32 are rounded to fp16 in place as well (injected factors)
};

// max |G| of a cell in kCoreMaxParts partial maxima (one CTA each); store_factors_kernel finishes the reduction
constexpr int kCoreMaxParts = 32;
__global__ void core_exponent_kernel(const StoreJob *jobs) {
  const StoreJob j = jobs[blockIdx.y];
  float mx = 0.f;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < j.nG; i += (long long)gridDim.x * blockDim.x)
    mx = fmaxf(mx, fabsf(j.G32[i]));
  for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  __shared__ float red[32];
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = mx;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int i = 0; i < (int)blockDim.x / 32; ++i) mx = fmaxf(mx, red[i]);
    j.pmax[blockIdx.x] = mx;
  }
}

__global__ void store_factors_kernel(const StoreJob *jobs) {
  const StoreJob j = jobs[blockIdx.y];
  __shared__ int s_e;
  if (threadIdx.x == 0) {
    float mx = 0.f;
    for (int i = 0; i < kCoreMaxParts; ++i) mx = fmaxf(mx, j.pmax[i]);
    int e = 0;
    if (mx > 0.f && isfinite(mx)) e = ilogbf(mx) - kCoreTargetExp;
    s_e = e;
    if (blockIdx.x == 0) *j.e = e;
  }
  __syncthreads();
  const int e = s_e;
  const long long stride = (long long)gridDim.x * blockDim.x;
  const long long i0 = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  for (long long i = i0; i < j.nG; i += stride) j.G16[i] = __float2half_rn(ldexpf(j.G32[i], -e));
  for (long long i = i0; i < j.nUT; i += stride) j.UT16[i] = __float2half_rn(j.UT32[i]);
  for (long long i = i0; i < j.nUF; i += stride) j.UF16[i] = __float2half_rn(j.UF32[i]);
}

// P_h[k][f] = fp16( sum_s G_h[k][s] U_F[f][s] ), the projected core of the decoder in the core's scaled units, for every
// (head, k) row of a cell: [m * r_t][128].  Formed once, when the stored factors exist, and kept with the handle: the
// residual pass, the decode pass and the attention kernels all read THIS array, so the backbone the residual was taken
// against is bit for bit the backbone the decoder adds back (closed loop).  grid (row blocks of 32, cells), 128 threads
// (thread = feature); dynamic shared memory: 128 * r_f halves (U_F, staged as [s][f]).
struct ProjJob { const __half *G, *UF; __half *P; int rows, r_f; };
__global__ void __launch_bounds__(128) project_core_kernel(const ProjJob *__restrict__ jobs) {
  const ProjJob j = jobs[blockIdx.y];
  const int r0 = blockIdx.x * 32, f = threadIdx.x;
  if (r0 >= j.rows) return;
  extern __shared__ __half pc_uf[];
  for (int e = f; e < 128 * j.r_f; e += 128) { const int ff = e / j.r_f, s = e - ff * j.r_f; pc_uf[s * 128 + ff] = j.UF[e]; }
  __syncthreads();
  // fp64 accumulation: products of two fp16 numbers are exact in it and the sum of <= 128 of them is far inside its
  // precision, so the one rounding to fp16 is the rounding of the exact value (the definition), not of an fp32 sum
  // that may sit on the other side of a rounding boundary
  // eight rows of G at a time, staged in shared memory (read straight from global memory the loop waited for one
  // broadcast load per row and step: 76 us for three small cells on the critical chain of the call)
  __shared__ __half gs[8][128];
  for (int rb = r0; rb < min(r0 + 32, j.rows); rb += 8) {
    __syncthreads();
    for (int e = f; e < 8 * j.r_f; e += 128) {
      const int r = e / j.r_f, s = e - r * j.r_f;
      gs[r][s] = rb + r < j.rows ? j.G[(size_t)(rb + r) * j.r_f + s] : __float2half(0.f);
    }
    __syncthreads();
    double acc[8];
#pragma unroll
    for (int r = 0; r < 8; ++r) acc[r] = 0.0;
    for (int s = 0; s < j.r_f; ++s) {
      const double u = (double)__half2float(pc_uf[s * 128 + f]);
#pragma unroll
      for (int r = 0; r < 8; ++r) acc[r] = fma((double)__half2float(gs[r][s]), u, acc[r]);
    }
#pragma unroll
    for (int r = 0; r < 8; ++r)
      if (rb + r < j.rows) j.P[(size_t)(rb + r) * 128 + f] = __double2half(acc[r]);
  }
}

__global__ void round_to_half_inplace_kernel(float *const *ptrs, const long long *counts) {
  const int ci = blockIdx.y;
  float *p = ptrs[ci];
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < counts[ci]; i += (long long)gridDim.x * blockDim.x)
    p[i] = __half2float(__float2half_rn(p[i]));
}

}  // namespace jolt

// ------------------------------------------------------------------ handle
struct CellStore {
  CellDesc c;          // X is null after compress
  __half *G16 = nullptr, *UT16 = nullptr, *UF16 = nullptr;
  int *e = nullptr;
  uint32_t *words = nullptr;
  __half *scales = nullptr;
  float *sigma = nullptr;  // k (or T for the exact path)
  float *lam = nullptr;    // 128
  int n_sigma = 0;
  const float *dbg_UT32 = nullptr;   // fp32 token factor in the workspace (valid until the next library call)
  __half *P16 = nullptr;   // projected core [m * r_t][128] (decode-side scratch kept with the handle, not part of the stored bytes)
  bool tc_ok = false;      // tensor maps below are valid
  alignas(64) CUtensorMap tmUT, tmP;
};

struct jolt_handle {
  int device = 0;
  int n_layers = 0, n_kv_heads = 0, T = 0, n_groups = 0;
  std::vector<int> group_start;
  std::vector<CellStore> cells;
  void *blob = nullptr;
  size_t blob_bytes = 0;
  uint64_t seed = 0;
  int64_t stored_bytes = 0;
  bool subspace = false;     // token factors came from the converged block iteration (exact mode, large T)
  int *d_status = nullptr;   // 4 words per cell, written by the decode kernels of the last call on this handle (jolt_check_status)
  mutable cudaStream_t last_stream = nullptr;   // stream of the last call that read the handle's buffers (jolt_free orders after it)
  __half *P_all = nullptr;   // the projected cores P_h = fp16(G_h U_F^T) of every cell (CellStore::P16 point into it)
};

// ------------------------------------------------------------------ validation
static int check_layout(const jolt_layout *L) {
  if (!L) return fail(JOLT_EINVAL, "layout is null");
  if (L->head_dim != kD) return fail(L->head_dim > 0 ? JOLT_EUNSUPPORTED : JOLT_EINVAL, "head_dim %d (only 128 is built)", L->head_dim);
  if (L->n_layers <= 0 || L->n_kv_heads <= 0 || L->seq_len <= 0) return fail(JOLT_EINVAL, "non-positive shape");
  if (L->seq_len % 128) return fail(JOLT_EUNSUPPORTED, "seq_len %d is not a multiple of 128", L->seq_len);
  if (L->dtype != JOLT_F16 && L->dtype != JOLT_F32) return fail(JOLT_EINVAL, "dtype %d", L->dtype);
  if (L->mem_space != JOLT_MEM_DEVICE && L->mem_space != JOLT_MEM_HOST) return fail(JOLT_EINVAL, "mem_space %d", L->mem_space);
  if (L->stride_token < kD || L->stride_token % 8) return fail(JOLT_EINVAL, "stride_token %lld", (long long)L->stride_token);
  if (L->stride_head % 8 || L->stride_layer % 8 || L->stride_head <= 0 || L->stride_layer <= 0) return fail(JOLT_EINVAL, "strides must be positive multiples of 8");
  if (L->n_groups <= 0 || !L->group_start) return fail(JOLT_EINVAL, "layer grouping missing");
  if (L->group_start[0] != 0 || L->group_start[L->n_groups] != L->n_layers) return fail(JOLT_EINVAL, "group_start must run from 0 to n_layers");
  for (int g = 0; g < L->n_groups; ++g)
    if (L->group_start[g + 1] <= L->group_start[g]) return fail(JOLT_EINVAL, "group_start must ascend");
  return JOLT_OK;
}

// Device tensors are read and written with 16-byte vector accesses (strides are multiples of 8 elements already).
static int check_device_alignment(const jolt_layout *L, const void *a, const void *b) {
  if (L->mem_space == JOLT_MEM_DEVICE && ((((uintptr_t)a) | ((uintptr_t)b)) & 15))
    return fail(JOLT_EINVAL, "device tensors must start on a 16-byte boundary");
  return JOLT_OK;
}

static size_t layout_span_elems(const jolt_layout *L) {
  return (size_t)(L->n_layers - 1) * L->stride_layer + (size_t)(L->n_kv_heads - 1) * L->stride_head +
         (size_t)(L->seq_len - 1) * L->stride_token + kD;
}

static int check_options(const jolt_options *o) {
  if (!o) return fail(JOLT_EINVAL, "options are null");
  if (o->token_mode != JOLT_TOKEN_EXACT && o->token_mode != JOLT_TOKEN_RANDOMIZED) return fail(JOLT_EINVAL, "token_mode %d", o->token_mode);
  if (o->oversample < 0 || o->power_iters < 0 || o->power_iters > 8) return fail(JOLT_EINVAL, "oversample / power_iters out of range");
  if (o->quant_group != kGroup) return fail(JOLT_EUNSUPPORTED, "quant_group %d (only 32 is built)", o->quant_group);
  return JOLT_OK;
}

static bool bits_ok(int b) { return b == 0 || b == 1 || b == 2 || b == 3 || b == 4 || b == 8; }

#define CU(x)                                                                                   \
  do {                                                                                          \
    cudaError_t e__ = (x);                                                                      \
    if (e__ != cudaSuccess) return fail(JOLT_ECUDA, "%s: %s", #x, cudaGetErrorString(e__));      \
  } while (0)
#define LAUNCHED() (++g_launches)

// ------------------------------------------------------------------ launch program
// All argument tables of a call are built on the host first, uploaded with one copy, and then the
// kernels are launched back to back: the stream never waits for the host between stages.
namespace {

struct Program {
  std::vector<char> host;
  struct Step { int stage; std::function<void(char *, cudaStream_t)> run; };
  std::vector<Step> steps;
  template <typename T> size_t push(const std::vector<T> &v) {
    size_t off = (host.size() + 127) & ~(size_t)127;
    host.resize(off + v.size() * sizeof(T));
    if (!v.empty()) memcpy(host.data() + off, v.data(), v.size() * sizeof(T));
    return off;
  }
  void add(int stage, std::function<void(char *, cudaStream_t)> f) { steps.push_back({stage, std::move(f)}); }
};

GemmTask mk(const void *A, int ta, long long a_rs, long long a_cs, const void *B, int tb, long long b_rs, long long b_cs,
            void *C, int tc, long long c_rs, int M, int N, int K) {
  GemmTask t;
  memset(&t, 0, sizeof t);
  t.A = A; t.B = B; t.C = C; t.M = M; t.N = N; t.K = K; t.nseg = 1; t.seg_inner = 1;
  t.a_rs = a_rs; t.a_cs = a_cs; t.b_rs = b_rs; t.b_cs = b_cs; t.c_rs = c_rs; t.c_cs = 1;
  t.ta = ta; t.tb = tb; t.tc = tc; t.alpha = 1.f; t.alpha_exp = nullptr; t.accumulate = 0;
  return t;
}

void add_gemm(Program &P, int stage, const std::vector<GemmTask> &all_tasks, bool f64) {
  if (all_tasks.empty()) return;
  // one launch per tile-count class: a grid sized for the largest task would start mostly empty CTAs for the rest.
  // Plain fp32 tasks take the register-tiled kernel (128 x 64 tiles), everything else the generic one (64 x 64).
  struct Bucket { long long key; bool fast; std::vector<GemmTask> tasks; };
  std::vector<Bucket> buckets;
  for (auto &t : all_tasks) {
    if (t.M <= 0 || t.N <= 0) continue;
    const bool fastk = !f64 && sgemm_fast_ok(t);
    const int bm = fastk ? 128 : 64;
    const long long key = ((long long)((t.M + bm - 1) / bm) << 32) | (long long)((t.N + 63) / 64);
    size_t b = 0;
    for (; b < buckets.size(); ++b) if (buckets[b].key == key && buckets[b].fast == fastk) break;
    if (b == buckets.size()) buckets.push_back({key, fastk, {}});
    buckets[b].tasks.push_back(t);
  }
  for (auto &bk : buckets) {
    const std::vector<GemmTask> &tasks = bk.tasks;
    const int tm = (int)(bk.key >> 32), tn = (int)(bk.key & 0xffffffff);
    const bool fastk = bk.fast;
    const size_t off = P.push(tasks);
    const int n = (int)tasks.size();
    P.add(stage, [=](char *dev, cudaStream_t s) {
      const GemmTask *d = (const GemmTask *)(dev + off);
      for (int z0 = 0; z0 < n; z0 += 32768) {
        dim3 grid(tn, tm, std::min(32768, n - z0));
        if (f64) simt_gemm_kernel<double><<<grid, 256, 0, s>>>(d + z0);
        else if (fastk) simt_sgemm_kernel<<<grid, 256, 0, s>>>(d + z0);
        else simt_gemm_kernel<float><<<grid, 256, 0, s>>>(d + z0);
        LAUNCHED();
      }
    });
  }
}

void add_eig(Program &P, int stage, const std::vector<EigTask> &tasks, int bj_sweeps) {
  if (tasks.empty()) return;
  // problems that fit one CTA's shared memory take the resident kernel, the rest the global-memory one
  std::vector<EigTask> small64, small32, big;
  std::vector<BJTask> bj;
  std::vector<CholFactorTask> cf;          // Cholesky factor for the cluster solver: work matrix in global memory (n > 152)
  std::vector<tc::CholInvTask> cfs;        // ... in shared memory
  std::vector<CJTask> cj;                  // one launch: rows per lane follow the largest matrix
  std::vector<PresolveTask> pre;           // block-solver problems that start from a single-precision basis
  for (auto &t : tasks) {
    // singular values of B (w_sqrt): single-precision cluster solver; the mode-3 Gram, whose spectrum spans 1e6 and more
    // when the cache has outlier channels, stays on the fp64 block solver
    if (t.bjA && t.w_sqrt && t.n > 32 && t.n <= kCJMaxN && (g_fast.load() & 16)) {
      // Cholesky factor in the block solver's scratch, then the cluster-resident one-sided Jacobi on its columns
      if (t.n <= tc::kCholInvMaxN) cfs.push_back({nullptr, 0, 0, t.A, t.n, nullptr, nullptr, nullptr, t.bjA, t.status, 1e-13});
      else cf.push_back({t.A, t.bjA, t.n, t.status});
      CJTask c; memset(&c, 0, sizeof c);
      c.L = t.bjA; c.n = t.n; c.U_out = t.U_out; c.ld_out = t.ld_out; c.r_out = t.r_out; c.w_out = t.w_out; c.w_sqrt = t.w_sqrt;
      c.status = t.status; c.sweeps_out = t.bjDone;
      cj.push_back(c);
      continue;
    }
    if (t.bjA && t.n > 32 && g_eig_smem.load() != 2) {
      BJTask b; memset(&b, 0, sizeof b);
      const bool presolve = t.preL && !t.w_sqrt && t.n <= tc::kCholInvMaxN && (g_fast.load() & 16);
      if (presolve) {
        // A + shift -> Cholesky factor -> single-precision one-sided Jacobi: U; then A' = U^T A U, block solver from V = U
        pre.push_back({t.A, t.preA, t.preU, t.preT, t.n});
        cfs.push_back({nullptr, 0, 0, t.preA, t.n, nullptr, nullptr, nullptr, t.preL, nullptr, 0.0});
        CJTask c; memset(&c, 0, sizeof c);
        c.L = t.preL; c.n = t.n; c.U_out = t.preU; c.ld_out = t.n; c.r_out = t.n;
        c.status = nullptr;      // only a starting basis: if this iteration stops short, the block solver sweeps more
        cj.push_back(c);
        b.V0 = t.preU;
      }
      b.A_in = presolve ? t.preA : t.A; b.A = t.bjA; b.V = t.bjV; b.J = t.bjJ; b.off = t.bjOff; b.done = t.bjDone; b.ticket = (unsigned *)(t.bjDone + 1);
      b.n = t.n; b.nbe = (((t.n + kBJBlock - 1) / kBJBlock) + 1) & ~1; b.nP = b.nbe * kBJBlock;
      b.w = t.w; b.U_out = t.U_out; b.ld_out = t.ld_out; b.r_out = t.r_out; b.w_out = t.w_out; b.w_sqrt = t.w_sqrt; b.status = t.status;
      b.tol = kBJTol;
      bj.push_back(b);
      continue;
    }
    if (!g_eig_smem.load() || t.n > kEigSmemMaxN) big.push_back(t);
    else if (eig_smem_bytes(t.n, 8) <= kSmemOptIn - 1024) small64.push_back(t);   // fp64 eigenvector accumulator fits
    else if (eig_smem_bytes(t.n, 4) <= kSmemOptIn - 1024) small32.push_back(t);
    else big.push_back(t);
  }
  const size_t o_pre = P.push(pre);
  const int n_pre = (int)pre.size();
  int pre_n = 0;
  for (auto &q : pre) pre_n = std::max(pre_n, q.n);
  if (n_pre) P.add(stage, [=](char *dev, cudaStream_t s) {
    presolve_shift_kernel<<<dim3(16, n_pre), 256, 0, s>>>((const PresolveTask *)(dev + o_pre)); LAUNCHED();
  });
  if (!cfs.empty()) {
    const size_t off = P.push(cfs);
    const int n = (int)cfs.size();
    int cmn = 0;
    for (auto &c : cfs) cmn = std::max(cmn, c.k);
    const size_t cshm = tc::cholinv_smem_bytes(cmn);
    static bool cattr = false;
    if (!cattr) { cudaFuncSetAttribute(tc::cholinv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tc::cholinv_smem_bytes(tc::kCholInvMaxN)); cattr = true; }
    P.add(stage, [=](char *dev, cudaStream_t s) {
      tc::cholinv_kernel<<<n, tc::kCholInvThreads, cshm, s>>>((const tc::CholInvTask *)(dev + off)); LAUNCHED();
    });
  }
  if (!cf.empty()) {
    const size_t off = P.push(cf);
    const int n = (int)cf.size();
    int cmn = 0;
    for (auto &c : cf) cmn = std::max(cmn, c.n);
    const size_t cshm = std::max(chol_factor_smem_bytes(kCholFactorSmemN), chol_factor_smem_bytes(cmn));
    static bool cattr = false;
    if (!cattr) { cudaFuncSetAttribute(chol_factor_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(kSmemOptIn - 2048)); cattr = true; }
    P.add(stage, [=](char *dev, cudaStream_t s) {
      chol_factor_kernel<<<n, kCholFactorThreads, cshm, s>>>((const CholFactorTask *)(dev + off)); LAUNCHED();
    });
  }
  if (!cj.empty()) {
    static bool cjattr = false;
    if (!cjattr) { cj_opt_in_smem(); cjattr = true; }
    {
      int mn = 0;
      for (auto &c : cj) mn = std::max(mn, c.n);
      const int nr = cj_rows_per_lane(mn), nt = (int)cj.size();
      const size_t o2 = P.push(cj);
      P.add(stage, [=](char *dev, cudaStream_t s) { cj_launch((const CJTask *)(dev + o2), nt, mn, nr, s); LAUNCHED(); });
    }
  }
  if (n_pre) P.add(stage, [=](char *dev, cudaStream_t s) {
    const dim3 grid((pre_n + 15) / 16, n_pre);
    presolve_mul_kernel<false><<<grid, 256, 0, s>>>((const PresolveTask *)(dev + o_pre)); LAUNCHED();
    presolve_mul_kernel<true><<<grid, 256, 0, s>>>((const PresolveTask *)(dev + o_pre)); LAUNCHED();
  });
  if (!bj.empty()) {
    // with a single-precision starting basis for every problem one sweep converges (measured: relative off-diagonal
    // mass 1e-12 .. 1e-13 before it, rank-deficient matrices included); four are allowed, and the launches after
    // convergence are no-ops of a few microseconds each
    if (n_pre == (int)bj.size()) bj_sweeps = std::min(bj_sweeps, 4);
    int max_nbe = 0, max_nP = 0;
    for (auto &b : bj) { max_nbe = std::max(max_nbe, b.nbe); max_nP = std::max(max_nP, b.nP); }
    const size_t off = P.push(bj);
    const int n = (int)bj.size();
    std::vector<BJTask> copy = bj;
    P.add(stage, [=](char *dev, cudaStream_t s) {
      const BJTask *d = (const BJTask *)(dev + off);
      for (auto &b : copy) { cudaMemsetAsync(b.off, 0, 4 * sizeof(double), s); cudaMemsetAsync(b.done, 0, 4 * sizeof(int), s); }
      bj_init_kernel<<<dim3(64, n), 256, 0, s>>>(d); LAUNCHED();
      const int np = max_nbe / 2;
      const int gx = np * (np + 1) / 2 + np * (max_nP / 32);
      const int n_steps = bj_sweeps * (max_nbe - 1);
      cudaLaunchAttribute pdl; pdl.id = cudaLaunchAttributeProgrammaticStreamSerialization; pdl.val.programmaticStreamSerializationAllowed = 1;
      cudaLaunchConfig_t cfg; memset(&cfg, 0, sizeof cfg);
      cfg.gridDim = dim3(gx + np, n); cfg.blockDim = dim3(kBJThreads); cfg.stream = s; cfg.attrs = &pdl; cfg.numAttrs = 1;
      for (int step = 0; step <= n_steps; ++step) { cudaLaunchKernelEx(&cfg, bj_round_kernel, d, step, n_steps, gx); LAUNCHED(); }
      bj_finish_kernel<<<n, 256, 0, s>>>(d, n_steps & 1); LAUNCHED();
    });
  }
  static bool attr_done = false;
  if (!attr_done) {
    cudaFuncSetAttribute(jacobi_eig_smem_kernel<double>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(kSmemOptIn - 1024));
    cudaFuncSetAttribute(jacobi_eig_smem_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(kSmemOptIn - 1024));
    attr_done = true;
  }
  for (int pass = 0; pass < 2; ++pass) {
    const std::vector<EigTask> &small = pass == 0 ? small64 : small32;
    if (small.empty()) continue;
    int mn = 0;
    for (auto &t : small) mn = std::max(mn, t.n);
    const size_t shm = eig_smem_bytes(mn, pass == 0 ? 8 : 4);
    const size_t off = P.push(small);
    const int n = (int)small.size();
    const bool dbl = pass == 0;
    P.add(stage, [=](char *dev, cudaStream_t s) {
      if (dbl) jacobi_eig_smem_kernel<double><<<n, kEigThreads, shm, s>>>((const EigTask *)(dev + off));
      else jacobi_eig_smem_kernel<float><<<n, kEigThreads, shm, s>>>((const EigTask *)(dev + off));
      LAUNCHED();
    });
  }
  if (!big.empty()) {
    int mn = 0;
    for (auto &t : big) mn = std::max(mn, t.n);
    const size_t off = P.push(big);
    const int n = (int)big.size();
    const size_t shm = (size_t)(2 * ((mn + 1) / 2) + 32) * sizeof(double);
    P.add(stage, [=](char *dev, cudaStream_t s) {
      jacobi_eig_kernel<<<n, kEigThreads, shm, s>>>((const EigTask *)(dev + off));
      LAUNCHED();
    });
  }
}


inline const void *x_head(const CellDesc &c, int h) {
  const int l = h / c.n_heads, hd = h % c.n_heads;
  const long long off = (long long)l * c.sl + (long long)hd * c.sh;
  return (const char *)c.X + off * (c.dtype == DT_F16 ? 2 : 4);
}

struct CellWork {      // device scratch of one cell
  CellDesc c;
  bool active = false;       // has a backbone to compute
  double *gram_part = nullptr, *C = nullptr, *Cv = nullptr, *Cw = nullptr;
  float *UF32 = nullptr, *lam = nullptr;
  float *omega = nullptr, *PF = nullptr, *W = nullptr, *S = nullptr, *Zp = nullptr, *Z = nullptr;
  double *Gs = nullptr, *Lwork = nullptr;      // Gram of the basis, Cholesky work matrix (k x (k+1)) for k > kCholSmemMaxN
  double *gpart = nullptr; float *LT32 = nullptr, *invd = nullptr;
  double *bjA = nullptr, *bjV = nullptr, *bjJ = nullptr, *bjOff = nullptr; int *bjDone = nullptr;
  // eigen-solver scratch of the feature stage: its own, since the probe runs that stage concurrently with the token stage
  double *bjfA = nullptr, *bjfV = nullptr, *bjfJ = nullptr, *bjfOff = nullptr; int *bjfDone = nullptr;
  double *preL = nullptr, *preT = nullptr, *preA = nullptr; float *preU = nullptr;      // pre-solve of the feature eigenproblem
  double *BBt = nullptr, *BBv = nullptr, *BBw = nullptr;
  float *Ut = nullptr, *sigma = nullptr;
  float *UT32 = nullptr, *G32 = nullptr;
  float *Y = nullptr; double *Gt = nullptr, *Gtv = nullptr, *Gtw = nullptr;
  float *Zpart = nullptr;    // per-token-segment partials of the projection sweep (T > 4096 on tensor cores)
  __half *P16 = nullptr;
  float *Xt = nullptr;
  int *status = nullptr;
  float *pmax = nullptr;     // partial maxima of |G| for the core exponent
  float *rho = nullptr;      // where the residual of the converged-subspace check goes (exact mode at large T)
  int n_sigma = 0;
  // tensor-core sweeps
  bool tc = false;           // sketch / projection sweeps run on tcgen05
  bool tc_gram = false;      // mode-3 Gram runs on tcgen05
  bool ufI = false;          // r_f = d: U_F = I, the token factor is computed in the original feature coordinates
  bool skip_feat = false;    // no mode-3 Gram / eigen-solve needed
  int kp = 0;                // sketch width padded to a multiple of 16
  __half *Bhi = nullptr, *Blo = nullptr;
  // CholeskyQR on tensor cores: Gram partials, L^-1 as fp16 hi + lo, its exponent, slots for measured magnitudes
  float *orthPart = nullptr; __half *orthLhi = nullptr, *orthLlo = nullptr; int *orthExp = nullptr;
  unsigned *orthMax = nullptr; int orthMaxUsed = 0; bool absmax_ready = false;
  int split_ready = 0;       // 1 / 2: Bhi, Blo already hold the split of S / Z (written by the last triangular solve)
};

enum FactorMode { FM_RANDOMIZED = 0, FM_EXACT = 1, FM_INJECTED = 2 };
constexpr int kOrthMaxSlots = 32;
constexpr int kGramChunks = 32;   // row chunks of a tall Gram (fp64 partial per chunk, summed in order)

// Scratch layout of one cell; run with b.base == nullptr to size it.
void carve(Bump &b, CellWork &w, int mode, bool need_backbone_scratch) {
  const bool real = b.base != nullptr;
  const CellDesc &c = w.c;
  const size_t M = (size_t)c.m * c.T * kD;
  if (w.active) {
    const size_t k = c.k, N = c.N, T = c.T;
    w.UF32 = b.take<float>(kD * (size_t)c.r_f);
    if (!(real && w.lam)) w.lam = b.take<float>(kD);
    w.UT32 = b.take<float>(T * c.r_t);
    w.G32 = b.take<float>((size_t)c.m * c.r_t * c.r_f);
    w.pmax = b.take<float>(32);
    w.Zp = b.take<float>((size_t)c.m * kD * std::max<size_t>(k, c.r_t));
    if (mode != FM_INJECTED) {
      {
        const size_t nmax = std::max<size_t>(kD, mode == FM_EXACT ? T : k);
        const size_t nbe = (((nmax + kBJBlock - 1) / kBJBlock) + 1) & ~(size_t)1, nP = nbe * kBJBlock;
        w.bjA = b.take<double>(2 * nP * nP); w.bjV = b.take<double>(nP * nP); w.bjJ = b.take<double>(2 * (nbe / 2) * 1024);
        w.bjOff = b.take<double>(4); w.bjDone = b.take<int>(4);
      }
      {
        const size_t nbe = (((kD + kBJBlock - 1) / kBJBlock) + 1) & ~(size_t)1, nP = nbe * kBJBlock;
        w.bjfA = b.take<double>(2 * nP * nP); w.bjfV = b.take<double>(nP * nP); w.bjfJ = b.take<double>(2 * (nbe / 2) * 1024);
        w.bjfOff = b.take<double>(4); w.bjfDone = b.take<int>(4);
        w.preL = b.take<double>(kD * kD + 8); w.preT = b.take<double>(kD * kD); w.preA = b.take<double>(kD * kD);
        w.preU = b.take<float>(kD * kD);
      }
      w.gram_part = b.take<double>((size_t)c.m * kD * kD * std::max(1, (tok_segments(c.T) + 1) / 2));
      w.C = b.take<double>(kD * kD); w.Cv = b.take<double>(kD * kD); w.Cw = b.take<double>(kD);
    }
    if (mode == FM_RANDOMIZED) {
      w.omega = b.take<float>((size_t)c.m * kD * k);
      w.PF = b.take<float>(kD * kD);
      w.W = b.take<float>((size_t)c.m * kD * k);
      w.S = b.take<float>(T * k);
      if (w.ufI) w.Z = w.Zp; else w.Z = b.take<float>(N * k);
      if (w.tc) {
        w.kp = (c.k + 15) & ~15;
        const size_t nb = std::max((size_t)c.m * w.kp * kD, (size_t)w.kp * T);
        w.Bhi = b.take<__half>(nb); w.Blo = b.take<__half>(nb);
        if (tok_segments(c.T) > 1) w.Zpart = b.take<float>((size_t)tok_segments(c.T) * c.m * kD * k);
        if (w.ufI && k <= 152 && w.kp <= 160) {
          const size_t steps = std::max((size_t)T / 64, (size_t)c.m * 2);
          w.orthPart = b.take<float>(((steps + 7) / 8) * w.kp * w.kp);
          w.orthLhi = b.take<__half>((size_t)w.kp * w.kp); w.orthLlo = b.take<__half>((size_t)w.kp * w.kp);
          w.orthExp = b.take<int>(4); w.orthMax = b.take<unsigned>(kOrthMaxSlots);
        }
      }
      w.Gs = b.take<double>(k * k); w.Lwork = k > (size_t)kCholSmemMaxN ? b.take<double>(k * (k + 1)) : nullptr;
      w.gpart = b.take<double>(kGramChunks * k * k); w.LT32 = b.take<float>(k * (k + 8)); w.invd = b.take<float>(k + 8);
      w.BBt = b.take<double>(k * k); w.BBv = b.take<double>(k * k); w.BBw = b.take<double>(k);
      w.Ut = b.take<float>(k * std::max<size_t>(c.r_t, 1));
      if (!(real && w.sigma)) w.sigma = b.take<float>(k);
      w.n_sigma = (int)k;
    } else if (mode == FM_EXACT) {
      w.Y = b.take<float>((size_t)c.m * T * c.r_f);
      w.Gt = b.take<double>(T * T); w.Gtv = b.take<double>(T * T); w.Gtw = b.take<double>(T);
      if (!(real && w.sigma)) w.sigma = b.take<float>(T);
      w.n_sigma = (int)T;
    }
  }
  if (need_backbone_scratch && c.r_t > 0) {
    w.P16 = b.take<__half>((size_t)c.m * c.r_t * kD);
    w.Xt = b.take<float>(M);
  }
}

}  // namespace
#include "fast_path.cuh"
namespace {

// G = M^T M (k x k, fp64) of tall fp32 matrices, split over row chunks so that the grid fills the GPU;
// the partials are summed in a fixed order.
struct TallGram { const float *M; int rows, k; double *part, *out; };
void add_tall_gram(Program &P, int stage, const std::vector<TallGram> &jobs) {
  std::vector<ReduceJob> rj;
  std::vector<TallGramJob> fastj[6];        // register-tiled kernel, column blocks of width <= 48 / 96 / 144; +3: off-diagonal blocks
  int fast_chunks[3] = {0, 0, 0};
  for (auto &j : jobs) {
    int chunk = std::max(128, (j.rows + kGramChunks - 1) / kGramChunks);
    chunk = (chunk + 15) & ~15;
    const int n = (j.rows + chunk - 1) / chunk;
    const int nb = (j.k + 143) / 144, bw = (j.k + nb - 1) / nb;          // column blocks of at most 144
    const int cls = bw <= 48 ? 0 : (bw <= 96 ? 1 : 2);
    for (int bi = 0; bi < nb; ++bi)
      for (int bj = 0; bj <= bi; ++bj)
        fastj[cls + (bi == bj ? 0 : 3)].push_back({j.M, j.rows, j.k, chunk, j.part, bi * bw, std::min(bw, j.k - bi * bw), bj * bw, std::min(bw, j.k - bj * bw)});
    fast_chunks[cls] = std::max(fast_chunks[cls], n);
    rj.push_back({j.part, j.out, n, j.k * j.k});
  }
  for (int q = 0; q < 6; ++q) {
    if (fastj[q].empty()) continue;
    const size_t off = P.push(fastj[q]);
    const int n = (int)fastj[q].size(), cls = q % 3, nch = fast_chunks[cls];
    const bool diag = q < 3;
    P.add(stage, [=](char *dev, cudaStream_t s) {
      const TallGramJob *d = (const TallGramJob *)(dev + off);
      const dim3 grid(nch, n);
      if (cls == 0) { if (diag) tall_gram_kernel<3, true><<<grid, 256, 0, s>>>(d); else tall_gram_kernel<3, false><<<grid, 256, 0, s>>>(d); }
      else if (cls == 1) { if (diag) tall_gram_kernel<6, true><<<grid, 256, 0, s>>>(d); else tall_gram_kernel<6, false><<<grid, 256, 0, s>>>(d); }
      else { if (diag) tall_gram_kernel<9, true><<<grid, 256, 0, s>>>(d); else tall_gram_kernel<9, false><<<grid, 256, 0, s>>>(d); }
      LAUNCHED();
    });
  }
  if (rj.empty()) return;
  const size_t off = P.push(rj);
  const int n = (int)rj.size();
  P.add(stage, [=](char *dev, cudaStream_t s) {
    reduce_partials_var_kernel<<<dim3(32, n), 256, 0, s>>>((const ReduceJob *)(dev + off));
    LAUNCHED();
  });
}

// orth(S) for every active cell by CholeskyQR2: twice {Gs = S^T S (fp64), Gs = L L^T, S <- S L^-T}.
// token_side selects S (T rows) or Z (N rows); the result is left in the source buffer.
void add_orth(Program &P, int stage, std::vector<CellWork> &ws, bool token_side, int passes, bool final_basis = false) {
  std::vector<int> on_tc;
  if (g_fast.load() & 32)
    for (size_t i = 0; i < ws.size(); ++i) if (orth_tc_ok(ws[i])) on_tc.push_back((int)i);
  add_orth_tc(P, stage, ws, on_tc, token_side, passes, final_basis);
  for (int pass = 0; pass < 2; ++pass) {
    // cls 0: Cholesky work matrix and L^T resident in shared memory (k <= kCholSmemMaxN); cls 1: both in global memory
    std::vector<TallGram> tg;
    std::vector<CholSmemTask> chs[2];
    std::vector<TrsmJob> tj[2];
    int max_k[2] = {0, 0};
    if (pass >= passes) continue;          // the triangular solve works in place, so one pass is possible
    for (auto &w : ws) {
      if (!w.active) continue;
      if ((g_fast.load() & 32) && orth_tc_ok(w)) continue;
      const int k = w.c.k, rows = token_side ? w.c.T : w.c.N;
      const int cls = k <= kCholSmemMaxN ? 0 : 1;
      float *buf = token_side ? w.S : w.Z;
      tg.push_back({buf, rows, k, w.gpart, w.Gs});
      chs[cls].push_back({w.Gs, w.LT32, w.invd, k, w.status, w.Lwork});
      TrsmJob tjob{buf, buf, rows, k, w.LT32, w.invd, nullptr, nullptr, 0, 0, 0};
      w.split_ready = 0;
      if (w.tc && pass == passes - 1 && (token_side || w.ufI)) {
        // the next sweep reads this basis as its dense operand: emit the hi + lo fp16 split here
        tjob.hi = w.Bhi; tjob.lo = w.Blo; tjob.split_mode = token_side ? 1 : 2; tjob.kp16 = w.kp;
        tjob.scale_exp = ilog2_floor(token_side ? (long long)w.c.T : (long long)w.c.N) / 2;
        w.split_ready = tjob.split_mode;
      }
      tj[cls].push_back(tjob);
      max_k[cls] = std::max(max_k[cls], k);
    }
    add_tall_gram(P, stage, tg);
    static bool attr_done = false;
    if (!attr_done) {
      cudaFuncSetAttribute(cholesky_smem_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)chol_smem_bytes(kCholSmemMaxN));
      cudaFuncSetAttribute(trsm_rows_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(kSmemOptIn - 1024));
      cudaFuncSetAttribute(trsm_rows_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(kSmemOptIn - 1024));
      cudaFuncSetAttribute(trsm_rows_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(kSmemOptIn - 1024));
      attr_done = true;
    }
    for (int cls = 0; cls < 2; ++cls) {
      if (chs[cls].empty()) continue;
      const size_t o1 = P.push(chs[cls]), o2 = P.push(tj[cls]);
      const int n = (int)chs[cls].size(), glob = cls;
      int max_rows = 0;
      for (auto &t : tj[cls]) max_rows = std::max(max_rows, t.rows);
      int rb = 256;
      while (rb > 64 && trsm_smem_bytes(max_k[cls], rb, glob) > kSmemOptIn - 1024) rb >>= 1;
      const size_t sh1 = chol_smem_bytes(max_k[cls], glob), sh2 = trsm_smem_bytes(max_k[cls], rb, glob);
      P.add(stage, [=](char *dev, cudaStream_t s) {
        cholesky_smem_kernel<<<n, 512, sh1, s>>>((const CholSmemTask *)(dev + o1), glob); LAUNCHED();
        const dim3 grid((max_rows + rb - 1) / rb, n);
        const TrsmJob *jobs = (const TrsmJob *)(dev + o2);
        if (rb == 256) trsm_rows_kernel<256><<<grid, 128, sh2, s>>>(jobs, glob);
        else if (rb == 128) trsm_rows_kernel<128><<<grid, 64, sh2, s>>>(jobs, glob);
        else trsm_rows_kernel<64><<<grid, 32, sh2, s>>>(jobs, glob);
        LAUNCHED();
      });
    }
  }
}

// S = sum_h X_h W_h.  First sketch: W_h = (U_F U_F^T) Omega'_h with the Gaussian Omega' drawn in the
// original feature coordinates (W_h = Omega'_h when r_f = d).  Power iteration: W_h = U_F Z_h.
void add_sketch(Program &P, int stage, std::vector<CellWork> &ws, bool from_omega) {
  std::vector<GemmTask> g0, g1, g2;
  std::vector<int> src(ws.size(), 0);
  for (size_t i = 0; i < ws.size(); ++i) {
    CellWork &w = ws[i];
    if (!w.active) continue;
    const CellDesc &c = w.c;
    const float *Wsrc = w.W;
    if (from_omega) {
      if (w.tc && w.ufI) src[i] = 0;                 // fp16 sketch already in the operand layout
      else if (w.ufI) Wsrc = w.omega;
      else {
        src[i] = 1;
        g0.push_back(mk(w.UF32, DT_F32, c.r_f, 1, w.UF32, DT_F32, 1, c.r_f, w.PF, DT_F32, kD, kD, kD, c.r_f));
        for (int h = 0; h < c.m; ++h)
          g1.push_back(mk(w.PF, DT_F32, kD, 1, w.omega + (size_t)h * kD * c.k, DT_F32, c.k, 1,
                          w.W + (size_t)h * kD * c.k, DT_F32, c.k, kD, c.k, kD));
      }
    } else {
      src[i] = 2;
      if (w.ufI) Wsrc = w.Z;
      else
        for (int h = 0; h < c.m; ++h)
          g1.push_back(mk(w.UF32, DT_F32, c.r_f, 1, w.Z + (size_t)h * c.r_f * c.k, DT_F32, c.k, 1,
                          w.W + (size_t)h * kD * c.k, DT_F32, c.k, kD, c.k, c.r_f));
    }
    if (w.tc) continue;
    GemmTask t = mk(c.X, c.dtype, c.st, 1, Wsrc, DT_F32, c.k, 1, w.S, DT_F32, c.k, c.T, c.k, kD);
    t.nseg = c.m; t.seg_inner = c.n_heads;
    t.a_so = c.sl; t.a_si = c.sh;
    t.b_so = (long long)c.n_heads * kD * c.k; t.b_si = (long long)kD * c.k;
    g2.push_back(t);
  }
  add_gemm(P, stage, g0, false);
  add_gemm(P, stage, g1, false);
  add_gemm(P, stage, g2, false);
  add_tok_tc(P, stage, ws, src);
}

// Z_h = U_F^T (X_h^T Q) for every head: rows h*r_f.. of the N x k matrix Z.  Q (T x cols) is `Qsel`.
void add_project(Program &P, int stage, std::vector<CellWork> &ws) {
  std::vector<GemmTask> g1, g2;
  for (auto &w : ws) {
    if (!w.active) continue;
    const CellDesc &c = w.c;
    for (int h = 0; h < c.m; ++h) {
      if (!w.tc)
        g1.push_back(mk(x_head(c, h), c.dtype, 1, c.st, w.S, DT_F32, c.k, 1, w.Zp + (size_t)h * kD * c.k, DT_F32, c.k,
                        kD, c.k, c.T));
      if (!w.ufI)
        g2.push_back(mk(w.UF32, DT_F32, 1, c.r_f, w.Zp + (size_t)h * kD * c.k, DT_F32, c.k, 1,
                        w.Z + (size_t)h * c.r_f * c.k, DT_F32, c.k, c.r_f, c.k, kD));
    }
  }
  add_feat_tc(P, stage, ws);
  add_gemm(P, stage, g1, false);
  add_gemm(P, stage, g2, false);
}

// ---- exact token factor at sizes where the T x T eigen-solve is out of reach (Sec. 5 calls the exact token SVD
// the dominant cost): block subspace iteration, i.e. the range finder with a wider block and enough power
// iterations to converge, followed by Rayleigh-Ritz (the small SVD).  The residual || A V - U Sigma ||_F /
// || U Sigma ||_F, V = A^T U Sigma^-1, of the returned factor is measured with two more sweeps and stored with
// the cell (V has unit columns, which is what the fp16 operand split of the sweeps is scaled for).
constexpr int kSubspaceOversample = 32;
constexpr int kSubspaceIters = 8;
constexpr float kSubspaceTol = 5e-4f;
constexpr int kExactEigMaxT = 1024;        // largest T for which the T x T Gram is diagonalised directly

struct ResidJob { float *S; const float *UT; const float *sigma; int T, k, r_t; float *rho; int *status; float *Z; int N; };

__global__ void pad_copy_kernel(const ResidJob *__restrict__ jobs) {      // S (T x k) <- [U_T | 0]
  const ResidJob j = jobs[blockIdx.y];
  for (long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x; e < (long long)j.T * j.k; e += (long long)gridDim.x * blockDim.x) {
    const int t = (int)(e / j.k), c = (int)(e - (long long)t * j.k);
    j.S[e] = c < j.r_t ? j.UT[(size_t)t * j.r_t + c] : 0.f;
  }
}

__global__ void scale_columns_kernel(const ResidJob *__restrict__ jobs) {  // Z (N x k) <- Z Sigma^-1 on the first r_t columns
  const ResidJob j = jobs[blockIdx.y];
  for (long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x; e < (long long)j.N * j.k; e += (long long)gridDim.x * blockDim.x) {
    const int c = (int)(e % j.k);
    const float sg = c < j.r_t ? j.sigma[c] : 0.f;
    j.Z[e] = sg > 0.f ? j.Z[e] / sg : 0.f;
  }
}

__global__ void __launch_bounds__(1024) subspace_residual_kernel(const ResidJob *__restrict__ jobs) {   // S holds A V
  const ResidJob j = jobs[blockIdx.x];
  double num = 0, den = 0;
  for (long long e = threadIdx.x; e < (long long)j.T * j.r_t; e += blockDim.x) {
    const int t = (int)(e / j.r_t), c = (int)(e - (long long)t * j.r_t);
    const double u = (double)j.sigma[c] * j.UT[e], d = (double)j.S[(size_t)t * j.k + c] - u;
    num += d * d; den += u * u;
  }
  __shared__ double rn[32], rd[32];
  for (int o = 16; o; o >>= 1) { num += __shfl_xor_sync(0xffffffffu, num, o); den += __shfl_xor_sync(0xffffffffu, den, o); }
  if ((threadIdx.x & 31) == 0) { rn[threadIdx.x >> 5] = num; rd[threadIdx.x >> 5] = den; }
  __syncthreads();
  if (threadIdx.x == 0) {
    num = 0; den = 0;
    for (int i = 0; i < (int)blockDim.x / 32; ++i) { num += rn[i]; den += rd[i]; }
    const float rho = den > 0 ? (float)sqrt(num / den) : 0.f;
    if (j.rho) *j.rho = rho;
    if (!(rho <= kSubspaceTol) && j.status) atomicOr(j.status, 16);
  }
}

// Stages that produce U_F (fp32), U_T (fp32) and the core (fp32) of every active cell.
// parts: 1 = the feature stage (mode-3 Gram, eigen-solve), 2 = the token stage and the core, 3 = both.  The two halves
// may go into different programs only where the token stage does not read U_F (the randomized probe).
void build_factor_program(Program &P, std::vector<CellWork> &ws, int mode, bool probe, int power_iters, uint64_t seed, bool fast,
                          bool check_subspace = false, int parts = 3) {
  (void)fast;
  std::vector<int> act;
  for (size_t i = 0; i < ws.size(); ++i) if (ws[i].active) act.push_back((int)i);
  if (act.empty()) return;
  const int na = (int)act.size();
  if (mode == FM_RANDOMIZED && (parts & 2)) {
    std::vector<unsigned *> slots;
    for (int i : act) if (ws[i].orthMax) slots.push_back(ws[i].orthMax);
    if (!slots.empty())
      P.add(ST_SKGEN, [=](char *, cudaStream_t s) { for (unsigned *p : slots) cudaMemsetAsync(p, 0, sizeof(unsigned) * kOrthMaxSlots, s); });
    std::vector<CellDesc> cd; std::vector<float *> om; std::vector<long long> cnt;
    for (int i : act) {
      if (ws[i].tc && ws[i].ufI) continue;
      cd.push_back(ws[i].c); om.push_back(ws[i].omega); cnt.push_back((long long)ws[i].c.m * kD * ws[i].c.k);
    }
    const size_t o1 = P.push(cd), o2 = P.push(om), o3 = P.push(cnt);
    const int sid = probe ? STREAM_PROBE : STREAM_SKETCH;
    const int ng = (int)cd.size();
    add_sketch_gen_tc(P, ST_SKGEN, ws, sid, seed);
    if (ng) P.add(ST_SKGEN, [=](char *dev, cudaStream_t s) {
      gen_sketch_kernel<<<dim3(148, ng), 256, 0, s>>>((const CellDesc *)(dev + o1), (float *const *)(dev + o2),
                                                      (const long long *)(dev + o3), sid, seed);
      LAUNCHED();
    });
  }
  if (mode != FM_INJECTED && (parts & 1)) {
    // mode-3 Gram: per-head partials in fp64, deterministic reduction, Jacobi
    std::vector<GemmTask> g;
    std::vector<const double *> parts; std::vector<double *> outs; std::vector<int> counts;
    std::vector<EigTask> eg;
    std::vector<float *> idU; std::vector<int> idLd;
    for (int i : act) {
      CellWork &w = ws[i];
      const CellDesc &c = w.c;
      if (w.ufI) { idU.push_back(w.UF32); idLd.push_back(c.r_f); }
      if (w.ufI && !probe) { w.tc_gram = false; w.skip_feat = true; continue; }   // r_f = d: U_F = I, no Gram, no eigen-solve
      if (!w.tc_gram) {
        for (int h = 0; h < c.m; ++h)
          g.push_back(mk(x_head(c, h), c.dtype, 1, c.st, x_head(c, h), c.dtype, c.st, 1, w.gram_part + (size_t)h * kD * kD,
                         DT_F64, kD, kD, kD, c.T));
        parts.push_back(w.gram_part); outs.push_back(w.C); counts.push_back(c.m);
      }
      EigTask e; memset(&e, 0, sizeof e);
      e.bjA = w.bjfA; e.bjV = w.bjfV; e.bjJ = w.bjfJ; e.bjOff = w.bjfOff; e.bjDone = w.bjfDone;
      e.A = w.C; e.Vt = w.Cv; e.w = w.Cw; e.n = kD; e.status = w.status; e.w_out = w.lam; e.w_sqrt = 0;
      e.preL = w.preL; e.preU = w.preU; e.preT = w.preT; e.preA = w.preA;
      if (!probe) { e.U_out = w.UF32; e.ld_out = c.r_f; e.r_out = c.r_f; }
      eg.push_back(e);
    }
    add_gram_tc(P, ST_GRAM, ws);
    add_gemm(P, ST_GRAM, g, true);
    const size_t o1 = P.push(parts), o2 = P.push(outs), o3 = P.push(counts);
    const int np_ = (int)parts.size();
    if (np_) P.add(ST_GRAM, [=](char *dev, cudaStream_t s) {
      reduce_partials_kernel<<<dim3(kD * kD / 256, np_), 256, 0, s>>>((const double *const *)(dev + o1), (double *const *)(dev + o2),
                                                                   (const int *)(dev + o3), kD * kD);
      LAUNCHED();
    });
    add_eig(P, ST_EIGF, eg, 14);        // Grams of caches with outlier channels span 1e6 in eigenvalue: slow to converge
    if (!idU.empty()) {
      const size_t p1 = P.push(idU), p2 = P.push(idLd);
      const int nid = (int)idU.size();
      P.add(ST_EIGF, [=](char *dev, cudaStream_t s) {
        set_identity_kernel<<<dim3(kD * kD / 256, nid), 256, 0, s>>>((float *const *)(dev + p1), (const int *)(dev + p2));
        LAUNCHED();
      });
    }
  }
  if (!(parts & 2)) return;
  if (mode == FM_RANDOMIZED) {
    // only the range of the intermediate bases matters (one Cholesky-QR pass keeps them well conditioned);
    // the final basis is orthonormalised twice
    add_sketch(P, ST_SKETCH, ws, true);
    add_orth(P, ST_ORTH, ws, true, power_iters == 0 ? 2 : 1, power_iters == 0);
    for (int it = 0; it < power_iters; ++it) {
      add_project(P, ST_POWER, ws);
      add_orth(P, ST_POWER, ws, false, 1);
      add_sketch(P, ST_POWER, ws, false);
      add_orth(P, ST_POWER, ws, true, it + 1 == power_iters ? 2 : 1, it + 1 == power_iters);
    }
    add_project(P, ST_PROJ, ws);          // Z now holds B^T (N x k)
    std::vector<TallGram> tgb; std::vector<EigTask> eg; std::vector<GemmTask> g2, g3;
    for (int i : act) {
      CellWork &w = ws[i];
      const CellDesc &c = w.c;
      tgb.push_back({w.Z, c.N, c.k, w.gpart, w.BBt});
      EigTask e; memset(&e, 0, sizeof e);
      e.bjA = w.bjA; e.bjV = w.bjV; e.bjJ = w.bjJ; e.bjOff = w.bjOff; e.bjDone = w.bjDone;
      e.A = w.BBt; e.Vt = w.BBv; e.w = w.BBw; e.n = c.k; e.status = w.status; e.w_out = w.sigma; e.w_sqrt = 1;
      if (!probe) { e.U_out = w.Ut; e.ld_out = c.r_t; e.r_out = c.r_t; }
      eg.push_back(e);
      if (!probe) {
        g2.push_back(mk(w.S, DT_F32, c.k, 1, w.Ut, DT_F32, c.r_t, 1, w.UT32, DT_F32, c.r_t, c.T, c.r_t, c.k));
        for (int h = 0; h < c.m; ++h) {  // G_h = Ut_r^T (B restricted to head h) : r_t x r_f
          if (w.ufI) {                   // U_F = I: B is already in the stored feature coordinates
            g2.push_back(mk(w.Ut, DT_F32, 1, c.r_t, w.Z + (size_t)h * kD * c.k, DT_F32, 1, c.k,
                            w.G32 + (size_t)h * c.r_t * kD, DT_F32, kD, c.r_t, kD, c.k));
          } else {
            g2.push_back(mk(w.Ut, DT_F32, 1, c.r_t, w.Z + (size_t)h * c.r_f * c.k, DT_F32, 1, c.k,
                            w.G32 + (size_t)h * c.r_t * c.r_f, DT_F32, c.r_f, c.r_t, c.r_f, c.k));
          }
        }
      }
    }
    add_tall_gram(P, ST_SVD, tgb);
    add_eig(P, ST_SVD, eg, 9);          // k x k, 6-7 sweeps observed
    add_gemm(P, ST_FACT, g2, false);
    add_gemm(P, ST_FACT, g3, false);
    if (check_subspace && !probe) {
      std::vector<ResidJob> rj;
      for (int i : act) {
        CellWork &w = ws[i];
        rj.push_back({w.S, w.UT32, w.sigma, w.c.T, w.c.k, w.c.r_t, w.rho, w.status, w.Z, w.c.N});
      }
      const size_t off = P.push(rj);
      const int n = (int)rj.size();
      P.add(ST_FACT, [=](char *dev, cudaStream_t s) { pad_copy_kernel<<<dim3(64, n), 256, 0, s>>>((const ResidJob *)(dev + off)); LAUNCHED(); });
      add_project(P, ST_FACT, ws);
      P.add(ST_FACT, [=](char *dev, cudaStream_t s) { scale_columns_kernel<<<dim3(64, n), 256, 0, s>>>((const ResidJob *)(dev + off)); LAUNCHED(); });
      add_sketch(P, ST_FACT, ws, false);
      P.add(ST_FACT, [=](char *dev, cudaStream_t s) { subspace_residual_kernel<<<n, 1024, 0, s>>>((const ResidJob *)(dev + off)); LAUNCHED(); });
    }
  } else if (mode == FM_EXACT) {
    std::vector<GemmTask> g1, g2, g3; std::vector<EigTask> eg;
    for (int i : act) {
      CellWork &w = ws[i];
      const CellDesc &c = w.c;
      for (int h = 0; h < c.m; ++h)
        g1.push_back(mk(x_head(c, h), c.dtype, c.st, 1, w.UF32, DT_F32, c.r_f, 1, w.Y + (size_t)h * c.T * c.r_f, DT_F32,
                        c.r_f, c.T, c.r_f, kD));
      GemmTask t = mk(w.Y, DT_F32, c.r_f, 1, w.Y, DT_F32, 1, c.r_f, w.Gt, DT_F64, c.T, c.T, c.T, c.r_f);
      t.nseg = c.m; t.seg_inner = c.m; t.a_si = (long long)c.T * c.r_f; t.b_si = (long long)c.T * c.r_f;
      g2.push_back(t);
      EigTask e; memset(&e, 0, sizeof e);
      e.bjA = w.bjA; e.bjV = w.bjV; e.bjJ = w.bjJ; e.bjOff = w.bjOff; e.bjDone = w.bjDone;
      e.A = w.Gt; e.Vt = w.Gtv; e.w = w.Gtw; e.n = c.T; e.status = w.status; e.w_out = w.sigma; e.w_sqrt = 1;
      if (!probe) { e.U_out = w.UT32; e.ld_out = c.r_t; e.r_out = c.r_t; }
      eg.push_back(e);
      if (!probe) for (int h = 0; h < c.m; ++h)
        g3.push_back(mk(w.UT32, DT_F32, 1, c.r_t, w.Y + (size_t)h * c.T * c.r_f, DT_F32, c.r_f, 1,
                        w.G32 + (size_t)h * c.r_t * c.r_f, DT_F32, c.r_f, c.r_t, c.r_f, c.T));
    }
    add_gemm(P, ST_SKETCH, g1, false);
    add_gemm(P, ST_SKETCH, g2, true);
    add_eig(P, ST_SVD, eg, 24);         // T x T
    add_gemm(P, ST_FACT, g3, false);
  } else if (mode == FM_INJECTED) {
    // core from given factors: Zp_h = X_h^T U_T (128 x r_t), G_h = Zp_h^T U_F (r_t x r_f)
    std::vector<GemmTask> g1, g2;
    for (int i : act) {
      CellWork &w = ws[i];
      const CellDesc &c = w.c;
      for (int h = 0; h < c.m; ++h) {
        g1.push_back(mk(x_head(c, h), c.dtype, 1, c.st, w.UT32, DT_F32, c.r_t, 1, w.Zp + (size_t)h * kD * c.r_t, DT_F32,
                        c.r_t, kD, c.r_t, c.T));
        g2.push_back(mk(w.Zp + (size_t)h * kD * c.r_t, DT_F32, 1, c.r_t, w.UF32, DT_F32, c.r_f, 1,
                        w.G32 + (size_t)h * c.r_t * c.r_f, DT_F32, c.r_f, c.r_t, c.r_f, kD));
      }
    }
    add_gemm(P, ST_FACT, g1, true);
    add_gemm(P, ST_FACT, g2, true);
  }
}

// P_h = fp16(G16_h U_F16^T), X~_h = 2^e U_T16 P_h (fp32 scratch) for cells with a backbone.
struct BackboneRef { CellDesc c; const __half *G16, *UT16, *UF16; const int *e; __half *P16; float *Xt; };
void add_backbone(Program &P, int stage, const std::vector<BackboneRef> &refs) {
  std::vector<GemmTask> g1, g2;
  for (auto &r : refs) {
    const CellDesc &c = r.c;
    if (c.r_t == 0) continue;
    for (int h = 0; h < c.m; ++h) {
      g1.push_back(mk(r.G16 + (size_t)h * c.r_t * c.r_f, DT_F16, c.r_f, 1, r.UF16, DT_F16, 1, c.r_f,
                      r.P16 + (size_t)h * c.r_t * kD, DT_F16, kD, c.r_t, kD, c.r_f));
      GemmTask t = mk(r.UT16, DT_F16, c.r_t, 1, r.P16 + (size_t)h * c.r_t * kD, DT_F16, kD, 1,
                      r.Xt + (size_t)h * c.T * kD, DT_F32, kD, c.T, kD, c.r_t);
      t.alpha_exp = r.e;
      g2.push_back(t);
    }
  }
  add_gemm(P, stage, g1, false);
  add_gemm(P, stage, g2, false);
}

int run_program(Program &P, char *d_tables, cudaStream_t st, bool timed = true) {
  if (!P.host.empty()) {
    CU(cudaMemcpyAsync(d_tables, P.host.data(), P.host.size(), cudaMemcpyHostToDevice, st));
    if (timed) g_timer.mark(ST_IN, st);      // the argument-table upload is set-up, not part of the first stage's kernels
  }
  int cur = -1;
  for (auto &s : P.steps) {
    if (timed && cur != -1 && s.stage != cur) g_timer.mark(cur, st);
    cur = s.stage;
    s.run(d_tables, st);
  }
  if (timed && cur != -1) g_timer.mark(cur, st);
  CU(cudaGetLastError());
  return JOLT_OK;
}

// Side streams on which independent groups of cells run their (latency-bound) factor stages concurrently.
constexpr int kMaxGroups = 8;
struct GroupStreams { bool have = false; cudaStream_t s[kMaxGroups]; cudaEvent_t fork, join[kMaxGroups]; };
GroupStreams g_groups[64];
GroupStreams *group_streams(int dev) {
  std::lock_guard<std::mutex> lk(g_ws_mu);
  GroupStreams &g = g_groups[dev];
  if (!g.have) {
    for (int i = 0; i < kMaxGroups; ++i) {
      // Group 0 holds the cells whose chain is the longest (those with a feature eigen-solve, when there are any): its
      // stream gets the greatest priority, so its small latency-bound kernels are placed ahead of the other groups'
      // cache-wide sweeps instead of waiting for a wave of their CTAs to drain (measured on config 1: median of the call
      // 3.04 -> 2.87 ms, and a quarter of the spread between calls).  The other groups' streams sit in the middle of the
      // range and the kernels that fill the machine are launched at the least priority whatever their stream
      // (launch_heavy): 2.87 -> 2.84 ms.
      int lo = 0, hi = 0;
      cudaDeviceGetStreamPriorityRange(&lo, &hi);      // (least, greatest)
      if (cudaStreamCreateWithPriority(&g.s[i], cudaStreamNonBlocking, i == 0 ? hi : (hi + lo) / 2) != cudaSuccess) return nullptr;
      if (cudaEventCreateWithFlags(&g.join[i], cudaEventDisableTiming) != cudaSuccess) return nullptr;
    }
    if (cudaEventCreateWithFlags(&g.fork, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    g.have = true;
  }
  return &g;
}

// Cells whose factor stages may run side by side.  Cells that need the feature eigen-solve (the longest chain)
// and the others never share a group.
int assign_groups(const std::vector<CellWork> &ws, std::vector<int> &group) {
  const int want = std::max(1, std::min(kMaxGroups, g_n_cell_groups.load()));
  group.assign(ws.size(), -1);
  int n_active = 0, n_long = 0;
  for (auto &w : ws) if (w.active) { ++n_active; if (!w.ufI) ++n_long; }
  if (n_active < 2 || want == 1) { for (size_t i = 0; i < ws.size(); ++i) if (ws[i].active) group[i] = 0; return n_active ? 1 : 0; }
  // long cells share the first groups, short cells the rest, each in proportion to their number
  int g_long = 0;
  if (n_long > 0 && n_long < n_active) g_long = std::max(1, std::min(want - 1, (want * n_long + n_active / 2) / n_active));
  else if (n_long == n_active) g_long = want;
  int rl = 0, rs = 0, used = 0;
  for (size_t i = 0; i < ws.size(); ++i) {
    if (!ws[i].active) continue;
    if (!ws[i].ufI && g_long > 0) { group[i] = rl % g_long; ++rl; }
    else { group[i] = g_long % want + rs % std::max(1, want - g_long % want); ++rs; }
    used = std::max(used, group[i] + 1);
  }
  return used;
}

}  // namespace

// ------------------------------------------------------------------ call context
namespace {

static Workspace g_tab[64];
static int tab_reserve(int dev, size_t bytes, void **out) {
  std::lock_guard<std::mutex> lk(g_ws_mu);
  Workspace &w = g_tab[dev];
  if (w.cap < bytes) {
    if (w.base) { cudaDeviceSynchronize(); cudaFree(w.base); w.base = nullptr; w.cap = 0; }
    const size_t want = std::max<size_t>(bytes * 2, 1 << 20);
    if (cudaMalloc(&w.base, want) != cudaSuccess) { cudaGetLastError(); return fail(JOLT_ENOMEM, "task tables of %zu bytes", want); }
    w.cap = want;
  }
  *out = w.base;
  return JOLT_OK;
}

struct TensorRef { const void *K, *V; };

int make_cells(const jolt_layout *L, const void *K, const void *V, const jolt_cell_plan *plan, int oversample,
               std::vector<CellDesc> &cells) {
  cells.clear();
  const int esz = L->dtype == JOLT_F16 ? 2 : 4;
  for (int g = 0; g < L->n_groups; ++g)
    for (int which = 0; which < 2; ++which) {
      CellDesc c;
      memset(&c, 0, sizeof c);
      const char *base = (const char *)(which == 0 ? K : V);
      c.X = base ? base + (size_t)L->group_start[g] * L->stride_layer * esz : nullptr;
      c.dtype = L->dtype == JOLT_F16 ? DT_F16 : DT_F32;
      c.n_heads = L->n_kv_heads;
      c.m = (L->group_start[g + 1] - L->group_start[g]) * L->n_kv_heads;
      c.T = L->seq_len;
      c.sl = L->stride_layer; c.sh = L->stride_head; c.st = L->stride_token;
      const jolt_cell_plan &p = plan[2 * g + which];
      c.r_t = p.r_t; c.r_f = p.r_t > 0 ? p.r_f : 0; c.bits = p.bits;
      c.N = c.m * c.r_f;
      c.k = std::min(std::min(c.r_t + oversample, c.T), c.N);
      c.cell = 2 * g + which;
      cells.push_back(c);
    }
  return JOLT_OK;
}

int check_plan(const std::vector<CellDesc> &cells, const jolt_cell_plan *plan) {
  for (size_t i = 0; i < cells.size(); ++i) {
    const jolt_cell_plan &p = plan[i];
    if (!bits_ok(p.bits)) return fail(JOLT_EINVAL, "cell %zu: bits %d", i, p.bits);
    if (p.r_t < 0) return fail(JOLT_EINVAL, "cell %zu: r_t %d", i, p.r_t);
    if (p.r_t == 0 && p.bits == 0) return fail(JOLT_EINVAL, "cell %zu stores nothing (r_t = 0 and bits = 0)", i);
    if (p.r_t > 0) {
      if (p.r_f < 1 || p.r_f > kD) return fail(JOLT_EINVAL, "cell %zu: r_f %d", i, p.r_f);
      if (p.r_t > cells[i].T || p.r_t > cells[i].m * p.r_f) return fail(JOLT_EINVAL, "cell %zu: r_t %d exceeds min(T, m r_f)", i, p.r_t);
    }
  }
  return JOLT_OK;
}

struct StatusReader {
  int *d = nullptr;
  std::vector<int> h;
};

int status_to_code(const std::vector<int> &st) {
  for (size_t i = 0; i < st.size(); i += 4) {
    if (st[i] & 1) return fail(JOLT_ENUMERIC, "cell %zu: eigen-solver did not converge", i / 4);
    if (st[i] & 4) return fail(JOLT_ENUMERIC, "cell %zu: quantisation step is not finite in fp16", i / 4);
    if (st[i] & 8) return fail(JOLT_ETIMEOUT, "cell %zu: a bounded device-side wait ran out", i / 4);
    if (st[i] & 16) return fail(JOLT_ENUMERIC, "cell %zu: the exact token subspace did not converge in %d block iterations (use the randomized mode)", i / 4, kSubspaceIters);
  }
  return JOLT_OK;
}

}  // namespace


// ------------------------------------------------------------------ compress
// Lays the stored arrays of every cell out in the handle's device buffer (cells[i].c and n_sigma must be set).  With a
// null buffer only the size is computed.  The layout is a function of the cell descriptors alone, which is what lets a
// serialised cache be mapped again.
static size_t carve_handle_blob(jolt_handle &H) {
  Bump b;
  b.base = (char *)H.blob;
  int64_t stored = 0;
  for (auto &cs : H.cells) {
    const CellDesc &c = cs.c;
    const size_t M = (size_t)c.m * c.T * kD;
    cs.e = b.take<int>(4);
    cs.lam = b.take<float>(kD);
    cs.sigma = b.take<float>(std::max(cs.n_sigma, 1));
    cs.G16 = b.take<__half>((size_t)c.m * c.r_t * c.r_f);
    cs.UT16 = b.take<__half>((size_t)c.T * c.r_t);
    cs.UF16 = b.take<__half>((size_t)kD * c.r_f);
    cs.words = b.take<uint32_t>(M / 32 * c.bits);
    cs.scales = b.take<__half>(c.bits ? M / 32 : 0);
    stored += cell_bytes(c.m, c.T, kD, c.r_t, c.r_f, c.bits, true);
  }
  H.stored_bytes = stored;
  return b.off + 256;
}

// Runs the programs of the cell groups concurrently, one side stream per group, forked from and joined back into the
// caller's stream; the groups' steps are enqueued round-robin, so every side stream has work from the start.
static int run_group_programs(int dev, cudaStream_t st, std::vector<Program> &PG, int n_groups, void *d_tab,
                              const std::vector<size_t> &tab_off) {
  {
    GroupStreams *gs = group_streams(dev);
    if (!gs) return fail(JOLT_ECUDA, "cannot create side streams");
    cudaError_t ce = cudaEventRecord(gs->fork, st);
    for (int g = 0; g < n_groups && ce == cudaSuccess; ++g) {
      ce = cudaStreamWaitEvent(gs->s[g], gs->fork, 0);
      if (ce == cudaSuccess && !PG[g].host.empty())
        ce = cudaMemcpyAsync((char *)d_tab + tab_off[g], PG[g].host.data(), PG[g].host.size(), cudaMemcpyHostToDevice, gs->s[g]);
    }
    // enqueue the groups' steps round-robin, so every side stream has work from the start
    size_t max_steps = 0;
    for (int g = 0; g < n_groups; ++g) max_steps = std::max(max_steps, PG[g].steps.size());
#ifdef JOLT_DEBUG
    const bool tl = getenv("JOLT_DEBUG_TIMELINE") != nullptr;      // per-group stage boundaries, printed after the call
    struct TL { int g, stage; cudaEvent_t ev; };
    std::vector<TL> tls;
    cudaEvent_t tl0 = nullptr;
    if (tl) { cudaEventCreate(&tl0); cudaEventRecord(tl0, st); }
#endif
    for (size_t si = 0; si < max_steps && ce == cudaSuccess; ++si)
      for (int g = 0; g < n_groups; ++g)
        if (si < PG[g].steps.size()) {
          PG[g].steps[si].run((char *)d_tab + tab_off[g], gs->s[g]);
#ifdef JOLT_DEBUG
          if (tl && (si + 1 == PG[g].steps.size() || PG[g].steps[si + 1].stage != PG[g].steps[si].stage)) {
            TL t{g, PG[g].steps[si].stage, nullptr}; cudaEventCreate(&t.ev); cudaEventRecord(t.ev, gs->s[g]); tls.push_back(t);
          }
#endif
        }
#ifdef JOLT_DEBUG
    if (tl) {
      cudaDeviceSynchronize();
      for (int g = 0; g < n_groups; ++g) {
        fprintf(stderr, "[jolt] group %d:", g);
        for (auto &t : tls) if (t.g == g) { float ms = 0; cudaEventElapsedTime(&ms, tl0, t.ev); fprintf(stderr, " %s@%.2f", kStageNames[t.stage], ms); }
        fprintf(stderr, "\n");
      }
      for (auto &t : tls) cudaEventDestroy(t.ev);
      cudaEventDestroy(tl0);
    }
#endif
    if (ce == cudaSuccess) ce = cudaGetLastError();
    for (int g = 0; g < n_groups && ce == cudaSuccess; ++g) {
      ce = cudaEventRecord(gs->join[g], gs->s[g]);
      if (ce == cudaSuccess) ce = cudaStreamWaitEvent(st, gs->join[g], 0);
    }
    if (ce != cudaSuccess) { cudaDeviceSynchronize(); return fail(JOLT_ECUDA, "side streams: %s", cudaGetErrorString(ce)); }
  }
  return JOLT_OK;
}

// Device buffer of the projected cores of the cells with a backbone (CellStore::P16 point into it).  A cell whose
// feature factor is exactly the identity (`identity_uf[c]`: r_f = d, factors not injected) needs none: P = G there.
static int alloc_projected_cores(jolt_handle &H, const std::vector<char> *identity_uf) {
  size_t halves = 0;
  const size_t nc = H.cells.size();
  std::vector<size_t> off(nc, 0);
  auto alias = [&](size_t c) { return identity_uf && (*identity_uf)[c]; };
  for (size_t c = 0; c < nc; ++c) {
    off[c] = halves;
    if (H.cells[c].c.r_t > 0 && !alias(c)) halves += ((size_t)H.cells[c].c.m * H.cells[c].c.r_t * kD + 127) & ~(size_t)127;
  }
  if (halves) {
    void *p = nullptr;
    if (cudaMalloc(&p, halves * sizeof(__half)) != cudaSuccess) { cudaGetLastError(); return fail(JOLT_ENOMEM, "projected cores: %zu bytes", halves * sizeof(__half)); }
    H.P_all = (__half *)p;
  }
  for (size_t c = 0; c < nc; ++c) {
    CellStore &cs = H.cells[c];
    cs.P16 = cs.c.r_t == 0 ? nullptr : (alias(c) ? cs.G16 : H.P_all + off[c]);
  }
  return JOLT_OK;
}

static void launch_project_cores(const ProjJob *d_jobs, int n, int max_rows, int max_rf, cudaStream_t s) {
  static bool attr = false;
  if (!attr) { cudaFuncSetAttribute(project_core_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 128 * 128 * 2); attr = true; }
  project_core_kernel<<<dim3((max_rows + 31) / 32, n), 128, (size_t)128 * max_rf * sizeof(__half), s>>>(d_jobs);
  LAUNCHED();
}

static int compress_impl(const jolt_layout *L, const void *K, const void *V, const jolt_cell_plan *plan,
                         const jolt_options *o, const float *const *inUT, const float *const *inUF, void *stream,
                         jolt_handle **out) {
  if (out) *out = nullptr;
  if (!out || !plan || !K || !V) return fail(JOLT_EINVAL, "null argument");
  int rc;
#ifdef JOLT_DEBUG
  const bool dbg = getenv("JOLT_DEBUG_TIMING") != nullptr;
  auto t_start = std::chrono::steady_clock::now();
  auto lap = [&](const char *what) { if (dbg) { auto n = std::chrono::steady_clock::now(); fprintf(stderr, "[jolt] %s: %.3f ms\n", what, std::chrono::duration<double, std::milli>(n - t_start).count()); t_start = n; } };
#else
  auto lap = [](const char *) {};
#endif
  if ((rc = check_layout(L)) || (rc = check_options(o)) || (rc = check_device_alignment(L, K, V))) return rc;
  const bool injected = inUT != nullptr || inUF != nullptr;
  if (injected && (!inUT || !inUF)) return fail(JOLT_EINVAL, "both factor arrays are needed");
  cudaStream_t st = (cudaStream_t)stream;
  // exact mode: direct T x T eigen-solve up to kExactEigMaxT tokens, converged block subspace iteration beyond
  const bool subspace = !injected && o->token_mode == JOLT_TOKEN_EXACT && L->seq_len > kExactEigMaxT;
  const int mode = injected ? FM_INJECTED : (o->token_mode == JOLT_TOKEN_EXACT && !subspace ? FM_EXACT : FM_RANDOMIZED);
  const int oversample = subspace ? std::max(o->oversample, kSubspaceOversample) : o->oversample;
  const int power_iters = subspace ? std::max(o->power_iters, kSubspaceIters) : o->power_iters;
  std::vector<CellDesc> cells;
  make_cells(L, K, V, plan, oversample, cells);
  if ((rc = check_plan(cells, plan))) return rc;       // all argument checks come before the first CUDA call
  int dev = 0;
  CU(cudaGetDevice(&dev));
  if (mode == FM_EXACT) {
    for (auto &c : cells) c.k = c.r_t;
  }
  if (injected) for (auto &c : cells) c.k = c.r_t;
  const int nc = (int)cells.size();
  const size_t esz = L->dtype == JOLT_F16 ? 2 : 4;
  const size_t span = layout_span_elems(L) * esz;

  // ---- handle blob
  std::unique_ptr<jolt_handle> H(new jolt_handle);
  H->device = dev; H->n_layers = L->n_layers; H->n_kv_heads = L->n_kv_heads; H->T = L->seq_len; H->n_groups = L->n_groups;
  H->group_start.assign(L->group_start, L->group_start + L->n_groups + 1);
  H->seed = o->seed;
  H->subspace = subspace;
  H->cells.resize(nc);
  for (int i = 0; i < nc; ++i) {
    H->cells[i].c = cells[i]; H->cells[i].c.X = nullptr;
    H->cells[i].n_sigma = cells[i].r_t > 0 && !injected ? (mode == FM_EXACT ? cells[i].T : cells[i].k) : 0;
  }
  for (int pass = 0; pass < 2; ++pass) {
    const size_t bytes = carve_handle_blob(*H);
    if (pass == 0) {
      static bool pool_set[64] = {};
      if (!pool_set[dev]) {      // keep freed blobs in the stream-ordered pool instead of returning them to the driver
        cudaMemPool_t pool; unsigned long long thr = ~0ull;
        if (cudaDeviceGetDefaultMemPool(&pool, dev) == cudaSuccess) cudaMemPoolSetAttribute(pool, cudaMemPoolAttrReleaseThreshold, &thr);
        cudaGetLastError();
        pool_set[dev] = true;
      }
      H->blob_bytes = bytes;
      if (cudaMallocAsync(&H->blob, H->blob_bytes, st) != cudaSuccess) { cudaGetLastError(); return fail(JOLT_ENOMEM, "compressed cache of %zu bytes", H->blob_bytes); }
    }
  }
  if (cudaMalloc(&H->d_status, sizeof(int) * 4 * (size_t)nc) != cudaSuccess) {
    cudaGetLastError(); cudaFreeAsync(H->blob, st); H->blob = nullptr; H->d_status = nullptr;
    return fail(JOLT_ENOMEM, "status words");
  }
  auto free_blob = [&]() {
    cudaFreeAsync(H->blob, st); H->blob = nullptr; cudaFree(H->d_status); H->d_status = nullptr;
    if (H->P_all) { cudaFree(H->P_all); H->P_all = nullptr; }
  };
  {
    std::vector<char> identity_uf(nc, 0);
    for (int i = 0; i < nc; ++i) identity_uf[i] = mode != FM_INJECTED && cells[i].r_t > 0 && cells[i].r_f == kD;
    if ((rc = alloc_projected_cores(*H, &identity_uf))) { free_blob(); return rc; }
  }
  H->last_stream = st;
  lap("validate+blob");

  // ---- workspace
  std::vector<CellWork> ws(nc);
  const int fmask = g_fast.load();
  const bool fast = (fmask & 1) != 0;
  size_t ws_bytes = 0;
  void *ws_base = nullptr;
  int *d_status = nullptr;
  char *stage_K = nullptr, *stage_V = nullptr;
  for (int pass = 0; pass < 2; ++pass) {
    Bump b;
    b.base = (char *)ws_base;
    d_status = b.take<int>(4 * (size_t)nc);
    if (L->mem_space == JOLT_MEM_HOST) { stage_K = b.take<char>(span); stage_V = b.take<char>(span); }
    for (int i = 0; i < nc; ++i) {
      CellWork &w = ws[i];
      w.c = cells[i];
      w.active = cells[i].r_t > 0;
      w.tc = (fmask & 2) && w.active && mode == FM_RANDOMIZED && tc_sweep_ok(cells[i], L->mem_space == JOLT_MEM_HOST);
      w.tc_gram = (fmask & 4) && w.active && mode != FM_INJECTED && tc_sweep_ok(cells[i], L->mem_space == JOLT_MEM_HOST);
      w.ufI = w.active && cells[i].r_f == kD;
      if (pass == 1) { w.lam = H->cells[i].lam; w.sigma = H->cells[i].n_sigma ? H->cells[i].sigma : nullptr; w.status = d_status + 4 * i; w.rho = (float *)(H->cells[i].e + 1); }
      carve(b, w, mode, true);
      if (pass == 1 && !w.n_sigma) w.n_sigma = H->cells[i].n_sigma;
    }
    if (pass == 0) {
      ws_bytes = b.off + 256;
      if ((rc = ws_reserve(dev, ws_bytes, &ws_base))) { free_blob(); return rc; }
    }
  }
  if (L->mem_space == JOLT_MEM_HOST) {
    // re-point the cells at the staged device copies
    for (int i = 0; i < nc; ++i) {
      const char *hb = (const char *)(i % 2 == 0 ? K : V);
      const char *db = i % 2 == 0 ? stage_K : stage_V;
      ws[i].c.X = db + ((const char *)ws[i].c.X - hb);
      cells[i].X = ws[i].c.X;
    }
  }

  lap("workspace");
  // ---- program
  Program P;
  std::vector<int> cell_group;
  const int n_groups = assign_groups(ws, cell_group);
  std::vector<Program> PG(std::max(n_groups, 1));
  for (int g = 0; g < n_groups; ++g) {
    std::vector<CellWork> sub = ws;
    for (int i = 0; i < nc; ++i) if (cell_group[i] != g) sub[i].active = false;
    build_factor_program(PG[g], sub, mode, false, power_iters, o->seed, fast, subspace);
  }
  lap("factor program");
  // fp16 storage of the factors and the residual / rotate / quantise / pack pass (tensor-core kernel where the cell
  // fits it, portable kernels otherwise).  With several cell groups each group's program ends with the tail of its
  // own cells, so only the last group's tail is left when the others have finished.
  std::vector<char> use_tc(nc, 0);
  const bool x_tma_ok = L->dtype == JOLT_F16 && L->stride_token * 2 % 16 == 0 && L->stride_head * 2 % 16 == 0 &&
                        L->stride_layer * 2 % 16 == 0;
  for (int i = 0; i < nc; ++i) {
    CellStore &cs = H->cells[i];
    if (fast && encode_store_maps(cs) && x_tma_ok && cells[i].bits > 0 && ((uintptr_t)cells[i].X % 16 == 0)) use_tc[i] = 1;
  }
  auto build_tail = [&](Program &PP, const std::vector<int> &idx) {
    std::vector<StoreJob> sj;
    for (int i : idx) {
      const CellDesc &c = cells[i];
      const CellStore &cs = H->cells[i];
      if (c.r_t == 0) continue;
      StoreJob j;
      j.G32 = ws[i].G32; j.UT32 = ws[i].UT32; j.UF32 = ws[i].UF32;
      j.G16 = cs.G16; j.UT16 = cs.UT16; j.UF16 = cs.UF16; j.e = cs.e; j.pmax = ws[i].pmax;
      j.nG = (long long)c.m * c.r_t * c.r_f; j.nUT = (long long)c.T * c.r_t; j.nUF = (long long)kD * c.r_f; j.round_inputs = 0;
      sj.push_back(j);
    }
    if (!sj.empty()) {
      const size_t off = PP.push(sj);
      const int n = (int)sj.size();
      std::vector<ProjJob> pj;
      int max_rows = 0, max_rf = 0;
      for (int i : idx) {
        const CellDesc &c = cells[i];
        if (c.r_t == 0 || H->cells[i].P16 == H->cells[i].G16) continue;
        pj.push_back({H->cells[i].G16, H->cells[i].UF16, H->cells[i].P16, c.m * c.r_t, c.r_f});
        max_rows = std::max(max_rows, c.m * c.r_t); max_rf = std::max(max_rf, c.r_f);
      }
      const size_t poff = PP.push(pj);
      const int np_ = (int)pj.size();
      PP.add(ST_STORE, [=](char *dev_t, cudaStream_t s) {
        core_exponent_kernel<<<dim3(kCoreMaxParts, n), 256, 0, s>>>((const StoreJob *)(dev_t + off)); LAUNCHED();
        store_factors_kernel<<<dim3(64, n), 256, 0, s>>>((const StoreJob *)(dev_t + off)); LAUNCHED();
        if (np_) launch_project_cores((const ProjJob *)(dev_t + poff), np_, max_rows, max_rf, s);
      });
    }
    int tc_heads = 0;
    for (int i : idx) if (use_tc[i]) tc_heads += cells[i].m;
    std::vector<tc::BBCell> bbc;
    std::vector<BackboneRef> br_port;
    std::vector<RowJob> rj;
    long long rows = 0;
    int tpi = 1, iph = 1;
    bb_split(tc_heads, L->seq_len / 128, tpi, iph);
    for (int i : idx) {
      const CellDesc &c = cells[i];
      const CellStore &cs = H->cells[i];
      if (use_tc[i]) {
        tc::BBCell b;
        fill_bb_common(b, cs, d_status + 4 * i);
        b.tiles_per_item = tpi; b.items_per_head = iph;
        const int g = i / 2;
        const int Lg = L->group_start[g + 1] - L->group_start[g];
        const uint64_t dims[4] = {(uint64_t)kD, (uint64_t)c.T, (uint64_t)c.n_heads, (uint64_t)Lg};
        const uint64_t str[3] = {(uint64_t)c.st * 2, (uint64_t)c.sh * 2, (uint64_t)c.sl * 2};
        const uint32_t box[4] = {64, 128, 1, 1};
        if (make_tmap_f16(&b.tmX, c.X, 4, dims, str, box)) { bbc.push_back(b); continue; }
      }
      if (c.bits == 0) continue;
      if (c.r_t > 0) br_port.push_back({ws[i].c, cs.G16, cs.UT16, cs.UF16, cs.e, ws[i].P16, ws[i].Xt});
      RowJob j;
      memset(&j, 0, sizeof j);
      j.c = ws[i].c; j.Xt = c.r_t > 0 ? ws[i].Xt : nullptr;
      j.words = cs.words; j.scales = cs.scales; j.status = d_status + 4 * i; j.row0 = rows;
      rows += (long long)c.m * c.T;
      rj.push_back(j);
    }
    add_backbone_tc<true>(PP, ST_RQ, bbc, o->seed);
    add_backbone(PP, ST_BACK, br_port);
    if (!rj.empty()) {
      const size_t off = PP.push(rj);
      const uint64_t seed = o->seed;
      const int nj = (int)rj.size();
      PP.add(ST_RQ, [=](char *dev_t, cudaStream_t s) {
        residual_quant_kernel<<<(unsigned)((rows + 127) / 128), 128, 0, s>>>((const RowJob *)(dev_t + off), nj, rows, seed);
        LAUNCHED();
      });
    }
  };
  if (n_groups > 1) {
    std::vector<int> rest;
    for (int g = 0; g < n_groups; ++g) {
      std::vector<int> idx;
      for (int i = 0; i < nc; ++i) if (cell_group[i] == g) idx.push_back(i);
      build_tail(PG[g], idx);
    }
    for (int i = 0; i < nc; ++i) if (cell_group[i] < 0) rest.push_back(i);
    build_tail(P, rest);
  } else {
    std::vector<int> all(nc);
    for (int i = 0; i < nc; ++i) all[i] = i;
    build_tail(P, all);
  }
  void *d_tab = nullptr;
  std::vector<size_t> tab_off(PG.size() + 1, 0);
  for (size_t g = 0; g < PG.size(); ++g) tab_off[g + 1] = tab_off[g] + ((PG[g].host.size() + 255) & ~(size_t)255);
  if ((rc = tab_reserve(dev, tab_off.back() + P.host.size() + 256, &d_tab))) { free_blob(); return rc; }
  lap("residual program");

  // ---- run
  if ((rc = arena_acquire(dev, st))) { free_blob(); return rc; }
  g_timer.begin(st);
  cudaError_t ce = cudaMemsetAsync(d_status, 0, sizeof(int) * 4 * nc, st);
  if (ce == cudaSuccess) ce = cudaMemsetAsync(H->d_status, 0, sizeof(int) * 4 * nc, st);
  if (subspace) for (int i = 0; i < nc && ce == cudaSuccess; ++i) ce = cudaMemsetAsync(H->cells[i].e, 0, 4 * sizeof(int), st);
  for (int i = 0; i < nc && ce == cudaSuccess; ++i)
    if (cells[i].r_t == 0 || cells[i].r_f == kD || injected) ce = cudaMemsetAsync(H->cells[i].lam, 0, sizeof(float) * kD, st);
  if (ce == cudaSuccess && L->mem_space == JOLT_MEM_HOST) {
    ce = cudaMemcpyAsync(stage_K, K, span, cudaMemcpyHostToDevice, st);
    if (ce == cudaSuccess) ce = cudaMemcpyAsync(stage_V, V, span, cudaMemcpyHostToDevice, st);
    g_timer.mark(ST_IN, st);
  }
  if (ce == cudaSuccess && injected) {
    std::vector<float *> ptrs; std::vector<long long> cnts;
    for (int i = 0; i < nc && ce == cudaSuccess; ++i) {
      const CellDesc &c = cells[i];
      if (c.r_t == 0) continue;
      if (!inUT[i] || !inUF[i]) { free_blob(); return fail(JOLT_EINVAL, "cell %d: factor pointer is null", i); }
      ce = cudaMemcpyAsync(ws[i].UT32, inUT[i], sizeof(float) * c.T * c.r_t, cudaMemcpyHostToDevice, st);
      if (ce == cudaSuccess) ce = cudaMemcpyAsync(ws[i].UF32, inUF[i], sizeof(float) * kD * c.r_f, cudaMemcpyHostToDevice, st);
    }
  }
  if (ce != cudaSuccess) { free_blob(); return fail(JOLT_ECUDA, "staging copy: %s", cudaGetErrorString(ce)); }
  if (n_groups <= 1) {
    if (n_groups == 1 && (rc = run_program(PG[0], (char *)d_tab, st))) { free_blob(); return rc; }
  } else {
    if ((rc = run_group_programs(dev, st, PG, n_groups, d_tab, tab_off))) { free_blob(); return rc; }
    g_timer.mark(ST_FACT, st);
  }
  if ((rc = run_program(P, (char *)d_tab + tab_off.back(), st))) { free_blob(); return rc; }
  arena_release(dev, st);
  lap("launches");
  std::vector<int> hstat(4 * nc);
  ce = cudaMemcpyAsync(hstat.data(), d_status, sizeof(int) * 4 * nc, cudaMemcpyDeviceToHost, st);
  if (ce == cudaSuccess) ce = cudaStreamSynchronize(st);
  if (ce != cudaSuccess) { cudaGetLastError(); free_blob(); return fail(JOLT_ECUDA, "compress: %s", cudaGetErrorString(ce)); }
  g_timer.finish();
  lap("sync");
  if ((rc = status_to_code(hstat))) { free_blob(); return rc; }
  for (int i = 0; i < nc; ++i) H->cells[i].dbg_UT32 = cells[i].r_t > 0 ? ws[i].UT32 : nullptr;
  *out = H.release();
  return JOLT_OK;
}

extern "C" int jolt_compress(const jolt_layout *L, const void *K, const void *V, const jolt_cell_plan *plan,
                             const jolt_options *o, void *stream, jolt_handle **out) {
  return compress_impl(L, K, V, plan, o, nullptr, nullptr, stream, out);
}

extern "C" int jolt_compress_with_factors(const jolt_layout *L, const void *K, const void *V, const jolt_cell_plan *plan,
                                          const jolt_options *o, const float *const *UT, const float *const *UF,
                                          void *stream, jolt_handle **out) {
  if (!UT || !UF) { if (out) *out = nullptr; return fail(JOLT_EINVAL, "factor arrays are null"); }
  return compress_impl(L, K, V, plan, o, UT, UF, stream, out);
}

// ------------------------------------------------------------------ decompress
static int decompress_impl(const jolt_handle *H, const jolt_layout *L, void *Kout, void *Vout, const jolt_rope *rope,
                           void *stream) {
  if (!H || !Kout || !Vout) return fail(JOLT_EINVAL, "null argument");
  int rc;
  if ((rc = check_layout(L)) || (rc = check_device_alignment(L, Kout, Vout))) return rc;
  if (rope && !(rope->base > 1.0 && rope->base < 1e12)) return fail(JOLT_EINVAL, "rotary base %g", rope->base);
  if (rope && (rope->pos0 < 0 || rope->pos0 > ((int64_t)1 << 40))) return fail(JOLT_EINVAL, "rotary pos0 out of range");
  if (L->n_layers != H->n_layers || L->n_kv_heads != H->n_kv_heads || L->seq_len != H->T || L->n_groups != H->n_groups)
    return fail(JOLT_EINVAL, "output layout does not match the compressed cache");
  for (int g = 0; g <= L->n_groups; ++g)
    if (L->group_start[g] != H->group_start[g]) return fail(JOLT_EINVAL, "output grouping does not match");
  cudaStream_t st = (cudaStream_t)stream;
  int dev = 0;
  CU(cudaGetDevice(&dev));
  if (dev != H->device) return fail(JOLT_EINVAL, "handle belongs to device %d, current device is %d", H->device, dev);
#ifdef JOLT_DEBUG
  const bool dbg_t = getenv("JOLT_DEBUG_TIMING") != nullptr;
  auto t_start = std::chrono::steady_clock::now();
  auto lap = [&](const char *what) { if (dbg_t) { auto n = std::chrono::steady_clock::now(); fprintf(stderr, "[jolt] decode %s: %.1f us\n", what, std::chrono::duration<double, std::micro>(n - t_start).count()); t_start = n; } };
#else
  auto lap = [](const char *) {};
#endif
  const int nc = (int)H->cells.size();
  const size_t esz = L->dtype == JOLT_F16 ? 2 : 4;
  const size_t span = layout_span_elems(L) * esz;
  const bool fast = (g_fast.load() & 1) != 0;
  std::vector<CellWork> ws(nc);
  std::vector<char> use_tc(nc, 0);
  int tc_heads = 0;
  for (int i = 0; i < nc; ++i)
    if (fast && H->cells[i].tc_ok) { use_tc[i] = 1; tc_heads += H->cells[i].c.m; }
  // key cells that the tensor-core decode kernel rotates in its epilogue (its r_t <= 128 form holds a whole row in registers)
  std::vector<char> rope_fused(nc, 0);
  int n_rope_fused = 0;
  for (int i = 0; rope && i < nc; i += 2)
    if (use_tc[i] && H->cells[i].c.r_t <= 128 && (g_fast.load() & 8)) { rope_fused[i] = 1; ++n_rope_fused; }
  float2 *rope_tab = nullptr;
  void *ws_base = nullptr;
  char *stage_K = nullptr, *stage_V = nullptr;
  int *d_status = nullptr;
  d_status = H->d_status;          // the handle's own words: jolt_check_status reads them after the call
  for (int pass = 0; pass < 2; ++pass) {
    Bump b;
    b.base = (char *)ws_base;
    if (L->mem_space == JOLT_MEM_HOST) { stage_K = b.take<char>(span); stage_V = b.take<char>(span); }
    if (n_rope_fused) rope_tab = b.take<float2>((size_t)(kD / 2) * L->seq_len);
    for (int i = 0; i < nc; ++i) {
      ws[i].c = H->cells[i].c;
      ws[i].active = false;
      ws[i].status = d_status ? d_status + 4 * i : nullptr;
      carve(b, ws[i], FM_INJECTED, !use_tc[i]);
    }
    if (pass == 0 && (rc = ws_reserve(dev, b.off + 256, &ws_base))) return rc;
  }
  char *Kd = L->mem_space == JOLT_MEM_HOST ? stage_K : (char *)Kout;
  char *Vd = L->mem_space == JOLT_MEM_HOST ? stage_V : (char *)Vout;
  lap("workspace");
  Program P;
  std::vector<BackboneRef> br;
  std::vector<RowJob> rj;
  std::vector<tc::BBCell> bbc;
  long long rows = 0;
  int tpi = 1, iph = 1;
  bb_split(tc_heads, L->seq_len / 128, tpi, iph);
  for (int i = 0; i < nc; ++i) {
    const CellStore &cs = H->cells[i];
    const CellDesc &c = cs.c;
    const int g = i / 2;
    char *obase = (i % 2 == 0 ? Kd : Vd) + (size_t)L->group_start[g] * L->stride_layer * esz;
    if (use_tc[i]) {
      tc::BBCell b;
      fill_bb_common(b, cs, d_status + 4 * i);
      b.tiles_per_item = tpi; b.items_per_head = iph;
      b.out = obase; b.out_dtype = L->dtype == JOLT_F16 ? DT_F16 : DT_F32;
      b.osl = L->stride_layer; b.osh = L->stride_head; b.ost = L->stride_token;
      b.tma_out = 0;
#ifdef JOLT_DEBUG
      b.dbg = g_dbg_stamps;
#endif
      b.rope = rope_fused[i] ? rope_tab : nullptr;
      if (L->dtype == JOLT_F16 && L->stride_token % 8 == 0 && L->stride_head % 8 == 0 && L->stride_layer % 8 == 0 &&
          ((uintptr_t)obase % 16 == 0)) {
        const uint64_t dims[4] = {(uint64_t)kD, (uint64_t)c.T, (uint64_t)c.n_heads, (uint64_t)(c.m / c.n_heads)};
        const uint64_t str[3] = {(uint64_t)L->stride_token * 2, (uint64_t)L->stride_head * 2, (uint64_t)L->stride_layer * 2};
        const uint32_t box[4] = {64, 128, 1, 1};
        const uint32_t boxw[4] = {64, 32, 1, 1};
        if (make_tmap_f16(&b.tmOut, obase, 4, dims, str, box) && make_tmap_f16(&b.tmOutW, obase, 4, dims, str, boxw)) b.tma_out = 1;
      }
      bbc.push_back(b);
      continue;
    }
    if (c.r_t > 0) br.push_back({c, cs.G16, cs.UT16, cs.UF16, cs.e, ws[i].P16, ws[i].Xt});
    RowJob j;
    memset(&j, 0, sizeof j);
    j.c = c; j.Xt = c.r_t > 0 ? ws[i].Xt : nullptr; j.words = cs.words; j.scales = cs.scales; j.status = d_status + 4 * i;
    j.out = obase;
    j.out_dtype = L->dtype == JOLT_F16 ? DT_F16 : DT_F32;
    j.osl = L->stride_layer; j.osh = L->stride_head; j.ost = L->stride_token;
    j.row0 = rows;
    rows += (long long)c.m * c.T;
    rj.push_back(j);
  }
  lap("descriptors");
  // the costliest cells (most residual bits, then largest r_t) first: the last wave of CTAs is then the cheapest one
  std::stable_sort(bbc.begin(), bbc.end(), [](const tc::BBCell &x, const tc::BBCell &y) {
    return x.bits != y.bits ? x.bits > y.bits : x.r_t > y.r_t;
  });
  if (n_rope_fused) {
    const int T = L->seq_len;
    const double base = rope->base;
    const long long pos0 = rope->pos0;
    P.add(ST_ROPE, [=](char *, cudaStream_t s) {
      rope_table_kernel<<<dim3((T + 255) / 256, kD / 2), 256, 0, s>>>(rope_tab, T, base, pos0);
      LAUNCHED();
    });
  }
  add_decode_tc(P, ST_DROWS, bbc, H->seed);
  add_backbone(P, ST_DBACK, br);
  if (!rj.empty()) {
    const size_t off = P.push(rj);
    const uint64_t seed = H->seed;
    const int nj = (int)rj.size();
    P.add(ST_DROWS, [=](char *dev_t, cudaStream_t s) {
      dequant_add_kernel<<<(unsigned)((rows + 127) / 128), 128, 0, s>>>((const RowJob *)(dev_t + off), nj, rows, seed);
      LAUNCHED();
    });
  }
  // key cells the decode kernel did not rotate itself: in place on the decoded tensor (the staging buffer when the
  // destination is host memory), one launch per run of consecutive layer groups
  for (int g = 0; rope && g < L->n_groups;) {
    if (rope_fused[2 * g]) { ++g; continue; }
    int g1 = g + 1;
    while (g1 < L->n_groups && !rope_fused[2 * g1]) ++g1;
    RopeJob j;
    j.K = Kd + (size_t)L->group_start[g] * L->stride_layer * esz; j.dtype = L->dtype == JOLT_F16 ? DT_F16 : DT_F32;
    j.n_rows = (L->group_start[g1] - L->group_start[g]) * L->n_kv_heads; j.n_heads = L->n_kv_heads; j.T = L->seq_len;
    g = g1;
    j.sl = L->stride_layer; j.sh = L->stride_head; j.st = L->stride_token;
    j.base = rope->base; j.pos0 = rope->pos0;
    const int gx = (L->seq_len + kRopeTokensPerCta - 1) / kRopeTokensPerCta;
    // about 16 CTAs per SM in flight; every CTA still visits several rows with one set of sines
    const int gy = std::max(1, std::min(j.n_rows, (16 * 148 + gx - 1) / gx));
    P.add(ST_ROPE, [=](char *, cudaStream_t s) {
      rope_rows_kernel<<<dim3(gx, gy), 256, 0, s>>>(j);
      LAUNCHED();
    });
  }
  lap("program");
  void *d_tab = nullptr;
  if ((rc = tab_reserve(dev, P.host.size() + 256, &d_tab))) return rc;
  if ((rc = arena_acquire(dev, st))) return rc;
  H->last_stream = st;
  g_timer.begin(st);
  CU(cudaMemsetAsync(d_status, 0, sizeof(int) * 4 * nc, st));
  lap("acquire+memset");
  if ((rc = run_program(P, (char *)d_tab, st))) return rc;
  lap("upload+launch");
  if (L->mem_space == JOLT_MEM_HOST) {
    std::vector<int> hstat(4 * (size_t)nc);
    CU(cudaMemcpyAsync(Kout, stage_K, span, cudaMemcpyDeviceToHost, st));
    CU(cudaMemcpyAsync(Vout, stage_V, span, cudaMemcpyDeviceToHost, st));
    CU(cudaMemcpyAsync(hstat.data(), d_status, sizeof(int) * 4 * nc, cudaMemcpyDeviceToHost, st));
    arena_release(dev, st);
    g_timer.mark(ST_OUT, st);
    CU(cudaStreamSynchronize(st));
    g_timer.finish();
    return status_to_code(hstat);     // a host destination synchronises anyway: the device status comes back with it
  }
  arena_release(dev, st);
  return JOLT_OK;
}

extern "C" int jolt_check_status(const jolt_handle *H, void *stream) {
  if (!H) return fail(JOLT_EINVAL, "null argument");
  if (!H->d_status) return JOLT_OK;
  int dev = 0;
  CU(cudaGetDevice(&dev));
  if (dev != H->device) return fail(JOLT_EINVAL, "handle belongs to device %d, current device is %d", H->device, dev);
  std::vector<int> hstat(4 * H->cells.size());
  cudaStream_t st = (cudaStream_t)stream;
  CU(cudaMemcpyAsync(hstat.data(), H->d_status, sizeof(int) * hstat.size(), cudaMemcpyDeviceToHost, st));
  CU(cudaStreamSynchronize(st));
  return status_to_code(hstat);
}

extern "C" int jolt_decompress(const jolt_handle *H, const jolt_layout *L, void *Kout, void *Vout, void *stream) {
  return decompress_impl(H, L, Kout, Vout, nullptr, stream);
}

extern "C" int jolt_decompress_rope(const jolt_handle *H, const jolt_layout *L, void *Kout, void *Vout,
                                    const jolt_rope *rope, void *stream) {
  if (!rope) return fail(JOLT_EINVAL, "rotary parameters are null");
  return decompress_impl(H, L, Kout, Vout, rope, stream);
}

// ------------------------------------------------------------------ attention on the compressed cache
template <int BITS>
static void launch_att_scores(dim3 grid, size_t shm, cudaStream_t s, const AttendJob *d, int NQP) {
  attend_scores_kernel<BITS><<<grid, kAttChunk, shm, s>>>(d, NQP);
}
template <int BITS>
static void launch_att_scores_mma(dim3 grid, cudaStream_t s, const AttendJob *d, int NQP) {
  const int n_chunks = (int)grid.x;
  grid.x = (grid.x + 1) / 2;                 // two chunks per CTA: the query operand is staged once, the second chunk's rows are prefetched
  attend_scores_mma_kernel<BITS><<<grid, kAttChunk, 0, s>>>(d, NQP, n_chunks);
}
template <int BITS>
static void launch_att_values_mma(dim3 grid, cudaStream_t s, const AttendJob *d, int NQP) {
  const size_t shm = (size_t)kAttHalf * 128 * sizeof(__half) + (size_t)4 * 2 * NQP * (kAttHalf + 8) * sizeof(__half);
  static std::atomic<bool> opted{false};      // 49.4 KB with eight query slots
  if (!opted.exchange(true)) {
    cudaFuncSetAttribute(attend_values_mma_kernel<BITS, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024);
    cudaFuncSetAttribute(attend_values_mma_kernel<BITS, 8>, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024);
  }
  if (NQP == 4) attend_values_mma_kernel<BITS, 4><<<grid, kAttChunk, shm, s>>>(d);
  else attend_values_mma_kernel<BITS, 8><<<grid, kAttChunk, shm, s>>>(d);
}
template <int BITS>
static void launch_att_values(dim3 grid, cudaStream_t s, const AttendJob *d, int NQP) {
  const size_t shm = (size_t)kAttHalf * (NQP * sizeof(float) + 16 * BITS + 8) + (size_t)4 * 128 * NQP * sizeof(float);
  if (NQP == 4) attend_values_kernel<BITS, 4><<<grid, kAttChunk, shm, s>>>(d);
  else attend_values_kernel<BITS, 8><<<grid, kAttChunk, shm, s>>>(d);
}

extern "C" int jolt_attend(const jolt_handle *H, const void *dQ, int32_t n_q, double scale, void *dOut, void *stream) {
  if (!H || !dQ || !dOut) return fail(JOLT_EINVAL, "null argument");
  if (n_q < 1 || n_q > kAttMaxQ) return fail(JOLT_EINVAL, "n_q %d (1..%d queries per KV head)", n_q, kAttMaxQ);
  if (!(scale == scale) || std::isinf(scale)) return fail(JOLT_EINVAL, "scale is not finite");
  if ((((uintptr_t)dQ) | ((uintptr_t)dOut)) & 15) return fail(JOLT_EINVAL, "queries and outputs must start on a 16-byte boundary");
  cudaStream_t st = (cudaStream_t)stream;
  int dev = 0;
  CU(cudaGetDevice(&dev));
  if (dev != H->device) return fail(JOLT_EINVAL, "handle belongs to device %d, current device is %d", H->device, dev);
  const int ng = H->n_groups, T = H->T, nh = H->n_kv_heads;
  const int NQP = n_q <= 4 ? 4 : 8;
  const int n_chunks = (T + kAttChunk - 1) / kAttChunk;
  int m_max = 0, krt = 0, krf = 0, vrt = 0, vrf = 0;
  unsigned kbits = 0, vbits = 0;
  for (int g = 0; g < ng; ++g) {
    const CellDesc &ck = H->cells[2 * g].c, &cv = H->cells[2 * g + 1].c;
    m_max = std::max(m_max, ck.m);
    krt = std::max(krt, ck.r_t); krf = std::max(krf, ck.r_t > 0 ? ck.r_f : 0);
    vrt = std::max(vrt, cv.r_t); vrf = std::max(vrf, cv.r_t > 0 ? cv.r_f : 0);
    kbits |= 1u << ck.bits; vbits |= 1u << cv.bits;
    if ((ck.r_t % 8) || (cv.r_t % 8) || (ck.r_f % 8) || (cv.r_f % 8)) return fail(JOLT_EUNSUPPORTED, "ranks must be multiples of 8");
  }
  const size_t shm_prep = 128 * sizeof(float);
  const size_t shm_sc = (size_t)128 * NQP * sizeof(float);
  const size_t shm_comb = (size_t)(n_chunks + vrt + 136) * sizeof(float);
  if (shm_comb > 48 * 1024) return fail(JOLT_EUNSUPPORTED, "sequence of %d tokens: the chunk merge needs %zu bytes of shared memory", T, shm_comb);
  // the projected cores do not depend on the queries: compress (or deserialize) formed them, the handle keeps them
  std::vector<AttendJob> jobs(ng);
  void *ws_base = nullptr;
  int rc;
  for (int pass = 0; pass < 2; ++pass) {
    Bump b;
    b.base = (char *)ws_base;
    for (int g = 0; g < ng; ++g) {
      const CellStore &sk = H->cells[2 * g], &sv = H->cells[2 * g + 1];
      AttendJob &j = jobs[g];
      auto fill = [](AttendCell &a, const CellStore &cs) {
        a.G = cs.G16; a.UT = cs.UT16; a.UF = cs.UF16; a.e = cs.e; a.words = cs.words; a.scales = cs.scales;
        a.r_t = cs.c.r_t; a.r_f = cs.c.r_t > 0 ? cs.c.r_f : 0; a.bits = cs.c.bits; a.cell = cs.c.cell;
      };
      fill(j.k, sk); fill(j.v, sv);
      j.m = sk.c.m; j.T = T;
      const size_t row0 = (size_t)H->group_start[g] * nh * n_q * kD;
      j.q = (const float *)dQ + row0; j.out = (float *)dOut + row0;
      j.kP = sk.P16;
      j.vP = sv.P16;
      j.wh = b.take<__half>((size_t)j.m * NQP * std::max(j.k.r_t, 8));
      j.wl = b.take<__half>((size_t)j.m * NQP * std::max(j.k.r_t, 8));
      j.we = b.take<float>((size_t)j.m * NQP);
      j.qt = b.take<float>((size_t)j.m * kD * NQP);
      j.qh = b.take<__half>((size_t)j.m * kAttMaxQ * kD);
      j.ql = b.take<__half>((size_t)j.m * kAttMaxQ * kD);
      j.qe = b.take<float>((size_t)j.m * kAttMaxQ);
      j.p = b.take<float>((size_t)j.m * T * NQP);
      j.ml = b.take<float>((size_t)j.m * n_chunks * 2 * NQP);
      j.y = b.take<float>((size_t)j.m * n_chunks * std::max(j.v.r_t, 1) * NQP);
      j.a = b.take<float>((size_t)j.m * n_chunks * kD * NQP);
    }
    if (pass == 0 && (rc = ws_reserve(dev, b.off + 256, &ws_base))) return rc;
  }
  Program P;
  const size_t off = P.push(jobs);
  const uint64_t seed = H->seed;
  const float fscale = (float)scale;
  const bool mma = (g_fast.load() & 1) != 0;        // warp-MMA forms of the two code streams (the CUDA-core forms stay as the portable path)
  const bool vmma = mma;
  P.add(ST_ATT, [=](char *dev_t, cudaStream_t s) {
    const AttendJob *d = (const AttendJob *)(dev_t + off);
    attend_prep_kernel<<<dim3(m_max, ng, NQP), 128, shm_prep, s>>>(d, n_q, NQP, fscale, seed);
    LAUNCHED();
    const dim3 grid(n_chunks, m_max, ng);
    const int n_tiles = (m_max * NQP + 127) / 128;
    if (krt > 0) {
      attend_bscore_kernel<<<dim3((T + 63) / 64, n_tiles, ng), 256, 0, s>>>(d, NQP);
      LAUNCHED();
    }
    for (int b = 0; b <= 8; ++b) {
      if (!((kbits >> b) & 1)) continue;
      switch (b) {
        case 0: launch_att_scores<0>(grid, shm_sc, s, d, NQP); break;
        case 1: if (mma) launch_att_scores_mma<1>(grid, s, d, NQP); else launch_att_scores<1>(grid, shm_sc, s, d, NQP); break;
        case 2: if (mma) launch_att_scores_mma<2>(grid, s, d, NQP); else launch_att_scores<2>(grid, shm_sc, s, d, NQP); break;
        case 3: launch_att_scores<3>(grid, shm_sc, s, d, NQP); break;
        case 4: if (mma) launch_att_scores_mma<4>(grid, s, d, NQP); else launch_att_scores<4>(grid, shm_sc, s, d, NQP); break;
        default: if (mma) launch_att_scores_mma<8>(grid, s, d, NQP); else launch_att_scores<8>(grid, shm_sc, s, d, NQP); break;
      }
      LAUNCHED();
    }
    for (int b = 1; b <= 8; ++b) {                 // b = 0: no residual, nothing to stream
      if (!((vbits >> b) & 1)) continue;
      switch (b) {
        case 1: if (vmma) launch_att_values_mma<1>(grid, s, d, NQP); else launch_att_values<1>(grid, s, d, NQP); break;
        case 2: if (vmma) launch_att_values_mma<2>(grid, s, d, NQP); else launch_att_values<2>(grid, s, d, NQP); break;
        case 3: launch_att_values<3>(grid, s, d, NQP); break;
        case 4: if (vmma) launch_att_values_mma<4>(grid, s, d, NQP); else launch_att_values<4>(grid, s, d, NQP); break;
        default: if (vmma) launch_att_values_mma<8>(grid, s, d, NQP); else launch_att_values<8>(grid, s, d, NQP); break;
      }
      LAUNCHED();
    }
    if (vrt > 0) {
      const int KT = (vrt + 63) / 64;
      attend_bvalue_kernel<<<dim3(n_chunks * KT, n_tiles, ng), 256, 0, s>>>(d, NQP, n_chunks, KT);
      LAUNCHED();
    }
    attend_combine_kernel<<<dim3(m_max, ng, n_q), 128, shm_comb, s>>>(d, n_q, NQP, n_chunks, seed);
    LAUNCHED();
  });
  void *d_tab = nullptr;
  if ((rc = tab_reserve(dev, P.host.size() + 256, &d_tab))) return rc;
  if ((rc = arena_acquire(dev, st))) return rc;
  H->last_stream = st;
  g_timer.begin(st);
  if ((rc = run_program(P, (char *)d_tab, st))) return rc;
  arena_release(dev, st);
  return JOLT_OK;
}

// ------------------------------------------------------------------ serialisation
namespace {
constexpr uint64_t kBlobMagic = 0x314C424F544C4F4Aull;      // "JOLTOBL1"
struct BlobHeader {
  uint64_t magic;
  uint32_t version, head_dim;
  int32_t n_layers, n_kv_heads, T, n_groups, n_cells, subspace;
  uint64_t seed, blob_bytes;
};
struct BlobCell { CellDesc c; int32_t n_sigma, pad; };
size_t blob_image_bytes(const jolt_handle *H) {
  return sizeof(BlobHeader) + sizeof(int32_t) * (H->n_groups + 1) + sizeof(BlobCell) * H->cells.size() + H->blob_bytes;
}
}  // namespace

extern "C" int jolt_serialized_bytes(const jolt_handle *H, int64_t *bytes) {
  if (!H || !bytes) return fail(JOLT_EINVAL, "null argument");
  *bytes = (int64_t)blob_image_bytes(H);
  return JOLT_OK;
}

extern "C" int jolt_serialize(const jolt_handle *H, void *host_dst, int64_t cap, void *stream) {
  if (!H || !host_dst) return fail(JOLT_EINVAL, "null argument");
  const size_t need = blob_image_bytes(H);
  if (cap < (int64_t)need) return fail(JOLT_EINVAL, "buffer of %lld bytes, %zu needed", (long long)cap, need);
  int dev = 0;
  CU(cudaGetDevice(&dev));
  if (dev != H->device) return fail(JOLT_EINVAL, "handle belongs to device %d, current device is %d", H->device, dev);
  char *p = (char *)host_dst;
  BlobHeader hd;
  memset(&hd, 0, sizeof hd);
  hd.magic = kBlobMagic; hd.version = 1; hd.head_dim = kD;
  hd.n_layers = H->n_layers; hd.n_kv_heads = H->n_kv_heads; hd.T = H->T; hd.n_groups = H->n_groups;
  hd.n_cells = (int32_t)H->cells.size(); hd.subspace = H->subspace ? 1 : 0; hd.seed = H->seed; hd.blob_bytes = H->blob_bytes;
  memcpy(p, &hd, sizeof hd); p += sizeof hd;
  memcpy(p, H->group_start.data(), sizeof(int32_t) * (H->n_groups + 1)); p += sizeof(int32_t) * (H->n_groups + 1);
  for (auto &cs : H->cells) {
    BlobCell bc;
    memset(&bc, 0, sizeof bc);
    bc.c = cs.c; bc.c.X = nullptr; bc.n_sigma = cs.n_sigma;
    memcpy(p, &bc, sizeof bc); p += sizeof bc;
  }
  cudaStream_t st = (cudaStream_t)stream;
  CU(cudaMemcpyAsync(p, H->blob, H->blob_bytes, cudaMemcpyDeviceToHost, st));
  CU(cudaStreamSynchronize(st));
  return JOLT_OK;
}

extern "C" int jolt_deserialize(const void *host_src, int64_t bytes, void *stream, jolt_handle **out) {
  if (out) *out = nullptr;
  if (!host_src || !out) return fail(JOLT_EINVAL, "null argument");
  const char *p = (const char *)host_src;
  BlobHeader hd;
  if (bytes < (int64_t)sizeof hd) return fail(JOLT_EINVAL, "image of %lld bytes is shorter than its header", (long long)bytes);
  memcpy(&hd, p, sizeof hd); p += sizeof hd;
  if (hd.magic != kBlobMagic || hd.version != 1 || hd.head_dim != (uint32_t)kD) return fail(JOLT_EINVAL, "not a compressed-cache image of this library version");
  if (hd.n_groups <= 0 || hd.n_cells != 2 * hd.n_groups || hd.n_layers <= 0 || hd.n_kv_heads <= 0 || hd.T <= 0) return fail(JOLT_EINVAL, "corrupt image header");
  if (hd.blob_bytes > (uint64_t)bytes) return fail(JOLT_EINVAL, "image of %lld bytes, header names a payload of %llu", (long long)bytes, (unsigned long long)hd.blob_bytes);
  const size_t need = sizeof hd + sizeof(int32_t) * ((size_t)hd.n_groups + 1) + sizeof(BlobCell) * (size_t)hd.n_cells + (size_t)hd.blob_bytes;
  if ((size_t)bytes < need) return fail(JOLT_EINVAL, "image of %lld bytes, header asks for %zu", (long long)bytes, need);
  int dev = 0;
  CU(cudaGetDevice(&dev));
  std::unique_ptr<jolt_handle> H(new jolt_handle);
  H->device = dev; H->n_layers = hd.n_layers; H->n_kv_heads = hd.n_kv_heads; H->T = hd.T; H->n_groups = hd.n_groups;
  H->seed = hd.seed; H->subspace = hd.subspace != 0;
  H->group_start.resize(hd.n_groups + 1);
  memcpy(H->group_start.data(), p, sizeof(int32_t) * (hd.n_groups + 1)); p += sizeof(int32_t) * (hd.n_groups + 1);
  if (H->group_start[0] != 0 || H->group_start[hd.n_groups] != hd.n_layers) return fail(JOLT_EINVAL, "corrupt layer grouping");
  for (int g = 0; g < hd.n_groups; ++g)
    if (H->group_start[g + 1] <= H->group_start[g]) return fail(JOLT_EINVAL, "corrupt layer grouping (not ascending)");
  H->cells.resize(hd.n_cells);
  for (int i = 0; i < hd.n_cells; ++i) {
    BlobCell bc;
    memcpy(&bc, p, sizeof bc); p += sizeof bc;
    const CellDesc &c = bc.c;
    const int g = i / 2;
    if (c.T != hd.T || c.n_heads != hd.n_kv_heads || c.m != (H->group_start[g + 1] - H->group_start[g]) * hd.n_kv_heads || c.cell != i ||
        c.r_t < 0 || c.r_t > c.T || c.r_f < 0 || c.r_f > kD || !bits_ok(c.bits) || bc.n_sigma < 0 || bc.n_sigma > c.T)
      return fail(JOLT_EINVAL, "corrupt descriptor of cell %d", i);
    H->cells[i].c = c; H->cells[i].c.X = nullptr; H->cells[i].n_sigma = bc.n_sigma;
  }
  if (carve_handle_blob(*H) != hd.blob_bytes) return fail(JOLT_EINVAL, "image payload size does not match its descriptors");
  H->blob_bytes = hd.blob_bytes;
  cudaStream_t st = (cudaStream_t)stream;
  if (cudaMallocAsync(&H->blob, H->blob_bytes, st) != cudaSuccess) { cudaGetLastError(); return fail(JOLT_ENOMEM, "compressed cache of %zu bytes", H->blob_bytes); }
  carve_handle_blob(*H);
  cudaError_t ce = cudaMemcpyAsync(H->blob, p, H->blob_bytes, cudaMemcpyHostToDevice, st);
  if (ce == cudaSuccess) ce = cudaStreamSynchronize(st);
  if (ce != cudaSuccess) { cudaGetLastError(); cudaFreeAsync(H->blob, st); return fail(JOLT_ECUDA, "upload: %s", cudaGetErrorString(ce)); }
  if (cudaMalloc(&H->d_status, sizeof(int) * 4 * (size_t)hd.n_cells) != cudaSuccess) { cudaGetLastError(); cudaFreeAsync(H->blob, st); return fail(JOLT_ENOMEM, "status words"); }
  cudaMemset(H->d_status, 0, sizeof(int) * 4 * (size_t)hd.n_cells);
  H->last_stream = st;
  {  // projected cores of the uploaded cells (not part of the image: a function of the stored core and feature factor)
    int rc = alloc_projected_cores(*H, nullptr);
    std::vector<ProjJob> pj;
    int max_rows = 0, max_rf = 0;
    for (auto &cs : H->cells)
      if (cs.c.r_t > 0) {
        pj.push_back({cs.G16, cs.UF16, cs.P16, cs.c.m * cs.c.r_t, cs.c.r_f});
        max_rows = std::max(max_rows, cs.c.m * cs.c.r_t); max_rf = std::max(max_rf, cs.c.r_f);
      }
    void *d_jobs = nullptr;
    if (rc == JOLT_OK && !pj.empty()) {
      ce = cudaMalloc(&d_jobs, pj.size() * sizeof(ProjJob));
      if (ce == cudaSuccess) ce = cudaMemcpyAsync(d_jobs, pj.data(), pj.size() * sizeof(ProjJob), cudaMemcpyHostToDevice, st);
      if (ce == cudaSuccess) { launch_project_cores((const ProjJob *)d_jobs, (int)pj.size(), max_rows, max_rf, st); ce = cudaStreamSynchronize(st); }
      if (d_jobs) cudaFree(d_jobs);
      if (ce != cudaSuccess) { cudaGetLastError(); rc = fail(JOLT_ECUDA, "projected cores: %s", cudaGetErrorString(ce)); }
    }
    if (rc != JOLT_OK) {
      if (H->P_all) cudaFree(H->P_all);
      cudaFree(H->d_status); cudaFreeAsync(H->blob, st);
      return rc;
    }
  }
  for (auto &cs : H->cells) encode_store_maps(cs);          // tensor maps point into the new buffers
  *out = H.release();
  return JOLT_OK;
}

extern "C" int jolt_free(jolt_handle *H) {
  if (!H) return JOLT_OK;
  if (H->blob) {
    int cur = 0;
    cudaGetDevice(&cur);
    if (cur != H->device) cudaSetDevice(H->device);
    if (H->P_all) { cudaFree(H->P_all); H->P_all = nullptr; }       // cudaFree waits for the kernels that read it
    if (H->d_status) { cudaFree(H->d_status); H->d_status = nullptr; }
    // ordered after the last call that read the buffers (its stream may be gone by now: then wait for the device)
    if (cudaFreeAsync(H->blob, H->last_stream) != cudaSuccess) { cudaGetLastError(); cudaDeviceSynchronize(); cudaFreeAsync(H->blob, 0); }
    if (cur != H->device) cudaSetDevice(cur);
  }
  delete H;
  return JOLT_OK;
}

extern "C" int jolt_compressed_bytes(const jolt_handle *H, int64_t *bytes) {
  if (!H || !bytes) return fail(JOLT_EINVAL, "null argument");
  *bytes = H->stored_bytes;
  return JOLT_OK;
}

extern "C" int jolt_get_component(const jolt_handle *H, int32_t cell, int32_t which, void *dst, int64_t cap, int64_t *written) {
  if (!H || !written) return fail(JOLT_EINVAL, "null argument");
  if (cell < 0 || cell >= (int)H->cells.size()) return fail(JOLT_EINVAL, "cell %d out of range", cell);
  const CellStore &cs = H->cells[cell];
  const CellDesc &c = cs.c;
  const size_t M = (size_t)c.m * c.T * kD;
  const void *src = nullptr;
  size_t n = 0;
  switch (which) {
    case 0: src = cs.G16; n = 2 * (size_t)c.m * c.r_t * c.r_f; break;
    case 1: src = cs.UT16; n = 2 * (size_t)c.T * c.r_t; break;
    case 2: src = cs.UF16; n = 2 * (size_t)kD * c.r_f; break;
    case 3: src = cs.words; n = 4 * (M / 32 * c.bits); break;
    case 4: src = cs.scales; n = c.bits ? 2 * (M / 32) : 0; break;
    case 5: src = cs.e; n = 4; break;
    case 6: src = cs.sigma; n = 4 * (size_t)cs.n_sigma; break;
    case 7: src = cs.lam; n = 4 * (size_t)kD; break;
    case 8: src = cs.dbg_UT32; n = cs.dbg_UT32 ? 4 * (size_t)c.T * c.r_t : 0; break;
    case 9: src = cs.e + 1; n = (H->subspace && c.r_t > 0) ? 4 : 0; break;   // residual of the converged-subspace check
    default: return fail(JOLT_EINVAL, "component %d", which);
  }
  *written = (int64_t)n;
  if (!dst) return JOLT_OK;
  if ((int64_t)n > cap) return fail(JOLT_EINVAL, "destination holds %lld bytes, component has %zu", (long long)cap, n);
  if (n) CU(cudaMemcpy(dst, src, n, cudaMemcpyDeviceToHost));
  return JOLT_OK;
}

// ------------------------------------------------------------------ plan
static void fill_defaults(jolt_options *o) {
  memset(o, 0, sizeof *o);
  o->token_mode = JOLT_TOKEN_RANDOMIZED; o->oversample = 10; o->power_iters = 1; o->quant_group = kGroup; o->seed = 0;
  o->bits_set = nullptr; o->n_bits = 0; o->rank_step = 16; o->r_t_min = 16; o->r_f_min = 16; o->q_cap = 0; o->eps2 = nullptr;
  o->count_scale_bytes = 1;
  o->allocator = JOLT_ALLOC_DUAL;
}
extern "C" void jolt_default_options(jolt_options *o) { if (o) fill_defaults(o); }

extern "C" int64_t jolt_cell_bytes(int32_t m, int32_t T, int32_t d, int32_t r_t, int32_t r_f, int32_t bits, int32_t scales) {
  return cell_bytes(m, T, d, r_t, r_f, bits, scales != 0);
}
extern "C" int32_t jolt_cap_policy(int32_t T, double ratio) { return cap_policy(T, ratio); }

static const double *builtin_eps2() {
  static double tab[9];
  static std::once_flag once;
  std::call_once(once, [] { eps2_calibration(tab); });
  return tab;
}
extern "C" int jolt_eps2_table(double out[9]) {
  if (!out) return fail(JOLT_EINVAL, "null argument");
  memcpy(out, builtin_eps2(), sizeof(double) * 9);
  return JOLT_OK;
}

extern "C" int jolt_allocate(int32_t n_cells, const int32_t *m, int32_t T, int32_t d, const double *lam3, const double *sig2sq,
                             const int64_t *sig2_off, const int32_t *sig2_len, const double *total_sq, const int32_t *r_t_max,
                             double budget, const jolt_options *o, jolt_cell_plan *out, double *achieved) {
  if (n_cells <= 0 || !m || !lam3 || !sig2sq || !sig2_off || !sig2_len || !total_sq || !r_t_max || !o || !out)
    return fail(JOLT_EINVAL, "null argument");
  if (d != kD) return fail(JOLT_EUNSUPPORTED, "head_dim %d", d);
  static const int32_t def_bits[4] = {0, 2, 4, 8};
  const int32_t *bits = o->bits_set ? o->bits_set : def_bits;
  const int nb = o->bits_set ? o->n_bits : 4;
  if (nb <= 0) return fail(JOLT_EINVAL, "empty bits set");
  for (int i = 0; i < nb; ++i) if (!bits_ok(bits[i])) return fail(JOLT_EINVAL, "bits %d", bits[i]);
  const int step = o->rank_step > 0 ? o->rank_step : 16;
  const int rt0 = o->r_t_min > 0 ? o->r_t_min : step, rf0 = o->r_f_min > 0 ? o->r_f_min : step;
  const double *eps2 = o->eps2 ? o->eps2 : builtin_eps2();
  std::vector<CellOptions> cells(n_cells);
  for (int c = 0; c < n_cells; ++c) {
    const double *l3 = lam3 + (size_t)c * kD;
    const double *s2 = sig2sq + sig2_off[c];
    const int ns = sig2_len[c];
    if (!(total_sq[c] > 0)) return fail(JOLT_EINVAL, "cell %d has zero energy", c);
    for (int rt = rt0; rt <= r_t_max[c]; rt += step) {
      double t2 = 0;
      for (int i = rt; i < ns; ++i) t2 += s2[i];
      for (int rf = rf0; rf <= kD; rf += step) {
        if (rt > m[c] * rf) continue;
        double t3 = 0;
        for (int i = rf; i < kD; ++i) t3 += l3[i];
        const double tau = std::min(1.0, (t2 + t3) / total_sq[c]);
        for (int bi = 0; bi < nb; ++bi) {
          cells[c].err.push_back(eps2[bits[bi]] * tau);
          cells[c].cost.push_back((double)cell_bytes(m[c], T, d, rt, rf, bits[bi], o->count_scale_bytes != 0));
          cells[c].trip.push_back({rt, rf, bits[bi]});
        }
      }
    }
    if (cells[c].err.empty()) return fail(JOLT_EINVAL, "cell %d: empty rank grid (r_t_max %d)", c, r_t_max[c]);
  }
  std::vector<size_t> choice;
  double total = 0;
  if (o->allocator < JOLT_ALLOC_DUAL || o->allocator > JOLT_ALLOC_UNIFORM) return fail(JOLT_EINVAL, "allocator %d", o->allocator);
  const bool ok = o->allocator == JOLT_ALLOC_GREEDY ? greedy_allocate(cells, budget, choice, total)
                  : o->allocator == JOLT_ALLOC_UNIFORM ? uniform_allocate(cells, budget, choice, total)
                                                       : dual_allocate(cells, budget, choice, total);
  for (int c = 0; c < n_cells; ++c) out[c] = cells[c].trip[choice[c]];
  if (achieved) *achieved = total;
  return ok ? JOLT_OK : fail(JOLT_EBUDGET, "cheapest allocation needs %.0f bytes, budget is %.0f", total, budget);
}

// The measured spectra of a cache (host memory): what the allocator needs, kept so that the cache can be planned again
// at another budget or with another allocator without touching the GPU.
struct jolt_spectra {
  int32_t nc = 0, T = 0, q_cap = 0;
  bool exact = false, cap_from_policy = false;
  double raw = 0;                              // bytes of the uncompressed fp16 cache
  std::vector<double> lam3, s2all, total;
  std::vector<int64_t> off;
  std::vector<int32_t> len, mm, rtmax;
};

namespace {
struct PackJob { const float *src; float *dst; int n; };
__global__ void pack_spectra_kernel(const PackJob *__restrict__ jobs) {
  const PackJob j = jobs[blockIdx.x];
  for (int i = threadIdx.x; i < j.n; i += blockDim.x) j.dst[i] = j.src[i];
}
}  // namespace

extern "C" int jolt_probe(const jolt_layout *L, const void *K, const void *V, double ratio_hint, const jolt_options *o, void *stream,
                          jolt_spectra **out) {
  if (out) *out = nullptr;
  if (!out || !K || !V) return fail(JOLT_EINVAL, "null argument");
  int rc;
  if ((rc = check_layout(L)) || (rc = check_options(o)) || (rc = check_device_alignment(L, K, V))) return rc;
  if (!(ratio_hint > 0) && o->q_cap <= 0) return fail(JOLT_EINVAL, "the cap needs a compression ratio or opts->q_cap");
  cudaStream_t st = (cudaStream_t)stream;
  int dev = 0;
  CU(cudaGetDevice(&dev));
  const double raw = 2.0 * 2.0 * (double)L->n_layers * L->n_kv_heads * L->seq_len * kD;
  const int nc = 2 * L->n_groups;
  // exact spectra come from the T x T eigen-solve up to kExactEigMaxT tokens; beyond, the probe is the converged
  // block iteration at the cap with the tail-mass accounting of the randomized probe
  const bool subspace = o->token_mode == JOLT_TOKEN_EXACT && L->seq_len > kExactEigMaxT;
  const bool exact = o->token_mode == JOLT_TOKEN_EXACT && !subspace;
  const int oversample = subspace ? std::max(o->oversample, kSubspaceOversample) : o->oversample;
  const int power_iters = subspace ? std::max(o->power_iters, kSubspaceIters) : o->power_iters;
  const int q_cap = o->q_cap > 0 ? o->q_cap : cap_policy(L->seq_len, ratio_hint);
  std::vector<jolt_cell_plan> probe(nc);
  std::vector<CellDesc> cells;
  for (int i = 0; i < nc; ++i) {
    const int m = (L->group_start[i / 2 + 1] - L->group_start[i / 2]) * L->n_kv_heads;
    const int lim = std::min(L->seq_len, m * kD);
    probe[i] = {exact ? lim : std::min(q_cap, lim), kD, 0};
  }
  make_cells(L, K, V, probe.data(), oversample, cells);
  if (exact) for (auto &c : cells) c.k = c.r_t;
  const int mode = exact ? FM_EXACT : FM_RANDOMIZED;
  const size_t esz = L->dtype == JOLT_F16 ? 2 : 4;
  const size_t span = layout_span_elems(L) * esz;
  const int fmask = g_fast.load();
  const bool fast = (fmask & 1) != 0;
  std::vector<CellWork> ws(nc);
  void *ws_base = nullptr;
  int *d_status = nullptr;
  float *d_pack = nullptr;
  char *stage_K = nullptr, *stage_V = nullptr;
  size_t pack_floats = 0;
  for (int pass = 0; pass < 2; ++pass) {
    Bump b;
    b.base = (char *)ws_base;
    d_status = b.take<int>(4 * (size_t)nc);
    if (L->mem_space == JOLT_MEM_HOST) { stage_K = b.take<char>(span); stage_V = b.take<char>(span); }
    for (int i = 0; i < nc; ++i) {
      ws[i].c = cells[i]; ws[i].active = true; ws[i].status = d_status ? d_status + 4 * i : nullptr;
      ws[i].lam = nullptr; ws[i].sigma = nullptr;
      ws[i].tc = (fmask & 2) && mode == FM_RANDOMIZED && tc_sweep_ok(cells[i], L->mem_space == JOLT_MEM_HOST);
      ws[i].tc_gram = (fmask & 4) && tc_sweep_ok(cells[i], L->mem_space == JOLT_MEM_HOST);
      ws[i].ufI = true;
      carve(b, ws[i], mode, false);
    }
    if (pass == 0) { pack_floats = 0; for (int i = 0; i < nc; ++i) pack_floats += kD + (size_t)ws[i].n_sigma; }
    d_pack = b.take<float>(pack_floats);
    if (pass == 0 && (rc = ws_reserve(dev, b.off + 256, &ws_base))) return rc;
  }
  if (L->mem_space == JOLT_MEM_HOST)
    for (int i = 0; i < nc; ++i) {
      const char *hb = (const char *)(i % 2 == 0 ? K : V);
      ws[i].c.X = (i % 2 == 0 ? stage_K : stage_V) + ((const char *)ws[i].c.X - hb);
    }
  // one program per cell group, run on concurrent streams like the factor stage of jolt_compress; then the spectra of
  // all cells are gathered into one buffer and leave the device in a single copy
  std::vector<int> cell_group(nc, -1);
  int n_groups = assign_groups(ws, cell_group);
  // the randomized token probe runs on X itself, so the feature spectra (Gram + eigen-solve of all cells) form a
  // program of their own on one more stream instead of lengthening every group's chain
  const bool split = mode == FM_RANDOMIZED && n_groups > 1 && n_groups < kMaxGroups;
  std::vector<Program> PG(std::max(n_groups, 1) + (split ? 1 : 0));
  for (int g = 0; g < n_groups; ++g) {
    std::vector<CellWork> sub = ws;
    for (int i = 0; i < nc; ++i) if (cell_group[i] != g) sub[i].active = false;
    build_factor_program(PG[g], sub, mode, true, power_iters, o->seed, fast, false, split ? 2 : 3);
  }
  if (split) {
    std::vector<CellWork> sub = ws;
    build_factor_program(PG[n_groups], sub, mode, true, power_iters, o->seed, fast, false, 1);
    ++n_groups;
  }
  Program P;
  {
    std::vector<PackJob> pj;
    size_t at = 0;
    for (int i = 0; i < nc; ++i) {
      pj.push_back({ws[i].lam, d_pack + at, kD}); at += kD;
      pj.push_back({ws[i].sigma, d_pack + at, ws[i].n_sigma}); at += ws[i].n_sigma;
    }
    const size_t poff = P.push(pj);
    const int n = (int)pj.size();
    P.add(ST_SVD, [=](char *dev_t, cudaStream_t s) { pack_spectra_kernel<<<n, 128, 0, s>>>((const PackJob *)(dev_t + poff)); LAUNCHED(); });
  }
  void *d_tab = nullptr;
  std::vector<size_t> tab_off(PG.size() + 1, 0);
  for (size_t g = 0; g < PG.size(); ++g) tab_off[g + 1] = tab_off[g] + ((PG[g].host.size() + 255) & ~(size_t)255);
  if ((rc = tab_reserve(dev, tab_off.back() + P.host.size() + 256, &d_tab))) return rc;
  if ((rc = arena_acquire(dev, st))) return rc;
  g_timer.begin(st);
  CU(cudaMemsetAsync(d_status, 0, sizeof(int) * 4 * nc, st));
  if (L->mem_space == JOLT_MEM_HOST) {
    CU(cudaMemcpyAsync(stage_K, K, span, cudaMemcpyHostToDevice, st));
    CU(cudaMemcpyAsync(stage_V, V, span, cudaMemcpyHostToDevice, st));
  }
  if (n_groups <= 1) {
    if (n_groups == 1 && (rc = run_program(PG[0], (char *)d_tab, st))) return rc;
  } else if ((rc = run_group_programs(dev, st, PG, n_groups, d_tab, tab_off))) return rc;
  if ((rc = run_program(P, (char *)d_tab + tab_off.back(), st))) return rc;
  arena_release(dev, st);
  std::vector<int> hstat(4 * nc);
  std::vector<float> pack(pack_floats);
  CU(cudaMemcpyAsync(hstat.data(), d_status, sizeof(int) * 4 * nc, cudaMemcpyDeviceToHost, st));
  CU(cudaMemcpyAsync(pack.data(), d_pack, sizeof(float) * pack_floats, cudaMemcpyDeviceToHost, st));
  CU(cudaStreamSynchronize(st));
  g_timer.finish();
  if ((rc = status_to_code(hstat))) return rc;
  // spectra -> allocator inputs (tail-mass accounting of Sec. 5 for the randomized probe)
  std::unique_ptr<jolt_spectra> S(new jolt_spectra);
  S->nc = nc; S->T = L->seq_len; S->q_cap = q_cap; S->exact = exact; S->cap_from_policy = o->q_cap <= 0; S->raw = raw;
  S->lam3.resize((size_t)nc * kD); S->total.resize(nc); S->off.resize(nc); S->len.resize(nc); S->mm.resize(nc); S->rtmax.resize(nc);
  size_t at = 0;
  for (int i = 0; i < nc; ++i) {
    const float *lam = pack.data() + at; at += kD;
    const float *sig = pack.data() + at; at += ws[i].n_sigma;
    double tot = 0;
    for (int j = 0; j < kD; ++j) { S->lam3[(size_t)i * kD + j] = lam[j]; tot += lam[j]; }
    S->total[i] = tot;
    S->off[i] = (int64_t)S->s2all.size();
    const int keep = exact ? ws[i].n_sigma : std::min(ws[i].n_sigma, cells[i].r_t);
    double acc = 0;
    for (int j = 0; j < keep; ++j) { const double v = (double)sig[j] * sig[j]; S->s2all.push_back(v); acc += v; }
    if (!exact) S->s2all.push_back(std::max(0.0, tot - acc));
    S->len[i] = keep + (exact ? 0 : 1);
    S->mm[i] = cells[i].m;
    S->rtmax[i] = cells[i].r_t;
  }
  *out = S.release();
  return JOLT_OK;
}

extern "C" int jolt_plan_from_spectra(const jolt_spectra *S, double budget, const jolt_options *o, jolt_cell_plan *out, double *achieved) {
  if (!S || !out || !o) return fail(JOLT_EINVAL, "null argument");
  if (!(budget > 0)) return fail(JOLT_EINVAL, "byte budget must be positive");
  // the probe stopped at its cap: a budget whose own cap (Sec. 5 "Cap selection") is larger needs a new probe
  if (S->cap_from_policy && !S->exact && o->q_cap <= 0 && cap_policy(S->T, S->raw / budget) > S->q_cap)
    return fail(JOLT_EINVAL, "this budget's cap %d exceeds the probed cap %d", cap_policy(S->T, S->raw / budget), S->q_cap);
  return jolt_allocate(S->nc, S->mm.data(), S->T, kD, S->lam3.data(), S->s2all.data(), S->off.data(), S->len.data(), S->total.data(),
                       S->rtmax.data(), budget, o, out, achieved);
}

extern "C" int jolt_spectra_free(jolt_spectra *S) { delete S; return JOLT_OK; }

extern "C" int jolt_plan(const jolt_layout *L, const void *K, const void *V, double budget, const jolt_options *o, void *stream,
                         jolt_cell_plan *out, double *achieved) {
  if (!out || !K || !V) return fail(JOLT_EINVAL, "null argument");
  int rc;
  if ((rc = check_layout(L)) || (rc = check_options(o))) return rc;
  if (!(budget > 0)) return fail(JOLT_EINVAL, "byte budget must be positive");
  const double raw = 2.0 * 2.0 * (double)L->n_layers * L->n_kv_heads * L->seq_len * kD;
  jolt_spectra *S = nullptr;
  if ((rc = jolt_probe(L, K, V, raw / budget, o, stream, &S))) return rc;
  rc = jolt_plan_from_spectra(S, budget, o, out, achieved);
  delete S;
  return rc;
}

// ------------------------------------------------------------------ misc exports
extern "C" int jolt_sketch_host(uint64_t seed, int32_t cell, int32_t stream_id, int64_t n_rows, int32_t n_cols, float *out) {
  if (!out || n_rows < 0 || n_cols < 0) return fail(JOLT_EINVAL, "bad argument");
  const uint64_t base = stream_base(seed, cell, stream_id);
  for (int64_t i = 0; i < n_rows * n_cols; ++i) out[i] = __half2float(__double2half(gaussian_from_u64(mix64(base + (uint64_t)i))));
  return JOLT_OK;
}
extern "C" int jolt_signs_host(uint64_t seed, int32_t cell, float out[128]) {
  if (!out) return fail(JOLT_EINVAL, "null argument");
  const uint64_t base = stream_base(seed, cell, STREAM_SIGNS);
  const uint64_t w[2] = {mix64(base + 0), mix64(base + 1)};
  for (int f = 0; f < 128; ++f) out[f] = ((w[f / 64] >> (f % 64)) & 1) ? -1.f : 1.f;
  return JOLT_OK;
}
extern "C" int jolt_release_workspace(void) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return JOLT_OK; }
  std::lock_guard<std::mutex> lk(g_ws_mu);
  cudaDeviceSynchronize();
  if (g_ws[dev].base) { cudaFree(g_ws[dev].base); g_ws[dev] = Workspace(); }
  if (g_tab[dev].base) { cudaFree(g_tab[dev].base); g_tab[dev] = Workspace(); }
  return JOLT_OK;
}
#ifdef JOLT_DEBUG
extern "C" int jolt_debug_stamps(long long *host_out, int n) {
  // n > 0 and host_out == nullptr: (re)allocate and zero a device stamp buffer of n entries; host_out != nullptr: read it back
  if (!host_out) {
    if (g_dbg_stamps) { cudaFree(g_dbg_stamps); g_dbg_stamps = nullptr; }
    if (n > 0) { if (cudaMalloc(&g_dbg_stamps, sizeof(long long) * n) != cudaSuccess) return JOLT_ENOMEM; cudaMemset(g_dbg_stamps, 0, sizeof(long long) * n); }
    return JOLT_OK;
  }
  if (!g_dbg_stamps) return JOLT_EINVAL;
  return cudaMemcpy(host_out, g_dbg_stamps, sizeof(long long) * n, cudaMemcpyDeviceToHost) == cudaSuccess ? JOLT_OK : JOLT_ECUDA;
}
#endif
extern "C" int64_t jolt_launch_count(void) { return g_launches.load(); }
extern "C" int jolt_test_set_wait_limit(int64_t cycles, int32_t skip_first_load) {
  const long long lim = cycles > 0 ? (long long)cycles : tc::kSpinCycles;
  const int skip = skip_first_load == 2 ? 2 : (skip_first_load ? 1 : 0);
  CU(cudaMemcpyToSymbol(tc::g_spin_limit, &lim, sizeof lim));
  CU(cudaMemcpyToSymbol(tc::g_test_skip_first_load, &skip, sizeof skip));
  return JOLT_OK;
}
extern "C" int jolt_test_set_decode_tail(int32_t percent, int32_t chunk_tiles) {
  if (percent < 0 || percent > 100 || (percent > 0 && chunk_tiles < 1)) return fail(JOLT_EINVAL, "decode tail %d %% in chunks of %d", percent, chunk_tiles);
  g_dec_tail_pct.store(percent);
  g_dec_tail_chunk.store(percent > 0 ? chunk_tiles : 8);
  return JOLT_OK;
}
extern "C" int jolt_set_stream_groups(int n) { return g_n_cell_groups.exchange(std::max(1, std::min(8, n))); }
extern "C" int jolt_set_fast_path(int enabled) { return g_fast.exchange(enabled & 255); }
extern "C" int jolt_last_stage_ms(float *out, int32_t cap, int32_t *n) {
  if (!out || !n) return fail(JOLT_EINVAL, "null argument");
  *n = std::min<int>(cap, kNumStages);
  if (g_timer.have) g_timer.finish();
  for (int i = 0; i < *n; ++i) out[i] = g_timer.ms[i];
  return JOLT_OK;
}
extern "C" const char *jolt_stage_name(int32_t i) { return (i >= 0 && i < kNumStages) ? kStageNames[i] : ""; }
extern "C" const char *jolt_strerror(int s) {
  switch (s) {
    case JOLT_OK: return "ok";
    case JOLT_EINVAL: return "invalid argument";
    case JOLT_EUNSUPPORTED: return "not supported by this build";
    case JOLT_EBUDGET: return "byte budget below the cheapest allocation";
    case JOLT_ENUMERIC: return "numerical failure";
    case JOLT_ENOMEM: return "out of memory";
    case JOLT_ECUDA: return "CUDA error";
    case JOLT_ETIMEOUT: return "bounded device wait ran out";
    default: return "unknown status";
  }
}
extern "C" const char *jolt_last_error(void) { return g_err.c_str(); }

#include "decode_static.cuh"
