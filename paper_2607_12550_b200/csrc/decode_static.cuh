// jolt_decompress_static: the decode path for callers that must not allocate device memory.
//
// Some callers cannot call cudaMalloc while they decode: a serving loop that has handed all free
// memory to its own pool and forbids further driver allocations, a thread inside a region where a
// device allocation would synchronise the whole context, or a host process whose allocator hooks
// reject anything outside start-up.  For them this entry point keeps ALL of its scratch (the per-head
// projected core, the fp32 backbone tile buffer and the kernel argument tables) in one fixed array that
// is part of the loaded library image.  The status words its kernels write are the handle's own (made
// with the handle), so a numerical failure seen by these kernels is reported by jolt_check_status.
#pragma once

namespace {

// Fixed scratch of the allocation-free decode: 16 MiB per GPU that loads the library, held until exit.
constexpr size_t kStaticScratchBytes = (size_t)16 << 20;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// In host code `g_static_scratch` is only a stand-in symbol, not a device address; the address a
// kernel may use is looked up once per device, with that device current.
static std::mutex g_static_mu;
static void *g_static_ptr[64] = {};

int static_scratch_address(int dev, char **out) {
  std::lock_guard<std::mutex> lk(g_static_mu);
  if (!g_static_ptr[dev]) {
    void *p = nullptr;
    const cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess || !p) { cudaGetLastError(); return fail(JOLT_ECUDA, "cudaGetSymbolAddress(static scratch): %s", cudaGetErrorString(e)); }
    g_static_ptr[dev] = p;
  }
  *out = (char *)g_static_ptr[dev];
  return JOLT_OK;
}

}  // namespace

extern "C" int jolt_decompress_static(const jolt_handle *H, const jolt_layout *L, void *Kout, void *Vout, void *stream) {
  if (!H || !Kout || !Vout) return fail(JOLT_EINVAL, "null argument");
  int rc;
  if ((rc = check_layout(L)) || (rc = check_device_alignment(L, Kout, Vout))) return rc;
  if (L->mem_space != JOLT_MEM_DEVICE) return fail(JOLT_EUNSUPPORTED, "the allocation-free decode writes device memory only");
  if (L->n_layers != H->n_layers || L->n_kv_heads != H->n_kv_heads || L->seq_len != H->T || L->n_groups != H->n_groups)
    return fail(JOLT_EINVAL, "output layout does not match the compressed cache");
  for (int g = 0; g <= L->n_groups; ++g)
    if (L->group_start[g] != H->group_start[g]) return fail(JOLT_EINVAL, "output grouping does not match");
  cudaStream_t st = (cudaStream_t)stream;
  int dev = 0;
  CU(cudaGetDevice(&dev));
  if (dev != H->device) return fail(JOLT_EINVAL, "handle belongs to device %d, current device is %d", H->device, dev);
  if (dev < 0 || dev >= 64) return fail(JOLT_EUNSUPPORTED, "device index %d", dev);
  const int nc = (int)H->cells.size();
  const size_t esz = L->dtype == JOLT_F16 ? 2 : 4;

  // size the scratch before touching the GPU: per cell P (fp16) and the fp32 backbone (the status words live with the
  // handle, allocated when it was made, so that jolt_check_status can report what these kernels saw)
  std::vector<CellWork> ws(nc);
  size_t work_bytes = 0;
  {
    Bump b;
    for (int i = 0; i < nc; ++i) { ws[i].c = H->cells[i].c; ws[i].active = false; carve(b, ws[i], FM_INJECTED, true); }
    work_bytes = (b.off + 255) & ~(size_t)255;
  }
  if (work_bytes > kStaticScratchBytes)
    return fail(JOLT_EINVAL, "cache needs %zu bytes of decode scratch, the static scratch holds %zu", work_bytes, kStaticScratchBytes);
  char *base = nullptr;
  if ((rc = static_scratch_address(dev, &base))) return rc;
  Bump b;
  b.base = base;
  int *d_status = H->d_status;
  for (int i = 0; i < nc; ++i) { ws[i].status = d_status + 4 * i; carve(b, ws[i], FM_INJECTED, true); }

  Program P;
  std::vector<BackboneRef> br;
  std::vector<RowJob> rj(nc);
  long long rows = 0;
  for (int i = 0; i < nc; ++i) {
    const CellStore &cs = H->cells[i];
    const CellDesc &c = cs.c;
    if (c.r_t > 0) br.push_back({c, cs.G16, cs.UT16, cs.UF16, cs.e, ws[i].P16, ws[i].Xt});
    RowJob &j = rj[i];
    memset(&j, 0, sizeof j);
    j.c = c; j.Xt = c.r_t > 0 ? ws[i].Xt : nullptr; j.words = cs.words; j.scales = cs.scales; j.status = d_status + 4 * i;
    j.out = (char *)(i % 2 == 0 ? Kout : Vout) + (size_t)L->group_start[i / 2] * L->stride_layer * esz;
    j.out_dtype = L->dtype == JOLT_F16 ? DT_F16 : DT_F32;
    j.osl = L->stride_layer; j.osh = L->stride_head; j.ost = L->stride_token;
    j.row0 = rows;
    rows += (long long)c.m * c.T;
  }
  add_backbone(P, ST_DBACK, br);
  {
    const size_t off = P.push(rj);
    const uint64_t seed = H->seed;
    P.add(ST_DROWS, [=](char *dev_t, cudaStream_t s) {
      dequant_add_kernel<<<(unsigned)((rows + 127) / 128), 128, 0, s>>>((const RowJob *)(dev_t + off), nc, rows, seed);
      LAUNCHED();
    });
  }
  const size_t total = work_bytes + ((P.host.size() + 255) & ~(size_t)255);
  if (total > kStaticScratchBytes)
    return fail(JOLT_EINVAL, "cache needs %zu bytes of decode scratch, the static scratch holds %zu", total, kStaticScratchBytes);
  char *d_tab = base + work_bytes;
  // the array keeps the previous call's contents; every region of it is fully written before it is read.  The status
  // words (the handle's) start at zero.
  H->last_stream = st;
  CU(cudaMemsetAsync(d_status, 0, sizeof(int) * 4 * nc, st));
  if (!P.host.empty()) CU(cudaMemcpyAsync(d_tab, P.host.data(), P.host.size(), cudaMemcpyHostToDevice, st));
  for (auto &s : P.steps) s.run(d_tab, st);
  CU(cudaGetLastError());
  return JOLT_OK;
}
