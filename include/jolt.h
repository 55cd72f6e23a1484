/*
 * jolt.h -- C ABI of the B200 (sm_100a) JoLT / FlashJoLT KV-cache compressor.
 *
 * One *cell* is a (layer group g, tensor t in {K, V}) pair (paper Sec. 4, first paragraph).  Its data is
 * the tensor X in R^{m x T x d_h}, m = (layers in the group) * n_kv_heads, merged index
 * h = layer_in_group * n_kv_heads + head.  Cell index everywhere: 2*g + (0 for K, 1 for V).
 *
 * Every function returns 0 (JOLT_OK) or a negative jolt_status.  No exception, abort or trap crosses
 * this boundary.  Device pointers are borrowed; the handle owns every compressed buffer.
 * All work is issued on the CUDA stream passed in (a cudaStream_t cast to void*, NULL = default
 * stream); jolt_plan and jolt_compress synchronise that stream before they return (they read back
 * spectra / a status word), jolt_decompress only when the destination is host memory.
 *
 * Concurrency.  Scratch memory and kernel argument tables are one cached arena per device.  Calls may be issued on
 * different streams: every call makes its stream wait (an event, no host synchronisation) for the last launch of the
 * previous call that used the arena, so the GPU work of two library calls on one device never overlaps.  Calls from
 * several host threads on one device must still be serialised by the caller (the event is recorded when a call
 * returns; a second thread that enters in between would build its tables in the same arena).  jolt_decompress_static
 * has a scratch array of its own and the rules stated there.
 */
#ifndef JOLT_H
#define JOLT_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  JOLT_OK = 0,
  JOLT_EINVAL = -1,        /* bad argument (null pointer, shape, plan outside its range)            */
  JOLT_EUNSUPPORTED = -2,  /* valid request that this build does not implement (e.g. head_dim != 128) */
  JOLT_EBUDGET = -3,       /* even the cheapest grid point exceeds the byte budget; plan = cheapest   */
  JOLT_ENUMERIC = -4,      /* Cholesky pivot <= 0, eigen-solver not converged, non-finite scale       */
  JOLT_ENOMEM = -5,        /* host or device allocation failed                                        */
  JOLT_ECUDA = -6,         /* a CUDA runtime / driver call failed (see jolt_last_error)               */
  JOLT_ETIMEOUT = -7       /* a bounded device-side wait ran out (kernel returned, context is usable) */
} jolt_status;

enum { JOLT_F16 = 0, JOLT_F32 = 1 };                 /* element type of the K / V tensors           */
enum { JOLT_MEM_DEVICE = 0, JOLT_MEM_HOST = 1 };      /* where the K / V tensors live                */
enum { JOLT_TOKEN_EXACT = 0, JOLT_TOKEN_RANDOMIZED = 1 };
enum { JOLT_K = 0, JOLT_V = 1 };

/* Shape and strides shared by the K and the V tensor (paper Sec. 4: "partition the L layers into G
 * contiguous groups").  Element (layer l, head n, token t, feature f) sits at
 * l*stride_layer + n*stride_head + t*stride_token + f (in elements; the feature stride is 1).
 * head_dim must be 128; seq_len a multiple of 128; all strides multiples of 8 elements; device tensors must start on
 * a 16-byte boundary (JOLT_EINVAL otherwise: the kernels use 16-byte vector accesses); host tensors are staged and
 * may start anywhere.
 * group_start has n_groups + 1 ascending entries, group_start[0] = 0, group_start[n_groups] = n_layers. */
typedef struct {
  int32_t n_layers, n_kv_heads, seq_len, head_dim;
  int32_t dtype;                    /* JOLT_F16 | JOLT_F32 */
  int32_t mem_space;                /* JOLT_MEM_DEVICE | JOLT_MEM_HOST (host: the call stages the copies) */
  int64_t stride_layer, stride_head, stride_token;
  int32_t n_groups;
  const int32_t *group_start;       /* host array */
} jolt_layout;

/* Ranks and residual bit-width of one cell: the (r_T, r_d, b) of paper Eq. (1).
 * r_t in [0, min(T, m*r_f)], r_t = 0 means no backbone (R = X); r_f in [1, 128] (ignored when r_t = 0);
 * bits in {0, 1, 2, 3, 4, 8}, 0 = no residual stored.  r_t = 0 together with bits = 0 is JOLT_EINVAL. */
typedef struct { int32_t r_t, r_f, bits; } jolt_cell_plan;

/* Options of the token-mode solver (paper Sec. 5) and of the allocator's grid (paper Sec. 4, Eq. (3)). */
typedef struct {
  int32_t token_mode;               /* JOLT_TOKEN_EXACT | JOLT_TOKEN_RANDOMIZED (see below)               */
  int32_t oversample;               /* p: sketch width k = min(r_t + p, T, m*r_f); default 10             */
  int32_t power_iters;              /* q >= 0 power iterations of the range finder                        */
  int32_t quant_group;              /* must be 32                                                         */
  uint64_t seed;                    /* seeds the Gaussian sketch and the rotation signs                   */
  const int32_t *bits_set;          /* host array of allowed bit-widths for jolt_plan; NULL = {0,2,4,8}   */
  int32_t n_bits;
  int32_t rank_step;                /* rank grid = multiples of rank_step (default 16)                    */
  int32_t r_t_min, r_f_min;         /* floors of the grid (default rank_step)                             */
  int32_t q_cap;                    /* <= 0: the paper's cap policy min(max(q_min(R), ceil(T/32)), 512)   */
  const double *eps2;               /* host table eps^2(b) for b = 0..8 (Eq. (2)); NULL = built-in        */
  int32_t count_scale_bytes;        /* 1 (default): the fp16 group scales count toward the budget         */
  int32_t allocator;                /* JOLT_ALLOC_DUAL (default) | JOLT_ALLOC_GREEDY | JOLT_ALLOC_UNIFORM  */
} jolt_options;

/* Allocators of jolt_plan / jolt_allocate.  JOLT_ALLOC_DUAL is the paper's method: the Lagrangian relaxation of
 * Eq. (3) with one multiplier, bisected (Eq. (4)).  The other two are the alternatives its ablations compare against
 * (Sec. 6), described there in one sentence each; the readings taken:
 * JOLT_ALLOC_GREEDY -- every cell starts at its cheapest option; each step applies, among all moves of one cell to a
 *   costlier option with a smaller modelled error that still fits the remaining budget, the one with the largest
 *   error reduction per extra byte; stops when no move is left.
 * JOLT_ALLOC_UNIFORM -- ranks and bits are shared: one (r_t, r_f, bits) for all key cells and one for all value
 *   cells, the pair with the smallest summed modelled error that fits the budget (exhaustive over the grid).
 * All three return JOLT_EBUDGET with the cheapest allocation when nothing fits. */
enum { JOLT_ALLOC_DUAL = 0, JOLT_ALLOC_GREEDY = 1, JOLT_ALLOC_UNIFORM = 2 };

/* JOLT_TOKEN_EXACT (the exact token-mode SVD that Sec. 5 replaces): up to T = 1024 the T x T Gram of the
 * projected unfolding is diagonalised in fp64.  Beyond that the dominant r_t subspace is computed by block
 * subspace iteration on the unfolding (block r_t + max(p, 32), max(q, 8) iterations, Rayleigh-Ritz), and the
 * residual || A V - U S ||_F / || U S ||_F, V = A^T U S^-1, of the result is stored with the cell (component 9);
 * a residual above 5e-4 fails the call with JOLT_ENUMERIC.  jolt_plan in exact mode at T > 1024 probes the
 * top q_cap singular values the same way and accounts the tail mass like the randomized probe. */
typedef struct jolt_handle jolt_handle;

/* Fill *o with the defaults listed above (randomized token mode, p = 10, q = 1, seed 0). */
void jolt_default_options(jolt_options *o);

/* jolt_plan -- paper Sec. 4 "Joint Lagrangian allocation", Eq. (1)-(4), with the spectra of Sec. 5.
 * Measures, per cell, the mode-3 Gram eigenvalues and the leading q_cap token-mode singular values
 * (randomized, plus the tail-mass value) on the GPU, copies them to the host, and runs the Lagrangian
 * dual by bisection so that sum of stored bytes <= byte_budget.
 * dK, dV: the tensors described by `layout`.  out: host array of 2*n_groups plans.
 * achieved_bytes (may be NULL): total stored bytes of the returned plan.
 * Errors: JOLT_EBUDGET leaves the cheapest plan in `out`; other errors leave `out` untouched. */
int jolt_plan(const jolt_layout *layout, const void *dK, const void *dV, double byte_budget,
              const jolt_options *opts, void *stream, jolt_cell_plan *out, double *achieved_bytes);

/* The two halves of jolt_plan, for callers that plan one cache at several budgets or with several allocators (the
 * ratio sweeps and allocator ablations of Sec. 6): the spectra are measured once and every further plan is host work.
 * jolt_probe -- Sec. 5: mode-3 Gram eigenvalues and the leading q_cap token-mode singular values of every cell (plus the
 *   tail-mass value of the randomized probe), measured by one GPU program per cell group on concurrent streams and
 *   copied to the host in one transfer.  q_cap = opts->q_cap if positive, else the cap policy at `ratio_hint`
 *   (uncompressed bytes over the byte budget the caller has in mind).  *out: a host object, free with
 *   jolt_spectra_free; NULL on error.
 * jolt_plan_from_spectra -- Sec. 4, Eq. (3)/(4) on the kept spectra; no GPU work, token ranks bounded by the probed cap.
 *   JOLT_EINVAL if the cap policy of this budget asks for more token directions than were probed (probe again with a
 *   larger q_cap); JOLT_EBUDGET as jolt_plan.
 * jolt_plan(budget) == jolt_probe(ratio of that budget) followed by jolt_plan_from_spectra(budget). */
typedef struct jolt_spectra jolt_spectra;
int jolt_probe(const jolt_layout *layout, const void *dK, const void *dV, double ratio_hint, const jolt_options *opts,
               void *stream, jolt_spectra **out);
int jolt_plan_from_spectra(const jolt_spectra *spectra, double byte_budget, const jolt_options *opts,
                           jolt_cell_plan *out, double *achieved_bytes);
int jolt_spectra_free(jolt_spectra *spectra);

/* jolt_compress -- paper Sec. 4 "Partial Tucker backbone" + "Rotated residual", Sec. 5 for the
 * randomized token factor.  For every cell: U_F from the mode-3 Gram, U_T (exact or randomized),
 * core G, residual against the stored fp16 backbone, sign-flip + 128-point Hadamard rotation along
 * features, per-32-feature absmax mid-rise quantisation to `bits` bits, bit-packing.
 * plan: host array of 2*n_groups cell plans.  *out receives a new handle (free with jolt_free).
 * On error *out is NULL. */
int jolt_compress(const jolt_layout *layout, const void *dK, const void *dV, const jolt_cell_plan *plan,
                  const jolt_options *opts, void *stream, jolt_handle **out);

/* Test hook: as jolt_compress but with the factors given instead of computed.
 * UT[c], UF[c]: host fp32 arrays, row-major T x r_t and 128 x r_f, for cell c (entries for cells
 * with r_t = 0 are ignored).  The library rounds them to fp16, forms the core and proceeds. */
int jolt_compress_with_factors(const jolt_layout *layout, const void *dK, const void *dV,
                               const jolt_cell_plan *plan, const jolt_options *opts,
                               const float *const *UT, const float *const *UF, void *stream,
                               jolt_handle **out);

/* jolt_decompress -- paper Sec. 4 "decoding simply inverts the rotation", Sec. 7 (decode reconstructs
 * the cache from its factors): X^ = U_T (G U_F^T) + s . H(dequant(codes)) / sqrt(d), written in
 * out_layout->dtype to dK_out / dV_out (shape must equal the compressed shape; strides may differ). */
int jolt_decompress(const jolt_handle *h, const jolt_layout *out_layout, void *dK_out, void *dV_out,
                    void *stream);

/* jolt_decompress_rope -- paper App. "RoPE pre vs. post on K": keys are decomposed before the rotary
 * position embedding, which is applied again when the cache is decoded.  The paper names the operation
 * without a formula; this entry point takes the common rotate-half form on head_dim 128: for token t at
 * position p = pos0 + t and feature j < 64, with angle p * base^(-j/64),
 *     K_out[.., t, j]      = K^[.., t, j] cos - K^[.., t, j + 64] sin
 *     K_out[.., t, j + 64] = K^[.., t, j + 64] cos + K^[.., t, j] sin
 * where K^ is the decoded key before it is rounded to the destination type.  V is written as by
 * jolt_decompress.  Angles are evaluated in fp64, the rotation in fp32.  Key cells decoded by the tensor-core
 * kernel with r_t <= 128 are rotated inside that kernel and rounded once; the other key cells are rotated by a
 * separate in-place pass over the decoded tensor, so an fp16 destination is rounded after decoding and again
 * after the rotation (jolt_set_fast_path bit 3 off sends every cell that way).  rope: host pointer; 1 < base < 1e12, 0 <= pos0 <= 2^40 (JOLT_EINVAL otherwise).  All other
 * arguments, the result and the error behaviour are those of jolt_decompress. */
typedef struct {
  double base;   /* frequency base (10000 in the original formulation) */
  int64_t pos0;  /* position of token 0 of this cache */
} jolt_rope;
int jolt_decompress_rope(const jolt_handle *h, const jolt_layout *out_layout, void *dK_out, void *dV_out,
                         const jolt_rope *rope, void *stream);

/* jolt_attend -- paper Sec. 7 and closing discussion: attention "directly on the factors, without materializing
 * the cache" is named as the route to decode parity; no algorithm is given.  This entry point computes single-step
 * softmax attention over the compressed cache, for every layer and KV head at once:
 *     O[l, h, i, :] = sum_t softmax_t( scale * <Q[l, h, i, :], K^[l, h, t, :]> ) V^[l, h, t, :]
 * where K^, V^ are the decoded cells before their rounding to an output type (what jolt_decompress would write to an
 * fp32 destination, up to fp32 rounding).  Neither is formed: the backbone terms are contracted with the small factors
 * first, the residual terms against a query rotated once per head, so the call reads the compressed bytes once.
 *   dQ, dOut: device, fp32, contiguous [n_layers][n_kv_heads][n_q][128], 16-byte aligned; n_q = queries per KV head,
 *   1..8 (the grouped-query group size).  Keys are used as stored: a cache whose keys were compressed before a rotary
 *   embedding needs jolt_decompress_rope instead (the rotation differs per token and does not commute with the
 *   contraction).  Scratch comes from the library's per-device workspace (grown on first use).  The first call on a
 *   handle also forms the projected cores P_h = fp16(G_h U_F^T) of all cells (m * r_t * 128 fp16 values per cell,
 *   about 5 % of the compressed size on the benchmark workload) in a device buffer that stays with the handle
 *   until jolt_free; later calls, on any stream, reuse them (a first call that fails leaves nothing behind; the next
 *   call forms them again).  Errors: JOLT_EINVAL
 *   (null / misaligned pointers, n_q out of range, wrong device), JOLT_EUNSUPPORTED (ranks that are not multiples
 *   of 8; sequences beyond about 3 million tokens), JOLT_ENOMEM, JOLT_ECUDA.  Asynchronous on `stream`.  Arithmetic:
 *   fp32; the contractions that run on the tensor cores take their fp32 operand as hi + lo fp16 (about 22 bits) and
 *   accumulate in fp32. */
int jolt_attend(const jolt_handle *h, const void *dQ, int32_t n_q, double scale, void *dOut, void *stream);

/* jolt_decompress_static -- the paper has no counterpart; this is a deployment variant of jolt_decompress
 * for callers that cannot allocate device memory while decoding (a serving process that has given all free
 * memory to its own pool, a thread for which a driver allocation would stall the context, a host whose
 * allocator policy forbids cudaMalloc after start-up).  It calls no cudaMalloc / cudaFree and no allocating
 * library routine: all scratch (projected cores, the fp32 backbone buffer, status words, kernel argument
 * tables) lives in one fixed 16 MiB device array that is part of the library image, so every GPU that loads
 * the library holds those 16 MiB until the process exits.
 *   - Arguments and result as jolt_decompress, device destinations only (JOLT_MEM_HOST -> JOLT_EUNSUPPORTED).
 *   - A cache whose decode scratch (about 4 bytes per cache element of cells with a backbone, plus
 *     2*m*r_t*128 bytes per such cell) exceeds 16 MiB is rejected with JOLT_EINVAL and a message that names
 *     both sizes; nothing is launched.
 *   - The first call on a device looks up the device address of the array (one cudaGetSymbolAddress with
 *     that device current); make that first call before any stream capture.
 *   - Every call shares the one array and finds the previous call's contents in it; the call clears what must
 *     start at zero.  Two calls that overlap on the GPU (different streams, or different threads) race on
 *     the array: issue them on one stream, or serialise them yourself. */
int jolt_decompress_static(const jolt_handle *h, const jolt_layout *out_layout, void *dK_out, void *dV_out,
                           void *stream);

/* Persistence of a compressed cache (paper Sec. 7: the footprint that shrinks is "the persistent state ... what matters
 * for prompt-caching deployments that keep many cached prefixes resident"; no format is given).  jolt_serialize writes a
 * self-describing image -- header, layer grouping, cell descriptors, then the stored arrays exactly as they sit in device
 * memory -- into host memory; jolt_deserialize maps such an image back into a new handle on the current device, with
 * which jolt_decompress / jolt_attend give bit-identical results.  The image is tied to this library version and to the
 * host's byte order.  host_dst / host_src: host pointers (pinned memory makes the copy asynchronous up to the final
 * synchronisation; both calls return after the copy has finished).  Errors: JOLT_EINVAL (null pointers, a buffer
 * smaller than jolt_serialized_bytes, an image that is truncated or fails its consistency checks), JOLT_ENOMEM,
 * JOLT_ECUDA; on error *out is NULL. */
int jolt_serialized_bytes(const jolt_handle *h, int64_t *bytes);
int jolt_serialize(const jolt_handle *h, void *host_dst, int64_t cap, void *stream);
int jolt_deserialize(const void *host_src, int64_t bytes, void *stream, jolt_handle **out);

/* Release a handle and all buffers it owns.  NULL is accepted.  The compressed buffers are returned to the
 * stream-ordered pool after the last call that read them (ordered on that call's stream; if that stream no longer
 * exists, after the device has gone idle), so a decode that is still running keeps its data. */
int jolt_free(jolt_handle *h);

/* Stored bytes of the compressed cache: factors + core + packed codes + scales, i.e. Eq. (1) plus
 * the scale term, summed over cells. */
int jolt_compressed_bytes(const jolt_handle *h, int64_t *bytes);

/* Read one stored component of one cell back to host memory (tests, serialisation).
 * which: 0 = core (fp16 bits, [m][r_t][r_f]), 1 = U_T (fp16, [T][r_t]), 2 = U_F (fp16, [128][r_f]),
 * 3 = packed codes (uint32, [m][T][4*bits]), 4 = scales (fp16, [m][T][4]), 5 = core exponent (int32),
 * 6 = token-mode singular values (fp32, k entries, 0 entries if injected), 7 = mode-3 eigenvalues
 * (fp32, 128; zeros when r_f = 128), 8 = the token factor before fp16 rounding (fp32, [T][r_t]; a view of
 * scratch memory, valid only until the next library call on the device; for tests), 9 = residual of the
 * converged-subspace check (fp32, one value; 0 bytes unless the handle was made in exact mode at T > 1024).
 * dst_bytes is the capacity of dst; *written gets the size of the component. */
int jolt_get_component(const jolt_handle *h, int32_t cell, int32_t which, void *dst, int64_t dst_bytes,
                       int64_t *written);

/* Host-only allocator (no GPU): the Lagrangian dual of Eq. (3)/(4) on caller-supplied spectra.
 * For cell c: lam3[c*128 .. +128) mode-3 Gram eigenvalues (descending); sig2sq + sig2_off[c] points at
 * sig2_len[c] squared token-mode singular values (descending; last one may be the synthetic tail
 * value); total_sq[c] = ||X||^2.  m[c], T, d describe the cell.  Grid and eps2 come from opts.
 * r_t_max[c] bounds the token rank grid.  out: n_cells plans. */
int jolt_allocate(int32_t n_cells, const int32_t *m, int32_t T, int32_t d, const double *lam3,
                  const double *sig2sq, const int64_t *sig2_off, const int32_t *sig2_len,
                  const double *total_sq, const int32_t *r_t_max, double byte_budget,
                  const jolt_options *opts, jolt_cell_plan *out, double *achieved_bytes);

/* Stored bytes of one cell at a given plan (Eq. (1), c = 2, plus 2*M/32 scale bytes if bits > 0 and
 * count_scale_bytes). */
int64_t jolt_cell_bytes(int32_t m, int32_t T, int32_t d, int32_t r_t, int32_t r_f, int32_t bits,
                        int32_t count_scale_bytes);

/* The cap policy of paper Sec. 5: min(max(q_min(R), ceil(T/32)), 512). */
int32_t jolt_cap_policy(int32_t T, double ratio);

/* Built-in eps^2(b) calibration (Gaussian round trip through the quantiser), b = 0..8; entries for
 * unsupported widths are NaN. */
int jolt_eps2_table(double out[9]);

/* Seeded draws of the method, exposed so that tests can compare them with an independent
 * implementation: n_rows x n_cols Gaussian sketch (host fp32 out) and the 128 rotation signs. */
int jolt_sketch_host(uint64_t seed, int32_t cell, int32_t stream_id, int64_t n_rows, int32_t n_cols, float *out);
int jolt_signs_host(uint64_t seed, int32_t cell, float out[128]);

/* Free cached device workspace held by the library for the current device. */
int jolt_release_workspace(void);

/* Number of kernel launches the library has issued since load (all streams). */
int64_t jolt_launch_count(void);

/* Selects the kernel family by bit mask: 0 = portable SIMT kernels only; bit 0 = fused tcgen05 backbone
 * kernels (decode, residual) and the tensor-core forms of jolt_attend's code streams, bit 1 = tcgen05 factor sweeps (sketch, projection), bit 2 = tcgen05 mode-3
 * Gram, bit 3 = rotary embedding inside the decode kernel (jolt_decompress_rope; otherwise a separate pass),
 * bit 4 = eigen-solver resident in a thread-block cluster (otherwise one launch per Jacobi round),
 * bit 5 = CholeskyQR of the range finder on tensor cores (otherwise fp64 SIMT Gram and row-wise triangular solve),
 * bit 6 = factor sweeps with two output tiles per CTA (otherwise one);
 * bit 7 = persistent decode kernel (one CTA per SM walks a share of all tiles; otherwise one CTA per 16-tile item;
 *         launches with a cell of r_t > 128, with keys rotated at decode or with cells of different sequence
 *         lengths always take the per-item kernel);
 * 255 (default) = all, where the shapes allow.  Returns the previous mask. */
int jolt_set_fast_path(int enabled);

/* Number of cell groups whose factor stages jolt_compress runs side by side on internal streams (1..8, default 4):
 * the small solvers between the sweeps are latency chains, which overlap with the GPU-filling kernels of other groups.
 * 1 runs every stage for all cells before the next one starts (the setting under which jolt_last_stage_ms attributes
 * the whole call to its stages).  Returns the previous value. */
int jolt_set_stream_groups(int n);

/* jolt_check_status -- device-side outcome of the last decode on this handle (jolt_decompress, jolt_decompress_rope,
 * jolt_decompress_static; these are asynchronous and return before their kernels have run).  Every device-side wait of
 * the kernels is bounded (a wait that runs out raises a status bit, the kernel drains and exits), and a quantisation step that is not finite in fp16 raises another.  Copies the handle's status
 * words back on `stream`, synchronises that stream, and returns JOLT_OK, JOLT_ETIMEOUT or JOLT_ENUMERIC.  Decodes into
 * host memory synchronise anyway and return this status themselves. */
int jolt_check_status(const jolt_handle *h, void *stream);

/* Test hook.  cycles > 0 replaces the limit of every bounded device-side wait (default 10^9 SM cycles, about half a
 * second).  skip_first_load = 1 makes the TMA thread of the two-tile sweep kernel leave out its first load, so that the
 * consumer's wait runs out: the kernel must drain, release its tensor memory and report JOLT_ETIMEOUT through
 * jolt_compress, and the next call on the same context must work.  skip_first_load = 2 does the same to the U_T thread
 * of the persistent decode kernel: the launch ends, jolt_check_status reports JOLT_ETIMEOUT, the next decode works.
 * cycles <= 0 and skip_first_load = 0 restore the defaults.  Applies to the current device. */
int jolt_test_set_wait_limit(int64_t cycles, int32_t skip_first_load);

/* Test hook for the persistent decode kernel.  Its CTAs take fixed shares of the launch's tile list; the kernel can
 * also hand the last `percent` % of the list out in chunks of `chunk_tiles` tiles to whichever CTA asks first.  The
 * library leaves that tail empty (it measured slower); this switch turns it on so that tests cover the path.
 * percent in [0, 100], chunk_tiles >= 1; (0, anything) restores the default.  Returns JOLT_EINVAL otherwise. */
int jolt_test_set_decode_tail(int32_t percent, int32_t chunk_tiles);

/* Wall-clock-free per-stage device timing of the last compress / decompress on this thread
 * (milliseconds, CUDA events): out[0..n) in stage order, names via jolt_stage_name. */
int jolt_last_stage_ms(float *out, int32_t cap, int32_t *n);
const char *jolt_stage_name(int32_t i);

const char *jolt_strerror(int status);
const char *jolt_last_error(void);   /* thread-local detail of the last failure */

#ifdef __cplusplus
}
#endif
#endif /* JOLT_H */
