"""ctypes binding of the C ABI in include/jolt.h: argument marshalling only.

Every step of the path runs in the CUDA library; there is no Python or CPU fallback.  Importing
this module without the built library raises.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libjolt.so")
if not os.path.exists(_LIB_PATH):
    raise ImportError(f"{_LIB_PATH} is missing: run `python -m paper_2607_12550_b200.build` (nvcc, sm_100a)")
lib = C.CDLL(_LIB_PATH)

OK, EINVAL, EUNSUPPORTED, EBUDGET, ENUMERIC, ENOMEM, ECUDA, ETIMEOUT = 0, -1, -2, -3, -4, -5, -6, -7
F16, F32 = 0, 1
MEM_DEVICE, MEM_HOST = 0, 1
TOKEN_EXACT, TOKEN_RANDOMIZED = 0, 1
ALLOC_DUAL, ALLOC_GREEDY, ALLOC_UNIFORM = 0, 1, 2


class Layout(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("n_kv_heads", C.c_int32), ("seq_len", C.c_int32), ("head_dim", C.c_int32),
                ("dtype", C.c_int32), ("mem_space", C.c_int32),
                ("stride_layer", C.c_int64), ("stride_head", C.c_int64), ("stride_token", C.c_int64),
                ("n_groups", C.c_int32), ("group_start", C.POINTER(C.c_int32))]


class CellPlan(C.Structure):
    _fields_ = [("r_t", C.c_int32), ("r_f", C.c_int32), ("bits", C.c_int32)]


class Options(C.Structure):
    _fields_ = [("token_mode", C.c_int32), ("oversample", C.c_int32), ("power_iters", C.c_int32),
                ("quant_group", C.c_int32), ("seed", C.c_uint64),
                ("bits_set", C.POINTER(C.c_int32)), ("n_bits", C.c_int32),
                ("rank_step", C.c_int32), ("r_t_min", C.c_int32), ("r_f_min", C.c_int32), ("q_cap", C.c_int32),
                ("eps2", C.POINTER(C.c_double)), ("count_scale_bytes", C.c_int32), ("allocator", C.c_int32)]


_vp = C.c_void_p
lib.jolt_default_options.argtypes = [C.POINTER(Options)]
lib.jolt_default_options.restype = None
lib.jolt_plan.argtypes = [C.POINTER(Layout), _vp, _vp, C.c_double, C.POINTER(Options), _vp, C.POINTER(CellPlan),
                          C.POINTER(C.c_double)]
lib.jolt_probe.argtypes = [C.POINTER(Layout), _vp, _vp, C.c_double, C.POINTER(Options), _vp, C.POINTER(_vp)]
lib.jolt_plan_from_spectra.argtypes = [_vp, C.c_double, C.POINTER(Options), C.POINTER(CellPlan), C.POINTER(C.c_double)]
lib.jolt_spectra_free.argtypes = [_vp]
lib.jolt_compress.argtypes = [C.POINTER(Layout), _vp, _vp, C.POINTER(CellPlan), C.POINTER(Options), _vp, C.POINTER(_vp)]
lib.jolt_compress_with_factors.argtypes = [C.POINTER(Layout), _vp, _vp, C.POINTER(CellPlan), C.POINTER(Options),
                                           C.POINTER(_vp), C.POINTER(_vp), _vp, C.POINTER(_vp)]
lib.jolt_decompress.argtypes = [_vp, C.POINTER(Layout), _vp, _vp, _vp]
lib.jolt_free.argtypes = [_vp]


class Rope(C.Structure):
    _fields_ = [("base", C.c_double), ("pos0", C.c_int64)]


lib.jolt_decompress_rope.argtypes = [_vp, C.POINTER(Layout), _vp, _vp, C.POINTER(Rope), _vp]
lib.jolt_decompress_static.argtypes = [_vp, C.POINTER(Layout), _vp, _vp, _vp]
lib.jolt_attend.argtypes = [_vp, _vp, C.c_int32, C.c_double, _vp, _vp]
lib.jolt_serialized_bytes.argtypes = [_vp, C.POINTER(C.c_int64)]
lib.jolt_serialize.argtypes = [_vp, _vp, C.c_int64, _vp]
lib.jolt_deserialize.argtypes = [_vp, C.c_int64, _vp, C.POINTER(_vp)]
lib.jolt_compressed_bytes.argtypes = [_vp, C.POINTER(C.c_int64)]
lib.jolt_get_component.argtypes = [_vp, C.c_int32, C.c_int32, _vp, C.c_int64, C.POINTER(C.c_int64)]
lib.jolt_allocate.argtypes = [C.c_int32, C.POINTER(C.c_int32), C.c_int32, C.c_int32, C.POINTER(C.c_double),
                              C.POINTER(C.c_double), C.POINTER(C.c_int64), C.POINTER(C.c_int32), C.POINTER(C.c_double),
                              C.POINTER(C.c_int32), C.c_double, C.POINTER(Options), C.POINTER(CellPlan),
                              C.POINTER(C.c_double)]
lib.jolt_cell_bytes.argtypes = [C.c_int32] * 7
lib.jolt_cell_bytes.restype = C.c_int64
lib.jolt_cap_policy.argtypes = [C.c_int32, C.c_double]
lib.jolt_cap_policy.restype = C.c_int32
lib.jolt_eps2_table.argtypes = [C.POINTER(C.c_double)]
lib.jolt_sketch_host.argtypes = [C.c_uint64, C.c_int32, C.c_int32, C.c_int64, C.c_int32, C.POINTER(C.c_float)]
lib.jolt_signs_host.argtypes = [C.c_uint64, C.c_int32, C.POINTER(C.c_float)]
lib.jolt_release_workspace.argtypes = []
lib.jolt_launch_count.argtypes = []
lib.jolt_launch_count.restype = C.c_int64
lib.jolt_set_fast_path.argtypes = [C.c_int]
lib.jolt_set_stream_groups.argtypes = [C.c_int]
lib.jolt_check_status.argtypes = [_vp, _vp]
lib.jolt_test_set_wait_limit.argtypes = [C.c_int64, C.c_int32]
lib.jolt_test_set_decode_tail.argtypes = [C.c_int32, C.c_int32]
lib.jolt_last_stage_ms.argtypes = [C.POINTER(C.c_float), C.c_int32, C.POINTER(C.c_int32)]
lib.jolt_stage_name.argtypes = [C.c_int32]
lib.jolt_stage_name.restype = C.c_char_p
lib.jolt_strerror.argtypes = [C.c_int]
lib.jolt_strerror.restype = C.c_char_p
lib.jolt_last_error.argtypes = []
lib.jolt_last_error.restype = C.c_char_p


class JoltError(RuntimeError):
    def __init__(self, status: int):
        self.status = status
        super().__init__(f"{lib.jolt_strerror(status).decode()} ({status}): {lib.jolt_last_error().decode()}")


def _check(status: int, allow=()):
    if status != OK and status not in allow:
        raise JoltError(status)
    return status


@dataclass
class _Keep:
    layout: Layout
    gs: object


def make_layout(K: torch.Tensor, group_start: Sequence[int], V: torch.Tensor | None = None) -> Layout:
    """Layout of a [n_layers, n_kv_heads, T, 128] tensor (any strides with unit feature stride).

    The C ABI describes K and V by ONE layout: when V is given it must match K in shape, strides, dtype and device."""
    assert K.dim() == 4 and K.stride(3) == 1
    if V is not None and (V.shape != K.shape or V.stride() != K.stride() or V.dtype != K.dtype or V.device != K.device):
        raise ValueError("K and V must share shape, strides, dtype and device (one jolt_layout describes both)")
    gs = (C.c_int32 * len(group_start))(*group_start)
    lay = Layout(K.shape[0], K.shape[1], K.shape[2], K.shape[3],
                 F16 if K.dtype == torch.float16 else F32,
                 MEM_DEVICE if K.is_cuda else MEM_HOST,
                 K.stride(0), K.stride(1), K.stride(2), len(group_start) - 1, gs)
    lay._gs = gs  # keep alive
    return lay


def default_options(**kw) -> Options:
    o = Options()
    lib.jolt_default_options(C.byref(o))
    keep = []
    for k, v in kw.items():
        if k == "bits_set":
            arr = (C.c_int32 * len(v))(*v)
            keep.append(arr)
            o.bits_set = arr
            o.n_bits = len(v)
        elif k == "eps2":
            arr = (C.c_double * 9)(*v)
            keep.append(arr)
            o.eps2 = arr
        else:
            setattr(o, k, v)
    o._keep = keep
    return o


def _stream_ptr(stream):
    if stream is None:
        return None
    return C.c_void_p(stream.cuda_stream)


def _plans(plans) -> C.Array:
    arr = (CellPlan * len(plans))()
    for i, p in enumerate(plans):
        arr[i] = CellPlan(*p)
    return arr


def jolt_plan(K, V, group_start, byte_budget: float, opts: Options | None = None, stream=None, allow_budget=False):
    lay = make_layout(K, group_start, V)
    opts = opts or default_options()
    out = (CellPlan * (2 * lay.n_groups))()
    ach = C.c_double(0)
    st = lib.jolt_plan(C.byref(lay), K.data_ptr(), V.data_ptr(), byte_budget, C.byref(opts), _stream_ptr(stream), out,
                       C.byref(ach))
    _check(st, allow=(EBUDGET,) if allow_budget else ())
    return [(p.r_t, p.r_f, p.bits) for p in out], ach.value


class Spectra:
    """The measured spectra of a cache (host object); plan it at any budget with `plan`."""

    def __init__(self, ptr, n_cells):
        self.ptr = ptr
        self.n_cells = n_cells

    def plan(self, byte_budget: float, opts: Options | None = None, allow_budget=False):
        opts = opts or default_options()
        out = (CellPlan * self.n_cells)()
        ach = C.c_double(0)
        st = lib.jolt_plan_from_spectra(self.ptr, byte_budget, C.byref(opts), out, C.byref(ach))
        _check(st, allow=(EBUDGET,) if allow_budget else ())
        return [(p.r_t, p.r_f, p.bits) for p in out], ach.value

    def free(self):
        if self.ptr:
            lib.jolt_spectra_free(self.ptr)
            self.ptr = None

    def __del__(self):
        if lib is not None:
            self.free()


def jolt_probe(K, V, group_start, ratio_hint: float, opts: Options | None = None, stream=None) -> Spectra:
    lay = make_layout(K, group_start, V)
    opts = opts or default_options()
    ptr = C.c_void_p()
    _check(lib.jolt_probe(C.byref(lay), K.data_ptr(), V.data_ptr(), float(ratio_hint), C.byref(opts), _stream_ptr(stream),
                          C.byref(ptr)))
    return Spectra(ptr, 2 * lay.n_groups)


class Handle:
    """Owns a compressed cache; freed on `free()` or garbage collection."""

    def __init__(self, ptr, n_cells):
        self.ptr = ptr
        self.n_cells = n_cells

    def free(self):
        if self.ptr:
            lib.jolt_free(self.ptr)
            self.ptr = None

    def __del__(self):
        self.free()

    def bytes(self) -> int:
        b = C.c_int64(0)
        _check(lib.jolt_compressed_bytes(self.ptr, C.byref(b)))
        return b.value

    _DT = {0: np.float16, 1: np.float16, 2: np.float16, 3: np.uint32, 4: np.float16, 5: np.int32, 6: np.float32,
           7: np.float32, 8: np.float32, 9: np.float32}

    def component(self, cell: int, which: int) -> np.ndarray:
        n = C.c_int64(0)
        _check(lib.jolt_get_component(self.ptr, cell, which, None, 0, C.byref(n)))
        buf = np.empty(n.value // np.dtype(self._DT[which]).itemsize, dtype=self._DT[which])
        if n.value:
            _check(lib.jolt_get_component(self.ptr, cell, which, buf.ctypes.data, n.value, C.byref(n)))
        return buf


def jolt_compress(K, V, group_start, plans, opts: Options | None = None, stream=None, factors=None) -> Handle:
    lay = make_layout(K, group_start, V)
    opts = opts or default_options()
    arr = _plans(plans)
    h = C.c_void_p(None)
    if factors is None:
        st = lib.jolt_compress(C.byref(lay), K.data_ptr(), V.data_ptr(), arr, C.byref(opts), _stream_ptr(stream), C.byref(h))
    else:
        UT, UF = factors
        uts = [np.ascontiguousarray(u, dtype=np.float32) if u is not None else None for u in UT]
        ufs = [np.ascontiguousarray(u, dtype=np.float32) if u is not None else None for u in UF]
        pt = (C.c_void_p * len(uts))(*[u.ctypes.data if u is not None else None for u in uts])
        pf = (C.c_void_p * len(ufs))(*[u.ctypes.data if u is not None else None for u in ufs])
        st = lib.jolt_compress_with_factors(C.byref(lay), K.data_ptr(), V.data_ptr(), arr, C.byref(opts), pt, pf,
                                            _stream_ptr(stream), C.byref(h))
    _check(st)
    return Handle(h.value, len(plans))


def jolt_decompress(handle: Handle, K_out, V_out, group_start, stream=None):
    lay = make_layout(K_out, group_start, V_out)
    _check(lib.jolt_decompress(handle.ptr, C.byref(lay), K_out.data_ptr(), V_out.data_ptr(), _stream_ptr(stream)))


def jolt_decompress_rope(handle: Handle, K_out, V_out, group_start, base=10000.0, pos0=0, stream=None):
    """Decode and re-apply the rotary embedding to the keys (rotate-half form); see include/jolt.h."""
    lay = make_layout(K_out, group_start, V_out)
    rope = Rope(float(base), int(pos0))
    _check(lib.jolt_decompress_rope(handle.ptr, C.byref(lay), K_out.data_ptr(), V_out.data_ptr(), C.byref(rope),
                                    _stream_ptr(stream)))


def jolt_decompress_static(handle: Handle, K_out, V_out, group_start, stream=None):
    """Decode without any device allocation (fixed 16 MiB scratch inside the library); see include/jolt.h."""
    lay = make_layout(K_out, group_start, V_out)
    _check(lib.jolt_decompress_static(handle.ptr, C.byref(lay), K_out.data_ptr(), V_out.data_ptr(), _stream_ptr(stream)))


def jolt_attend(handle: Handle, Q, scale=None, stream=None):
    """Single-step attention of Q [n_layers, n_kv_heads, n_q, 128] (fp32, CUDA) over the compressed cache; see include/jolt.h."""
    assert Q.dim() == 4 and Q.dtype == torch.float32 and Q.is_cuda and Q.is_contiguous()
    out = torch.empty_like(Q)
    sc = float(scale) if scale is not None else 1.0 / (Q.shape[-1] ** 0.5)
    _check(lib.jolt_attend(handle.ptr, Q.data_ptr(), Q.shape[2], sc, out.data_ptr(), _stream_ptr(stream)))
    return out


def jolt_serialize(handle: Handle, stream=None) -> np.ndarray:
    """The compressed cache as a self-describing byte image (host numpy array); see include/jolt.h."""
    n = C.c_int64(0)
    _check(lib.jolt_serialized_bytes(handle.ptr, C.byref(n)))
    buf = np.empty(n.value, dtype=np.uint8)
    _check(lib.jolt_serialize(handle.ptr, buf.ctypes.data, n.value, _stream_ptr(stream)))
    return buf


def jolt_deserialize(image: np.ndarray, stream=None) -> Handle:
    image = np.ascontiguousarray(image, dtype=np.uint8)
    h = _vp()
    _check(lib.jolt_deserialize(image.ctypes.data, image.size, _stream_ptr(stream), C.byref(h)))
    hd = np.frombuffer(image[:48].tobytes(), dtype=np.int32)
    return Handle(h.value, int(hd[8]))


def jolt_free(handle: Handle):
    handle.free()


def jolt_allocate(m, T, d, lam3, sig2sq_list, total_sq, r_t_max, byte_budget, opts: Options | None = None,
                  allow_budget=False):
    n = len(m)
    opts = opts or default_options()
    lam = np.ascontiguousarray(np.asarray(lam3, dtype=np.float64).reshape(n, 128))
    offs, lens, flat = [], [], []
    for s in sig2sq_list:
        offs.append(len(flat))
        lens.append(len(s))
        flat.extend(float(x) for x in s)
    flat = np.asarray(flat, dtype=np.float64)
    out = (CellPlan * n)()
    ach = C.c_double(0)
    st = lib.jolt_allocate(n, (C.c_int32 * n)(*m), T, d, lam.ctypes.data_as(C.POINTER(C.c_double)),
                           flat.ctypes.data_as(C.POINTER(C.c_double)), (C.c_int64 * n)(*offs), (C.c_int32 * n)(*lens),
                           (C.c_double * n)(*total_sq), (C.c_int32 * n)(*r_t_max), byte_budget, C.byref(opts), out,
                           C.byref(ach))
    _check(st, allow=(EBUDGET,) if allow_budget else ())
    return [(p.r_t, p.r_f, p.bits) for p in out], ach.value, st


def cell_bytes(m, T, d, r_t, r_f, bits, scales=True) -> int:
    return lib.jolt_cell_bytes(m, T, d, r_t, r_f, bits, 1 if scales else 0)


def cap_policy(T, ratio) -> int:
    return lib.jolt_cap_policy(T, ratio)


def eps2_table():
    t = (C.c_double * 9)()
    _check(lib.jolt_eps2_table(t))
    return list(t)


def sketch_host(seed, cell, stream_id, n_rows, n_cols) -> np.ndarray:
    out = np.empty((n_rows, n_cols), dtype=np.float32)
    _check(lib.jolt_sketch_host(seed, cell, stream_id, n_rows, n_cols, out.ctypes.data_as(C.POINTER(C.c_float))))
    return out


def signs_host(seed, cell) -> np.ndarray:
    out = np.empty(128, dtype=np.float32)
    _check(lib.jolt_signs_host(seed, cell, out.ctypes.data_as(C.POINTER(C.c_float))))
    return out


def stage_ms() -> dict:
    buf = (C.c_float * 32)()
    n = C.c_int32(0)
    _check(lib.jolt_last_stage_ms(buf, 32, C.byref(n)))
    return {lib.jolt_stage_name(i).decode(): buf[i] for i in range(n.value) if buf[i] > 0}


def launch_count() -> int:
    return lib.jolt_launch_count()


def set_fast_path(enabled) -> int:
    """False / 0: portable kernels only; True / 255: every sm_100a kernel; other ints: bit mask
    (1 = fused backbone kernels, 2 = factor sweeps, 4 = Gram, 8 = rotary embedding inside the decode kernel,
    16 = cluster-resident eigen-solver, 32 = CholeskyQR on tensor cores, 64 = two output tiles per CTA in the factor sweeps,
    128 = persistent decode kernel).  Returns the previous mask."""
    if enabled is True:
        enabled = 255
    return lib.jolt_set_fast_path(int(enabled))


def set_stream_groups(n: int) -> int:
    """Number of cell groups jolt_compress runs side by side (1 = stage by stage); returns the previous value."""
    return lib.jolt_set_stream_groups(int(n))


def check_status(handle: "Handle", stream=None):
    """Device-side outcome of the last decode on the handle (synchronises the stream); raises JoltError on failure."""
    _check(lib.jolt_check_status(handle.ptr, _stream_ptr(stream)))


def set_test_wait_limit(cycles: int = 0, skip_first_load=False):
    """Test hook of the bounded device-side waits (skip_first_load: False / True = the sweep kernel / 2 = the persistent
    decode kernel); see include/jolt.h."""
    _check(lib.jolt_test_set_wait_limit(int(cycles), int(skip_first_load)))


def set_test_decode_tail(percent: int = 0, chunk_tiles: int = 8):
    """Test hook: chunked tail of the persistent decode kernel's tile list; see include/jolt.h."""
    _check(lib.jolt_test_set_decode_tail(int(percent), int(chunk_tiles)))


def release_workspace():
    lib.jolt_release_workspace()
