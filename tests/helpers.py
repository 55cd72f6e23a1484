"""Shared helpers of the parity tests: run the oracle cell by cell on the same bytes the library got."""
import math

import numpy as np

from oracle import jolt_oracle as O


def cell_view(K, V, group_start, cell):
    g, which = divmod(cell, 2)
    t = (K, V)[which][group_start[g]:group_start[g + 1]]
    L, nh, T, d = t.shape
    return t.reshape(L * nh, T, d)


def oracle_cache(Knp, Vnp, group_start, plans, *, seed, token_mode, oversample=10, power_iters=1, out_dtype="f16",
                 factors=None):
    cells = []
    for c, (rt, rf, b) in enumerate(plans):
        X = cell_view(Knp, Vnp, group_start, c).astype(np.float64)
        fac = None
        if factors is not None and rt > 0:
            fac = (factors[0][c].astype(np.float64), factors[1][c].astype(np.float64))
        cells.append(O.compress_cell(X, rt, rf, b, seed=seed, cell=c, token_mode=token_mode, oversample=oversample,
                                     power_iters=power_iters, out_dtype=out_dtype, factors=fac))
    return cells


def projector_distance(U, U0):
    """|| U U^T - U0 U0^T ||_F without forming T x T matrices."""
    a = np.linalg.norm(U.T @ U) ** 2 + np.linalg.norm(U0.T @ U0) ** 2 - 2 * np.linalg.norm(U.T @ U0) ** 2
    return math.sqrt(max(a, 0.0))


def code_mismatch(codes_gpu, codes_ref):
    """(fraction of differing codes, max |difference|)."""
    d = codes_gpu.astype(np.int32) - codes_ref.astype(np.int32)
    nz = d != 0
    return float(nz.mean()), int(np.abs(d).max()) if d.size else 0


def cell_from_handle(h, c, m, T, plan, seed, out_dtype="f16"):
    """The oracle's CompressedCell built from the library's OWN stored components of cell c (core, exponent, factors,
    packed words, scales); the rotation signs come from the oracle's generator.  Decoding it with the oracle pins the
    library's decode kernels with no quantisation ambiguity: both sides then hold identical stored numbers."""
    rt, rf, b = plan
    if rt > 0:
        G = h.component(c, 0).astype(np.float64).reshape(m, rt, rf)
        e = int(h.component(c, 5)[0])
        UT = h.component(c, 1).astype(np.float64).reshape(T, rt)
        UF = h.component(c, 2).astype(np.float64).reshape(128, rf)
    else:
        G, e, UT, UF = np.zeros((m, 0, 0)), 0, np.zeros((T, 0)), np.zeros((128, 0))
        rf = 0
    words = scales = None
    if b > 0:
        words = h.component(c, 3).reshape(m, T, 4 * b)
        scales = h.component(c, 4).reshape(m, T, 4)
    return O.CompressedCell(m, T, 128, rt, rf, b, 32, e, G, UT, UF, O.rotation_signs(seed, c), words, scales, out_dtype)


def fp16_ulp(x):
    """Spacing of fp16 numbers at |x| (subnormal spacing 2^-24 below 2^-14)."""
    a = np.maximum(np.abs(np.asarray(x, dtype=np.float64)), 2.0 ** -14)
    return 2.0 ** (np.floor(np.log2(a)) - 10)


def decode_elementwise_bound(oc, out_dtype="f16"):
    """Per-entry bound on |library decode - oracle decode| for identical stored components.

    The library forms each output entry as ONE fp32 tensor-core accumulation of the backbone terms U_T[t,k] P[k,f] and
    of the dequantised residual (rounded to fp16, relative 2^-11 per term) times the +-1 rotation, then rounds once to
    the output type; the oracle does the same sum in float64.  Hence, per entry:
      one rounding step of the output type
      + 2^-11 * ||r^'_row||_2            (fp16 operand rounding of the residual; Cauchy-Schwarz over the 128 terms / sqrt(128))
      + 2^-17 * sum_k |U_T[t,k] P[k,f]| 2^e   (fp32 accumulation of the tensor core, which truncates: ~2^-24 per MMA step,
                                               taken with a wide margin)
      + 2^-10 * max_k |U_T[t,k]| max_k |P[k,f]| 2^e   (one entry of the fp16 projected core one step off)."""
    m, T, d = oc.m, oc.T, oc.d
    Xo = O.decoded_unrounded(oc)
    step = fp16_ulp(Xo) if out_dtype == "f16" else np.abs(Xo) * 2.0 ** -23 + 1e-30
    res = 0.0
    if oc.bits > 0:
        codes = O.unpack_codes(oc.words, oc.bits, d)
        rp = O.dequantize_rows(codes, oc.scales, oc.bits, oc.group)
        res = 2.0 ** -11 * np.linalg.norm(rp, axis=-1, keepdims=True)
    bb = 0.0
    if oc.r_t > 0:
        P = np.abs(O.fp16_round(np.einsum("hrs,fs->hrf", oc.Gs16, oc.UF16, optimize=True)))
        bb = 2.0 ** -17 * math.ldexp(1.0, oc.e) * np.einsum("tr,hrf->htf", np.abs(oc.UT16), P, optimize=True)
        # the projected core P = fp16(G U_F^T) is itself rounded from an fp32 sum on the device: an entry that sits on a
        # rounding boundary may come out one fp16 step away, which moves the output by 2^-11 of one term
        bb = bb + 2.0 ** -10 * math.ldexp(1.0, oc.e) * np.abs(oc.UT16).max(axis=1)[None, :, None] * P.max(axis=1)[:, None, :]
    return step + res + bb


def oracle_codes_for_stored_backbone(X, oc):
    """Codes and scales the definition gives for the residual of X against the backbone stored in `oc` (a cell built by
    cell_from_handle): R = X - X~(stored), rotate, quantise (Sec. 4 "Rotated residual")."""
    Xt = O.stored_backbone(oc.Gs16, oc.e, oc.UT16, oc.UF16) if oc.r_t > 0 else 0.0
    Rp = O.rotate(np.asarray(X, dtype=np.float64) - Xt, oc.signs)
    return O.quantize_rows(Rp, oc.bits, oc.group)
