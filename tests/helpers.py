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
