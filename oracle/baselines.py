"""Error-context baselines of the reconstruction table (Sec. 6, "Reconstruction fidelity"), restated from their
one-line descriptions.  TEST INFRASTRUCTURE: plain numpy float64, written to be checked by eye; only tests/, the smoke
check and the CPU-baseline leg of bench.py may import it.  Nothing here is a port of the cited systems' code.

  int4 per-channel      every (head, feature channel) of a cell keeps one fp16 step and one fp16 zero point for all of
                        its T tokens; entries become 4-bit codes (asymmetric min/max quantiser).  Its rate is fixed:
                        16 / (4 + 32 / T) x, the "native floor" of about 3.97x the table's footnote quotes at T = 1024.
  cross-layer SVD       the layers of a group are stacked along the feature axis into one T x (layers * heads * d)
                        matrix, which is replaced by its best rank-r approximation; both factors are kept in fp16 and r
                        is the largest rank whose bytes stay within the target ratio.

Both functions return the reconstruction and the bytes they store, so the caller can report the achieved ratio beside
the error (the table compares errors at matched budgets only where a method can reach the budget).
"""
from __future__ import annotations

import numpy as np


def fp16_round(x):
    return np.asarray(x, dtype=np.float64).astype(np.float16).astype(np.float64)


def int4_per_channel(X):
    """X[m][T][d] -> (X^, stored bytes).  Channel = (head, feature): min/max over the T tokens, 16 levels."""
    X = np.asarray(X, dtype=np.float64)
    m, T, d = X.shape
    lo = X.min(axis=1, keepdims=True)
    hi = X.max(axis=1, keepdims=True)
    step = fp16_round((hi - lo) / 15.0)
    zero = fp16_round(lo)
    safe = np.where(step > 0, step, 1.0)
    codes = np.clip(np.rint((X - zero) / safe), 0, 15)
    Xh = zero + codes * step
    stored = m * T * d * 4 // 8 + m * d * 2 * 2          # 4-bit codes + fp16 (step, zero) per channel
    return Xh, stored


def int4_per_channel_ratio(T: int) -> float:
    """Compression ratio of the scheme above against an fp16 cache: 16 bits over 4 bits plus 32 bits per T tokens."""
    return 16.0 / (4.0 + 32.0 / T)


def cross_layer_rank(T: int, N: int, ratio: float) -> int:
    """Largest r with fp16 factors U[T][r], W[N][r] inside the byte budget 2 T N / ratio."""
    return max(1, int(np.floor(T * N / (ratio * (T + N)))))


def cross_layer_svd(Xg, ratio: float):
    """Xg[layers][heads][T][d] (one layer group, K or V) -> (X^ of the same shape, stored bytes, r).

    The group is unfolded to A[T][layers * heads * d]; A ~ U_r diag(s_r) V_r^T with the singular values folded into the
    right factor, both factors rounded to fp16."""
    Xg = np.asarray(Xg, dtype=np.float64)
    L, nh, T, d = Xg.shape
    N = L * nh * d
    A = Xg.transpose(2, 0, 1, 3).reshape(T, N)
    r = min(cross_layer_rank(T, N, ratio), min(T, N))
    U, s, Vt = np.linalg.svd(A, full_matrices=False)
    U16 = fp16_round(U[:, :r])
    W16 = fp16_round((s[:r, None] * Vt[:r]).T)            # N x r
    Ah = U16 @ W16.T
    Xh = Ah.reshape(T, L, nh, d).transpose(1, 2, 0, 3)
    stored = 2 * r * (T + N)
    return Xh, stored, r


def rel_frobenius(X, Xh):
    X = np.asarray(X, dtype=np.float64)
    return float(np.linalg.norm(X - np.asarray(Xh, dtype=np.float64)) / max(np.linalg.norm(X), 1e-300))
