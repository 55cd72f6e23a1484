"""Pins of the error-context baselines (Sec. 6, reconstruction table): closed forms, exact cases, brute force."""
import itertools

import numpy as np

from oracle import baselines as BL


def test_int4_rate_is_the_papers_native_floor():
    # Sec. 6, footnote of the reconstruction table: the fixed-rate 4-bit quantiser achieves about 3.97x at T = 1024
    assert abs(BL.int4_per_channel_ratio(1024) - 3.97) < 0.005
    X = np.random.default_rng(0).standard_normal((3, 1024, 128))
    _, stored = BL.int4_per_channel(X)
    assert abs(X.size * 2 / stored - BL.int4_per_channel_ratio(1024)) < 1e-12


def test_int4_reproduces_a_sixteen_level_channel_exactly():
    rng = np.random.default_rng(1)
    m, T, d = 2, 64, 8
    lo = rng.integers(-8, 8, size=(m, 1, d)) / 4.0                 # fp16-exact zero points
    step = 2.0 ** rng.integers(-6, 2, size=(m, 1, d))              # fp16-exact steps
    codes = rng.integers(0, 16, size=(m, T, d))
    codes[:, 0, :] = 0
    codes[:, 1, :] = 15                                            # the channel spans all sixteen levels
    X = lo + codes * step
    Xh, _ = BL.int4_per_channel(X)
    assert np.array_equal(Xh, X)
    C = np.full((1, 16, 4), 0.375)                                 # a constant channel has step 0 and is exact too
    assert np.array_equal(BL.int4_per_channel(C)[0], C)


def test_int4_matches_brute_force_nearest_level():
    rng = np.random.default_rng(2)
    X = rng.standard_normal((1, 9, 3))
    Xh, _ = BL.int4_per_channel(X)
    for f in range(3):
        col = X[0, :, f]
        lo, hi = col.min(), col.max()
        step = float(np.float16((hi - lo) / 15.0)); zero = float(np.float16(lo))
        levels = zero + step * np.arange(16)
        for t in range(9):
            best = levels[np.argmin(np.abs(levels - col[t]))]
            # ties between two levels may round either way: accept any level at the minimum distance
            assert abs(abs(Xh[0, t, f] - col[t]) - abs(best - col[t])) < 1e-12
    # error bound: half a step plus the rounding of the zero point pushed through 15 levels
    step = np.float16((X.max(axis=1) - X.min(axis=1)) / 15.0).astype(np.float64)
    assert np.all(np.abs(Xh - X) <= 0.5 * step[:, None, :] + 2.0 ** -10 * (np.abs(X).max() + 15 * step.max()))


def test_cross_layer_rank_fills_the_budget():
    for T, N, ratio in itertools.product((256, 1024), (1024, 8192), (2.0, 3.0)):
        r = BL.cross_layer_rank(T, N, ratio)
        budget = 2 * T * N / ratio
        assert 2 * r * (T + N) <= budget < 2 * (r + 1) * (T + N)


def test_cross_layer_svd_error_is_the_discarded_spectrum():
    rng = np.random.default_rng(3)
    L, nh, T, d = 2, 2, 48, 8
    N = L * nh * d
    U, _ = np.linalg.qr(rng.standard_normal((T, N)))
    V, _ = np.linalg.qr(rng.standard_normal((N, N)))
    s = 2.0 ** -np.arange(N, dtype=np.float64) * 8.0
    A = (U * s) @ V.T
    Xg = A.reshape(T, L, nh, d).transpose(1, 2, 0, 3)
    Xh, stored, r = BL.cross_layer_svd(Xg, 2.0)
    assert r == BL.cross_layer_rank(T, N, 2.0) and stored == 2 * r * (T + N)
    want = np.sqrt((s[r:] ** 2).sum() / (s ** 2).sum())            # Eckart-Young, from the constructed spectrum
    got = BL.rel_frobenius(Xg, Xh)
    assert abs(got - want) <= 2.0 ** -9 + 1e-3 * want              # fp16 rounding of the two stored factors


def test_cross_layer_svd_stacks_layers_along_features():
    # every layer and head carries the SAME T x d matrix of rank 3: the stacked matrix still has rank 3, so any
    # budget with r >= 3 reproduces the group up to the fp16 rounding of the factors; stacking along tokens instead
    # would not change that, but folding back in the wrong order would scramble the entries
    rng = np.random.default_rng(4)
    L, nh, T, d = 3, 2, 40, 16
    B = rng.standard_normal((T, 3)) @ rng.standard_normal((3, d))
    Xg = np.broadcast_to(B, (L, nh, T, d)) * (1.0 + np.arange(L * nh).reshape(L, nh, 1, 1))
    Xh, _, r = BL.cross_layer_svd(Xg, 2.0)
    assert r >= 3
    assert np.max(np.abs(Xh - Xg)) <= 2.0 ** -8 * np.abs(Xg).max()
