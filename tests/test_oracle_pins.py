"""Pins for the CPU oracle: what the paper and the mathematics fix, independent of the oracle's own code."""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import jolt_oracle as O

RNG = np.random.default_rng(1234)


def _golden():
    vals = {}
    with open(os.path.join(os.path.dirname(__file__), "golden", "paper_values.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if "=" in line:
                k, v = line.split("=")
                vals[k.strip()] = float(v)
    return vals


# ----------------------------------------------------------------------------- RNG
def test_mix64_is_splitmix64():
    # SplitMix64 started from state 0 emits these words (Steele, Lea, Flood 2014; widely tabulated).
    state, outs = 0, []
    for _ in range(3):
        outs.append(int(O.mix64(np.uint64(state))))
        state = (state + 0x9E3779B97F4A7C15) & (2 ** 64 - 1)
    assert outs == [0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F]


def test_gaussian_moments_and_fp16_grid():
    g = O.gaussian_sketch(7, 3, 4096, 64)
    assert g.shape == (4096, 64)
    assert np.array_equal(g, g.astype(np.float16).astype(np.float64))     # defined on the fp16 grid
    n = g.size
    assert abs(g.mean()) < 4 / math.sqrt(n)
    assert abs(g.var() - 1) < 4 * math.sqrt(2 / n) + 1e-6
    assert abs((g ** 4).mean() - 3) < 0.1
    # columns nearly uncorrelated
    c = np.corrcoef(g.T)
    assert np.abs(c - np.eye(64)).max() < 0.1
    # different cells / seeds give different streams
    assert not np.array_equal(g, O.gaussian_sketch(7, 4, 4096, 64))
    assert not np.array_equal(g, O.gaussian_sketch(8, 3, 4096, 64))


def test_signs_balanced_and_pm1():
    s = np.stack([O.rotation_signs(5, c) for c in range(200)])
    assert set(np.unique(s)) == {-1.0, 1.0}
    assert abs(s.mean()) < 0.03


# ----------------------------------------------------------------------------- rotation
def test_hadamard_matches_sylvester_recursion():
    H = np.array([[1.0]])
    while H.shape[0] < 128:
        H = np.block([[H, H], [H, -H]])
    assert np.array_equal(H, O.hadamard_matrix(128))
    assert np.array_equal(H @ H, 128 * np.eye(128))
    assert np.array_equal(H, H.T)


def test_rotation_is_orthogonal_involution():
    s = O.rotation_signs(1, 0)
    R = RNG.standard_normal((3, 17, 128))
    Rp = O.rotate(R, s)
    assert np.allclose(np.linalg.norm(Rp, axis=-1), np.linalg.norm(R, axis=-1), rtol=1e-13)
    assert np.abs(O.unrotate(Rp, s) - R).max() < 1e-14
    # a single outlier channel is spread evenly: |r'_j| = |r_c| / sqrt(d) for all j
    e = np.zeros(128)
    e[5] = 3.0
    assert np.allclose(np.abs(O.rotate(e, s)), 3.0 / math.sqrt(128))


# ----------------------------------------------------------------------------- quantiser
@pytest.mark.parametrize("bits", [1, 2, 3, 4, 8])
def test_quantiser_error_bound_and_range(bits):
    x = RNG.standard_normal((500, 128)) * np.exp(RNG.standard_normal((500, 1)) * 3)
    codes, sc = O.quantize_rows(x, bits)
    assert codes.min() >= 0 and codes.max() <= (1 << bits) - 1
    xh = O.dequantize_rows(codes, sc, bits)
    g = x.reshape(500, 4, 32)
    a = np.abs(g).max(-1, keepdims=True)
    delta = sc.astype(np.float64)[..., None]
    err = np.abs(g - xh.reshape(500, 4, 32))
    # half a step, plus the clamped top bin after fp16 rounding of the step (relative 2^-11 for a
    # normal step, absolute 2^-25 per level for a subnormal one)
    assert np.all(err <= delta / 2 + a * 2.0 ** -10 + (1 << bits) * 2.0 ** -25)


def test_quantiser_is_floor_of_ratio():
    # brute-force restatement on a group whose step is exactly representable: absmax 4, b = 3 -> Delta = 1
    x = np.zeros((1, 128))
    vals = np.array([-4.0, -3.5, -2.01, -1.0, -0.25, 0.0, 0.25, 0.99, 1.0, 2.5, 3.999, 4.0])
    x[0, :12] = vals
    codes, sc = O.quantize_rows(x, 3)
    assert float(sc[0, 0]) == 1.0
    expect = np.clip(np.floor(vals), -4, 3) + 4
    assert np.array_equal(codes[0, :12], expect.astype(np.uint8))
    xh = O.dequantize_rows(codes, sc, 3)
    assert np.array_equal(xh[0, :12], expect - 4 + 0.5)
    # all-zero groups: mid code, dequantises to 0
    assert np.all(codes[0, 32:] == 4) and np.all(xh[0, 32:] == 0)


def test_single_precision_reciprocal_form_is_within_the_code_tolerance():
    """The definition takes floor(r' / Delta) in float64.  A kernel that multiplies by a single-precision reciprocal
    lands in the neighbouring bin only where r' / Delta is within rounding distance of an integer: never by more
    than one code, and on far fewer than the 0.1 % of entries the code-parity gate allows."""
    x = np.random.default_rng(77).standard_normal((4096, 128)) * 0.37
    for bits in (1, 2, 3, 4, 8):
        codes, sc = O.quantize_rows(x, bits)
        half = float(1 << (bits - 1))
        g = x.reshape(4096, 4, 32).astype(np.float32)
        d32 = sc.astype(np.float32)
        inv = (np.float32(1.0) / d32).astype(np.float32)
        q = np.clip(np.floor(g * inv[..., None]), -half, half - 1.0) + half
        diff = np.abs(q.reshape(4096, 128).astype(np.int64) - codes.astype(np.int64))
        assert diff.max() <= 1
        assert (diff != 0).mean() <= 2e-4


def test_one_bit_is_sign_quantiser():
    x = RNG.standard_normal((10, 128))
    codes, sc = O.quantize_rows(x, 1)
    assert np.array_equal(codes, (x >= 0).astype(np.uint8))


def test_eps2_decreasing_and_four_per_bit():
    e = O.eps2_table([0, 1, 2, 3, 4, 8], n=1 << 16)
    assert e[0] == _golden()["eps2_zero_bits"]
    assert e[0] > e[1] > e[2] > e[3] > e[4] > e[8]
    assert 3.5 < e[2] / e[3] < 4.5 and 3.5 < e[3] / e[4] < 4.5
    assert 200 < e[4] / e[8] < 300


@pytest.mark.parametrize("bits", [1, 2, 3, 4, 8])
def test_pack_matches_bitstring_definition(bits):
    codes = RNG.integers(0, 1 << bits, size=(6, 128), dtype=np.uint8)
    words = O.pack_codes(codes, bits)
    assert words.shape == (6, 4 * bits) and words.dtype == np.uint32
    for r in range(6):
        for g in range(4):
            big = 0
            for j in range(32):
                big |= int(codes[r, g * 32 + j]) << (j * bits)
            for w in range(bits):
                assert int(words[r, g * bits + w]) == (big >> (32 * w)) & 0xFFFFFFFF
    assert np.array_equal(O.unpack_codes(words, bits, 128), codes)


def test_pack_exhaustive_single_positions():
    for bits in (1, 2, 3, 4, 8):
        for j in range(32):
            for v in {1, (1 << bits) - 1}:
                codes = np.zeros((1, 32), dtype=np.uint8)
                codes[0, j] = v
                w = O.pack_codes(codes, bits)
                big = sum(int(x) << (32 * i) for i, x in enumerate(w[0]))
                assert big == v << (j * bits)
                assert np.array_equal(O.unpack_codes(w, bits, 32), codes)


# ----------------------------------------------------------------------------- Tucker backbone
def _lowrank(m, T, d, rt, rf, noise=0.0, rng=RNG):
    G = rng.standard_normal((m, rt, rf))
    UT = np.linalg.qr(rng.standard_normal((T, rt)))[0]
    UF = np.linalg.qr(rng.standard_normal((d, rf)))[0]
    X = O.reconstruct(G, UT, UF)
    return X + noise * rng.standard_normal(X.shape)


def test_feature_factor_is_eigenbasis_of_gram():
    X = RNG.standard_normal((3, 50, 128))
    U, lam = O.feature_factor(X, 128)
    C = O.mode3_gram(X)
    assert np.allclose(C, np.einsum("htf,htg->fg", X, X))
    assert np.linalg.norm(U.T @ U - np.eye(128)) < 1e-12
    assert np.linalg.norm(C @ U - U * lam) < 1e-10 * np.linalg.norm(C)
    assert np.all(np.diff(lam) <= 1e-9)
    # eigenvalues are the squared singular values of the mode-3 unfolding (library special case)
    sv = np.linalg.svd(X.reshape(-1, 128), compute_uv=False)
    assert np.allclose(lam, sv ** 2, rtol=1e-10)


def test_full_rank_reconstructs_exactly():
    X = RNG.standard_normal((2, 24, 128))
    U_F, _ = O.feature_factor(X, 128)
    A = O.token_unfold(np.einsum("htf,fs->hts", X, U_F))
    U_T, _ = O.token_factor_exact(A, 24)
    G = O.core_tensor(X, U_T, U_F)
    assert np.abs(O.reconstruct(G, U_T, U_F) - X).max() < 1e-12


def test_unfold_index_convention():
    Y = RNG.standard_normal((3, 5, 4))
    A = O.token_unfold(Y)
    assert A.shape == (5, 12)
    assert A[2, 1 * 4 + 3] == Y[1, 2, 3]


def test_exact_lowrank_input_truncates_to_zero_error():
    X = _lowrank(4, 64, 128, 6, 9)
    c = O.compress_cell(X, 6, 9, 0, token_mode="exact")
    i = c.ideal
    assert np.abs(O.reconstruct(i["G"], i["U_T"], i["U_F"]) - X).max() < 1e-11
    c2 = O.compress_cell(X, 6, 9, 0, token_mode="randomized", oversample=4, power_iters=0)
    i2 = i2 = c2.ideal
    assert np.abs(O.reconstruct(i2["G"], i2["U_T"], i2["U_F"]) - X).max() < 1e-10


@pytest.mark.parametrize("mode", ["exact", "randomized"])
def test_orthonormal_factors_and_energy_split(mode):
    X = _lowrank(4, 96, 128, 20, 30, noise=0.3)
    c = O.compress_cell(X, 12, 16, 0, token_mode=mode, seed=3, cell=1)
    U_T, U_F, G = c.ideal["U_T"], c.ideal["U_F"], c.ideal["G"]
    assert np.linalg.norm(U_T.T @ U_T - np.eye(12)) < 1e-12
    assert np.linalg.norm(U_F.T @ U_F - np.eye(16)) < 1e-12
    R = X - O.reconstruct(G, U_T, U_F)
    assert abs(np.sum(X ** 2) - np.sum(G ** 2) - np.sum(R ** 2)) < 1e-10 * np.sum(X ** 2)


def test_sthosvd_sandwich_bound():
    X = _lowrank(4, 96, 128, 30, 40, noise=0.2)
    rt, rf = 10, 24
    c = O.compress_cell(X, rt, rf, 0, token_mode="exact")
    i = c.ideal
    R2 = np.sum((X - O.reconstruct(i["G"], i["U_T"], i["U_F"])) ** 2)
    lam = i["lam"]
    s2 = np.linalg.svd(O.token_unfold(X), compute_uv=False) ** 2
    tail3, tail2 = lam[rf:].sum(), s2[rt:].sum()
    assert max(tail2, tail3) * (1 - 1e-10) <= R2 <= (tail2 + tail3) * (1 + 1e-10)


def test_randomized_equals_exact_when_sketch_covers_rank():
    X = _lowrank(3, 80, 128, 7, 128)
    A = O.token_unfold(X)  # rank 7
    Ue, _ = O.token_factor_exact(A, 7)
    Om = O.gaussian_sketch(0, 0, A.shape[1], 12)
    for q in (0, 1):
        Ur = O.token_factor_randomized(A, 7, Om, q)[0]
        assert np.linalg.norm(Ue @ Ue.T - Ur @ Ur.T) < 1e-10


def test_randomized_error_decreases_with_power_iterations_and_ignores_qr_variant():
    X = _lowrank(4, 128, 128, 60, 128, noise=0.0)
    A = O.token_unfold(X) * 1.0
    U, s, Vt = np.linalg.svd(A, full_matrices=False)
    A = (U * (np.arange(1, len(s) + 1) ** -0.7)) @ Vt          # slow decay: the hard case
    Om = O.gaussian_sketch(1, 0, A.shape[1], 20)
    errs = []
    for q in (0, 1, 2):
        Ur = O.token_factor_randomized(A, 10, Om, q)[0]
        errs.append(np.linalg.norm(A - Ur @ (Ur.T @ A)))
    best = np.linalg.norm(A - U[:, :10] @ (U[:, :10].T @ A))
    assert errs[0] > errs[1] > errs[2] >= best * (1 - 1e-12)
    # same range with an SVD-based orthonormalisation instead of QR
    old = O._orth
    try:
        O._orth = lambda S: np.linalg.svd(S, full_matrices=False)[0]
        Ur2 = O.token_factor_randomized(A, 10, Om, 1)[0]
    finally:
        O._orth = old
    Ur1 = O.token_factor_randomized(A, 10, Om, 1)[0]
    assert np.linalg.norm(Ur1 @ Ur1.T - Ur2 @ Ur2.T) < 1e-8


def test_core_equals_projected_b_in_randomized_path():
    X = _lowrank(3, 64, 128, 20, 128, noise=0.1)
    A = O.token_unfold(X)
    Om = O.gaussian_sketch(0, 0, A.shape[1], 18)
    U_T, s, Q, Ut, B = O.token_factor_randomized(A, 8, Om, 1)
    G = O.core_tensor(X, U_T, np.eye(128))
    assert np.allclose(O.token_unfold(np.transpose(G, (0, 1, 2))).reshape(8, -1), Ut[:, :8].T @ B, atol=1e-10)
    assert np.allclose(np.sum(G ** 2), np.sum(s[:8] ** 2))


def test_core_scale_exponent():
    for mx in (1e-3, 0.7, 1.0, 1023.0, 1024.0, 5e4, 3e7):
        e = O.core_scale_exponent(np.array([mx, -mx / 3]))
        assert 2 ** 10 <= mx * 2.0 ** -e < 2 ** 11
    assert O.core_scale_exponent(np.zeros(3)) == 0


@pytest.mark.parametrize("bits", [1, 2, 4, 8])
def test_closed_loop_roundtrip_error_is_quantisation_only(bits):
    X = _lowrank(2, 64, 128, 10, 20, noise=0.2) * 3
    c = O.compress_cell(X, 8, 16, bits, seed=11, cell=2, out_dtype="f32")
    Xh = O.decompress_cell(c)
    # per row: ||x^ - x|| = ||r^' - r'|| <= sqrt(d) * (Delta_max/2 + clamp slack), rotation is orthogonal
    delta = c.scales.astype(np.float64).max(-1)
    amax = np.abs(O.rotate(c.ideal["R_stored"], c.signs)).max(-1)
    bound = math.sqrt(128) * (delta / 2 + amax * 2.0 ** -10) + 1e-5
    assert np.all(np.linalg.norm(Xh - X, axis=-1) <= bound)
    # and rank-0 mode (no backbone) is a pure rotated quantiser
    c0 = O.compress_cell(X, 0, 0, bits, seed=11, cell=2, out_dtype="f32")
    assert c0.UT16.shape[1] == 0
    e0, e1 = O.rel_frobenius(X, O.decompress_cell(c0)), O.rel_frobenius(X, Xh)
    assert e1 < e0


def test_bits_zero_stores_no_residual():
    X = _lowrank(2, 32, 128, 4, 8, noise=0.1)
    c = O.compress_cell(X, 4, 8, 0, out_dtype="f32")
    assert c.words is None and c.scales is None
    Xh = O.decompress_cell(c)
    assert np.allclose(Xh, O.stored_backbone(c.Gs16, c.e, c.UT16, c.UF16).astype(np.float32))


def test_stored_backbone_decodes_an_exactly_low_rank_cell_at_any_magnitude():
    """bits = 0 and an input of exact multilinear rank (r_t, r_f): the stored backbone IS the decode, so it must give
    X back to fp16-storage accuracy -- also when the core has to be scaled down (entries above the fp16 range) or up
    (entries below the fp16 normal range) by the per-cell exponent, which a wrong sign or offset of that exponent
    would miss by orders of magnitude."""
    base = _lowrank(3, 96, 128, 6, 12, noise=0.0, rng=np.random.default_rng(5))
    for scale in (1.0, 3.0e4, 2.0e-7):
        X = base * scale
        c = O.compress_cell(X, 6, 12, 0, token_mode="exact", out_dtype="f32")
        mx = np.abs(c.ideal["G"]).max()
        if scale > 1e3:
            assert mx > 65504 and c.e > 0          # would overflow fp16 unscaled
        if scale < 1e-3:
            assert mx < 2.0 ** -14 and c.e < 0     # would be subnormal unscaled
        assert np.abs(c.Gs16).max() < 2048 and np.abs(c.Gs16).max() >= 1024
        Xh = O.stored_backbone(c.Gs16, c.e, c.UT16, c.UF16)
        # three fp16 roundings (core, two factors) and one of P_h: a few 2^-11 relative
        assert O.rel_frobenius(X, Xh) <= 2.5e-3
        assert O.rel_frobenius(X, O.decompress_cell(c)) <= 2.5e-3
    # independent restatement with explicit loops on a tiny cell
    c = O.compress_cell(base[:, :16] * 50.0, 4, 8, 0, token_mode="exact", out_dtype="f32")
    Xh = O.stored_backbone(c.Gs16, c.e, c.UT16, c.UF16)
    h, t, f = 1, 5, 77
    P = [float(np.float16(sum(c.Gs16[h, r, s_] * c.UF16[f, s_] for s_ in range(8)))) for r in range(4)]
    assert abs(Xh[h, t, f] - 2.0 ** c.e * sum(c.UT16[t, r] * P[r] for r in range(4))) <= 1e-12 * abs(Xh[h, t, f]) + 1e-300


def test_plan_spectra_are_the_mode_spectra():
    """What the allocator consumes: exact mode gives the squared singular values of the two unfoldings (both sum to
    ||X||^2); the randomized probe gives the same leading values plus a zero tail once its cap covers the rank."""
    X = _lowrank(3, 64, 128, 9, 128, noise=0.0, rng=np.random.default_rng(8)) * 2.0
    tot = float(np.sum(X * X))
    lam, s2, total = O.plan_spectra(X, 16, token_mode="exact")
    assert abs(total - tot) <= 1e-12 * tot
    assert abs(np.sum(s2) - tot) <= 1e-10 * tot and abs(np.sum(lam) - tot) <= 1e-10 * tot
    s3 = np.linalg.svd(X.reshape(-1, 128), compute_uv=False)
    assert np.allclose(lam, s3 ** 2, rtol=1e-9, atol=1e-9 * tot)
    s2_ref = np.linalg.svd(np.transpose(X, (1, 0, 2)).reshape(64, -1), compute_uv=False) ** 2
    assert np.allclose(s2[:9], s2_ref[:9], rtol=1e-10)
    lam_r, s2_r, total_r = O.plan_spectra(X, 16, token_mode="randomized", seed=3, cell=1, power_iters=1)
    assert len(s2_r) == 17 and total_r == total
    assert np.allclose(s2_r[:9], s2_ref[:9], rtol=1e-9)          # the cap (16) covers the token rank (9)
    assert np.all(s2_r[9:] <= 1e-9 * tot)                        # nothing is left for the synthetic tail value
    # with a cap below the rank the tail value carries exactly the omitted mass
    lam_c, s2_c, _ = O.plan_spectra(X, 4, token_mode="randomized", seed=3, cell=1, power_iters=2)
    assert len(s2_c) == 5 and abs(np.sum(s2_c) - tot) <= 1e-10 * tot
    assert s2_c[4] >= np.sum(s2_ref[4:9]) * (1 - 1e-6)


# ----------------------------------------------------------------------------- bytes, cap policy
def test_eq1_closed_form_and_printed_cache_size():
    g = _golden()
    L, nh, d = int(g["mistral_layers"]), int(g["mistral_kv_heads"]), int(g["head_dim"])
    T = 2048
    # full-rank, 16-bit "residual" with no factors == raw fp16 cache: (b/8) m T d term alone
    raw = 2 * sum(O.eq1_bytes(4 * nh, T, d, 0, 0, 16) for _ in range(L // 4))
    assert raw == 268435456
    assert round(raw / 1e6, 1) == g["mistral_ctx2048_cache_MB"]
    m, rt, rf, b = 32, 48, 64, 4
    assert O.eq1_bytes(m, T, d, rt, rf, b) == (m * rt * rf + T * rt + d * rf) * 2 + b * m * T * d // 8
    assert O.stored_bytes(m, T, d, rt, rf, b) - O.eq1_bytes(m, T, d, rt, rf, b) == 2 * m * T * d // 32
    assert O.stored_bytes(m, T, d, rt, rf, 0) == O.eq1_bytes(m, T, d, rt, rf, 0)


def test_cap_policy_printed_values():
    g = _golden()
    assert O.cap_policy(1024, 3) == g["cap_T1024"]
    for T in (128, 512, 1024):
        assert O.cap_policy(T, 2) == g["cap_qmin_low_ratio"]      # no-op for T <= 1024
        assert O.cap_policy(T, 5) == g["cap_qmin_high_ratio"]
    assert O.cap_policy(4096, 2) == 128 and O.cap_policy(8192, 3) == 256
    assert O.cap_policy(32768, 2.5) == g["cap_max"] and O.cap_policy(10 ** 6, 8) == g["cap_max"]
    assert O.cap_policy(2049, 4) == 65


def test_tail_mass_accounting_conserves_energy():
    s = np.array([5.0, 3.0, 1.0])
    spec = O.tail_mass_spectrum(s, 40.0)
    assert len(spec) == 4 and abs(np.sum(spec ** 2) - 40.0) < 1e-12
    assert O.tail_mass_spectrum(s, 34.0)[-1] == 0.0


def test_tau_table_limits():
    lam = np.array([4.0, 2.0, 1.0, 1.0])
    s2 = np.array([5.0, 2.0, 1.0])
    tau = O.tau_table(lam, s2, 8.0, [0, 1, 3], [0, 2, 4])
    assert tau[0, 0] == 1.0                       # nothing kept
    assert tau[2, 2] == 0.0                       # everything kept
    assert tau[1, 1] == (3.0 + 2.0) / 8.0


# ----------------------------------------------------------------------------- dual
def _brute(cells, budget):
    best, best_e = None, math.inf
    for combo in itertools.product(*[range(len(c[0])) for c in cells]):
        cost = sum(c[1][i] for c, i in zip(cells, combo))
        if cost <= budget:
            e = sum(c[0][i] for c, i in zip(cells, combo))
            if e < best_e:
                best, best_e = combo, e
    return best, best_e


def test_dual_everett_optimality_by_brute_force():
    rng = np.random.default_rng(5)
    for trial in range(6):
        cells = []
        for _ in range(4):
            costs = np.sort(rng.integers(10, 400, size=9)).astype(np.float64)
            errs = np.sort(rng.random(9))[::-1].copy()
            cells.append((errs, costs))
        lo = sum(c[1].min() for c in cells)
        hi = sum(c[1].max() for c in cells)
        for budget in np.linspace(lo, hi, 7):
            ch, cost, lam, ok = O.dual_allocate(cells, budget)
            assert ok and cost <= budget
            e_dual = sum(c[0][i] for c, i in zip(cells, ch))
            # Everett: optimal among all allocations that cost no more than the dual's own cost
            _, e_best = _brute(cells, cost)
            assert e_dual <= e_best + 1e-12
            # and no cheaper-than-budget allocation beats it by more than the duality gap lam * slack
            _, e_b = _brute(cells, budget)
            assert e_dual - e_b <= lam * (budget - cost) + 1e-12


def test_dual_cost_monotone_and_infeasible_budget():
    rng = np.random.default_rng(6)
    cells = [(np.sort(rng.random(8))[::-1].copy(), np.sort(rng.integers(5, 90, 8)).astype(float)) for _ in range(3)]
    prev = math.inf
    for lam in (0, 1e-4, 1e-3, 1e-2, 1e-1, 1.0, 10.0):
        cost = sum(c[1][O._argmin_lagrangian(c[0], c[1], lam)] for c in cells)
        assert cost <= prev
        prev = cost
    ch, cost, lam, ok = O.dual_allocate(cells, 1.0)
    assert not ok and cost == sum(c[1].min() for c in cells)
    ch, cost, lam, ok = O.dual_allocate(cells, 1e9)
    assert ok and lam == 0.0


def test_dual_moves_bits_to_flat_spectrum_cell():
    # two cells of equal size: one with a fast-decaying spectrum (keys), one flat (values);
    # with a budget that cannot give both cells 4 bits, the flat one gets at least as many
    m, T, d = 2, 64, 128
    eps2 = {0: 1.0, 2: 0.126, 4: 0.0079}
    rt_grid, rf_grid = [8, 16, 32], [32, 64, 128]
    lamK = 100.0 * np.arange(1, 129) ** -3.0
    lamV = np.ones(128)
    sK = 100.0 * np.arange(1, 65) ** -3.0
    sV = np.ones(64) * 2
    cells, trips = [], []
    for lam, s2 in ((lamK, sK * lamK.sum() / sK.sum()), (lamV, sV)):
        tau = O.tau_table(lam, s2, lam.sum(), rt_grid, rf_grid)
        e, c, t = O.cell_options(m, T, d, tau, rt_grid, rf_grid, [0, 2, 4], eps2)
        cells.append((e, c))
        trips.append(t)
    raw = 2 * m * T * d * 2
    ch, cost, lam, ok = O.dual_allocate(cells, raw / 3)
    assert ok and cost <= raw / 3
    bK, bV = trips[0][ch[0]][2], trips[1][ch[1]][2]
    assert bV >= bK


# ----------------------------------------------------------------------------- rotary embedding at decode
def test_rope_is_the_textbook_rotation():
    # d = 4: pairs (0, 2) and (1, 3), frequencies 1 and base^(-1/2); written out by hand
    x = np.array([[1.0, 2.0, 3.0, 4.0], [0.5, -1.0, 2.0, 0.25]])
    y = O.rope_rotate(x, base=100.0, pos0=3)
    for t in range(2):
        p = 3 + t
        for j, th in enumerate([1.0, 0.1]):
            c, s = math.cos(p * th), math.sin(p * th)
            assert abs(y[t, j] - (x[t, j] * c - x[t, j + 2] * s)) < 1e-14
            assert abs(y[t, j + 2] - (x[t, j + 2] * c + x[t, j] * s)) < 1e-14


def test_rope_invariants():
    X = RNG.standard_normal((3, 40, 128))
    Y = O.rope_rotate(X, base=10000.0, pos0=17)
    # orthogonal per token: norms kept, inverse undoes it, position 0 is the identity
    assert np.allclose(np.linalg.norm(Y, axis=-1), np.linalg.norm(X, axis=-1), rtol=1e-13)
    assert np.allclose(O.rope_rotate(Y, 10000.0, 17, inverse=True), X, atol=1e-13)
    assert np.allclose(O.rope_rotate(X[:, :1], 10000.0, 0), X[:, :1], atol=0)
    # the defining property: <rope(q, m), rope(k, n)> depends on m - n only
    q, k = RNG.standard_normal((1, 128)), RNG.standard_normal((1, 128))
    def score(m, n):
        return float((O.rope_rotate(q, 10000.0, m) @ O.rope_rotate(k, 10000.0, n).T).item())
    assert abs(score(5, 2) - score(105, 102)) < 1e-10
    assert abs(score(5, 2) - score(5, 3)) > 1e-6
    # composition of shifts: rotating by a then by b is rotating by a + b
    assert np.allclose(O.rope_rotate(O.rope_rotate(X[:, :1], 10000.0, 7), 10000.0, 5), O.rope_rotate(X[:, :1], 10000.0, 12), atol=1e-12)


# --------------------------------------------------------------------------- attention on the compressed cache
def _attend_case(seed=5, m=2, T=24, n_q=3, bits_k=4, bits_v=2, r_t=8, r_f=64):
    rng = np.random.default_rng(seed)
    XK = rng.standard_normal((m, T, 128)) * np.exp(0.5 * rng.standard_normal((m, T, 1)))
    XV = rng.standard_normal((m, T, 128))
    cK = O.compress_cell(XK, r_t, r_f, bits_k, seed=1, cell=0, token_mode="exact")
    cV = O.compress_cell(XV, r_t, 128, bits_v, seed=1, cell=1, token_mode="exact")
    Q = rng.standard_normal((m, n_q, 128))
    return cK, cV, Q


def test_attend_matches_brute_force_loops():
    import math
    cK, cV, Q = _attend_case()
    scale = 1.0 / math.sqrt(128)
    Out = O.attend_cells(cK, cV, Q, scale)
    Kh, Vh = O.decoded_unrounded(cK), O.decoded_unrounded(cV)
    for h in range(cK.m):
        for i in range(Q.shape[1]):
            s = [scale * sum(float(Q[h, i, f]) * float(Kh[h, t, f]) for f in range(128)) for t in range(cK.T)]
            mx = max(s)
            w = [math.exp(v - mx) for v in s]
            z = sum(w)
            for f in range(0, 128, 17):
                ref = sum(w[t] * float(Vh[h, t, f]) for t in range(cK.T)) / z
                assert abs(Out[h, i, f] - ref) <= 1e-12 * max(1.0, abs(ref))


def test_attend_limits():
    cK, cV, Q = _attend_case(seed=6)
    Vh, Kh = O.decoded_unrounded(cV), O.decoded_unrounded(cK)
    # zero query: uniform weights, the output is the mean decoded value
    assert np.allclose(O.attend_cells(cK, cV, np.zeros_like(Q), 0.3), Vh.mean(axis=1, keepdims=True).repeat(Q.shape[1], 1))
    # zero scale: the same
    assert np.allclose(O.attend_cells(cK, cV, Q, 0.0), Vh.mean(axis=1, keepdims=True).repeat(Q.shape[1], 1))
    # very sharp softmax: the output is the decoded value at the best-scoring token
    Out = O.attend_cells(cK, cV, Q, 1e4)
    best = np.einsum("hif,htf->hit", Q, Kh).argmax(axis=-1)
    for h in range(cK.m):
        for i in range(Q.shape[1]):
            assert np.allclose(Out[h, i], Vh[h, best[h, i]], atol=1e-9)
    # the unrounded decode rounds to what decompress_cell returns
    assert np.array_equal(O.fp16_round(Kh), O.decompress_cell(cK))


def test_attend_scores_on_the_factors_identity():
    # The identity behind attention on the factors: with P_h the stored projected core,
    #   <q, K^[h, t]> = sum_k U_T[t, k] (P_h q)[k] 2^e  +  <H(s . q) / sqrt(d), r^'[h, t]>,
    # and for the values  sum_t p_t V^[h, t] = 2^e (p^T U_T) P_h + s . H(sum_t p_t r^'[h, t]) / sqrt(d).
    import math
    cK, cV, Q = _attend_case(seed=7, bits_k=3, bits_v=4)
    Kh, Vh = O.decoded_unrounded(cK), O.decoded_unrounded(cV)
    PK = O.fp16_round(np.einsum("hrs,fs->hrf", cK.Gs16, cK.UF16))
    rK = O.dequantize_rows(O.unpack_codes(cK.words, cK.bits, 128), cK.scales, cK.bits, cK.group)
    S_fact = math.ldexp(1.0, cK.e) * np.einsum("tk,hik->hit", cK.UT16, np.einsum("hkf,hif->hik", PK, Q)) \
        + np.einsum("hif,htf->hit", O.rotate(Q, cK.signs), rK)
    S_def = np.einsum("hif,htf->hit", Q, Kh)
    assert np.abs(S_fact - S_def).max() <= 1e-11 * np.abs(S_def).max()
    rng = np.random.default_rng(0)
    Pw = rng.random((cV.m, 2, cV.T))
    PV = O.fp16_round(np.einsum("hrs,fs->hrf", cV.Gs16, cV.UF16))
    rV = O.dequantize_rows(O.unpack_codes(cV.words, cV.bits, 128), cV.scales, cV.bits, cV.group)
    O_fact = math.ldexp(1.0, cV.e) * np.einsum("hik,hkf->hif", np.einsum("hit,tk->hik", Pw, cV.UT16), PV) \
        + O.unrotate(np.einsum("hit,htf->hif", Pw, rV), cV.signs)
    O_def = np.einsum("hit,htf->hif", Pw, Vh)
    assert np.abs(O_fact - O_def).max() <= 1e-11 * np.abs(O_def).max()


# --------------------------------------------------------------------------- ablation allocators
def test_greedy_hand_worked_sequence():
    # two cells, options (error, cost); budget 10.  Start: cheapest of each = (9, 1) and (8, 1), cost 2.
    # moves that fit: A: (4, 3): 5/2 = 2.5, (1, 8): 8/7;  B: (5, 2): 3/1 = 3, (2, 6): 6/5.  -> B to (5, 2), cost 3
    # then A (4, 3): 2.5, A (1, 8): 8/7 (fits: 3 + 7 = 10), B (2, 6): 3/4 -> A to (4, 3), cost 5
    # then A (1, 8): 3/5 = 0.6 (5 + 5 = 10 fits), B (2, 6): 3/4 = 0.75 (5 + 4 = 9 fits) -> B to (2, 6), cost 9
    # then A (1, 8): extra 5 does not fit (14 > 10): stop.
    A = (np.array([9.0, 4.0, 1.0]), np.array([1.0, 3.0, 8.0]))
    Bc = (np.array([8.0, 5.0, 2.0]), np.array([1.0, 2.0, 6.0]))
    ch, cost, ok = O.greedy_allocate([A, Bc], 10.0)
    assert ok and ch == [1, 2] and cost == 9.0
    # a budget below the cheapest allocation is reported, with the cheapest allocation
    ch, cost, ok = O.greedy_allocate([A, Bc], 1.5)
    assert not ok and ch == [0, 0] and cost == 2.0
    # a budget that covers everything ends at the smallest errors
    ch, cost, ok = O.greedy_allocate([A, Bc], 100.0)
    assert ok and ch == [2, 2]


def test_greedy_and_uniform_invariants_against_brute_force():
    import itertools
    rng = np.random.default_rng(11)
    for trial in range(20):
        n_opt = 5
        trips = [[(16 * (i + 1), 16, 4) for i in range(n_opt)] for _ in range(4)]
        cells = []
        for c in range(4):
            cost = np.sort(rng.uniform(1, 10, n_opt))
            err = np.sort(rng.uniform(0, 1, n_opt))[::-1] * rng.uniform(0.5, 2)
            cells.append((err, cost))
        lo = sum(c.min() for e, c in cells)
        hi = sum(c.max() for e, c in cells)
        for budget in (lo + (hi - lo) * f for f in (1e-6, 0.25, 0.5, 0.75, 1 + 1e-6)):   # off the exact end points
            all_alloc = list(itertools.product(range(n_opt), repeat=4))
            feas = [a for a in all_alloc if sum(cells[c][1][i] for c, i in enumerate(a)) <= budget + 1e-12]
            e_opt = min(sum(cells[c][0][i] for c, i in enumerate(a)) for a in feas)
            # greedy: feasible, no affordable improving single move left, never better than the optimum
            ch, cost, ok = O.greedy_allocate(cells, budget)
            assert ok and cost <= budget + 1e-12 and abs(cost - sum(cells[c][1][i] for c, i in enumerate(ch))) < 1e-9
            e_g = sum(cells[c][0][i] for c, i in enumerate(ch))
            assert e_g >= e_opt - 1e-12
            for c in range(4):
                for i in range(n_opt):
                    extra, gain = cells[c][1][i] - cells[c][1][ch[c]], cells[c][0][ch[c]] - cells[c][0][i]
                    assert not (extra > 0 and gain > 0 and cost + extra <= budget)
            # uniform: the best shared pair by independent enumeration; never better than the per-cell optimum
            chu, costu, oku = O.uniform_allocate(cells, trips, budget)
            pairs = [(a, b) for a in range(n_opt) for b in range(n_opt)
                     if cells[0][1][a] + cells[2][1][a] + cells[1][1][b] + cells[3][1][b] <= budget]
            if pairs:
                e_pairs = min(cells[0][0][a] + cells[2][0][a] + cells[1][0][b] + cells[3][0][b] for a, b in pairs)
                e_u = sum(cells[c][0][i] for c, i in enumerate(chu))
                assert oku and chu[0] == chu[2] and chu[1] == chu[3] and costu <= budget + 1e-12
                assert abs(e_u - e_pairs) < 1e-12 and e_u >= e_opt - 1e-12
            else:
                assert not oku and chu == [0, 0, 0, 0]
