"""CPU-side checks of the C ABI: the library loads, exports every declared symbol, validates its
arguments before touching a GPU, and its host allocator agrees with the oracle's dual."""
import ctypes
import os
import re

import numpy as np
import pytest
import torch

import __graft_entry__ as entry
from oracle import jolt_oracle as O

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    entry.build()
    import paper_2607_12550_b200 as pkg
    return pkg.load()


def test_every_declared_symbol_is_exported(B):
    hdr = open(os.path.join(ROOT, "include", "jolt.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    names = set(re.findall(r"\b(jolt_[a-z0-9_]+)\s*\(", hdr))
    assert {"jolt_plan", "jolt_compress", "jolt_decompress", "jolt_free"} <= names
    for n in sorted(names):
        assert hasattr(B.lib, n), n


def test_status_strings(B):
    assert B.lib.jolt_strerror(0) == b"ok"
    for s in range(-7, 0):
        assert B.lib.jolt_strerror(s) not in (b"", b"unknown status")


def _cpu_cache(L=2, nh=2, T=128, dtype=torch.float16):
    K = torch.zeros(L, nh, T, 128, dtype=dtype)
    return K, K.clone()


def test_argument_validation_needs_no_gpu(B):
    K, V = _cpu_cache()
    opts = B.default_options()
    plans = [(16, 16, 4)] * 2
    # bad head_dim
    K96 = torch.zeros(2, 2, 128, 96, dtype=torch.float16)
    with pytest.raises(B.JoltError) as e:
        B.jolt_compress(K96, K96, [0, 2], plans, opts)
    assert e.value.status == B.EUNSUPPORTED
    # seq_len not a multiple of 128
    Kb = torch.zeros(2, 2, 100, 128, dtype=torch.float16)
    with pytest.raises(B.JoltError) as e:
        B.jolt_compress(Kb, Kb, [0, 2], plans, opts)
    assert e.value.status == B.EUNSUPPORTED
    # grouping must cover all layers
    with pytest.raises(B.JoltError) as e:
        B.jolt_compress(K, V, [0, 1], plans, opts)
    assert e.value.status == B.EINVAL
    with pytest.raises(B.JoltError) as e:
        B.jolt_compress(K, V, [0, 2, 2], plans * 2, opts)
    assert e.value.status == B.EINVAL
    # quant group other than 32
    with pytest.raises(B.JoltError) as e:
        B.jolt_compress(K, V, [0, 2], plans, B.default_options(quant_group=64))
    assert e.value.status == B.EUNSUPPORTED
    # null handle
    assert B.lib.jolt_free(None) == 0
    lay = B.make_layout(K, [0, 2])
    assert B.lib.jolt_decompress(None, ctypes.byref(lay), K.data_ptr(), V.data_ptr(), None) == B.EINVAL


def test_image_checks_come_before_any_gpu_call(B):
    import numpy as np
    h = ctypes.c_void_p()
    assert B.lib.jolt_deserialize(None, 0, None, ctypes.byref(h)) == B.EINVAL
    junk = np.zeros(4096, dtype=np.uint8)
    assert B.lib.jolt_deserialize(junk.ctypes.data, junk.size, None, ctypes.byref(h)) == B.EINVAL and not h.value
    assert B.lib.jolt_deserialize(junk.ctypes.data, 8, None, ctypes.byref(h)) == B.EINVAL
    n = ctypes.c_int64(0)
    assert B.lib.jolt_serialized_bytes(None, ctypes.byref(n)) == B.EINVAL
    assert B.lib.jolt_serialize(None, junk.ctypes.data, junk.size, None) == B.EINVAL
    assert B.lib.jolt_attend(None, junk.ctypes.data, 4, 1.0, junk.ctypes.data, None) == B.EINVAL


def test_byte_model_and_cap_policy_match_oracle(B):
    for (m, T, rt, rf, b) in [(32, 4096, 128, 128, 4), (8, 512, 64, 64, 2), (160, 4096, 48, 112, 0), (32, 8192, 16, 16, 8)]:
        assert B.cell_bytes(m, T, 128, rt, rf, b, True) == O.stored_bytes(m, T, 128, rt, rf, b)
        assert B.cell_bytes(m, T, 128, rt, rf, b, False) == O.eq1_bytes(m, T, 128, rt, rf, b)
    for T in (128, 512, 1024, 2049, 4096, 8192, 32768, 10 ** 6):
        for R in (2, 2.5, 3, 4, 5, 8):
            assert B.cap_policy(T, R) == O.cap_policy(T, R)


def test_builtin_eps2_matches_oracle_calibration(B):
    t = B.eps2_table()
    ref = O.eps2_table([0, 1, 2, 3, 4, 8])
    # each side calibrates through its own evaluation of the quantiser (the library's is the kernel's single-precision
    # reciprocal-multiply, the oracle's the float64 definition); codes differ by one on a few samples in 10^5
    # (test_oracle_pins.py bounds that), which moves the Gaussian round-trip error in the sixth digit at most
    for b, v in ref.items():
        assert abs(t[b] - v) <= 1e-5 * max(v, 1e-30)


def test_seeded_draws_match_oracle(B):
    for seed, cell in [(0, 0), (7, 3), (2 ** 63 + 5, 11)]:
        g = B.sketch_host(seed, cell, 0, 64, 17)
        ref = O.gaussian_sketch(seed, cell, 64, 17)
        assert np.array_equal(g.astype(np.float64), ref)
        assert np.array_equal(B.signs_host(seed, cell).astype(np.float64), O.rotation_signs(seed, cell))
    g2 = B.sketch_host(7, 3, 2, 64, 17)
    assert np.array_equal(g2.astype(np.float64), O.gaussian_sketch(7, 3, 64, 17, stream=O.STREAM_PROBE))


def _grid(lo, hi, step):
    return list(range(lo, hi + 1, step))


@pytest.mark.parametrize("bits_set", [[0, 2, 4, 8], [1, 2, 3, 4]])
def test_library_dual_equals_oracle_dual_on_oracle_spectra(B, bits_set):
    rng = np.random.default_rng(3)
    m, T, d = 8, 512, 128
    n_cells = 6
    eps2 = O.eps2_table(sorted(set(bits_set) | {0}), n=1 << 14)
    eps_arr = [eps2.get(b, float("nan")) for b in range(9)]
    lam, sig2, tot, rtmax = [], [], [], []
    for c in range(n_cells):
        alpha = 1.0 if c % 2 == 0 else 0.4
        s = (np.arange(1, 65) ** -alpha) * rng.uniform(0.5, 2.0)
        l3 = np.sort(rng.random(128) ** 3)[::-1] * 5
        total = max(np.sum(s ** 2), l3.sum()) * 1.3
        l3 = l3 * total / l3.sum()
        spec = O.tail_mass_spectrum(s, total) ** 2
        lam.append(l3); sig2.append(spec); tot.append(float(total)); rtmax.append(64)
    raw = n_cells * m * T * d * 2
    for ratio in (1.5, 2.0, 3.0, 5.0, 9.0):
        budget = raw / ratio
        cells, trips = [], []
        for c in range(n_cells):
            rt_grid, rf_grid = _grid(16, rtmax[c], 16), _grid(16, 128, 16)
            tau = O.tau_table(lam[c], sig2[c], tot[c], rt_grid, rf_grid)
            e, s_, t = O.cell_options(m, T, d, tau, rt_grid, rf_grid, bits_set, eps2)
            cells.append((e, s_)); trips.append(t)
        ch, cost, _, ok = O.dual_allocate(cells, budget)
        ref = [trips[c][i] for c, i in enumerate(ch)]
        opts = B.default_options(bits_set=bits_set, eps2=eps_arr)
        got, ach, st = B.jolt_allocate([m] * n_cells, T, d, np.stack(lam), sig2, tot, rtmax, budget, opts, allow_budget=True)
        assert (st == 0) == ok
        assert got == ref, (ratio, got, ref)
        assert ach == cost
        if ok:
            assert ach <= budget


@pytest.mark.parametrize("which", ["greedy", "uniform"])
def test_library_ablation_allocators_equal_the_oracle(B, which):
    rng = np.random.default_rng(5)
    m, T, d = 8, 512, 128
    n_cells = 6
    bits_set = [0, 2, 4, 8]
    eps2 = O.eps2_table(bits_set, n=1 << 14)
    eps_arr = [eps2.get(b, float("nan")) for b in range(9)]
    lam, sig2, tot, rtmax = [], [], [], []
    for c in range(n_cells):
        alpha = 1.0 if c % 2 == 0 else 0.4
        s = (np.arange(1, 65) ** -alpha) * rng.uniform(0.5, 2.0)
        l3 = np.sort(rng.random(128) ** 3)[::-1] * 5
        total = max(np.sum(s ** 2), l3.sum()) * 1.3
        l3 = l3 * total / l3.sum()
        spec = O.tail_mass_spectrum(s, total) ** 2
        lam.append(l3); sig2.append(spec); tot.append(float(total)); rtmax.append(64 if c != 3 else 48)
    raw = n_cells * m * T * d * 2
    for ratio in (1.5, 2.0, 3.0, 5.0, 9.0, 400.0):
        budget = raw / ratio
        cells, trips = [], []
        for c in range(n_cells):
            rt_grid, rf_grid = _grid(16, rtmax[c], 16), _grid(16, 128, 16)
            tau = O.tau_table(lam[c], sig2[c], tot[c], rt_grid, rf_grid)
            e, s_, t = O.cell_options(m, T, d, tau, rt_grid, rf_grid, bits_set, eps2)
            cells.append((e, s_)); trips.append(t)
        if which == "greedy":
            ch, cost, ok = O.greedy_allocate(cells, budget)
        else:
            ch, cost, ok = O.uniform_allocate(cells, trips, budget)
        ref = [tuple(trips[c][i]) for c, i in enumerate(ch)]
        opts = B.default_options(bits_set=bits_set, eps2=eps_arr,
                                 allocator=B.ALLOC_GREEDY if which == "greedy" else B.ALLOC_UNIFORM)
        got, ach, st = B.jolt_allocate([m] * n_cells, T, d, np.stack(lam), sig2, tot, rtmax, budget, opts, allow_budget=True)
        assert (st == 0) == ok, (ratio, st, ok)
        assert got == ref, (ratio, got, ref)
        assert ach == cost
        if which == "uniform":
            assert len(set(got[0::2])) == 1 and len(set(got[1::2])) == 1
    bad = B.default_options(allocator=7)
    with pytest.raises(B.JoltError) as e:
        B.jolt_allocate([m] * n_cells, T, d, np.stack(lam), sig2, tot, rtmax, raw / 2, bad)
    assert e.value.status == B.EINVAL


def test_budget_below_minimum_reports_ebudget_and_cheapest_plan(B):
    lam = np.ones((2, 128)); sig2 = [np.ones(33), np.ones(33)]
    got, ach, st = B.jolt_allocate([4, 4], 256, 128, lam, sig2, [128.0, 128.0], [32, 32], 10.0, allow_budget=True)
    assert st == B.EBUDGET
    assert got == [(16, 16, 0)] * 2
    assert ach == 2 * B.cell_bytes(4, 256, 128, 16, 16, 0)


def test_plan_validation_needs_no_gpu(B):
    K, V = _cpu_cache(L=2, nh=2, T=128)
    opts = B.default_options()
    gs = [0, 2]
    bad_plans = [
        [(0, 0, 0), (16, 16, 4)],          # a cell that stores nothing
        [(16, 16, 5), (16, 16, 4)],        # unsupported bit width
        [(16, 0, 4), (16, 16, 4)],         # r_f out of range
        [(16, 129, 4), (16, 16, 4)],
        [(129, 128, 4), (16, 16, 4)],      # r_t > T
        [(65, 16, 4), (16, 16, 4)],        # r_t > m * r_f  (m = 4)
        [(-1, 16, 4), (16, 16, 4)],
    ]
    for plans in bad_plans:
        with pytest.raises(B.JoltError) as e:
            B.jolt_compress(K, V, gs, plans, opts)
        assert e.value.status == B.EINVAL, plans
    with pytest.raises(B.JoltError) as e:
        B.jolt_compress(K, V, gs, [(16, 16, 4)] * 2, B.default_options(power_iters=9))
    assert e.value.status == B.EINVAL
    with pytest.raises(B.JoltError) as e:
        B.jolt_plan(K, V, gs, -5.0, opts)
    assert e.value.status == B.EINVAL
