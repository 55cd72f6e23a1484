"""The allocation-free decode entry point (collected last on purpose: a failure here must not hide the
other tests under `pytest -x`).

jolt_decompress_static serves callers that may not allocate device memory while they decode, so its
scratch is a fixed array inside the library.  The test decodes the same compressed cache through the
regular entry point and twice in a row through the static one (the second call finds the first call's
contents in the shared array) and requires the same reconstruction within the parity tolerance."""
import pytest
import torch

import __graft_entry__ as entry

pytestmark = pytest.mark.gpu

REL_RECON = 1e-3


@pytest.fixture(scope="module")
def B():
    entry.build()
    import paper_2607_12550_b200 as pkg
    return pkg.load()


def _rel(a, b):
    return float((a.float() - b.float()).norm() / b.float().norm())


def test_static_decode_matches_regular_decode_twice(B):
    from paper_2607_12550_b200 import synth
    cfg = synth.CacheConfig("t", 4, 2, 2, 256, n_terms=24, seed=12)
    K, V = synth.make_cache(cfg, device="cuda")
    gs = [0, 2, 4]
    plans = [(32, 64, 4), (24, 128, 2), (0, 0, 8), (16, 96, 0)]
    opts = B.default_options(seed=9)
    h = B.jolt_compress(K, V, gs, plans, opts)
    Kr, Vr = torch.empty_like(K), torch.empty_like(V)
    B.jolt_decompress(h, Kr, Vr, gs)
    torch.cuda.synchronize()
    for call in range(2):
        Ks, Vs = torch.full_like(K, float("nan")), torch.full_like(V, float("nan"))
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        B.jolt_decompress_static(h, Ks, Vs, gs)
        torch.cuda.synchronize()
        if call == 1:
            # "allocates nothing": the driver's free-memory figure does not move across the call (the first call on a
            # device may still load the module and look the array's address up, so the second one is the one measured)
            assert torch.cuda.mem_get_info()[0] == free_before
        B.check_status(h)
        assert torch.isfinite(Ks).all() and torch.isfinite(Vs).all()
        assert _rel(Ks, Kr) <= REL_RECON, (call, _rel(Ks, Kr))
        assert _rel(Vs, Vr) <= REL_RECON, (call, _rel(Vs, Vr))
    # a second cache of another shape re-uses the same array
    cfg2 = synth.CacheConfig("t2", 2, 1, 4, 128, n_terms=8, seed=13)
    K2, V2 = synth.make_cache(cfg2, device="cuda")
    gs2 = [0, 1, 2]
    h2 = B.jolt_compress(K2, V2, gs2, [(8, 32, 3)] * 4, opts)
    K2r, V2r = torch.empty_like(K2), torch.empty_like(V2)
    B.jolt_decompress(h2, K2r, V2r, gs2)
    K2s, V2s = torch.empty_like(K2), torch.empty_like(V2)
    B.jolt_decompress_static(h2, K2s, V2s, gs2)
    torch.cuda.synchronize()
    assert _rel(K2s, K2r) <= REL_RECON and _rel(V2s, V2r) <= REL_RECON
    h.free(); h2.free()


def test_static_decode_rejects_oversized_cache(B):
    from paper_2607_12550_b200 import synth
    cfg = synth.CacheConfig("big", 4, 4, 8, 1024, n_terms=8, seed=14)     # 4 M elements per cell: 16 MiB of fp32 alone
    K, V = synth.make_cache(cfg, device="cuda")
    gs = [0, 4]
    h = B.jolt_compress(K, V, gs, [(16, 16, 2)] * 2, B.default_options(seed=1))
    Ko, Vo = torch.empty_like(K), torch.empty_like(V)
    with pytest.raises(B.JoltError) as e:
        B.jolt_decompress_static(h, Ko, Vo, gs)
    assert e.value.status == B.EINVAL and "static scratch holds" in str(e.value)
    B.jolt_decompress(h, Ko, Vo, gs)        # the regular entry point still serves it
    torch.cuda.synchronize()
    h.free()
