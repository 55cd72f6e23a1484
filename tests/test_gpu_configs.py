"""Full-size cells of the four large configurations (one layer group each: a K and a V cell at the real
m, T and sketch width), planned by the library, compared with the oracle run on the same plan."""
import numpy as np
import pytest
import torch

import __graft_entry__ as entry
from oracle import jolt_oracle as O
from tests.helpers import cell_view, oracle_cache, projector_distance
from tests.test_gpu_parity import REL_ERR, recon_gate

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    entry.build()
    import paper_2607_12550_b200 as pkg
    return pkg.load()


@pytest.mark.parametrize("name", ["c1", "c4", "c2", "c3"])
def test_first_group_of_config(B, name):
    from paper_2607_12550_b200 import synth
    cfg = synth.CONFIGS[name]
    K, V = synth.make_cache(cfg, device="cuda", n_groups=1)
    gs = [0, cfg.layers_per_group]
    raw = 2 * K.numel() * 2
    bits_set = [1, 2, 3, 4] if name == "c4" else [0, 2, 4, 8]
    opts = B.default_options(seed=cfg.seed, power_iters=cfg.power_iters, bits_set=bits_set)
    plans, planned = B.jolt_plan(K, V, gs, raw / cfg.ratio, opts)
    assert planned <= raw / cfg.ratio
    h = B.jolt_compress(K, V, gs, plans, opts)
    assert h.bytes() == planned
    UT32 = [h.component(c, 8).astype(np.float64) for c in range(2)]     # scratch view: read before the next call
    Ko, Vo = torch.empty_like(K), torch.empty_like(V)
    B.jolt_decompress(h, Ko, Vo, gs)
    torch.cuda.synchronize()
    # the same cache decoded with the rotary embedding re-applied to the keys (values must not change)
    Kr, Vr = torch.empty_like(K), torch.empty_like(V)
    B.jolt_decompress_rope(h, Kr, Vr, gs, base=10000.0, pos0=1000)
    torch.cuda.synchronize()
    assert torch.equal(Vr, Vo)
    Krnp = Kr.cpu().numpy()
    del Kr, Vr
    # attention on the compressed cache (4 queries per KV head), against attention over the library's fp32 decode here
    # and against the oracle on the oracle's own cells below
    gq = torch.Generator().manual_seed(3)
    Q = torch.randn(K.shape[0], K.shape[1], 4, 128, generator=gq)
    att = B.jolt_attend(h, Q.cuda())
    torch.cuda.synchronize()
    Knp, Vnp = K.cpu().numpy(), V.cpu().numpy()
    Konp, Vonp = Ko.cpu().numpy(), Vo.cpu().numpy()
    ocells, gates = [], []
    for c in range(2):
        rt, rf, b = plans[c]
        X = cell_view(Knp, Vnp, gs, c).astype(np.float64)
        o = O.compress_cell(X, rt, rf, b, seed=cfg.seed, cell=c, token_mode="randomized", power_iters=cfg.power_iters)
        Xo = O.decompress_cell(o)
        Xg = cell_view(Konp, Vonp, gs, c).astype(np.float64)
        eo, eg = O.rel_frobenius(X, Xo), O.rel_frobenius(X, Xg)
        rel = np.linalg.norm(Xg - Xo) / np.linalg.norm(Xo)
        assert abs(eg - eo) <= REL_ERR * eo, (name, c, plans[c], eg, eo)
        assert rel <= recon_gate(eo), (name, c, plans[c], rel, eo)
        if c == 0:
            Xro = O.decompress_cell_rope(o, 10000.0, 1000)
            Xrg = cell_view(Krnp, Vonp, gs, 0).astype(np.float64)
            relr = np.linalg.norm(Xrg - Xro) / np.linalg.norm(Xro)
            assert relr <= recon_gate(eo), (name, "rope", relr, eo)
            del Xro, Xrg
        if rt > 0:
            # projectors are compared before fp16 storage: independently rounded fp16 copies of two factors
            # that agree to 1e-5 are already ~2e-3 apart
            UT = UT32[c].reshape(o.UT16.shape)
            sig = o.ideal["sigma"]
            if (sig[rt - 1] - sig[rt]) / sig[0] > 1e-2:
                assert projector_distance(UT, o.ideal["U_T"]) <= 1e-3, (name, c)
            assert np.abs(h.component(c, 6)[:rt] - sig[:rt]).max() <= 1e-4 * sig[0], (name, c)
        ocells.append(o)
        gates.append(recon_gate(eo))
        del X, Xo, Xg
    ref = O.attend_cells(ocells[0], ocells[1], Q.reshape(-1, 4, 128).numpy(), 1.0 / 128 ** 0.5)
    got = att.cpu().numpy().astype(np.float64).reshape(-1, 4, 128)
    rel = np.linalg.norm(got - ref) / np.linalg.norm(ref)
    assert rel <= 3 * max(gates), (name, "attend", rel, gates)
    h.free()
