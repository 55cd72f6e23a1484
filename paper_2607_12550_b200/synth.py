"""Seeded synthetic KV caches shaped like the paper's GQA / MHA workloads.

Only input generation lives here (no arithmetic of the compression method), so that the
library, its tests and the CPU oracle can all be fed the very same bytes.

Recipe per cell (layer group g, tensor t in {K, V}), X in R^{m x T x d}, m = layers_in_group * n_heads:

    X = sum_{i=1..n} w_i * a_i (x) p_i (x) q_i + noise

* p_i: columns of the thin QR of a seeded T x n Gaussian, scaled by sqrt(T) (unit RMS);
* q_i: columns of a seeded d x d orthogonal matrix scaled by sqrt(d), index wrapped mod d;
* a_i in R^m ~ N(1, 0.1^2); w_i = i^-alpha, alpha = alpha_k for keys, alpha_v for values;
* noise ~ N(0, sigma^2), sigma = 0.05 for keys and 0.1 for values;
* keys only: the fixed feature channels OUTLIER_CHANNELS are multiplied by 10 after the noise is added.

These tensors stand in for real caches of Mistral-7B-v0.3 (GQA, 8 KV heads, 32 layers) and
LLaMA-2-13B (MHA, 40 heads, 40 layers): fast-decaying keys with a few outlier channels, flat values.
"""
from __future__ import annotations

from dataclasses import dataclass

import torch

OUTLIER_CHANNELS = (5, 37, 70, 101)


@dataclass(frozen=True)
class CacheConfig:
    name: str
    n_layers: int
    layers_per_group: int
    n_kv_heads: int
    seq_len: int
    head_dim: int = 128
    n_terms: int = 128
    alpha_k: float = 1.0
    alpha_v: float = 0.6
    seed: int = 0
    dtype: str = "f16"
    batch: int = 1
    ratio: float = 2.0
    power_iters: int = 1

    @property
    def n_groups(self):
        return self.n_layers // self.layers_per_group

    @property
    def m(self):
        return self.layers_per_group * self.n_kv_heads

    def cache_bytes_fp16(self):
        return 2 * 2 * self.n_layers * self.n_kv_heads * self.seq_len * self.head_dim


CONFIGS = {
    # tiny single group, oracle-sized; fixed ranks (64, 64), 2-bit residual
    "c0": CacheConfig("c0", 1, 1, 8, 512, n_terms=64, seed=0, dtype="f32"),
    # GQA-shaped (Mistral-7B-like), budget 2x; the benchmark workload
    "c1": CacheConfig("c1", 32, 4, 8, 4096, n_terms=128, seed=1, ratio=2.0),
    # MHA-shaped (LLaMA-2-13B-like), budgets 2x and 3x
    "c2": CacheConfig("c2", 40, 4, 40, 4096, n_terms=128, seed=2, ratio=2.0),
    # long-context GQA, budget 2.5x, two power iterations
    "c3": CacheConfig("c3", 32, 4, 8, 32768, n_terms=256, alpha_k=0.9, alpha_v=0.5, seed=3, ratio=2.5,
                      power_iters=2),
    # batched serving-shaped GQA: 16 sequences, seeds 4 + b, budget 3x
    "c4": CacheConfig("c4", 32, 4, 8, 8192, n_terms=128, seed=4, batch=16, ratio=3.0),
}


def _cpu_gen(seed: int, group: int, which: int, salt: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed((seed * 1000003 + group * 7919 + which * 104729 + salt) & 0x7FFFFFFFFFFFFFFF)
    return g


def make_cell(cfg: CacheConfig, group: int, which: int, *, seed: int | None = None,
              device: str | torch.device = "cpu", m: int | None = None) -> torch.Tensor:
    """One cell X [m, T, d] in fp32 on `device` (which: 0 = keys, 1 = values)."""
    seed = cfg.seed if seed is None else seed
    m = cfg.m if m is None else m
    T, d, n = cfg.seq_len, cfg.head_dim, cfg.n_terms
    g = _cpu_gen(seed, group, which, 1)
    n_tok = min(n, T)
    P, _ = torch.linalg.qr(torch.randn(T, n_tok, generator=g, dtype=torch.float64))
    P = P * (T ** 0.5)
    if n_tok < n:
        P = P[:, torch.arange(n) % n_tok]
    Qo, _ = torch.linalg.qr(torch.randn(d, d, generator=g, dtype=torch.float64))
    Qw = (Qo * (d ** 0.5))[:, torch.arange(n) % d]                      # d x n
    a = 1.0 + 0.1 * torch.randn(m, n, generator=g, dtype=torch.float64)
    alpha = cfg.alpha_k if which == 0 else cfg.alpha_v
    w = torch.arange(1, n + 1, dtype=torch.float64) ** (-alpha)
    coef = (a * w).to(torch.float32).to(device)                         # m x n
    P32 = P.to(torch.float32).to(device)
    Qw32 = Qw.to(torch.float32).to(device)
    X = torch.matmul(P32.unsqueeze(0) * coef.unsqueeze(1), Qw32.t())    # m x T x d
    sigma = 0.05 if which == 0 else 0.1
    dev = torch.device(device)
    gd = torch.Generator(device=dev)
    gd.manual_seed((seed * 1000003 + group * 7919 + which * 104729 + 2) & 0x7FFFFFFFFFFFFFFF)
    X += sigma * torch.randn(X.shape, generator=gd, dtype=torch.float32, device=dev)
    if which == 0:
        X[:, :, list(OUTLIER_CHANNELS)] *= 10.0
    return X


def make_cache(cfg: CacheConfig, *, seq: int = 0, device: str | torch.device = "cpu",
               n_groups: int | None = None):
    """K and V of one sequence, each [n_layers, n_kv_heads, T, d] contiguous in cfg.dtype.

    Cell g covers layers [g * layers_per_group, (g+1) * layers_per_group); its merged index is
    h = layer_in_group * n_kv_heads + head.  `n_groups` limits generation to the first groups."""
    ng = cfg.n_groups if n_groups is None else n_groups
    dt = torch.float16 if cfg.dtype == "f16" else torch.float32
    L = ng * cfg.layers_per_group
    out = []
    for which in (0, 1):
        buf = torch.empty(L, cfg.n_kv_heads, cfg.seq_len, cfg.head_dim, dtype=dt, device=device)
        for g in range(ng):
            X = make_cell(cfg, g, which, seed=cfg.seed + seq, device=device)
            buf[g * cfg.layers_per_group:(g + 1) * cfg.layers_per_group] = X.view(
                cfg.layers_per_group, cfg.n_kv_heads, cfg.seq_len, cfg.head_dim).to(dt)
            del X
        out.append(buf)
    return out[0], out[1]
