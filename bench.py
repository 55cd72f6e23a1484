#!/usr/bin/env python
"""Benchmark of the JoLT hot path on B200: one step = compress + decompress of one whole synthetic KV cache.

Workload (N = 1): the GQA-shaped cache of the headline metric (32 layers in groups of 4, 8 KV heads,
T = 4096, d_h = 128, fp16, budget 2x, randomized token factor, q = 1), ranks and bits from jolt_plan.
Prints ONE JSON line.  `--impl reference` times the CPU oracle on a bounded sample instead.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "KV compress+decompress GB/s of fp16 cache (2x budget)"
UNIT = "GB/s"


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm": d["hbm_gbs"], "tensor": d["bf16_tflops"], "tensor_sustained": d.get("bf16_tflops_sustained"),
                "source": "measured"}
    return {"hbm": 6650.0, "tensor": 1590.0, "tensor_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    Q = "index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown," \
        "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap"

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "50",
                                          "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=2)
            except Exception:
                self.proc.kill()
        sm = sorted(int(r[1]) for r in self.rows if len(r) >= 9 and r[1].isdigit())
        mx = [int(r[2]) for r in self.rows if len(r) >= 9 and r[2].isdigit()]
        reasons = set()
        for r in self.rows:
            if len(r) < 9:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def shard_of_rank(rank: int, world: int, base_seed: int):
    """Weak scaling: cells (and whole sequences) are independent, so rank r compresses its own sequence
    (generator seed base_seed + r) and no collective touches the data path."""
    return {"seq": rank, "seed": base_seed + rank}


def max_over_ranks(dist, values, device):
    """Element-wise maximum of per-rank timings (the job is as slow as its slowest rank)."""
    import torch
    if dist is None:
        return list(values)
    t = torch.tensor(list(values), device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def job_throughput(world: int, bytes_per_rank: int, ms: float) -> float:
    """Whole-job GB/s: every rank processed bytes_per_rank in ms (max over ranks)."""
    return world * bytes_per_rank / (ms * 1e-3) / 1e9


def cell_work(m, T, d, r_t, r_f, bits, k, q, in_bytes_per_elt):
    """Algorithmic flops / bytes of one cell (split-precision passes do not count)."""
    M = m * T * d
    X = M * in_bytes_per_elt
    out = 2 * (m * r_t * r_f + T * r_t + d * r_f) + bits * M // 8 + (2 * M // 32 if bits else 0)
    w = {}
    w["gram"] = (2 * M * d, X)
    w["sketch"] = (2 * M * k, X)
    w["power"] = (4 * M * k * q, 2 * q * X)
    w["project"] = (2 * M * k, X)
    w["residual_quant"] = (2 * M * r_t, X + out)
    w["compress"] = (2 * M * d + 2 * M * k * (2 + 2 * q) + 2 * M * r_t, (4 + 2 * q) * X + out)
    w["compress_strict_bytes"] = X + out
    w["decompress"] = (2 * M * r_t + 2 * m * r_t * r_f * d, 2 * M + out)
    return w


def roof_time(flops, nbytes, pk):
    return max(flops / (pk["tensor"] * 1e12), nbytes / (pk["hbm"] * 1e9))


# The plan jolt_plan gives for the c1 workload (seed 1, 2x budget, bits {0, 2, 4, 8}); the reference arm, which has no
# GPU to plan with, times the oracle on this plan, and the GPU arm reports whether its own plan equals it.
C1_PLAN = [(128, 128, 4), (96, 128, 8), (16, 48, 8), (96, 128, 8), (128, 128, 4), (96, 128, 8), (16, 64, 8), (96, 128, 8),
           (128, 128, 4), (96, 128, 8), (128, 128, 4), (96, 128, 8), (16, 48, 8), (96, 128, 8), (128, 128, 4), (96, 128, 8)]


def dram_traffic(kernel: str, workload: str):
    """DRAM bytes per launch of `kernel` on `workload`, from the table kept beside the ncu summaries
    (profiles/dram_traffic.txt: kernel, workload, cells captured, bytes read, bytes written); scaled by the caller."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.txt")
    if not os.path.exists(path):
        return None
    for line in open(path):
        f = line.split("#")[0].split()
        if len(f) >= 5 and f[0] == kernel and f[1] == workload:
            return {"cells": int(f[2]), "read": float(f[3]), "write": float(f[4])}
    return None


def run_reference(args):
    """The CPU oracle, as it stands, on a bounded sample of the same workload (rank 0 only)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import numpy as np
    import torch
    from oracle import jolt_oracle as O
    from paper_2607_12550_b200 import synth
    cfg = synth.CONFIGS["c1"]
    # sample: the K and the V cell of group 0, with plans typical of the 2x allocation
    plans = {0: C1_PLAN[0], 1: C1_PLAN[1]}
    cells = {w: synth.make_cell(cfg, 0, w).to(torch.float16).numpy() for w in (0, 1)}
    cell_bytes = cells[0].size * 2
    n_cells_total = 2 * cfg.n_groups

    def step():
        tc = td = 0.0
        for w, X in cells.items():
            t0 = time.perf_counter()
            oc = O.compress_cell(X, *plans[w], seed=cfg.seed, cell=w, token_mode="randomized", power_iters=1)
            t1 = time.perf_counter()
            O.decompress_cell(oc)
            t2 = time.perf_counter()
            tc += t1 - t0
            td += t2 - t1
        return tc, td

    for _ in range(args.warmup_ref):
        step()
    tcs, tds = [], []
    for _ in range(args.steps):
        a, b = step()
        tcs.append(a); tds.append(b)
    tc, td = sum(tcs) / len(tcs), sum(tds) / len(tds)
    sample_bytes = 2 * cell_bytes
    value = sample_bytes / (tc + td) / 1e9
    cores = os.cpu_count()
    try:
        cores = torch.get_num_threads()
    except Exception:
        pass
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup_ref, "ms_per_step": (tc + td) * 1e3 * n_cells_total / 2, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": "c1: GQA 32 layers / 4 per group, 8 KV heads, T=4096, d=128, fp16, 2x budget",
                       "sample": f"2 of 16 cells (group 0: K at {C1_PLAN[0]}, V at {C1_PLAN[1]}, the plan jolt_plan gives this cache); "
                                 "ms_per_step scaled to 16 cells", "plan": [list(p) for p in C1_PLAN]},
            "compress_gbs": sample_bytes / tc / 1e9, "decompress_gbs": sample_bytes / td / 1e9,
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": "group 0 K and V cells (2 of 16), numpy fp64"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def torch_rope(x, base):
    """Rotate-half rotary embedding of a [..., T, 128] tensor (accuracy bookkeeping of --rope only)."""
    import torch
    T = x.shape[-2]
    inv = base ** (-torch.arange(64, device=x.device, dtype=torch.float64) / 64)
    ang = torch.arange(T, device=x.device, dtype=torch.float64)[:, None] * inv[None, :]
    c, s_ = ang.cos().float(), ang.sin().float()
    a, b = x[..., :64], x[..., 64:]
    return torch.cat([a * c - b * s_, b * c + a * s_], dim=-1)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="jolt", choices=["jolt", "reference"])
    ap.add_argument("--workload", default="c1")
    ap.add_argument("--groups", type=int, default=0, help="limit the number of layer groups (profiling captures)")
    ap.add_argument("--token-mode", default="randomized", choices=["randomized", "exact"],
                    help="token-mode solver; exact at T > 1024 is the converged block iteration")
    ap.add_argument("--ratio", type=float, default=0.0, help="compression ratio of the byte budget (default: the workload's)")
    ap.add_argument("--rope", action="store_true",
                    help="decode through jolt_decompress_rope (keys rotated at decode; not the headline workload)")
    ap.add_argument("--attend", type=int, default=0, metavar="N_Q",
                    help="also time jolt_attend (attention on the compressed cache) with N_Q queries per KV head")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--portable", action="store_true", help="portable SIMT kernels only")
    ap.add_argument("--fast-mask", type=int, default=-1, help="kernel family bit mask (jolt_set_fast_path); default: all")
    args = ap.parse_args()
    args.warmup_ref = min(args.warmup, 1)
    if args.impl == "reference":
        args.steps = min(args.steps, 3)
        return run_reference(args)

    import numpy as np
    import torch
    import __graft_entry__ as entry
    entry.build()
    import paper_2607_12550_b200 as pkg
    B = pkg.load()
    synth = pkg.synth

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU fallback")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if args.portable:
        B.set_fast_path(False)
    elif args.fast_mask >= 0:
        B.set_fast_path(args.fast_mask)
    W = max(args.warmup, 3)
    pk = peaks()

    cfg = synth.CONFIGS[args.workload]
    ng = args.groups or cfg.n_groups
    # weak scaling: every rank compresses its own sequence (seed + rank); no data-path collective
    shard = shard_of_rank(rank, world, cfg.seed)
    K, V = synth.make_cache(cfg, seq=shard["seq"], device=f"cuda:{local}", n_groups=ng)
    gs = [g * cfg.layers_per_group for g in range(ng + 1)]
    cache_bytes = 2 * K.numel() * 2
    ratio = args.ratio or cfg.ratio
    opts = B.default_options(seed=shard["seed"], power_iters=cfg.power_iters,
                             token_mode=B.TOKEN_EXACT if args.token_mode == "exact" else B.TOKEN_RANDOMIZED)
    t0 = time.perf_counter()
    plans, planned_bytes = B.jolt_plan(K, V, gs, cache_bytes / ratio, opts)
    torch.cuda.synchronize()
    plan_ms = (time.perf_counter() - t0) * 1e3          # first call: includes one-time workspace and module set-up
    t0 = time.perf_counter()
    B.jolt_plan(K, V, gs, cache_bytes / ratio, opts)
    torch.cuda.synchronize()
    plan_ms_warm = (time.perf_counter() - t0) * 1e3
    Ko, Vo = torch.empty_like(K), torch.empty_like(V)

    ev = lambda: torch.cuda.Event(enable_timing=True)
    stage_acc = {}

    def step(record=None):
        e0, e1, e2 = ev(), ev(), ev()
        e0.record()
        h = B.jolt_compress(K, V, gs, plans, opts)
        e1.record()
        st_c = B.stage_ms()
        if args.rope:
            B.jolt_decompress_rope(h, Ko, Vo, gs, base=10000.0, pos0=0)
        else:
            B.jolt_decompress(h, Ko, Vo, gs)
        e2.record()
        torch.cuda.synchronize()
        st_d = B.stage_ms()
        h.free()
        if record is not None:
            record.append((e0.elapsed_time(e1), e1.elapsed_time(e2)))
            for k_, v_ in list(st_c.items()) + list(st_d.items()):
                stage_acc[k_] = stage_acc.get(k_, 0.0) + v_
        return h

    for _ in range(W):
        step()
    if dist:
        dist.barrier()
    torch.cuda.synchronize()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    n0 = B.launch_count()
    rec = []
    for _ in range(args.steps):
        step(rec)
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
    launches = B.launch_count() - n0
    clocks = sampler.stop() if rank == 0 else None
    tc_all = sorted(r[0] for r in rec)
    td_all = sorted(r[1] for r in rec)
    tc = sum(tc_all) / len(rec)
    td = sum(td_all) / len(rec)
    # decompress stage timing (device events inside the library need a sync, done in step())
    tc, td = max_over_ranks(dist, [tc, td], "cuda")
    ms = tc + td

    # per-kernel durations for the roofline entries: the same compress with one cell group, i.e. every stage for all
    # cells before the next one starts, so that the library's CUDA-event stage timer (on the launching stream)
    # attributes the call to its stages; not part of the timed steps above
    lock = {}
    prev_groups = B.set_stream_groups(1)
    try:
        n_lock = 3
        for i in range(n_lock + 1):
            h = B.jolt_compress(K, V, gs, plans, opts)
            torch.cuda.synchronize()
            if i:       # the first call warms the single-group path up
                for k_, v_ in B.stage_ms().items():
                    lock[k_] = lock.get(k_, 0.0) + v_ / n_lock
            h.free()
    finally:
        B.set_stream_groups(prev_groups)

    # accuracy of the benchmarked configuration (mean relative Frobenius error over cells)
    errs = []
    for c in range(2 * ng):
        g, w = divmod(c, 2)
        a = (K, V)[w][gs[g]:gs[g + 1]].float()
        b_ = (Ko, Vo)[w][gs[g]:gs[g + 1]].float()
        if args.rope and w == 0:
            a = torch_rope(a, 10000.0)
        errs.append(float((a - b_).norm() / a.norm()))
    rel_k = sum(errs[0::2]) / ng
    rel_v = sum(errs[1::2]) / ng

    # attention computed on the compressed cache (not part of the headline metric)
    attend = None
    if args.attend:
        h = B.jolt_compress(K, V, gs, plans, opts)
        Qa = torch.randn(K.shape[0], K.shape[1], args.attend, 128, device=K.device)
        for _ in range(3):
            B.jolt_attend(h, Qa)
        torch.cuda.synchronize()
        ts = []
        for _ in range(max(args.steps, 5)):
            a0, a1 = ev(), ev()
            a0.record()
            B.jolt_attend(h, Qa)
            a1.record()
            torch.cuda.synchronize()
            ts.append(a0.elapsed_time(a1))
        ts.sort()
        t_att = ts[len(ts) // 2]
        attend = {"n_q": args.attend, "ms": t_att, "compressed_bytes": planned_bytes,
                  "gbs_of_compressed": planned_bytes / (t_att * 1e-3) / 1e9,
                  "frac_of_hbm_peak": planned_bytes / (t_att * 1e-3) / 1e9 / pk["hbm"],
                  "decode_then_read_ms": td + cache_bytes / (pk["hbm"] * 1e9) * 1e3}
        h.free()

    # end to end through the public API with host buffers (pinned), copies inside the timed region
    e2e = None
    if not args.no_e2e:
        Kh, Vh = K.cpu().pin_memory(), V.cpu().pin_memory()
        Koh, Voh = torch.empty_like(Kh).pin_memory(), torch.empty_like(Vh).pin_memory()

        def step_host():
            h = B.jolt_compress(Kh, Vh, gs, plans, opts)
            B.jolt_decompress(h, Koh, Voh, gs)
            h.free()
        for _ in range(2):
            step_host()
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
        t0 = time.perf_counter()
        n_e2e = max(2, min(args.steps, 5))
        for _ in range(n_e2e):
            step_host()
        torch.cuda.synchronize()
        te = (time.perf_counter() - t0) / n_e2e
        te = max_over_ranks(dist, [te], "cuda")[0]
        e2e = {"value": job_throughput(world, cache_bytes, te * 1e3), "unit": UNIT, "h2d_bytes_per_step": cache_bytes,
               "d2h_bytes_per_step": cache_bytes, "ms_per_step": te * 1e3}
        del Kh, Vh, Koh, Voh

    if rank != 0:
        if dist:
            dist.destroy_process_group()
        return

    # roofline bookkeeping
    q = cfg.power_iters
    tot = {}
    for c, (rt, rf, b) in enumerate(plans):
        kk = min(rt + 10, cfg.seq_len, cfg.m * rf)
        w = cell_work(cfg.m, cfg.seq_len, cfg.head_dim, rt, rf, b, kk, q, 2)
        for name, val in w.items():
            if isinstance(val, tuple):
                f0, b0 = tot.get(name, (0, 0))
                tot[name] = (f0 + val[0], b0 + val[1])
            else:
                tot[name] = tot.get(name, 0) + val
    t_roof_c = sum(roof_time(*cell_work(cfg.m, cfg.seq_len, cfg.head_dim, rt, rf, b, min(rt + 10, cfg.seq_len, cfg.m * rf), q, 2)["compress"], pk)
                   for rt, rf, b in plans)
    t_roof_d = sum(roof_time(*cell_work(cfg.m, cfg.seq_len, cfg.head_dim, rt, rf, b, min(rt + 10, cfg.seq_len, cfg.m * rf), q, 2)["decompress"], pk)
                   for rt, rf, b in plans)
    stages = {k_: v_ / len(rec) for k_, v_ in stage_acc.items()}
    # roofline of the dominant kernel of the headline (decompress) call: the decode kernel (persistent form, or the
    # per-item one) is the only kernel of jolt_decompress; its duration is the library's own CUDA-event stage timer on the launching stream
    fd, bd = tot["decompress"]
    t_dec = stages.get("decode_rows", td)
    dec_bound = "hbm" if bd / (pk["hbm"] * 1e9) >= fd / (pk["tensor"] * 1e12) else "tensor"
    # DRAM traffic of one launch: ncu capture of a few cells (profiles/dram_traffic.txt), scaled by the cells of this run
    dec_kernel = "tc::decode_kernel" if args.rope else "tc::decode_persistent_kernel"
    tr = dram_traffic(dec_kernel, cfg.name)
    traffic = (tr["read"] + tr["write"]) * (2 * ng) / tr["cells"] if tr else None
    if dec_bound == "hbm":
        ach = bd / (t_dec * 1e-3) / 1e9
        roofline = {"kernel": dec_kernel, "bound": "hbm", "achieved": ach, "peak": pk["hbm"], "unit": "GB/s",
                    "frac": ach / pk["hbm"], "traffic": traffic, "algorithmic_bytes": bd, "kernel_ms": t_dec,
                    "peak_source": pk["source"] + " (MEASURED_PEAKS.json hbm_gbs)"}
    else:
        ach = fd / (t_dec * 1e-3) / 1e12
        roofline = {"kernel": dec_kernel, "bound": "tensor", "achieved": ach, "peak": pk["tensor"], "unit": "TFLOP/s",
                    "frac": ach / pk["tensor"], "traffic": traffic, "algorithmic_flops": fd, "kernel_ms": t_dec,
                    "peak_source": pk["source"] + " (MEASURED_PEAKS.json bf16_tflops, burst)"}

    # compress: its largest GPU-filling kernel is the fused residual pass (tc::backbone_kernel<true>: X in, codes and
    # scales out), HBM-bound; the factor sweeps (tc::tc_gemm2_kernel) read X once each and are bound by the tensor
    # pipe once the dense operand is split in hi + lo (two MMAs per K step)
    fr, br_ = tot["residual_quant"]
    t_res = lock.get("residual_quant")
    roof_c = None
    if t_res:
        tr = dram_traffic("tc::backbone_kernel<1>", cfg.name)
        ach = br_ / (t_res * 1e-3) / 1e9
        roof_c = {"kernel": "tc::backbone_kernel<1>", "bound": "hbm", "achieved": ach, "peak": pk["hbm"], "unit": "GB/s",
                  "frac": ach / pk["hbm"], "traffic": (tr["read"] + tr["write"]) * (2 * ng) / tr["cells"] if tr else None,
                  "algorithmic_bytes": br_, "kernel_ms": t_res,
                  "peak_source": pk["source"] + " (MEASURED_PEAKS.json hbm_gbs)"}
    roof_s = None
    t_sw = lock.get("project")
    if t_sw:
        fs, bs = tot["project"]
        # split operand: the sweep issues two MMAs per K step for every cell (the algorithmic count has one)
        t_hbm, t_tc = bs / (pk["hbm"] * 1e9), 2 * fs / (pk["tensor"] * 1e12)
        roof_s = {"kernel": "tc::tc_gemm2_kernel<FEAT> (projection sweep)", "bound": "tensor" if t_tc > t_hbm else "hbm",
                  "achieved_gbs": bs / (t_sw * 1e-3) / 1e9, "achieved_tflops_issued": 2 * fs / (t_sw * 1e-3) / 1e12,
                  "frac": max(t_hbm, t_tc) * 1e3 / t_sw, "kernel_ms": t_sw, "algorithmic_bytes": bs, "algorithmic_flops": fs}

    line = {"metric": METRIC, "value": job_throughput(world, cache_bytes, ms), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": W, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f16 operands, f32 accumulate (f64 Cholesky, f32 Jacobi)", "data": "synthetic",
            "config": {"workload": f"{cfg.name}: {ng * cfg.layers_per_group} layers / {cfg.layers_per_group} per group, "
                                   f"{cfg.n_kv_heads} KV heads, T={cfg.seq_len}, d=128, fp16, budget {ratio}x, "
                                   + (f"randomized q={q}" if args.token_mode == "randomized" else "exact (converged block iteration)"),
                       "cache_bytes": cache_bytes, "compressed_bytes": planned_bytes, "achieved_ratio": cache_bytes / planned_bytes,
                       "rope_at_decode": bool(args.rope), "plan": plans, "l2": f"inputs ({cache_bytes / 1e6:.0f} MB) exceed L2; no flush"},
            "compress_ms": tc, "decompress_ms": td, "plan_ms": plan_ms, "plan_ms_warm": plan_ms_warm,
            "compress_ms_min_med_max": [tc_all[0], tc_all[len(tc_all) // 2], tc_all[-1]],
            "decompress_ms_min_med_max": [td_all[0], td_all[len(td_all) // 2], td_all[-1]],
            "compress_gbs": world * cache_bytes / (tc * 1e-3) / 1e9, "decompress_gbs": world * cache_bytes / (td * 1e-3) / 1e9,
            "compress_roofline_frac": t_roof_c * 1e3 / tc, "decompress_roofline_frac": t_roof_d * 1e3 / td,
            "compress_roofline_ms": t_roof_c * 1e3, "decompress_roofline_ms": t_roof_d * 1e3,
            "rel_frobenius_error": {"K": rel_k, "V": rel_v},
            "stages_ms": stages, "compress_stages_ms_one_group": lock, "roofline": roofline, "roofline_compress": roof_c,
            "roofline_sweep": roof_s, "gpu_launches": launches, "clocks": clocks, "e2e": e2e,
            "same_plan_as_reference_arm": (cfg.name == "c1" and ng == cfg.n_groups and [tuple(p) for p in plans] == C1_PLAN)}
    if attend:
        line["attend"] = attend

    if not args.no_cpu_baseline and world == 1:
        from oracle import jolt_oracle as O
        t0 = time.perf_counter()
        sample = {}
        jolt_err = {}
        for w_ in (0, 1):
            X = (K, V)[w_][gs[0]:gs[1]].reshape(cfg.m, cfg.seq_len, 128).cpu().numpy()
            a = time.perf_counter()
            oc = O.compress_cell(X, *plans[w_], seed=cfg.seed, cell=w_, token_mode="randomized", power_iters=q)
            b_ = time.perf_counter()
            Xo = O.decompress_cell(oc)
            c_ = time.perf_counter()
            sample[w_] = (b_ - a, c_ - b_)
            jolt_err["KV"[w_]] = O.rel_frobenius(X, Xo)
        sc = sum(v[0] for v in sample.values()); sd = sum(v[1] for v in sample.values())
        sb = 2 * cfg.m * cfg.seq_len * 128 * 2
        line["cpu_baseline"] = {"value": sb / (sc + sd) / 1e9, "unit": UNIT, "cores": torch.get_num_threads(), "kind": "oracle",
                                "sample": "cells 0 and 1 (group 0, K and V) of the same cache and plan, numpy fp64",
                                "compress_gbs": sb / sc / 1e9, "decompress_gbs": sb / sd / 1e9}
        # error context of the paper's reconstruction table (Sec. 6): the two baselines it lists, restated in the oracle,
        # on the first 1024 tokens (the table's length) of layer group 0; not timed, not part of the metric
        from oracle import baselines as BL
        Tc = min(1024, cfg.seq_len)
        ctx = {"tokens": Tc, "ratio_target": ratio, "jolt_oracle_full_length": jolt_err,
               "int4_per_channel": {"ratio": BL.int4_per_channel_ratio(Tc)}, "cross_layer_svd": {}}
        for w_ in (0, 1):
            Xg = (K, V)[w_][gs[0]:gs[1], :, :Tc].cpu().numpy().astype("float64")
            Xh, _ = BL.int4_per_channel(Xg.reshape(-1, Tc, 128))
            ctx["int4_per_channel"]["KV"[w_]] = BL.rel_frobenius(Xg.reshape(-1, Tc, 128), Xh)
            Xs, stored, r = BL.cross_layer_svd(Xg, ratio)
            ctx["cross_layer_svd"]["KV"[w_]] = BL.rel_frobenius(Xg, Xs)
            ctx["cross_layer_svd"]["rank"] = r
            ctx["cross_layer_svd"]["ratio"] = Xg.size * 2 / stored
        line["cpu_baseline"]["error_context"] = ctx
    print(json.dumps(line))
    if dist:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
