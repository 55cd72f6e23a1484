"""The N > 1 path of the benchmark on CPU (gloo, world size 2): ranks take independent sequences, timings are
reduced with a maximum over ranks, throughput is the whole job's.  No data-path collective exists to test:
cells and sequences are independent."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        shard = bench.shard_of_rank(rank, world, base_seed=4)
        # every rank generates ITS sequence (tiny stand-in of the cache generator) and "times" a step
        from paper_2607_12550_b200 import synth
        cfg = synth.CacheConfig("t", 1, 1, 2, 128, n_terms=4, seed=4)
        K, _ = synth.make_cache(cfg, seq=shard["seq"])
        local_ms = [10.0 + 5.0 * rank, 1.0 + rank]
        dist.barrier()
        red = bench.max_over_ranks(dist, local_ms, "cpu")
        sums = torch.tensor([float(K.float().abs().sum())], dtype=torch.float64)
        gathered = [torch.zeros_like(sums) for _ in range(world)]
        dist.all_gather(gathered, sums)
        out[rank] = (shard, red, [float(g) for g in gathered])
    finally:
        dist.destroy_process_group()


def test_two_ranks_weak_scaling_helpers():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
    assert set(out.keys()) == {0, 1}
    (s0, r0, g0), (s1, r1, g1) = out[0], out[1]
    assert s0 == {"seq": 0, "seed": 4} and s1 == {"seq": 1, "seed": 5}
    assert r0 == r1 == [15.0, 2.0]                       # max over ranks, identical on every rank
    assert g0 == g1 and g0[0] != g0[1]                   # different ranks hold different sequences
    assert bench.job_throughput(2, 10 ** 9, 1000.0) == 2.0
    assert bench.max_over_ranks(None, [3.0, 4.0], "cpu") == [3.0, 4.0]
