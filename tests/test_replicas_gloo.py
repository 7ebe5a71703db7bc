"""world_size-2 test of the multi-GPU host logic on CPU (gloo): replicas get distinct seeded
workloads, throughput is summed over ranks and timed by the slowest rank."""
import os

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2509_19086_b200 import replicas
from paper_2509_19086_b200 import workloads as wl


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        spec = replicas.replica_spec(wl.scaled(wl.SPECS[0], n_jobs=8, fixed_len=32, n_gaps=4), rank)
        prof = wl.make_profiles(spec, threads=1)
        gaps = wl.make_gaps(spec)
        pairs = prof.n_jobs * gaps.shape[0]
        local_ms = [10.0 + 5.0 * rank, 100.0 - 30.0 * rank]
        total, mx = replicas.aggregate(pairs, local_ms, dist)
        out[rank] = dict(seed=spec.seed, d0=int(prof.dur_ms[:8].sum()), total=total, mx=mx,
                         value=replicas.throughput(total, 4, mx[0]))
    finally:
        dist.destroy_process_group()


def test_two_replicas_aggregate_with_gloo():
    world = 2
    port = 29500 + (os.getpid() % 2000)
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    r0, r1 = out[0], out[1]
    assert r0["seed"] == wl.BASE_SEED and r1["seed"] == wl.BASE_SEED + 1000
    assert r0["total"] == r1["total"] == 2 * 8 * 4            # work of both ranks
    assert r0["mx"] == r1["mx"] == [15.0, 100.0]              # slowest rank per timer
    assert r0["value"] == r1["value"] == 64 * 4 / 15e-3


def test_single_process_aggregate_is_identity():
    total, mx = replicas.aggregate(12.0, [3.0, 4.0], None)
    assert total == 12.0 and mx == [3.0, 4.0]
    assert replicas.replica_spec(wl.SPECS[2], 0) is wl.SPECS[2]
    assert replicas.replica_spec(wl.SPECS[2], 3).seed == wl.SPECS[2].seed + 3000
    assert replicas.throughput(10.0, 2, 0.0) == 0.0
