"""world_size-2 test of the sharded scheduler's host logic on CPU (gloo): the partition of the jobs, the
rebasing of a shard's arrays, and the all-gather that puts rank r's bids at row r.  The per-shard select and the
fold of the bids are played by the oracle and a few numpy lines here (on a GPU they are sja_select,
sja_get_bids and sja_reduce_bids); the result must equal the oracle's unsharded select."""
import os

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2509_19086_b200 import sharded
from paper_2509_19086_b200 import workloads as wl

BID = np.dtype([("key", "<u8"), ("job", "<u4"), ("end_step", "<u4"), ("dur_ms", "<u4"), ("rank", "<u4"),
                ("score", "<u8")])


def _bids_from_awards(aw, prio, policy, lo, rank):
    b = np.zeros(aw.shape[0], BID)
    has = aw["job"] != 0xFFFFFFFF
    key = aw["score"].astype(np.uint64) + np.uint64(1)
    if policy == 2:
        key = key + (prio[np.where(has, aw["job"], 0)].astype(np.uint64) << np.uint64(55))
    b["key"] = np.where(has, key, 0)
    b["job"] = np.where(has, aw["job"] + lo, 0xFFFFFFFF)
    b["end_step"], b["dur_ms"], b["score"], b["rank"] = aw["end_step"], aw["dur_ms"], aw["score"], rank
    return b


def _worker(rank, world, port, out):
    import oracle
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        res = {}
        for policy, base in ((0, 1), (2, 3)):
            spec = wl.scaled(wl.SPECS[base], n_jobs=301, fixed_len=60, n_gaps=40, policy=policy)
            prof = wl.make_profiles(spec, threads=1)
            gaps = wl.make_gaps(spec)
            lo, hi = sharded.shard_bounds(prof.n_jobs, world, rank)
            sp = sharded.shard_profiles(prof, lo, hi)
            z = np.zeros(hi - lo, np.uint32)
            local = oracle.select(sp, z, sp.ready_ms, gaps, policy)
            bids = _bids_from_awards(local, sp.prio, policy, lo, rank)
            allb = sharded.gather_bids(torch.from_numpy(bids.view(np.uint8).copy()), dist).numpy().view(BID)
            allb = allb.reshape(world, -1)
            assert (allb["rank"] == np.arange(world)[:, None]).all()          # rank r at row r
            best = np.zeros(gaps.shape[0], BID)
            for g in range(gaps.shape[0]):
                col = allb[:, g]
                k = col["key"].max()
                cand = col[col["key"] == k]
                best[g] = cand[np.argmin(cand["job"])]
            full = oracle.select(prof, np.zeros(prof.n_jobs, np.uint32), prof.ready_ms, gaps, policy)
            ok = all(np.array_equal(np.where(best["key"] > 0, best[f], full[f]), full[f])
                     for f in ("job", "end_step", "dur_ms", "score"))
            ok = ok and np.array_equal(best["key"] == 0, full["job"] == 0xFFFFFFFF)
            res[policy] = (bool(ok), lo, hi, int((best["rank"][best["key"] > 0] == rank).sum()))
        out[rank] = res
    finally:
        dist.destroy_process_group()


def test_two_shards_with_gloo():
    world = 2
    port = 31500 + (os.getpid() % 2000)
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    for policy in (0, 2):
        (ok0, lo0, hi0, w0), (ok1, lo1, hi1, w1) = out[0][policy], out[1][policy]
        assert ok0 and ok1
        assert (lo0, hi0, lo1, hi1) == (0, 151, 151, 301)
        assert w0 + w1 > 0


def test_shard_bounds_and_rebasing():
    for n, w in ((10, 3), (7, 7), (5, 8), (1000, 6)):
        b = [sharded.shard_bounds(n, w, r) for r in range(w)]
        assert b[0][0] == 0 and b[-1][1] == n
        assert all(b[r][1] == b[r + 1][0] for r in range(w - 1))
        sizes = [hi - lo for lo, hi in b]
        assert max(sizes) - min(sizes) <= 1 and sizes == sorted(sizes, reverse=True)
    spec = wl.scaled(wl.SPECS[3], n_jobs=50, zipf_max=200, n_gaps=4)
    prof = wl.make_profiles(spec, threads=1)
    sp = sharded.shard_profiles(prof, 17, 33)
    a, b = int(prof.off[17]), int(prof.off[33])
    assert sp.n_jobs == 16 and sp.off[0] == 0 and sp.n_steps == b - a
    assert np.array_equal(sp.dur_ms, prof.dur_ms[a:b]) and np.array_equal(sp.prio, prof.prio[17:33])
    assert np.array_equal(wl.unpack_safe_bits(sp.safe_bits, sp.n_steps), wl.unpack_safe_bits(prof.safe_bits, prof.n_steps)[a:b])
