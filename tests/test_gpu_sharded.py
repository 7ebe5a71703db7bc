"""One scheduler over several job shards, emulated on one GPU: every shard is a context of its own, run one
after the other (no kernel waits on another), the gathered bids are a concatenation.  Awards, grants and job
state must equal the oracle's for the unsharded problem, round after round."""
import numpy as np
import pytest

from paper_2509_19086_b200 import sharded
from paper_2509_19086_b200 import workloads as wl

pytestmark = pytest.mark.gpu
FIELDS = ("job", "end_step", "dur_ms", "score")
U32MAX = 0xFFFFFFFF


@pytest.mark.parametrize("base,changes,world", [
    (1, dict(n_jobs=1501, fixed_len=500, n_gaps=300), 2),
    (2, dict(n_jobs=2500, fixed_len=400, n_gaps=500), 4),
    (3, dict(n_jobs=1300, zipf_max=2500, n_gaps=400), 3),
])
def test_sharded_rounds_equal_the_unsharded_oracle(oracle_mod, base, changes, world):
    from paper_2509_19086_b200 import binding
    spec = wl.scaled(wl.SPECS[base], **changes)
    prof = wl.make_profiles(spec, threads=2)
    J = prof.n_jobs
    bounds = [sharded.shard_bounds(J, world, r) for r in range(world)]
    assert bounds[0][0] == 0 and bounds[-1][1] == J and all(bounds[r][1] == bounds[r + 1][0] for r in range(world - 1))
    progress = np.zeros(J, np.uint32)
    ready = prof.ready_ms.copy()
    ctxs = [binding.Sja() for _ in range(world)]
    try:
        for r, (lo, hi) in enumerate(bounds):
            sp = sharded.shard_profiles(prof, lo, hi)
            ctxs[r].load_profiles(sp.off, sp.dur_ms, sp.mem_MiB, sp.safe_bits, sp.ready_ms,
                                  wait_ms=sp.wait_ms, prio=sp.prio)
        for rnd in range(5):
            gaps = wl.make_gaps(spec, rnd)
            want = oracle_mod.select(prof, progress, ready, gaps, spec.policy)
            bids = []
            for r, (lo, hi) in enumerate(bounds):
                ctxs[r].advertise(gaps)
                ctxs[r].select(spec.policy)
                bids.append(ctxs[r].get_bids(lo, r))
            all_bids = np.concatenate(bids)                    # what an all-gather delivers: rank r at r * G
            n_total = 0
            for r in range(world):
                accept, glob = ctxs[r].reduce_bids(world, r, all_bids)
                for f in FIELDS:
                    assert np.array_equal(glob[f], want[f]), (rnd, r, f)
                owner = np.searchsorted([b[1] for b in bounds], want["job"], side="right")
                assert np.array_equal(accept == 1, (want["job"] != U32MAX) & (owner == r))
                n_total += ctxs[r].commit_masked(accept)
            assert n_total == oracle_mod.commit(progress, ready, gaps, want)
            for r, (lo, hi) in enumerate(bounds):
                p, rd = ctxs[r].get_state()
                assert np.array_equal(p, progress[lo:hi]) and np.array_equal(rd, ready[lo:hi])
    finally:
        for c in ctxs:
            c.close()


def test_sharded_scheduler_single_rank_with_device_buffers(oracle_mod):
    """The ShardedScheduler wrapper with one rank (no collective): device buffers all the way."""
    import torch
    from paper_2509_19086_b200 import binding
    spec = wl.scaled(wl.SPECS[2], n_jobs=2000, fixed_len=300, n_gaps=256)
    prof = wl.make_profiles(spec, threads=2)
    progress = np.zeros(prof.n_jobs, np.uint32)
    ready = prof.ready_ms.copy()
    with binding.Sja() as ctx:
        ctx.load_profiles(prof.off, prof.dur_ms, prof.mem_MiB, prof.safe_bits, prof.ready_ms,
                          wait_ms=prof.wait_ms, prio=prof.prio)
        sched = sharded.ShardedScheduler(ctx, 0, 0, 1)
        for rnd in range(3):
            gaps = wl.make_gaps(spec, rnd)
            glob, n = sched.round(gaps, spec.policy, want_count=True)
            torch.cuda.synchronize()
            got = glob.cpu().numpy().view(binding.AWARD_DTYPE)
            want = oracle_mod.select(prof, progress, ready, gaps, spec.policy)
            for f in FIELDS:
                assert np.array_equal(got[f], want[f]), (rnd, f)
            assert n == oracle_mod.commit(progress, ready, gaps, want)
