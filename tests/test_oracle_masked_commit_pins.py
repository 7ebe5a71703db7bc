"""Pin for the masked commit of the oracle: not taking up a grant is the same, for grants and job
state, as never having advertised that gap (select treats gaps independently)."""
import numpy as np

from paper_2509_19086_b200 import workloads as wl


def test_masked_commit_equals_round_without_the_masked_gaps(oracle_mod):
    oracle = oracle_mod
    spec = wl.scaled(wl.SPECS[4], n_jobs=70, fixed_len=90, n_gaps=48, n_rounds=1)
    prof = wl.make_profiles(spec, threads=1)
    gaps = wl.make_gaps(spec)
    rng = np.random.default_rng(9)
    for trial in range(10):
        accept = (rng.random(gaps.shape[0]) < 0.6).astype(np.uint8)
        p1, r1 = np.zeros(prof.n_jobs, np.uint32), prof.ready_ms.copy()
        aw = oracle.select(prof, p1, r1, gaps, 0)
        n1 = oracle.commit_masked(p1, r1, gaps, aw, accept)
        assert not aw["granted"][accept == 0].any()
        keep = np.nonzero(accept)[0]
        p2, r2 = np.zeros(prof.n_jobs, np.uint32), prof.ready_ms.copy()
        sub = np.ascontiguousarray(gaps[keep])
        aw2 = oracle.select(prof, p2, r2, sub, 0)
        n2 = oracle.commit(p2, r2, sub, aw2)
        assert n1 == n2 and n1 > 0
        assert np.array_equal(p1, p2) and np.array_equal(r1, r2)
        assert aw[keep].tobytes() == aw2.tobytes()
    # all accepted = plain commit; none accepted = nothing happens
    p3, r3 = np.zeros(prof.n_jobs, np.uint32), prof.ready_ms.copy()
    aw3 = oracle.select(prof, p3, r3, gaps, 0)
    plain = aw3.copy()
    p4, r4 = p3.copy(), r3.copy()
    assert oracle.commit_masked(p3, r3, gaps, aw3, np.ones(gaps.shape[0], np.uint8)) == oracle.commit(p4, r4, gaps, plain)
    assert aw3.tobytes() == plain.tobytes() and np.array_equal(p3, p4)
    p5, r5 = np.zeros(prof.n_jobs, np.uint32), prof.ready_ms.copy()
    aw5 = oracle.select(prof, p5, r5, gaps, 0)
    assert oracle.commit_masked(p5, r5, gaps, aw5, np.zeros(gaps.shape[0], np.uint8)) == 0
    assert not p5.any() and not aw5["granted"].any()
