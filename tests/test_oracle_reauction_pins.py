"""Pins for the re-auction round of the oracle (properties that do not mention its loop)."""
import numpy as np

from paper_2509_19086_b200 import workloads as wl
from tests.helpers import gaps_from_lists, profiles_from_lists, random_small_profiles

U32MAX = 0xFFFFFFFF


def _interested(oracle, prof, j, p, ready, gap):
    return oracle.brute_pair(prof, j, int(p), int(ready), int(gap["start_ms"]), int(gap["T_ms"]),
                             int(gap["C_MiB"]))


def test_reauction_fixpoint_is_stable_and_valid(oracle_mod):
    """At the fixpoint: every grant is a valid longest subjob from the pre-round state, no job
    is granted twice, and every unfilled gap has no interested job left that is still free."""
    oracle = oracle_mod
    rng = np.random.default_rng(21)
    for trial in range(25):
        jobs = random_small_profiles(rng, int(rng.integers(2, 10)), 14, p_safe=0.4, dmax=9, mmax=20)
        J = len(jobs)
        prof = profiles_from_lists(jobs, ready=rng.integers(0, 4, J), wait=rng.integers(0, 5000, J),
                                   prio=rng.integers(0, 3, J))
        G = int(rng.integers(2, 12))
        gaps = gaps_from_lists([(0, int(rng.integers(0, 6)), int(rng.integers(5, 40)), int(rng.integers(5, 22)))
                                for _ in range(G)])
        policy = trial % 3
        p0 = np.zeros(J, np.uint32)
        r0 = prof.ready_ms.copy()
        progress, ready = p0.copy(), r0.copy()
        aw, n, passes = oracle.round_with_reauction(prof, progress, ready, gaps, policy)
        granted = np.nonzero(aw["granted"] == 1)[0]
        assert n == granted.size and passes >= 1
        jobs_g = aw["job"][granted]
        assert np.unique(jobs_g).size == jobs_g.size
        for g in granted:
            j = int(aw["job"][g])
            want = _interested(oracle, prof, j, p0[j], r0[j], gaps[g])
            assert want is not None and (int(aw["end_step"][g]), int(aw["dur_ms"][g])) == want[:2]
            assert progress[j] == aw["end_step"][g] and ready[j] == gaps["start_ms"][g] + aw["dur_ms"][g]
        free = np.setdiff1d(np.arange(J), jobs_g)
        assert (progress[free] == 0).all()
        for g in np.nonzero(aw["granted"] == 0)[0]:
            for j in free:
                assert _interested(oracle, prof, int(j), p0[j], r0[j], gaps[g]) is None, (trial, g, j)


def test_reauction_first_pass_is_plain_round_and_max_passes(oracle_mod):
    oracle = oracle_mod
    spec = wl.scaled(wl.SPECS[4], n_jobs=60, fixed_len=80, n_gaps=40, n_rounds=1)
    prof = wl.make_profiles(spec, threads=1)
    gaps = wl.make_gaps(spec)
    p1, r1 = np.zeros(prof.n_jobs, np.uint32), prof.ready_ms.copy()
    plain = oracle.select(prof, p1, r1, gaps, 0)
    n_plain = oracle.commit(p1, r1, gaps, plain)
    p2, r2 = np.zeros(prof.n_jobs, np.uint32), prof.ready_ms.copy()
    aw1, n1, passes1 = oracle.round_with_reauction(prof, p2, r2, gaps, 0, max_passes=1)
    assert passes1 == 1 and n1 == n_plain and aw1.tobytes() == plain.tobytes()
    assert np.array_equal(p1, p2) and np.array_equal(r1, r2)
    p3, r3 = np.zeros(prof.n_jobs, np.uint32), prof.ready_ms.copy()
    aw, n, passes = oracle.round_with_reauction(prof, p3, r3, gaps, 0)
    assert passes > 1 and n > n_plain                       # orphaned gaps do get filled
    kept = plain["granted"] == 1
    assert aw[kept].tobytes() == plain[kept].tobytes()       # grants of pass 0 stand


def test_reauction_hand_example(oracle_mod):
    """Job 0 wins both gaps, takes the longer one; job 1 then fills the other (hand-computed)."""
    oracle = oracle_mod
    prof = profiles_from_lists([([10] * 6, [9] * 6, [1] * 6), ([10] * 6, [2] * 6, [1] * 6)])
    gaps = gaps_from_lists([(0, 0, 25, 50), (1, 0, 45, 50)])
    progress, ready = np.zeros(2, np.uint32), prof.ready_ms.copy()
    aw, n, passes = oracle.round_with_reauction(prof, progress, ready, gaps, 0)
    assert (n, passes) == (2, 2)
    assert aw["job"].tolist() == [1, 0] and aw["granted"].tolist() == [1, 1]
    assert aw["end_step"].tolist() == [2, 4] and aw["score"].tolist() == [40, 360]
    assert progress.tolist() == [4, 2] and ready.tolist() == [40, 20]
