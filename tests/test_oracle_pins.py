"""Pins for the CPU oracle: it is checked against things other than itself.

P1 exhaustive prefix enumeration on tiny inputs       P5 closed form
P2 invariants on every award                          P6 monotonicity / symmetry
P3 rigid-job special case (only the last step safe)   P7 the paper's illustrative scenario
P4 reductions to numpy cumsum / searchsorted          P8 hand-computed policy examples
A planted mistake in the walk (wrong sign, dropped term, off-by-one on a bound, a missed
boundary) fails at least one of these.
"""
import itertools
import json
import os

import numpy as np
import pytest

from paper_2509_19086_b200 import workloads as wl
from tests.helpers import gaps_from_lists, profiles_from_lists, random_small_profiles

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
U32MAX = 0xFFFFFFFF


def _select_all(oracle, prof, gaps, policy, progress=None, ready=None):
    J = prof.n_jobs
    progress = np.zeros(J, np.uint32) if progress is None else progress
    ready = prof.ready_ms if ready is None else ready
    return oracle.select(prof, progress, ready, gaps, policy)


# ---------------------------------------------------------------- P1 brute force
def test_p1_all_safe_masks_exhaustive(oracle_mod):
    """Every safe mask of a 7-step job, several (T, C, p): walk == enumeration."""
    oracle = oracle_mod
    d = [3, 1, 4, 1, 5, 9, 2]
    m = [5, 8, 2, 9, 3, 7, 6]
    n = len(d)
    for mask in range(1 << n):
        s = [(mask >> i) & 1 for i in range(n)]
        prof = profiles_from_lists([(d, m, s)])
        for p, T, C in itertools.product([0, 2, 6, 7], [0, 3, 8, 13, 25, 100], [1, 5, 8, 9]):
            got = oracle.pair(prof, 0, p, 0, 0, T, C)
            want = oracle.brute_pair(prof, 0, p, 0, 0, T, C)
            assert got == want, (mask, p, T, C)


def test_p1_random_tiny_select(oracle_mod):
    oracle = oracle_mod
    rng = np.random.default_rng(7)
    for trial in range(60):
        jobs = random_small_profiles(rng, int(rng.integers(1, 9)), 12,
                                     p_safe=float(rng.uniform(0.05, 0.9)),
                                     allow_zero=(trial % 3 == 0))
        J = len(jobs)
        prof = profiles_from_lists(
            jobs, ready=rng.integers(0, 6, J), wait=rng.integers(0, 5000, J),
            prio=rng.integers(0, 3, J))
        lens = np.diff(prof.off).astype(np.int64)
        progress = np.array([rng.integers(0, l + 1) for l in lens], dtype=np.uint32)
        gaps = gaps_from_lists([(int(rng.integers(0, 7)), int(rng.integers(0, 8)),
                                 int(rng.integers(0, 40)), int(rng.integers(0, 22)))
                                for _ in range(6)])
        for policy in (0, 1, 2, 3):
            aw = oracle.select(prof, progress, prof.ready_ms, gaps, policy)
            ref = oracle.brute_select(prof, progress, prof.ready_ms, gaps, policy)
            for g in range(len(gaps)):
                for key in ("job", "end_step", "dur_ms", "score"):
                    assert int(aw[key][g]) == ref[g][key], (trial, policy, g, key)


# ---------------------------------------------------------------- P2 invariants
def _check_award_invariants(prof, progress, ready, gaps, aw):
    for g in range(len(gaps)):
        j = int(aw["job"][g])
        if j == U32MAX:
            assert aw["end_step"][g] == 0 and aw["dur_ms"][g] == 0 and aw["score"][g] == 0
            continue
        s = int(prof.off[j])
        p, k = int(progress[j]), int(aw["end_step"][g])
        T, C, start = int(gaps["T_ms"][g]), int(gaps["C_MiB"][g]), int(gaps["start_ms"][g])
        length = int(prof.off[j + 1]) - s
        assert p < k <= length
        d = prof.dur_ms[s + p:s + k].astype(np.int64)
        m = prof.mem_MiB[s + p:s + k].astype(np.int64)
        assert d.sum() == aw["dur_ms"][g] <= T                      # I1
        assert m.max() <= C                                         # I2
        safe = wl.unpack_safe_bits(prof.safe_bits, prof.n_steps)
        assert safe[s + k - 1] == 1 or k == length                  # I3
        assert start >= int(ready[j])                               # I6
        # I4 maximal: the next safe boundary (if any) breaks T or C
        nxt = [i for i in range(k + 1, length + 1) if safe[s + i - 1] or i == length]
        if nxt:
            k2 = nxt[0]
            d2 = prof.dur_ms[s + p:s + k2].astype(np.int64).sum()
            m2 = prof.mem_MiB[s + p:s + k2].astype(np.int64).max()
            assert d2 > T or m2 > C


def test_p2_invariants_cfg0(oracle_mod):
    oracle = oracle_mod
    spec = wl.SPECS[0]
    prof = wl.make_profiles(spec, threads=1)
    gaps = wl.make_gaps(spec)
    progress = np.zeros(prof.n_jobs, np.uint32)
    aw = oracle.select(prof, progress, prof.ready_ms, gaps, spec.policy)
    assert (aw["job"] != U32MAX).any()
    _check_award_invariants(prof, progress, prof.ready_ms, gaps, aw)
    # I7: select has no side effects and is repeatable
    aw2 = oracle.select(prof, progress, prof.ready_ms, gaps, spec.policy)
    assert aw.tobytes() == aw2.tobytes()
    assert not progress.any()


def test_p2_commit_invariants_multi_round(oracle_mod):
    """I5 / I8: one grant per job and round; committed subjobs tile a prefix of each job."""
    oracle = oracle_mod
    spec = wl.scaled(wl.SPECS[4], n_jobs=40, fixed_len=64, n_gaps=24, n_rounds=12)
    prof = wl.make_profiles(spec, threads=1)
    progress = np.zeros(prof.n_jobs, np.uint32)
    ready = prof.ready_ms.copy()
    safe = wl.unpack_safe_bits(prof.safe_bits, prof.n_steps)
    log = []
    total = 0
    for r in range(spec.n_rounds):
        gaps = wl.make_gaps(spec, r)
        before_p, before_r = progress.copy(), ready.copy()
        aw = oracle.select(prof, progress, ready, gaps, spec.policy)
        _check_award_invariants(prof, progress, ready, gaps, aw)
        n = oracle.commit(progress, ready, gaps, aw)
        total += n
        granted_jobs = aw["job"][aw["granted"] == 1]
        assert len(set(granted_jobs.tolist())) == len(granted_jobs) == n       # I5
        winners = set(aw["job"][aw["job"] != U32MAX].tolist())
        assert winners == set(granted_jobs.tolist())     # every winning job gets exactly one gap
        assert (progress >= before_p).all() and (ready >= before_r).all()
        for g in np.nonzero(aw["granted"])[0]:
            j = int(aw["job"][g])
            same = aw[(aw["job"] == j)]
            assert aw["end_step"][g] == same["end_step"].max()                  # R6
            assert g == min(h for h in range(len(aw)) if aw["job"][h] == j
                            and aw["end_step"][h] == aw["end_step"][g])
            assert progress[j] == aw["end_step"][g]
            assert ready[j] == gaps["start_ms"][g] + aw["dur_ms"][g]
            log.append((j, int(before_p[j]), int(progress[j])))
        untouched = np.setdiff1d(np.arange(prof.n_jobs), granted_jobs)
        assert (progress[untouched] == before_p[untouched]).all()
    assert total > 0
    # replaying the log tiles [0, p_j) and every cut is a safe boundary
    replay = np.zeros(prof.n_jobs, np.int64)
    for j, a, b in log:
        assert replay[j] == a and b > a
        assert safe[int(prof.off[j]) + b - 1] == 1
        replay[j] = b
    assert (replay == progress).all()


# ---------------------------------------------------------------- P3 rigid job
def test_p3_only_last_step_safe_is_rigid_admission(oracle_mod):
    """Only the end is a boundary: interest iff total duration <= T and global max <= C
    (the monolithic job of Sections 1 and 3.5)."""
    oracle = oracle_mod
    rng = np.random.default_rng(11)
    for _ in range(200):
        n = int(rng.integers(1, 30))
        d = rng.integers(1, 20, n).tolist()
        m = rng.integers(1, 50, n).tolist()
        s = [0] * n
        if rng.random() < 0.5:
            s[-1] = 1            # the end counts as a boundary with or without its bit
        prof = profiles_from_lists([(d, m, s)])
        p = int(rng.integers(0, n))
        T, C = int(rng.integers(1, 250)), int(rng.integers(1, 60))
        got = oracle.pair(prof, 0, p, 0, 0, T, C)
        fits = sum(d[p:]) <= T and max(m[p:]) <= C
        assert (got is not None) == fits
        if fits:
            assert got == (n, sum(d[p:]), sum(x * y for x, y in zip(d[p:], m[p:])))


# ---------------------------------------------------------------- P4 library reductions
def test_p4_all_safe_unbounded_capacity_is_searchsorted(oracle_mod):
    oracle = oracle_mod
    rng = np.random.default_rng(3)
    for _ in range(100):
        n = int(rng.integers(1, 200))
        d = rng.integers(0, 30, n)
        m = rng.integers(0, 1000, n)
        prof = profiles_from_lists([(d.tolist(), m.tolist(), [1] * n)])
        T = int(rng.integers(0, 2500))
        cs = np.cumsum(d)
        k = int(np.searchsorted(cs, T, side="right"))
        got = oracle.pair(prof, 0, 0, 0, 0, T, U32MAX)
        if k == 0:
            assert got is None
        else:
            assert got == (k, int(cs[k - 1]), int(np.cumsum(d * m)[k - 1]))


def test_p4_all_safe_unbounded_time_is_first_violation(oracle_mod):
    oracle = oracle_mod
    rng = np.random.default_rng(4)
    for _ in range(100):
        n = int(rng.integers(1, 200))
        d = rng.integers(1, 30, n)
        m = rng.integers(1, 1000, n)
        prof = profiles_from_lists([(d.tolist(), m.tolist(), [1] * n)])
        C = int(rng.integers(1, 1100))
        over = np.nonzero(m > C)[0]
        k = int(over[0]) if over.size else n
        got = oracle.pair(prof, 0, 0, 0, 0, U32MAX, C)
        if k == 0:
            assert got is None
        else:
            assert got is not None and got[0] == k


def test_p4_dense_prefix_matches_walk(oracle_mod):
    """k* = L[min(k_T, k_C)] on the dense arrays (library cumsum / cummax / searchsorted)."""
    oracle = oracle_mod
    rng = np.random.default_rng(5)
    jobs = random_small_profiles(rng, 20, 60, p_safe=0.2, dmax=30, mmax=100)
    prof = profiles_from_lists(jobs)
    for j in range(prof.n_jobs):
        length = int(prof.off[j + 1] - prof.off[j])
        for _ in range(10):
            p = int(rng.integers(0, length))
            T, C = int(rng.integers(0, 400)), int(rng.integers(1, 110))
            D, M, L, W = oracle.dense_prefix(prof, j, p)
            kT = int(np.searchsorted(D, T, side="right")) - 1
            kC = int(np.searchsorted(M, C, side="right")) - 1
            k = int(L[min(kT, kC)])
            got = oracle.pair(prof, j, p, 0, 0, T, C)
            if k <= p:
                assert got is None
            else:
                assert got == (k, int(D[k - p]), int(W[k - p]))
        rows = oracle.boundary_table(prof, j, 0)
        D, M, L, W = oracle.dense_prefix(prof, j, 0)
        assert [r[0] for r in rows] == sorted(set(int(x) for x in L[1:] if x > 0))
        assert rows[-1][0] == length


def test_p4_boundary_table_segment_maximum(oracle_mod):
    """The segment-maximum column of the boundary rows.  Hand-computed example, then the property the column
    exists for: started at any boundary row r0, the running maximum of the segment maxima over rows r0..r is
    the window maximum max m[k_{r0-1} .. k_r), i.e. the M column of a scan that starts at progress k_{r0-1}
    (library maximum.accumulate on the raw steps, not on the table)."""
    oracle = oracle_mod
    #            step  0  1  2  3  4  5  6  7
    prof = profiles_from_lists([([1, 2, 3, 4, 5, 6, 7, 8], [5, 9, 2, 7, 7, 1, 8, 3], [0, 1, 0, 0, 1, 1, 0, 0])])
    rows = oracle.boundary_table(prof, 0, 0)
    assert [(r[0], r[3]) for r in rows] == [(2, 9), (5, 7), (6, 1), (8, 8)]          # (k, segment maximum)
    assert [(r[1], r[2], r[4]) for r in rows] == [(3, 9, 23), (15, 9, 92), (21, 9, 98), (36, 9, 178)]   # D, M, W
    rows = oracle.boundary_table(prof, 0, 3)          # from progress 3: the first segment is steps 3..4 only
    assert [(r[0], r[3], r[2]) for r in rows] == [(5, 7, 7), (6, 1, 7), (8, 8, 8)]   # (k, segment max, M)
    rng = np.random.default_rng(55)
    jobs = random_small_profiles(rng, 12, 80, p_safe=0.25, dmax=30, mmax=500)
    prof = profiles_from_lists(jobs)
    for j in range(prof.n_jobs):
        s = int(prof.off[j])
        length = int(prof.off[j + 1]) - s
        p0 = int(rng.integers(0, length))
        rows = oracle.boundary_table(prof, j, p0)
        ks = [p0] + [r[0] for r in rows]
        m = prof.mem_MiB[s:s + length]
        for r0 in range(len(rows)):
            start = ks[r0]                               # progress point after committing up to row r0 - 1
            run = 0
            win = np.maximum.accumulate(m[start:])
            for r in range(r0, len(rows)):
                k, seg = rows[r][0], rows[r][3]
                assert seg == int(m[ks[r]:k].max())      # the segment since the previous boundary, nothing else
                run = max(run, seg)
                assert run == int(win[k - start - 1]), (j, p0, r0, r)


# ---------------------------------------------------------------- P5 closed form
@pytest.mark.parametrize("a,b,q,n,T,wait", [
    (7, 11, 4, 100, 365, 0), (1, 1, 1, 50, 17, 999), (13, 5, 10, 95, 5000, 123456),
    (50, 81920, 3, 4096, 5000, 3600000), (9, 2, 8, 40, 10**6, 5000),
])
def test_p5_constant_profile_closed_form(oracle_mod, a, b, q, n, T, wait):
    """d = a, m = b <= C, a boundary every q-th step: k = q * floor(floor(T/a)/q), capped."""
    oracle = oracle_mod
    s = [1 if (i + 1) % q == 0 else 0 for i in range(n)]
    s[-1] = 0 if n % q else s[-1]
    prof = profiles_from_lists([([a] * n, [b] * n, s)], wait=[wait])
    steps = min(T // a, n)
    k = n if steps == n else q * (steps // q)      # the end of the job is always a boundary
    gaps = gaps_from_lists([(0, 0, T, b)])
    aw = oracle.select(prof, np.zeros(1, np.uint32), prof.ready_ms, gaps, 1)
    if k == 0:
        assert aw["job"][0] == U32MAX
    else:
        assert (int(aw["job"][0]), int(aw["end_step"][0]), int(aw["dur_ms"][0])) == (0, k, k * a)
        assert int(aw["score"][0]) == k * a * b * (1 + wait // 1000)
    # capacity one MiB too small: decline
    aw = oracle.select(prof, np.zeros(1, np.uint32), prof.ready_ms,
                       gaps_from_lists([(0, 0, T, b - 1)]), 0)
    assert aw["job"][0] == U32MAX


# ---------------------------------------------------------------- P6 monotonicity / symmetry
def test_p6_monotone_in_T_and_C(oracle_mod):
    oracle = oracle_mod
    rng = np.random.default_rng(6)
    jobs = random_small_profiles(rng, 10, 80, p_safe=0.15, dmax=40, mmax=200)
    prof = profiles_from_lists(jobs)
    for j in range(prof.n_jobs):
        prev_k = 0
        for T in range(0, 600, 13):
            r = oracle.pair(prof, j, 0, 0, 0, T, 150)
            k = 0 if r is None else r[0]
            assert k >= prev_k
            prev_k = k
        prev_k = 0
        for C in range(0, 220, 7):
            r = oracle.pair(prof, j, 0, 0, 0, 300, C)
            k = 0 if r is None else r[0]
            assert k >= prev_k
            prev_k = k


def test_p6_duplicate_job_and_permutations(oracle_mod):
    oracle = oracle_mod
    rng = np.random.default_rng(8)
    jobs = random_small_profiles(rng, 12, 40, p_safe=0.3, dmax=30, mmax=100)
    jobs_dup = jobs + [jobs[3]]                       # job 12 is a copy of job 3
    J = len(jobs_dup)
    wait = rng.integers(0, 9000, J)
    wait[12] = wait[3]
    prio = rng.integers(0, 3, J)
    prio[12] = prio[3]
    prof = profiles_from_lists(jobs_dup, wait=wait, prio=prio)
    gaps = gaps_from_lists([(0, 0, int(rng.integers(10, 300)), int(rng.integers(20, 110)))
                            for _ in range(30)])
    for policy in (0, 1, 2, 3):
        aw = _select_all(oracle, prof, gaps, policy)
        assert not (aw["job"] == 12).any()            # the copy never beats the lower id
        # permuting the gaps permutes the awards
        perm = rng.permutation(len(gaps))
        aw_p = _select_all(oracle, prof, gaps[perm], policy)
        assert aw_p.tobytes() == aw[perm].tobytes()
    # reversing job order: same scores; winners differ only through ties
    rev = list(reversed(jobs_dup))
    prof_r = profiles_from_lists(rev, wait=wait[::-1], prio=prio[::-1])
    for policy in (0, 1, 2, 3):
        a = _select_all(oracle, prof, gaps, policy)
        b = _select_all(oracle, prof_r, gaps, policy)
        assert (a["score"] == b["score"]).all()
        assert ((a["job"] == U32MAX) == (b["job"] == U32MAX)).all()


def test_tight_fit_winner_leaves_the_least_slack(oracle_mod):
    """Policy 3 (Section 3.9, slack-minimising): no interested job would leave less slack C - peak on the
    slice than the winner, the winner's subjob is still its longest one, and the score is its peak."""
    oracle = oracle_mod
    rng = np.random.default_rng(88)
    jobs = random_small_profiles(rng, 40, 30, p_safe=0.3, dmax=9, mmax=60)
    prof = profiles_from_lists(jobs, ready=rng.integers(0, 5, 40))
    gaps = gaps_from_lists([(0, int(rng.integers(0, 8)), int(rng.integers(5, 120)), int(rng.integers(5, 70)))
                            for _ in range(40)])
    z = np.zeros(40, np.uint32)
    aw = oracle.select(prof, z, prof.ready_ms, gaps, 3)
    won = 0
    for g in range(len(gaps)):
        start, T, C = int(gaps["start_ms"][g]), int(gaps["T_ms"][g]), int(gaps["C_MiB"][g])
        pairs = [oracle.brute_pair(prof, j, 0, int(prof.ready_ms[j]), start, T, C) for j in range(40)]
        peaks = [None if r is None else max(jobs[j][1][:r[0]]) for j, r in enumerate(pairs)]
        interested = [j for j in range(40) if pairs[j] is not None]
        if not interested:
            assert int(aw["job"][g]) == U32MAX
            continue
        w = int(aw["job"][g])
        won += 1
        assert w in interested and int(aw["end_step"][g]) == pairs[w][0] and int(aw["score"][g]) == peaks[w]
        assert all(C - peaks[w] <= C - peaks[j] for j in interested)
        assert all(peaks[j] < peaks[w] for j in interested if j < w)     # lowest id among the tightest
    assert won > 20


def test_ready_time_and_finished_jobs(oracle_mod):
    oracle = oracle_mod
    prof = profiles_from_lists([([5], [5], [1]), ([5], [6], [1])], ready=[10, 11])
    gaps = gaps_from_lists([(0, 9, 100, 100), (0, 10, 100, 100), (0, 11, 100, 100)])
    aw = _select_all(oracle, prof, gaps, 0)
    assert aw["job"].tolist() == [U32MAX, 0, 1]       # start >= ready, inclusive
    aw = oracle.select(prof, np.array([1, 1], np.uint32), prof.ready_ms, gaps, 0)
    assert (aw["job"] == U32MAX).all()                # p == len: finished jobs decline
    # inclusive bounds on T and C
    assert oracle.pair(prof, 0, 0, 0, 0, 5, 5) == (1, 5, 25)
    assert oracle.pair(prof, 0, 0, 0, 0, 4, 5) is None
    assert oracle.pair(prof, 0, 0, 0, 0, 5, 4) is None


def test_zero_work_interest_is_not_lost(oracle_mod):
    """d = 0 or m = 0 steps are legal; a zero score still wins over 'no job'."""
    oracle = oracle_mod
    prof = profiles_from_lists([([0, 0], [0, 7], [1, 1])])
    aw = _select_all(oracle, prof, gaps_from_lists([(0, 0, 0, 7)]), 0)
    assert (int(aw["job"][0]), int(aw["end_step"][0]), int(aw["score"][0])) == (0, 2, 0)


# ---------------------------------------------------------------- P7 paper scenario
def test_p7_paper_illustrative_scenario(oracle_mod):
    oracle = oracle_mod
    with open(os.path.join(GOLDEN, "paper_scenario.json")) as f:
        sc = json.load(f)
    d, m = [], []
    for ph in sc["profile"]["phases"]:
        d += [ph["duration_ms"]] * ph["steps"]
        m += [ph["mem_MiB"]] * ph["steps"]
    assert max(m) == sc["from_paper"]["declared_peak_MiB"]
    n = len(d)
    for case in sc["cases"]:
        q = sc["profile"]["safe_every"]
        s = [1 if (i + 1) % q == 0 else 0 for i in range(n)] if case["atomizable"] else [0] * n
        s[-1] = 1
        prof = profiles_from_lists([(d, m, s)])
        got = oracle.pair(prof, 0, 0, 0, 0, case["T_ms"], case["C_MiB"])
        exp = case["expect"]
        assert (got is not None) == exp["interest"], case["name"]
        if exp["interest"]:
            assert got == (exp["end_step"], exp["dur_ms"], exp["work"]), case["name"]


# ---------------------------------------------------------------- P8 policy examples
def test_p8_hand_computed_policy_examples(oracle_mod):
    oracle = oracle_mod
    with open(os.path.join(GOLDEN, "policy_examples.json")) as f:
        gold = json.load(f)
    g = gold["gap"]
    gaps = gaps_from_lists([(g["slice"], g["start_ms"], g["T_ms"], g["C_MiB"])])
    for ex in gold["examples"]:
        prof = profiles_from_lists([(j["d"], j["m"], j["safe"]) for j in ex["jobs"]],
                                   wait=ex.get("wait_ms"), prio=ex.get("prio"))
        aw = _select_all(oracle, prof, gaps, ex["policy"])
        for key, val in ex["expect"].items():
            assert int(aw[key][0]) == val, (ex["name"], key)
