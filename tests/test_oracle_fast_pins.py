"""Pins for the second CPU oracle (oracle/fast_oracle.c: prefix arrays + binary search).

It carries the full-size trajectories stored under tests/golden/, so it is pinned here against things it does
not share code with: the step-by-step walk (oracle/sja_oracle.c), the exhaustive enumerator (oracle/brute.py),
a closed form, and the walk's commit rule.  A planted mistake (a bound off by one, `<` for `<=`, a running
maximum that is not rebuilt when the progress point moves, a tie that goes to the higher job id, a commit that
prefers the lower end step) fails at least one of them.
"""
import numpy as np
import pytest

from paper_2509_19086_b200 import workloads as wl
from tests.helpers import gaps_from_lists, profiles_from_lists, random_small_profiles

U32MAX = 0xFFFFFFFF


@pytest.fixture(scope="module")
def fast_mod(oracle_mod):
    from oracle import fast
    fast.build()
    return fast


def _same(a, b, ctx=None):
    for f in ("job", "end_step", "dur_ms", "granted", "score"):
        bad = np.nonzero(a[f] != b[f])[0]
        assert bad.size == 0, (ctx, f, bad[:5], a[bad[:5]], b[bad[:5]])


def _rounds_against_walk(oracle, fast, spec, policies, n_rounds, threads=4):
    prof = wl.make_profiles(spec, threads=threads)
    with fast.FastOracle(prof) as fo:
        for policy in policies:
            p_w = np.zeros(prof.n_jobs, np.uint32)
            r_w = prof.ready_ms.copy()
            p_f, r_f = p_w.copy(), r_w.copy()
            total = 0
            for r in range(n_rounds):
                gaps = wl.make_gaps(spec, r)
                want = oracle.select(prof, p_w, r_w, gaps, policy)
                got = fo.select(p_f, r_f, gaps, policy)
                _same(got, want, (spec.name, policy, r, "select"))
                n_w = oracle.commit(p_w, r_w, gaps, want)
                n_f = fast.commit(p_f, r_f, gaps, got)
                assert n_w == n_f
                _same(got, want, (spec.name, policy, r, "commit"))
                assert np.array_equal(p_w, p_f) and np.array_equal(r_w, r_f)
                total += n_w
            assert total > 0


def test_fast_equals_walk_cfg0_cfg1(oracle_mod, fast_mod):
    """The two small published configurations in full, every policy their attributes allow."""
    _rounds_against_walk(oracle_mod, fast_mod, wl.SPECS[0], (0, 3), 3, threads=1)
    _rounds_against_walk(oracle_mod, fast_mod, wl.SPECS[1], (0, 3), 2)


@pytest.mark.parametrize("spec,policies,rounds", [
    (wl.scaled(wl.SPECS[2], n_jobs=1500, fixed_len=700, n_gaps=160), (0, 1, 3), 4),
    (wl.scaled(wl.SPECS[3], n_jobs=2500, zipf_max=3000, n_gaps=256), (0, 2, 3), 4),
    (wl.scaled(wl.SPECS[4], n_jobs=600, fixed_len=300, n_gaps=200, n_rounds=40), (0,), 40),
])
def test_fast_equals_walk_scaled_configs_over_committed_rounds(oracle_mod, fast_mod, spec, policies, rounds):
    """Scaled versions of the three large configurations; progress points move, jobs finish, the running
    maximum has to be rebuilt from every new progress point."""
    _rounds_against_walk(oracle_mod, fast_mod, spec, policies, rounds)


def test_fast_equals_enumeration_on_tiny_inputs(oracle_mod, fast_mod):
    """Random tiny rounds incl. zero-length jobs, zero durations and memory, progress anywhere in the job:
    every policy against the exhaustive enumerator (not against the walk)."""
    rng = np.random.default_rng(303)
    for trial in range(60):
        jobs = random_small_profiles(rng, int(rng.integers(1, 9)), 12, p_safe=float(rng.uniform(0.05, 0.9)),
                                     allow_zero=(trial % 3 == 0))
        J = len(jobs)
        prof = profiles_from_lists(jobs, ready=rng.integers(0, 6, J), wait=rng.integers(0, 5000, J),
                                   prio=rng.integers(0, 3, J))
        lens = np.diff(prof.off).astype(np.int64)
        progress = np.array([rng.integers(0, n + 1) for n in lens], dtype=np.uint32)
        gaps = gaps_from_lists([(int(rng.integers(0, 7)), int(rng.integers(0, 8)), int(rng.integers(0, 40)),
                                 int(rng.integers(0, 22))) for _ in range(6)])
        with fast_mod.FastOracle(prof) as fo:
            for policy in (0, 1, 2, 3):
                aw = fo.select(progress, prof.ready_ms, gaps, policy)
                ref = oracle_mod.brute_select(prof, progress, prof.ready_ms, gaps, policy)
                for g in range(len(gaps)):
                    for key in ("job", "end_step", "dur_ms", "score"):
                        assert int(aw[key][g]) == ref[g][key], (trial, policy, g, key)


def test_fast_all_safe_masks_exhaustive(oracle_mod, fast_mod):
    """Every safe mask of a 7-step job over a grid of (p, T, C): fast oracle == enumeration."""
    d = [3, 1, 4, 1, 5, 9, 2]
    m = [5, 8, 2, 9, 3, 7, 6]
    grid = [(T, C) for T in (0, 3, 8, 13, 25, 100) for C in (1, 5, 8, 9)]
    gaps = gaps_from_lists([(0, 0, T, C) for (T, C) in grid])
    for mask in range(1 << 7):
        s = [(mask >> i) & 1 for i in range(7)]
        prof = profiles_from_lists([(d, m, s)])
        with fast_mod.FastOracle(prof) as fo:
            for p in (0, 2, 6, 7):
                aw = fo.select(np.array([p], np.uint32), prof.ready_ms, gaps, 0)
                for g, (T, C) in enumerate(grid):
                    want = oracle_mod.brute_pair(prof, 0, p, 0, 0, T, C)
                    if want is None:
                        assert aw["job"][g] == U32MAX, (mask, p, T, C)
                    else:
                        assert (int(aw["end_step"][g]), int(aw["dur_ms"][g]), int(aw["score"][g])) == want, (mask, p, T, C)


@pytest.mark.parametrize("a,b,q,n,T,wait", [(7, 11, 4, 100, 365, 0), (13, 5, 10, 95, 5000, 123456),
                                            (50, 81920, 3, 4096, 5000, 3600000)])
def test_fast_constant_profile_closed_form(fast_mod, a, b, q, n, T, wait):
    """d = a, m = b <= C, a boundary every q-th step: k = q * floor(floor(T/a)/q), capped at the job's end."""
    s = [1 if (i + 1) % q == 0 else 0 for i in range(n)]
    prof = profiles_from_lists([([a] * n, [b] * n, s)], wait=[wait])
    steps = min(T // a, n)
    k = n if steps == n else q * (steps // q)
    with fast_mod.FastOracle(prof) as fo:
        aw = fo.select(np.zeros(1, np.uint32), prof.ready_ms, gaps_from_lists([(0, 0, T, b)]), 1)
    if k == 0:
        assert aw["job"][0] == U32MAX
    else:
        assert (int(aw["end_step"][0]), int(aw["dur_ms"][0])) == (k, k * a)
        assert int(aw["score"][0]) == k * a * b * (1 + wait // 1000)


def test_fast_eligibility_ties_and_inclusive_bounds(fast_mod):
    """Hand-computed: bounds are inclusive, a gap that opens before the job is ready is declined, a finished
    job declines, equal scores go to the lower job id, the SLA class outranks the work."""
    job = ([10, 10, 10], [4, 6, 8], [1, 1, 1])
    prof = profiles_from_lists([job, job, job, ([5], [1], [1])], ready=[0, 0, 7, 0], prio=[0, 0, 0, 2])
    gaps = gaps_from_lists([(0, 5, 20, 6),     # T = 20 admits two steps exactly, C = 6 admits m = 6
                            (0, 5, 19, 6),     # one step only
                            (0, 5, 30, 5),     # the second step's memory is above the capacity
                            (0, 6, 30, 8),     # job 2 (ready 7) still declines
                            (0, 7, 30, 8)])    # now it may bid; jobs 0 and 1 are finished below
    progress = np.array([0, 0, 0, 0], np.uint32)
    with fast_mod.FastOracle(prof) as fo:
        aw = fo.select(progress, prof.ready_ms, gaps, 0)
        assert aw["job"].tolist() == [0, 0, 0, 0, 0]
        assert aw["end_step"].tolist() == [2, 1, 1, 3, 3]
        assert aw["dur_ms"].tolist() == [20, 10, 10, 30, 30]
        assert aw["score"].tolist() == [100, 40, 40, 180, 180]
        sla = fo.select(progress, prof.ready_ms, gaps, 2)
        assert sla["job"].tolist() == [3, 3, 3, 3, 3] and sla["score"].tolist() == [5] * 5
        done = np.array([3, 3, 0, 1], np.uint32)
        aw = fo.select(done, prof.ready_ms, gaps, 0)
        assert aw["job"].tolist() == [U32MAX, U32MAX, U32MAX, U32MAX, 2]


def test_fast_commit_rule_against_walk_commit(oracle_mod, fast_mod):
    """R6 on hand-made award lists with multi-winners and equal end steps: the two commits agree, and the
    accepted gap is the one with the largest end step, then the lowest gap id."""
    rng = np.random.default_rng(11)
    for trial in range(40):
        J, G = int(rng.integers(1, 7)), int(rng.integers(1, 14))
        gaps = gaps_from_lists([(0, int(rng.integers(0, 50)), 100, 100) for _ in range(G)])
        aw = np.zeros(G, dtype=oracle_mod.AWARD_DTYPE)
        aw["job"] = rng.integers(0, J + 1, G)
        aw["job"][aw["job"] == J] = U32MAX
        aw["end_step"] = np.where(aw["job"] == U32MAX, 0, rng.integers(1, 4, G))
        aw["dur_ms"] = np.where(aw["job"] == U32MAX, 0, rng.integers(0, 30, G))
        a1, a2 = aw.copy(), aw.copy()
        p1, r1 = np.zeros(J, np.uint32), np.zeros(J, np.uint32)
        p2, r2 = p1.copy(), r1.copy()
        assert oracle_mod.commit(p1, r1, gaps, a1) == fast_mod.commit(p2, r2, gaps, a2)
        assert a1.tobytes() == a2.tobytes() and np.array_equal(p1, p2) and np.array_equal(r1, r2)
        for j in range(J):
            mine = [g for g in range(G) if aw["job"][g] == j]
            if not mine:
                continue
            best = max(mine, key=lambda g: (int(aw["end_step"][g]), -g))
            assert [g for g in mine if a2["granted"][g]] == [best]
            assert p2[j] == aw["end_step"][best] and r2[j] == gaps["start_ms"][best] + aw["dur_ms"][best]
