"""Pins for the window options of the oracle walk: late start inside a gap and per-job deadlines
(Section 4.4, item 2).  None of them retypes the walk: enumeration of every prefix, equivalence
with a plain pair on a transformed gap, closed forms and hand-computed examples."""
import numpy as np

from tests.helpers import gaps_from_lists, profiles_from_lists, random_small_profiles

U32MAX = 0xFFFFFFFF


def test_window_options_against_enumeration(oracle_mod):
    oracle = oracle_mod
    rng = np.random.default_rng(61)
    seen_late = seen_deadline = 0
    for trial in range(40):
        jobs = random_small_profiles(rng, 1, 14, p_safe=float(rng.uniform(0.1, 0.9)), dmax=9, mmax=20,
                                     allow_zero=(trial % 5 == 0))
        prof = profiles_from_lists(jobs)
        n = len(jobs[0][0])
        for _ in range(40):
            p = int(rng.integers(0, n + 1))
            ready, start = int(rng.integers(0, 40)), int(rng.integers(0, 40))
            T, C = int(rng.integers(0, 60)), int(rng.integers(1, 22))
            lo, hi = (0, U32MAX) if rng.random() < 0.7 else (int(rng.integers(0, 20)), int(rng.integers(0, 70)))
            late = bool(rng.integers(0, 2))
            deadline = U32MAX if rng.random() < 0.3 else int(rng.integers(0, 110))
            got = oracle.pair(prof, 0, p, ready, start, T, C, lo, hi, late, deadline)
            want = oracle.brute_pair(prof, 0, p, ready, start, T, C, lo, hi, late, deadline)
            assert got == want, (trial, p, ready, start, T, C, lo, hi, late, deadline)
            seen_late += got is not None and late and ready > start
            seen_deadline += got != oracle.pair(prof, 0, p, ready, start, T, C, lo, hi, late)
    assert seen_late > 20 and seen_deadline > 20      # both options actually decided something


def test_late_start_is_a_plain_pair_on_the_rest_of_the_window(oracle_mod):
    """A job that turns ready at time r inside [start, start + T] sees exactly the gap (r, T - (r - start));
    ready by the start: the option changes nothing; ready after the window has closed: decline."""
    oracle = oracle_mod
    rng = np.random.default_rng(62)
    jobs = random_small_profiles(rng, 6, 30, p_safe=0.4, dmax=9, mmax=20)
    prof = profiles_from_lists(jobs)
    for j in range(6):
        for _ in range(60):
            start, T, C = int(rng.integers(0, 50)), int(rng.integers(0, 90)), int(rng.integers(5, 22))
            ready = int(rng.integers(0, 160))
            got = oracle.pair(prof, j, 0, ready, start, T, C, late_start=True)
            if ready <= start:
                assert got == oracle.pair(prof, j, 0, ready, start, T, C)
            elif ready <= start + T:
                assert got == oracle.pair(prof, j, 0, ready, ready, T - (ready - start), C)
            else:
                assert got is None
    # no room left is still room for a subjob of zero duration (all bounds are inclusive)
    zero = profiles_from_lists([([0, 5], [1, 1], [1, 1])])
    assert oracle.pair(zero, 0, 0, 30, 10, 20, 5, late_start=True) == (1, 0, 0)
    assert oracle.pair(zero, 0, 0, 31, 10, 20, 5, late_start=True) is None
    assert oracle.pair(zero, 0, 0, 0, 10, 20, 5, deadline_ms=10) == (1, 0, 0)
    assert oracle.pair(zero, 0, 0, 0, 10, 20, 5, deadline_ms=9) is None
    # the largest representable times: start + T beyond 2^32 must not wrap
    one = profiles_from_lists([([7, 7], [1, 1], [1, 1])])
    assert oracle.pair(one, 0, 0, U32MAX - 3, U32MAX - 10, U32MAX, 5, late_start=True) == (2, 14, 14)
    assert oracle.pair(one, 0, 0, U32MAX - 3, U32MAX - 10, 14, 5, late_start=True) == (1, 7, 7)
    assert oracle.pair(one, 0, 0, U32MAX - 3, U32MAX - 10, 13, 5, late_start=True) is None


def test_deadline_is_a_cap_on_the_window(oracle_mod):
    """With begin = start: a deadline acts exactly like the window min(T, deadline - start); one that has
    passed declines; 2^32 - 1 is no deadline.  Closed form on a constant profile."""
    oracle = oracle_mod
    rng = np.random.default_rng(63)
    jobs = random_small_profiles(rng, 5, 30, p_safe=0.5, dmax=9, mmax=20)
    prof = profiles_from_lists(jobs)
    for j in range(5):
        for _ in range(60):
            start, T, C = int(rng.integers(0, 50)), int(rng.integers(0, 90)), int(rng.integers(5, 22))
            deadline = int(rng.integers(0, 150))
            got = oracle.pair(prof, j, 0, 0, start, T, C, deadline_ms=deadline)
            if deadline < start:
                assert got is None
            else:
                assert got == oracle.pair(prof, j, 0, 0, start, min(T, deadline - start), C)
            assert oracle.pair(prof, j, 0, 0, start, T, C, deadline_ms=U32MAX) == oracle.pair(prof, j, 0, 0, start, T, C)
    const = profiles_from_lists([([5] * 40, [3] * 40, [1] * 40)])
    for start in (0, 12):
        for ready in (0, 12, 20):
            for T in (4, 23, 100, 1000):
                for deadline in (3, 31, 64, 500, U32MAX):
                    begin = max(start, ready)
                    room = min(start + T, deadline) - begin
                    k = min(room // 5, 40) if room >= 0 else 0
                    got = oracle.pair(const, 0, 0, ready, start, T, 9, 0, U32MAX, True, deadline)
                    assert got == ((k, 5 * k, 15 * k) if k > 0 else None), (start, ready, T, deadline)


def test_window_options_in_select_and_commit(oracle_mod):
    """Hand example.  Gap: start 10, T 20, so [10, 30].  Job 0 (ready 0): steps of 8 ms, memory 10, all safe.
    Job 1 (ready 16): steps of 6 ms, memory 40, all safe.  Efficiency policy.
    plain: job 1 is not ready -> job 0 takes 2 steps (16 ms, work 160).
    late start: job 1 begins at 16, 14 ms left -> 2 steps (12 ms, work 480) and wins; its ready time
    becomes 16 + 12 = 28.  Deadline 25 for job 1: 9 ms left -> 1 step (work 240), still the winner.
    Deadline 21: 5 ms left -> nothing fits, job 0 wins again.  Deadline 17 for job 0 too: 7 ms -> nobody."""
    oracle = oracle_mod
    prof = profiles_from_lists([([8] * 5, [10] * 5, [1] * 5), ([6] * 5, [40] * 5, [1] * 5)], ready=[0, 16])
    gaps = gaps_from_lists([(0, 10, 20, 100)])
    z = np.zeros(2, np.uint32)

    def sel(**kw):
        a = oracle.select(prof, z, prof.ready_ms, gaps, 0, **kw)
        return int(a["job"][0]), int(a["end_step"][0]), int(a["dur_ms"][0]), int(a["score"][0])

    assert sel() == (0, 2, 16, 160)
    assert sel(late_start=True) == (1, 2, 12, 480)
    assert sel(late_start=True, deadline_ms=np.array([U32MAX, 25], np.uint32)) == (1, 1, 6, 240)
    assert sel(late_start=True, deadline_ms=np.array([U32MAX, 21], np.uint32)) == (0, 2, 16, 160)
    assert sel(late_start=True, deadline_ms=np.array([17, 21], np.uint32)) == (U32MAX, 0, 0, 0)
    assert sel(deadline_ms=np.array([18, U32MAX], np.uint32)) == (0, 1, 8, 80)

    aw = oracle.select(prof, z, prof.ready_ms, gaps, 0, late_start=True)
    progress, ready = z.copy(), prof.ready_ms.copy()
    assert oracle.commit(progress, ready, gaps, aw, late_start=True) == 1
    assert progress.tolist() == [0, 2] and ready.tolist() == [0, 28]
    # a job that was ready before the gap opened still counts from the gap's start
    aw = oracle.select(prof, z, prof.ready_ms, gaps, 0)
    progress, ready = z.copy(), prof.ready_ms.copy()
    assert oracle.commit(progress, ready, gaps, aw, late_start=True) == 1
    assert progress.tolist() == [2, 0] and ready.tolist() == [26, 16]
