"""Pins for the optional subjob duration thresholds (tau_min, tau_max) of the oracle walk."""
import numpy as np

from tests.helpers import gaps_from_lists, profiles_from_lists, random_small_profiles

U32MAX = 0xFFFFFFFF


def test_thresholds_against_enumeration(oracle_mod):
    oracle = oracle_mod
    rng = np.random.default_rng(31)
    for trial in range(40):
        jobs = random_small_profiles(rng, 1, 14, p_safe=float(rng.uniform(0.1, 0.9)), dmax=9, mmax=20)
        prof = profiles_from_lists(jobs)
        n = len(jobs[0][0])
        for _ in range(25):
            p = int(rng.integers(0, n + 1))
            T, C = int(rng.integers(0, 60)), int(rng.integers(1, 22))
            lo, hi = int(rng.integers(0, 30)), int(rng.integers(0, 70))
            got = oracle.pair(prof, 0, p, 0, 0, T, C, lo, hi)
            want = oracle.brute_pair(prof, 0, p, 0, 0, T, C, lo, hi)
            assert got == want, (trial, p, T, C, lo, hi)


def test_thresholds_closed_form_and_special_cases(oracle_mod):
    """d = 5 everywhere, every step safe, ample capacity: k = floor(min(T, tau_max) / 5), declined
    when that is shorter than tau_min; tau_max acts exactly like a shorter window."""
    oracle = oracle_mod
    prof = profiles_from_lists([([5] * 40, [3] * 40, [1] * 40)])
    for T in (0, 4, 5, 23, 100, 199, 200, 1000):
        for lo in (0, 5, 21, 60):
            for hi in (0, 7, 50, U32MAX):
                k = min(min(T, hi) // 5, 40)
                got = oracle.pair(prof, 0, 0, 0, 0, T, 9, lo, hi)
                if k == 0 or 5 * k < lo:
                    assert got is None, (T, lo, hi)
                else:
                    assert got == (k, 5 * k, 15 * k), (T, lo, hi)
                assert got == oracle.pair(prof, 0, 0, 0, 0, min(T, hi), 9, lo, U32MAX)
    # defaults switch the thresholds off
    assert oracle.pair(prof, 0, 0, 0, 0, 23, 9) == oracle.pair(prof, 0, 0, 0, 0, 23, 9, 0, U32MAX) == (4, 20, 60)


def test_thresholds_in_select(oracle_mod):
    """Hand example: job 0 has the larger work but its subjob is shorter than tau_min."""
    oracle = oracle_mod
    prof = profiles_from_lists([([4, 4], [50, 50], [1, 0]), ([3, 3, 3], [10, 10, 10], [1, 1, 1])])
    gaps = gaps_from_lists([(0, 0, 7, 100)])
    z = np.zeros(2, np.uint32)
    plain = oracle.select(prof, z, prof.ready_ms, gaps, 0)
    assert (int(plain["job"][0]), int(plain["dur_ms"][0]), int(plain["score"][0])) == (0, 4, 200)
    bounded = oracle.select(prof, z, prof.ready_ms, gaps, 0, 5, U32MAX)
    assert (int(bounded["job"][0]), int(bounded["end_step"][0]), int(bounded["dur_ms"][0])) == (1, 2, 6)
    capped = oracle.select(prof, z, prof.ready_ms, gaps, 0, 0, 3)
    assert (int(capped["job"][0]), int(capped["end_step"][0]), int(capped["score"][0])) == (1, 1, 30)
    none = oracle.select(prof, z, prof.ready_ms, gaps, 0, 8, U32MAX)
    assert int(none["job"][0]) == U32MAX
