"""Pins for the power envelope of the oracle walk (Section 4.4, item 1: offers carry a power cap, admission
keeps the maximum of the subjob's predicted power trace below it).  Enumeration of every prefix, the
symmetry with the memory channel, a closed form and a hand-computed select."""
import numpy as np

from tests.helpers import gaps_from_lists, profiles_from_lists, random_small_profiles

U32MAX = 0xFFFFFFFF


def test_power_cap_against_enumeration(oracle_mod):
    oracle = oracle_mod
    rng = np.random.default_rng(71)
    decided = 0
    for trial in range(40):
        jobs = random_small_profiles(rng, 3, 14, p_safe=float(rng.uniform(0.1, 0.9)), dmax=9, mmax=20,
                                     allow_zero=(trial % 5 == 0))
        prof = profiles_from_lists(jobs)
        power = rng.integers(0, 30, prof.n_steps).astype(np.uint32)
        for j in range(3):
            n = len(jobs[j][0])
            for _ in range(15):
                p = int(rng.integers(0, n + 1))
                T, C = int(rng.integers(0, 60)), int(rng.integers(1, 22))
                cap = U32MAX if rng.random() < 0.2 else int(rng.integers(0, 32))
                late, ready, start = bool(rng.integers(0, 2)), int(rng.integers(0, 12)), int(rng.integers(0, 12))
                got = oracle.pair(prof, j, p, ready, start, T, C, late_start=late, power_W=power, power_cap_W=cap)
                want = oracle.brute_pair(prof, j, p, ready, start, T, C, late_start=late, power_W=power, power_cap_W=cap)
                assert got == want, (trial, j, p, T, C, cap)
                decided += got != oracle.pair(prof, j, p, ready, start, T, C, late_start=late)
    assert decided > 30        # the cap actually changed answers


def test_power_channel_mirrors_the_memory_channel(oracle_mod):
    """The two envelopes enter the test the same way: with the arrays swapped and the bounds swapped the chosen
    subjob (k, dur) is the same; without a cap, or without a trace, nothing changes; a cap below the first
    step's power declines."""
    oracle = oracle_mod
    rng = np.random.default_rng(72)
    jobs = random_small_profiles(rng, 4, 30, p_safe=0.4, dmax=9, mmax=25)
    prof = profiles_from_lists(jobs)
    power = rng.integers(1, 26, prof.n_steps).astype(np.uint32)
    swapped = profiles_from_lists([(d, power[int(prof.off[j]):int(prof.off[j + 1])].tolist(), s)
                                   for j, (d, m, s) in enumerate(jobs)])
    for j in range(4):
        for _ in range(60):
            T, C, cap = int(rng.integers(0, 120)), int(rng.integers(1, 27)), int(rng.integers(1, 27))
            a = oracle.pair(prof, j, 0, 0, 0, T, C, power_W=power, power_cap_W=cap)
            b = oracle.pair(swapped, j, 0, 0, 0, T, cap, power_W=prof.mem_MiB, power_cap_W=C)
            assert (a is None) == (b is None) and (a is None or a[:2] == b[:2])
            plain = oracle.pair(prof, j, 0, 0, 0, T, C)
            assert oracle.pair(prof, j, 0, 0, 0, T, C, power_W=power, power_cap_W=U32MAX) == plain
            assert oracle.pair(prof, j, 0, 0, 0, T, C, power_W=None, power_cap_W=cap) == plain
            first = int(power[int(prof.off[j])])
            if first > 0:
                assert oracle.pair(prof, j, 0, 0, 0, T, C, power_W=power, power_cap_W=first - 1) is None


def test_power_cap_closed_form_and_select(oracle_mod):
    """Power rises by 10 W per step (10, 20, 30, ...), d = 5, every step safe, ample memory: the subjob ends
    where the power would exceed the cap or the window ends, k = min(floor(cap / 10), floor(T / 5)).
    Hand example: two gaps of equal window, caps 25 W and 100 W; job 0 (work 50 per step, power 30 W flat) is
    shut out of the first gap, job 1 (work 5 per step, power 20 W flat) takes it."""
    oracle = oracle_mod
    prof = profiles_from_lists([([5] * 20, [3] * 20, [1] * 20)])
    power = (10 * np.arange(1, 21)).astype(np.uint32)
    for T in (4, 23, 60, 1000):
        for cap in (0, 9, 10, 35, 200, 1000):
            k = min(cap // 10, T // 5, 20)
            got = oracle.pair(prof, 0, 0, 0, 0, T, 9, power_W=power, power_cap_W=cap)
            assert got == ((k, 5 * k, 15 * k) if k else None), (T, cap)
    two = profiles_from_lists([([4] * 5, [10] * 5, [1] * 5), ([4] * 5, [1] * 5, [1] * 5)])
    pw = np.array([30] * 5 + [20] * 5, np.uint32)
    gaps = gaps_from_lists([(0, 0, 9, 100), (0, 0, 9, 100)])
    z = np.zeros(2, np.uint32)
    aw = oracle.select(two, z, two.ready_ms, gaps, 0, power_W=pw, power_cap_W=np.array([25, 100], np.uint32))
    assert aw["job"].tolist() == [1, 0] and aw["end_step"].tolist() == [2, 2] and aw["score"].tolist() == [8, 80]
    none = oracle.select(two, z, two.ready_ms, gaps, 0, power_W=pw, power_cap_W=np.array([19, 19], np.uint32))
    assert (none["job"] == U32MAX).all()
