"""Seeded random rounds of widely varying shape (job counts from 1 to thousands, empty jobs, zero durations
and zero memory, no / all boundaries, one or many capacities, window lengths from 0 to 2^32-1, duration
thresholds): the three select kernels agree byte for byte and match the oracle wherever it is quick; a second
family mixes late start, deadlines, power caps, all four policies, commits and re-profiling."""
import numpy as np
import pytest

from paper_2509_19086_b200 import workloads as wl

pytestmark = pytest.mark.gpu
U = 0xFFFFFFFF
FIELDS = ("job", "end_step", "dur_ms", "score")


def _random_profiles(rng, J, maxlen, allow_empty, mmax):
    lens = rng.integers(0 if allow_empty else 1, maxlen + 1, J)
    N = int(lens.sum())
    off = np.zeros(J + 1, np.uint64)
    off[1:] = np.cumsum(lens)
    d = rng.integers(0 if rng.random() < 0.3 else 1, int(rng.choice([1, 9, 50, 1000])) + 1, N).astype(np.uint32)
    m = rng.integers(0 if rng.random() < 0.3 else 1, mmax + 1, N).astype(np.uint32)
    safe = (rng.random(N) < float(rng.choice([0.0, 0.02, 0.1, 0.5, 1.0]))).astype(np.uint8)
    bits = wl.pack_safe_bits(safe) if N else np.zeros(0, np.uint32)
    ready = rng.integers(0, int(rng.choice([1, 10, 1000, 100000])), J).astype(np.uint32)
    wait = rng.integers(0, 3600001, J).astype(np.uint32)
    prio = rng.integers(0, 3, J).astype(np.uint8)
    return wl.Profiles(off, d, m, bits, ready, wait, prio), lens


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_random_rounds_all_kernels(oracle_mod, seed):
    from paper_2509_19086_b200 import binding
    rng = np.random.default_rng(seed)
    with_oracle = 0
    with binding.Sja() as ctx:
        for case in range(120):
            J = int(rng.choice([1, 7, 33, 100, 513, 2000, 5000]))
            maxlen = int(rng.choice([1, 5, 40, 300, 2000]))
            mmax = int(rng.choice([1, 20, 100, 81920]))
            prof, lens = _random_profiles(rng, J, maxlen, rng.random() < 0.2, mmax)
            progress = (lens * rng.random(J) * (rng.random() < 0.5)).astype(np.uint32)
            G = int(rng.choice([1, 31, 32, 33, 100, 700, 3000]))
            ncls = int(rng.choice([1, 2, 4, 30]))
            Tmax = int(rng.choice([0, 10, 500, 5000, 200000]))
            gaps = np.zeros(G, wl.GAP_DTYPE)
            gaps["slice"] = rng.integers(0, 7, G)
            gaps["C_MiB"] = rng.integers(0, mmax + 2, ncls)[rng.integers(0, ncls, G)]
            gaps["T_ms"] = rng.integers(0, Tmax + 1, G) if rng.random() < 0.8 else int(rng.integers(0, Tmax + 1))
            gaps["start_ms"] = rng.integers(0, int(rng.choice([1, 12, 2000, 200000])), G)
            if rng.random() < 0.1:
                gaps["T_ms"][: G // 2] = U
            policy = int(rng.integers(0, 4))
            lo, hi = (0, U) if rng.random() < 0.7 else (int(rng.integers(0, 50)), int(rng.integers(50, 3000)))
            ctx.load_profiles(prof.off, prof.dur_ms, prof.mem_MiB, prof.safe_bits, prof.ready_ms,
                              progress=progress, wait_ms=prof.wait_ms, prio=prof.prio)
            ctx.set_duration_bounds(lo, hi)
            ctx.advertise(gaps)
            tile = ctx.select(policy, flags=binding.FLAG_FORCE_TILE, out="host")
            what = (seed, case, J, maxlen, G, ncls, Tmax, policy, lo, hi)
            assert ctx.select(policy, flags=binding.FLAG_FORCE_MERGE, out="host").tobytes() == tile.tobytes(), what
            assert ctx.select(policy, flags=binding.FLAG_FORCE_SEARCH, out="host").tobytes() == tile.tobytes(), what
            if J * G * max(1, maxlen) < 2e7:
                want = oracle_mod.select(prof, progress, prof.ready_ms, gaps, policy, lo, hi)
                for f in FIELDS:
                    assert np.array_equal(tile[f], want[f]), what + (f,)
                with_oracle += 1
    assert with_oracle > 60


@pytest.mark.parametrize("seed", [21, 22])
def test_random_rounds_with_options(oracle_mod, seed):
    from paper_2509_19086_b200 import binding
    rng = np.random.default_rng(seed)
    with binding.Sja() as ctx:
        for case in range(80):
            J = int(rng.choice([1, 7, 33, 100, 513, 1500]))
            maxlen = int(rng.choice([1, 5, 40, 300]))
            mmax = int(rng.choice([20, 100, 81920]))
            prof, lens = _random_profiles(rng, J, maxlen, False, mmax)
            prof.mem_MiB[:] = np.maximum(prof.mem_MiB, 1)
            prof.ready_ms[:] = rng.integers(0, int(rng.choice([10, 1000, 6000])), J)
            off = prof.off.astype(np.int64)
            progress = np.zeros(J, np.uint32)
            power = rng.integers(0, 500, prof.n_steps).astype(np.uint32)
            deadline = rng.integers(0, 12000, J).astype(np.uint32)
            deadline[rng.random(J) < 0.4] = U
            late, use_dl, use_pw = bool(rng.integers(0, 2)), rng.random() < 0.6, rng.random() < 0.6
            policy = int(rng.integers(0, 4))
            ctx.load_profiles(prof.off, prof.dur_ms, prof.mem_MiB, prof.safe_bits, prof.ready_ms,
                              wait_ms=prof.wait_ms, prio=prof.prio)
            ctx.set_duration_bounds(0, U)
            if use_pw:
                ctx.load_power(prof.off, power)
            ctx.set_window_options(late, deadline if use_dl else None)
            for rnd in range(3):
                what = (seed, case, rnd, J, maxlen, late, use_dl, use_pw, policy)
                G = int(rng.choice([1, 33, 200, 900]))
                gaps = np.zeros(G, wl.GAP_DTYPE)
                gaps["C_MiB"] = rng.choice(rng.integers(1, mmax + 2, 3), G)
                gaps["T_ms"] = rng.integers(0, int(rng.choice([500, 5000])) + 1, G)
                gaps["start_ms"] = rng.integers(0, 3000, G) + 1000 * rnd
                caps = rng.integers(0, 520, G).astype(np.uint32)
                caps[rng.random(G) < 0.2] = U
                ctx.advertise(gaps)
                if use_pw:
                    ctx.advertise_power_caps(caps)
                got = ctx.select(policy, out="host")
                want = oracle_mod.select(prof, progress, prof.ready_ms, gaps, policy, late_start=late,
                                         deadline_ms=deadline if use_dl else None,
                                         power_W=power if use_pw else None, power_cap_W=caps if use_pw else None)
                for f in FIELDS:
                    assert np.array_equal(got[f], want[f]), what + (f,)
                assert ctx.commit() == oracle_mod.commit(progress, prof.ready_ms, gaps, want, late_start=late), what
                p, r = ctx.get_state()
                assert np.array_equal(p, progress) and np.array_equal(r, prof.ready_ms), what
                for j in rng.integers(0, J, 3):                   # re-profile a few jobs between rounds
                    a, b = int(off[j]) + int(progress[j]), int(off[j + 1])
                    nd = rng.integers(1, 60, b - a).astype(np.uint32)
                    nm = rng.integers(1, mmax + 1, b - a).astype(np.uint32)
                    ctx.update_profile(int(j), nd, nm)
                    prof.dur_ms[a:b] = nd
                    prof.mem_MiB[a:b] = nm
