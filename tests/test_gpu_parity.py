"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle, element by element.

All quantities are integers, so the bar is bit-exact equality.
"""
import numpy as np
import pytest

from paper_2509_19086_b200 import workloads as wl
from tests.helpers import gaps_from_lists, profiles_from_lists, random_small_profiles

pytestmark = pytest.mark.gpu

U32MAX = 0xFFFFFFFF


@pytest.fixture(scope="module")
def sja_mod():
    from paper_2509_19086_b200 import binding
    return binding


def _load(ctx, prof, progress=None):
    ctx.load_profiles(prof.off, prof.dur_ms, prof.mem_MiB, prof.safe_bits, prof.ready_ms,
                      progress=progress, wait_ms=prof.wait_ms, prio=prof.prio)


def _assert_awards_equal(got, want, fields=("job", "end_step", "dur_ms", "score")):
    for f in fields:
        bad = np.nonzero(got[f] != want[f])[0]
        assert bad.size == 0, (f, bad[:5], got[bad[:5]], want[bad[:5]])


def _check_scan(oracle, ctx, prof, progress):
    sc = ctx.get_scan()
    J = prof.n_jobs
    for j in range(J):
        rows = oracle.boundary_table(prof, j, int(progress[j]))
        b0, b1 = int(sc["boff"][j]), int(sc["boff"][j + 1])
        assert b1 - b0 == len(rows), (j, b1 - b0, len(rows))
        if not rows:
            continue
        exp = np.array(rows, dtype=np.uint64)
        assert np.array_equal(sc["k"][b0:b1], exp[:, 0]), j
        assert np.array_equal(sc["D"][b0:b1], exp[:, 1]), j
        assert np.array_equal(sc["M"][b0:b1], exp[:, 2]), j
        assert np.array_equal(sc["S"][b0:b1], exp[:, 3]), j
        assert np.array_equal(sc["W"][b0:b1], exp[:, 4]), j


# ------------------------------------------------------------------ scan (a1)
def test_scan_matches_oracle_ragged_lengths(sja_mod, oracle_mod):
    """Job lengths around every tile edge of the scan (16-step lanes, 512-step warp blocks)."""
    rng = np.random.default_rng(101)
    lens = [1, 2, 15, 16, 17, 31, 32, 33, 100, 511, 512, 513, 1023, 1024, 1025, 1500, 2047, 4096, 5000, 3, 0, 7]
    jobs = []
    for n in lens:
        d = rng.integers(0, 60, n).tolist()
        m = rng.integers(0, 90000, n).tolist()
        s = (rng.random(n) < 0.12).astype(int).tolist()
        jobs.append((d, m, s))
    prof = profiles_from_lists(jobs, ready=rng.integers(0, 100, len(jobs)))
    progress = np.array([int(rng.integers(0, n + 1)) for n in lens], dtype=np.uint32)
    progress[:6] = 0
    with sja_mod.Sja() as ctx:
        _load(ctx, prof, progress)
        _check_scan(oracle_mod, ctx, prof, progress)
        # device-resident inputs take the same path without the staging copy
        import torch
        dev = {k: torch.from_numpy(np.ascontiguousarray(v).view(np.int64 if v.dtype == np.uint64 else np.int32)).cuda()
               for k, v in dict(off=prof.off, d=prof.dur_ms, m=prof.mem_MiB, s=prof.safe_bits,
                                r=prof.ready_ms, p=progress).items()}
        ctx.load_profiles(dev["off"], dev["d"], dev["m"], dev["s"], dev["r"], progress=dev["p"])
        _check_scan(oracle_mod, ctx, prof, progress)


def test_scan_matches_oracle_dense_boundaries_and_large_values(sja_mod, oracle_mod):
    """Every step safe (512 rows per warp block) and 32-bit-wide values (64-bit work sums)."""
    rng = np.random.default_rng(102)
    jobs = []
    for n in (700, 40, 1300):
        jobs.append((rng.integers(0, 2**20, n).tolist(), rng.integers(0, 2**32 - 1, n).tolist(), [1] * n))
    jobs.append(([5] * 600, [7] * 600, [0] * 600))          # no interior boundary at all
    prof = profiles_from_lists(jobs)
    progress = np.zeros(len(jobs), np.uint32)
    with sja_mod.Sja() as ctx:
        _load(ctx, prof, progress)
        _check_scan(oracle_mod, ctx, prof, progress)


def test_scan_matches_oracle_boundary_densities_around_the_row_buffer(sja_mod, oracle_mod):
    """Boundary densities on both sides of what the warp's row buffer holds per 512-step block (about 300 rows):
    blocks that leave through the buffer (in either of its two positions: even and odd blocks), blocks that
    overflow it, and jobs that switch between the two from block to block."""
    rng = np.random.default_rng(103)
    jobs = []
    for dens in (0.3, 0.36, 0.45, 0.52, 0.56, 0.58, 0.59, 0.6, 0.62, 0.7, 0.9):
        for n in (3000, 1111):
            d = rng.integers(0, 60, n).tolist()
            m = rng.integers(0, 90000, n).tolist()
            s = (rng.random(n) < dens).astype(int).tolist()
            jobs.append((d, m, s))
    # density that changes along the job: sparse, dense, sparse ... in 512-step stretches that do not align with the blocks
    n = 6000
    dens = np.where((np.arange(n) // 700) % 2 == 0, 0.05, 0.75)
    jobs.append((rng.integers(1, 50, n).tolist(), rng.integers(1, 81920, n).tolist(), (rng.random(n) < dens).astype(int).tolist()))
    prof = profiles_from_lists(jobs, ready=rng.integers(0, 100, len(jobs)))
    lens = np.diff(prof.off).astype(np.int64)
    progress = (lens * rng.random(len(jobs)) * (rng.random(len(jobs)) < 0.5)).astype(np.uint32)
    with sja_mod.Sja() as ctx:
        _load(ctx, prof, progress)
        _check_scan(oracle_mod, ctx, prof, progress)


def test_scan_long_jobs_counted_by_the_whole_cta(sja_mod, oracle_mod):
    """Jobs of more than 8192 steps (256 safe words) are counted by the whole counting CTA, two at a time, and jobs of
    more than 65 536 steps take several trips; an even and an odd number of them per block of 64 jobs, some entered
    at a progress point that is not word-aligned, between short jobs."""
    rng = np.random.default_rng(104)
    lens = [int(x) for x in rng.integers(1, 600, 140)]
    for pos, n in ((3, 150_000), (4, 70_000), (17, 9_000), (40, 8_225), (41, 66_000), (63, 12_345),   # six in block 0
                   (64, 65_536 + 31), (90, 8_193), (127, 30_000),                                     # three in block 1
                   (139, 100_001)):                                                                   # one in block 2
        lens[pos] = n
    jobs = []
    for n in lens:
        d = rng.integers(1, 50, n).astype(np.uint32)
        m = rng.integers(1, 81920, n).astype(np.uint32)
        s = (rng.random(n) < 0.1).astype(np.uint8)
        jobs.append((d, m, s))
    off = np.zeros(len(jobs) + 1, np.uint64)
    off[1:] = np.cumsum(lens)
    prof = wl.Profiles(off, np.concatenate([j[0] for j in jobs]), np.concatenate([j[1] for j in jobs]),
                       wl.pack_safe_bits(np.concatenate([j[2] for j in jobs])),
                       rng.integers(0, 100, len(jobs)).astype(np.uint32), None, None)
    progress = np.zeros(len(jobs), np.uint32)
    for pos, p in ((3, 70_001), (4, 33), (41, 500), (64, 31), (127, 21_000), (139, 99_990)):
        progress[pos] = p
    with sja_mod.Sja() as ctx:
        _load(ctx, prof, progress)
        _check_scan(oracle_mod, ctx, prof, progress)


def test_scan_cfg1_sampled_jobs(sja_mod, oracle_mod):
    spec = wl.SPECS[1]
    prof = wl.make_profiles(spec)
    progress = np.zeros(prof.n_jobs, np.uint32)
    with sja_mod.Sja() as ctx:
        _load(ctx, prof, progress)
        sc = ctx.get_scan()
        safe = wl.unpack_safe_bits(prof.safe_bits, prof.n_steps)
        assert ctx.scan_size() == int(safe.sum())
        rng = np.random.default_rng(5)
        for j in rng.choice(prof.n_jobs, 40, replace=False):
            rows = np.array(oracle_mod.boundary_table(prof, int(j), 0), dtype=np.uint64)
            b0, b1 = int(sc["boff"][j]), int(sc["boff"][j + 1])
            assert b1 - b0 == rows.shape[0]
            got = np.stack([sc["k"][b0:b1], sc["D"][b0:b1], sc["M"][b0:b1], sc["S"][b0:b1], sc["W"][b0:b1]], 1)
            assert np.array_equal(got.astype(np.uint64), rows)


# ------------------------------------------------------------------ select (a2-a5)
@pytest.mark.parametrize("flags", [0, 1, 2, 4])
@pytest.mark.parametrize("policy", [0, 1, 2, 3])
def test_select_tiny_random_vs_oracle(sja_mod, oracle_mod, policy, flags):
    rng = np.random.default_rng(200 + policy)
    with sja_mod.Sja() as ctx:
        for trial in range(12):
            jobs = random_small_profiles(rng, int(rng.integers(1, 70)), 40, p_safe=float(rng.uniform(0.05, 0.9)),
                                         dmax=30, mmax=100, allow_zero=(trial % 4 == 0))
            J = len(jobs)
            prof = profiles_from_lists(jobs, ready=rng.integers(0, 20, J), wait=rng.integers(0, 9000, J),
                                       prio=rng.integers(0, 3, J))
            lens = np.diff(prof.off).astype(np.int64)
            progress = np.array([rng.integers(0, n + 1) for n in lens], dtype=np.uint32)
            G = int(rng.integers(1, 90))
            gaps = gaps_from_lists([(int(rng.integers(0, 7)), int(rng.integers(0, 30)), int(rng.integers(0, 400)),
                                     int(rng.integers(0, 110))) for _ in range(G)])
            _load(ctx, prof, progress)
            ctx.advertise(gaps)
            got = ctx.select(policy, flags=flags, out="host")
            want = oracle_mod.select(prof, progress, prof.ready_ms, gaps, policy)
            _assert_awards_equal(got, want)
            assert not got["granted"].any()


@pytest.mark.parametrize("cfg", [0, 1])
def test_select_published_small_configs(sja_mod, oracle_mod, cfg):
    spec = wl.SPECS[cfg]
    prof = wl.make_profiles(spec)
    gaps = wl.make_gaps(spec)
    progress = np.zeros(prof.n_jobs, np.uint32)
    with sja_mod.Sja() as ctx:
        _load(ctx, prof)
        ctx.advertise(gaps)
        want = oracle_mod.select(prof, progress, prof.ready_ms, gaps, spec.policy)
        for flags in (0, 1, 2, 4):
            got = ctx.select(spec.policy, flags=flags, out="host")
            _assert_awards_equal(got, want)
        assert (got["job"] != U32MAX).sum() > 0
        # select is free of side effects and repeatable
        p, r = ctx.get_state()
        assert not p.any() and np.array_equal(r, prof.ready_ms)
        again = ctx.select(spec.policy, out="host")
        assert again.tobytes() == got.tobytes()


def test_select_fairness_and_sla_scaled_configs(sja_mod, oracle_mod):
    for base, changes in ((2, dict(n_jobs=3000, fixed_len=700, n_gaps=300)),
                          (3, dict(n_jobs=4000, zipf_max=6000, n_gaps=256))):
        spec = wl.scaled(wl.SPECS[base], **changes)
        prof = wl.make_profiles(spec)
        gaps = wl.make_gaps(spec)
        progress = np.zeros(prof.n_jobs, np.uint32)
        with sja_mod.Sja() as ctx:
            _load(ctx, prof)
            ctx.advertise(gaps)
            want = oracle_mod.select(prof, progress, prof.ready_ms, gaps, spec.policy)
            for flags in (0, 1, 2, 4):
                got = ctx.select(spec.policy, flags=flags, out="host")
                _assert_awards_equal(got, want)


def test_select_long_windows_and_many_capacity_classes(sja_mod, oracle_mod):
    """Windows far longer than any staged tile and hundreds of distinct capacities."""
    rng = np.random.default_rng(77)
    spec = wl.scaled(wl.SPECS[1], n_jobs=700, fixed_len=900, n_gaps=400)
    prof = wl.make_profiles(spec)
    gaps = wl.make_gaps(spec)
    gaps["T_ms"] = rng.integers(0, 40000, gaps.shape[0])
    gaps["T_ms"][:5] = U32MAX
    gaps["C_MiB"] = rng.integers(1, 90000, gaps.shape[0])
    gaps["C_MiB"][:3] = U32MAX
    progress = rng.integers(0, 900, prof.n_jobs).astype(np.uint32)
    with sja_mod.Sja() as ctx:
        _load(ctx, prof, progress)
        ctx.advertise(gaps)
        want = oracle_mod.select(prof, progress, prof.ready_ms, gaps, 0)
        for flags in (0, 1, 2, 4):
            got = ctx.select(0, flags=flags, out="host")
            _assert_awards_equal(got, want)


@pytest.mark.parametrize("policy", [0, 1, 2, 3])
def test_select_ties_duplicate_jobs_and_ready_boundaries(sja_mod, oracle_mod, policy):
    """Many exact ties (copies of the same profile), zero-work segments (a longer subjob with the
    same score), few distinct ready times met exactly by the gap starts, repeated T values, and
    job / gap counts that are not multiples of 32: every kernel against the oracle."""
    rng = np.random.default_rng(4100 + policy)
    base = random_small_profiles(rng, 9, 60, p_safe=0.4, dmax=12, mmax=50, allow_zero=True)
    jobs = [base[int(rng.integers(0, len(base)))] for _ in range(173)]
    J = len(jobs)
    prof = profiles_from_lists(jobs, ready=rng.choice([0, 5, 5, 10, 4000000000], J),
                               wait=rng.choice([0, 999, 1000, 2000], J), prio=rng.choice([0, 1, 1, 2], J))
    progress = np.zeros(J, np.uint32)
    rows = [(int(rng.integers(0, 7)), int(rng.choice([0, 4, 5, 9, 10, 11, 3999999999, 4000000000])),
             int(rng.choice([0, 3, 17, 17, 40, 90, 90, 250, U32MAX])), int(rng.choice([7, 25, 50])))
            for _ in range(77)]
    gaps = gaps_from_lists(rows)
    with sja_mod.Sja() as ctx:
        _load(ctx, prof, progress)
        for rnd in range(4):
            ctx.advertise(gaps)
            want = oracle_mod.select(prof, progress, prof.ready_ms, gaps, policy)
            assert (want["job"] != U32MAX).any()
            for flags in (0, 1, 2, 4):
                _assert_awards_equal(ctx.select(policy, flags=flags, out="host"), want)
            ctx.commit()
            oracle_mod.commit(progress, prof.ready_ms, gaps, want)
            p, r = ctx.get_state()
            assert np.array_equal(p, progress) and np.array_equal(r, prof.ready_ms)


def test_tight_fit_policy_committed_rounds_all_kernels(sja_mod, oracle_mod):
    """Policy 3 (least slack on the slice) at a size where the tile kernel is the default: awards of every
    kernel, grants and job state over committed rounds.  Many jobs share a peak, so ties are frequent."""
    spec = wl.scaled(wl.SPECS[4], n_jobs=3000, fixed_len=700, n_gaps=384)
    prof = wl.make_profiles(spec, threads=2)
    progress = np.zeros(prof.n_jobs, np.uint32)
    ready = prof.ready_ms.copy()
    with sja_mod.Sja() as ctx:
        _load(ctx, prof)
        for rnd in range(5):
            gaps = wl.make_gaps(spec, rnd)
            ctx.advertise(gaps)
            want = oracle_mod.select(prof, progress, ready, gaps, 3)
            assert (want["job"] != U32MAX).mean() > 0.5
            for flags in (0, 1, 2, 4):
                _assert_awards_equal(ctx.select(3, flags=flags, out="host"), want)
            assert ctx.commit() == oracle_mod.commit(progress, ready, gaps, want)
            p, r = ctx.get_state()
            assert np.array_equal(p, progress) and np.array_equal(r, ready)


# ------------------------------------------------------------------ commit (a6), multi-round
@pytest.mark.parametrize("flags", [0, 1, 2, 4])
def test_streaming_rounds_bit_exact(sja_mod, oracle_mod, flags):
    """Scaled streaming workload: per-round awards (with grants) and final state match the oracle."""
    spec = wl.scaled(wl.SPECS[4], n_jobs=1500, fixed_len=300, n_gaps=200, n_rounds=60)
    prof = wl.make_profiles(spec)
    progress = np.zeros(prof.n_jobs, np.uint32)
    ready = prof.ready_ms.copy()
    total = 0
    with sja_mod.Sja() as ctx:
        _load(ctx, prof)
        for r in range(spec.n_rounds):
            gaps = wl.make_gaps(spec, r)
            ctx.advertise(gaps)
            ctx.select(spec.policy, flags=flags)
            n_gpu = ctx.commit()
            got = ctx.get_awards()
            want = oracle_mod.select(prof, progress, ready, gaps, spec.policy)
            n_cpu = oracle_mod.commit(progress, ready, gaps, want)
            _assert_awards_equal(got, want, fields=("job", "end_step", "dur_ms", "score", "granted"))
            assert n_gpu == n_cpu
            total += n_cpu
        p, rdy = ctx.get_state()
        assert np.array_equal(p, progress) and np.array_equal(rdy, ready)
        assert total > spec.n_rounds          # the workload really grants subjobs
        assert (p == 300).any()               # and some jobs finish and must decline afterwards


def test_commit_resolves_multiple_wins(sja_mod, oracle_mod):
    """One dominant job wins every gap; it accepts the largest k, then the lowest gap id."""
    jobs = [([10] * 20, [100] * 20, [1] * 20), ([10] * 20, [1] * 20, [1] * 20)]
    prof = profiles_from_lists(jobs)
    gaps = gaps_from_lists([(0, 0, 50, 200), (1, 0, 120, 200), (2, 0, 120, 200), (3, 0, 30, 200)])
    with sja_mod.Sja() as ctx:
        _load(ctx, prof)
        ctx.advertise(gaps)
        ctx.select(0)
        assert ctx.commit() == 1
        aw = ctx.get_awards()
        assert aw["job"].tolist() == [0, 0, 0, 0]
        assert aw["granted"].tolist() == [0, 1, 0, 0]
        p, r = ctx.get_state()
        assert p.tolist() == [12, 0] and r.tolist() == [120, 0]
        want = oracle_mod.select(prof, np.zeros(2, np.uint32), prof.ready_ms, gaps, 0)
        pr, rd = np.zeros(2, np.uint32), prof.ready_ms.copy()
        oracle_mod.commit(pr, rd, gaps, want)
        _assert_awards_equal(aw, want, fields=("job", "end_step", "dur_ms", "score", "granted"))


# ------------------------------------------------------------------ host logic / errors
def test_error_paths(sja_mod):
    b = sja_mod
    prof = profiles_from_lists([([1, 2], [3, 4], [0, 1]), ([5], [6], [1])], wait=None, prio=None)
    gaps = gaps_from_lists([(0, 0, 10, 10)])
    with b.Sja() as ctx:
        with pytest.raises(b.SjaError) as e:
            ctx.advertise(gaps)
        assert e.value.status == 4                      # STATE: advertise before load
        with pytest.raises(b.SjaError) as e:
            ctx.commit()
        assert e.value.status == 4
        _load(ctx, prof)
        with pytest.raises(b.SjaError) as e:
            ctx.select(0)
        assert e.value.status == 4                      # select before advertise
        ctx.advertise(gaps)
        for policy, status in ((1, 1), (2, 1), (9, 1)):  # fairness w/o wait, SLA w/o prio, unknown
            with pytest.raises(b.SjaError) as e:
                ctx.select(policy)
            assert e.value.status == status
        got = ctx.select(0, out="host")
        assert got["job"][0] == 1                       # job1: work 30 > job0: 1*3+2*4 = 11
        assert ctx.commit() == 1
        with pytest.raises(b.SjaError) as e:
            ctx.commit()
        assert e.value.status == 4                      # twice
        # bad CSR leaves the loaded state untouched
        bad_off = np.array([0, 5, 3], dtype=np.uint64)
        with pytest.raises(b.SjaError) as e:
            ctx.load_profiles(bad_off, prof.dur_ms, prof.mem_MiB, prof.safe_bits, prof.ready_ms)
        assert e.value.status == 2
        with pytest.raises(b.SjaError) as e:
            ctx.load_profiles(prof.off, prof.dur_ms, prof.mem_MiB, prof.safe_bits, prof.ready_ms,
                              progress=np.array([3, 0], np.uint32))
        assert e.value.status == 2                      # progress > len
        p, r = ctx.get_state()
        assert p.tolist() == [0, 1]
        # duration overflow is reported at load
        big = profiles_from_lists([([2**31, 2**31], [1, 1], [1, 1])])
        with pytest.raises(b.SjaError) as e:
            _load(ctx, big)
        assert e.value.status == 3
        # fairness score overflow is reported at select
        huge = profiles_from_lists([([2**31 - 1], [2**32 - 1], [1])], wait=[4_000_000_000])
        _load(ctx, huge)
        ctx.advertise(gaps)
        ctx.select(0)
        with pytest.raises(b.SjaError) as e:
            ctx.select(1)
        assert e.value.status == 3


def test_failed_allocation_leaves_a_usable_context(sja_mod, oracle_mod):
    """A device allocation that fails inside sja_advertise (injected on the host: the n-th growing allocation
    reports out-of-memory without being tried) must leave no half-built batch behind: select and commit answer
    SJA_ERR_STATE and launch nothing, the loaded profiles stay usable, and the next advertise works."""
    spec = wl.scaled(wl.SPECS[1], n_jobs=400, fixed_len=300, n_gaps=64)
    prof = wl.make_profiles(spec, threads=1)
    small, large = wl.make_gaps(spec), wl.make_gaps(spec, 1, n_gaps=9000)
    zero = np.zeros(prof.n_jobs, np.uint32)
    with sja_mod.Sja() as ctx:
        _load(ctx, prof)
        ctx.advertise(small)
        want_small = oracle_mod.select(prof, zero, prof.ready_ms, small, spec.policy)
        _assert_awards_equal(ctx.select(spec.policy, out="host"), want_small)
        for nth in (1, 2, 3, 4, 5, 6):              # each of the six buffers a larger batch has to grow
            ctx.debug_fail_alloc(nth)
            with pytest.raises(sja_mod.SjaError) as e:
                ctx.advertise(large[:1500 * nth])   # larger than any batch before: all six grow again
            assert e.value.status == 5, nth         # SJA_ERR_OOM
            for call in (lambda: ctx.select(spec.policy), ctx.commit, ctx.get_awards):
                with pytest.raises(sja_mod.SjaError) as e:
                    call()
                assert e.value.status == 4, nth     # SJA_ERR_STATE: there is no batch
            ctx.debug_fail_alloc(0)
            ctx.advertise(small)                    # the context is still good
            _assert_awards_equal(ctx.select(spec.policy, out="host"), want_small)
        ctx.advertise(large)
        want_large = oracle_mod.select(prof, zero, prof.ready_ms, large, spec.policy)
        _assert_awards_equal(ctx.select(spec.policy, out="host"), want_large)
        # a failure while select grows its candidate rows: the batch stays advertised, the next select works
        ctx.advertise(wl.make_gaps(spec, 2, n_gaps=12000))
        ctx.debug_fail_alloc(1)
        with pytest.raises(sja_mod.SjaError) as e:
            ctx.select(spec.policy)
        assert e.value.status == 5
        with pytest.raises(sja_mod.SjaError) as e:
            ctx.commit()
        assert e.value.status == 4
        want = oracle_mod.select(prof, zero, prof.ready_ms, wl.make_gaps(spec, 2, n_gaps=12000), spec.policy)
        _assert_awards_equal(ctx.select(spec.policy, out="host"), want)
        assert ctx.commit() > 0


def test_empty_and_degenerate_inputs(sja_mod, oracle_mod):
    # all jobs empty; a job that is already finished; gaps nobody fits
    prof = profiles_from_lists([([], [], []), ([], [], [])])
    gaps = gaps_from_lists([(0, 0, 100, 100), (1, 5, 0, 0)])
    with sja_mod.Sja() as ctx:
        _load(ctx, prof)
        assert ctx.scan_size() == 0
        ctx.advertise(gaps)
        got = ctx.select(0, out="host")
        assert (got["job"] == U32MAX).all() and not got["score"].any()
        assert ctx.commit() == 0
        prof2 = profiles_from_lists([([4, 4], [9, 9], [1, 1]), ([0, 0], [0, 7], [1, 1])])
        progress = np.array([2, 0], np.uint32)
        _load(ctx, prof2, progress)
        ctx.advertise(gaps_from_lists([(0, 0, 0, 7), (0, 0, 0, 6)]))
        got = ctx.select(0, out="host")
        want = oracle_mod.select(prof2, progress, prof2.ready_ms, gaps_from_lists([(0, 0, 0, 7), (0, 0, 0, 6)]), 0)
        _assert_awards_equal(got, want)
        assert got["job"].tolist() == [1, 1] and got["end_step"].tolist() == [2, 1]   # zero-work interest


def test_select_very_large_gap_batch_unsorted_path(sja_mod, oracle_mod):
    """More gaps than the ranking kernel orders (65 536): the batch stays in the caller's order and
    the per-pair search kernel serves it."""
    spec = wl.scaled(wl.SPECS[1], n_jobs=300, fixed_len=200, n_gaps=70000)
    prof = wl.make_profiles(spec, threads=2)
    gaps = wl.make_gaps(spec)
    progress = np.zeros(prof.n_jobs, np.uint32)
    with sja_mod.Sja() as ctx:
        _load(ctx, prof)
        ctx.advertise(gaps)
        got = ctx.select(spec.policy, out="host")
        want = oracle_mod.select(prof, progress, prof.ready_ms, gaps, spec.policy)
        _assert_awards_equal(got, want)
        assert ctx.commit() == oracle_mod.commit(progress, prof.ready_ms.copy(), gaps, want)
        _assert_awards_equal(ctx.get_awards(), want, fields=("job", "end_step", "dur_ms", "score", "granted"))
        # exactly at the limit the ordered path runs
        ctx.load_profiles(prof.off, prof.dur_ms, prof.mem_MiB, prof.safe_bits, prof.ready_ms)
        ctx.advertise(gaps[:65536])
        got = ctx.select(spec.policy, out="host")
        _assert_awards_equal(got, want[:65536])


def test_very_many_capacity_classes_take_the_standby_search(sja_mod, oracle_mod):
    """More distinct capacities than max(64, G/16): the ordered-gap kernel that was queued returns at once and the
    per-pair search kernel queued behind it serves the round (the class count never leaves the device); device
    batches are read in place.  Plain rounds, a forced tile / merge request, and a re-auction (which reads the count
    once and then queues the search alone) all match the oracle."""
    import torch
    spec = wl.scaled(wl.SPECS[3], n_jobs=3000, zipf_max=2500, n_gaps=1000)
    prof = wl.make_profiles(spec, threads=2)
    gaps = wl.make_gaps(spec)
    rng = np.random.default_rng(808)
    gaps["C_MiB"] = rng.choice(np.arange(1500, 82000, 97), gaps.shape[0])      # several hundred distinct capacities
    assert np.unique(gaps["C_MiB"]).size > 200
    progress = np.zeros(prof.n_jobs, np.uint32)
    ready = prof.ready_ms.copy()
    dev_gaps = torch.from_numpy(gaps.view(np.uint8).reshape(-1).copy()).cuda()
    with sja_mod.Sja() as ctx:
        _load(ctx, prof)
        for policy, flags in ((0, 0), (2, 0), (3, sja_mod.FLAG_FORCE_TILE), (0, sja_mod.FLAG_FORCE_MERGE)):
            ctx.advertise(dev_gaps)
            want = oracle_mod.select(prof, progress, ready, gaps, policy)
            _assert_awards_equal(ctx.select(policy, flags=flags, out="host"), want)
        n_gpu, passes = ctx.round_reauction(2)
        aw_o, n_cpu, passes_o = oracle_mod.round_with_reauction(prof, progress, ready, gaps, 2)
        assert (n_gpu, passes) == (n_cpu, passes_o) and n_gpu > 0
        _assert_awards_equal(ctx.get_awards(), aw_o, fields=("job", "end_step", "dur_ms", "score", "granted"))
        p, r = ctx.get_state()
        assert np.array_equal(p, progress) and np.array_equal(r, ready)


def test_reloads_from_device_arrays(sja_mod, oracle_mod):
    """Loads from device-resident arrays into a context that already holds a load take the path with a
    single host wait (the validation verdict is checked on the device).  Covered here: a same-size reload,
    a rejected CSR (the previous load must stay usable, bit for bit), a larger load (the table outgrows
    the buffers and the scan is run again), a smaller one, and scan rows against the oracle after each."""
    import torch
    dev = torch.device("cuda", 0)

    def to_dev(prof, off=None):
        t = lambda a, dt: None if a is None else torch.from_numpy(np.ascontiguousarray(a).view(dt)).to(dev)
        return dict(off=t(prof.off if off is None else off, np.int64), d=t(prof.dur_ms, np.int32),
                    m=t(prof.mem_MiB, np.int32), s=t(prof.safe_bits, np.int32), ready=t(prof.ready_ms, np.int32),
                    wait=t(prof.wait_ms, np.int32), prio=t(prof.prio, np.uint8))

    def load_dev(ctx, d):
        ctx.load_profiles(d["off"], d["d"], d["m"], d["s"], d["ready"], wait_ms=d["wait"], prio=d["prio"])

    def check(ctx, prof, spec):
        gaps = wl.make_gaps(spec)
        ctx.advertise(gaps)
        z = np.zeros(prof.n_jobs, np.uint32)
        want = oracle_mod.select(prof, z, prof.ready_ms, gaps, spec.policy)
        _assert_awards_equal(ctx.select(spec.policy, out="host"), want)
        assert ctx.scan_size() == int(wl.unpack_safe_bits(prof.safe_bits, prof.n_steps).sum())
        return want

    small = wl.scaled(wl.SPECS[3], n_jobs=900, zipf_max=3000, n_gaps=300)
    large = wl.scaled(wl.SPECS[3], n_jobs=900, zipf_max=60000, n_gaps=300)     # same J, far more rows
    p_small, p_large = wl.make_profiles(small, threads=2), wl.make_profiles(large, threads=2)
    assert p_large.n_steps > 2 * p_small.n_steps
    with sja_mod.Sja() as ctx:
        d_small, d_large = to_dev(p_small), to_dev(p_large)
        load_dev(ctx, d_small)                      # first load: nothing to reuse yet
        check(ctx, p_small, small)
        load_dev(ctx, d_small)                      # reload: single-wait path
        want = check(ctx, p_small, small)
        bad = p_small.off.copy()
        bad[5], bad[6] = bad[6], bad[5]             # offsets not monotone
        with pytest.raises(sja_mod.SjaError) as e:
            load_dev(ctx, to_dev(p_small, off=bad))
        assert e.value.status == 2
        _assert_awards_equal(ctx.select(small.policy, out="host"), want)     # the old load still stands
        assert ctx.commit() > 0
        load_dev(ctx, d_large)                      # more rows than the table buffers hold
        check(ctx, p_large, large)
        load_dev(ctx, d_small)                      # and back
        check(ctx, p_small, small)


def test_select_is_deterministic_and_device_outputs_match(sja_mod):
    """The cross-CTA reduction is on a totally ordered key, so repeated selects give identical bytes;
    a device output buffer receives the same awards as a host buffer."""
    import torch
    spec = wl.scaled(wl.SPECS[2], n_jobs=5000, fixed_len=600, n_gaps=700)
    prof = wl.make_profiles(spec, threads=2)
    gaps = wl.make_gaps(spec)
    stream = torch.cuda.Stream()
    with sja_mod.Sja(stream=stream.cuda_stream) as ctx:
        _load(ctx, prof)
        ctx.advertise(gaps)
        first = ctx.select(spec.policy, out="host")
        for flags in (0, 1, 2, 4, 0, 1, 2, 4, 0):
            assert ctx.select(spec.policy, flags=flags, out="host").tobytes() == first.tobytes()
        dev = torch.zeros(24 * gaps.shape[0], dtype=torch.uint8, device="cuda")
        ctx.select(spec.policy, out=dev)
        stream.synchronize()
        assert dev.cpu().numpy().tobytes() == first.tobytes()
        t = ctx.profile_read()
        assert t["select_launches"] == 0          # profiling is off unless enabled
        ctx.profile_enable(True)
        ctx.select(spec.policy)
        t = ctx.profile_read()
        assert t["select_launches"] == 1 and t["select_ms"] > 0
