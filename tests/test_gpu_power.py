"""GPU parity for the power envelope (sja_load_power, sja_advertise_power_caps): selects and commits through
the C ABI against the oracle with the same trace and caps, bit for bit."""
import numpy as np
import pytest

from paper_2509_19086_b200 import workloads as wl
from tests.helpers import gaps_from_lists, profiles_from_lists, random_small_profiles

pytestmark = pytest.mark.gpu
FIELDS = ("job", "end_step", "dur_ms", "score")
U32MAX = 0xFFFFFFFF


def _load(ctx, prof, progress=None):
    ctx.load_profiles(prof.off, prof.dur_ms, prof.mem_MiB, prof.safe_bits, prof.ready_ms,
                      progress=progress, wait_ms=prof.wait_ms, prio=prof.prio)


def _same(got, want, fields=FIELDS):
    for f in fields:
        bad = np.nonzero(got[f] != want[f])[0]
        assert bad.size == 0, (f, bad[:5], got[bad[:5]], want[bad[:5]])


@pytest.mark.parametrize("policy", [0, 1, 2, 3])
def test_power_caps_tiny_random(oracle_mod, policy):
    from paper_2509_19086_b200 import binding
    rng = np.random.default_rng(1300 + policy)
    with binding.Sja() as ctx:
        for trial in range(10):
            jobs = random_small_profiles(rng, int(rng.integers(1, 80)), 40, p_safe=float(rng.uniform(0.05, 0.9)),
                                         dmax=30, mmax=100, allow_zero=(trial % 4 == 0))
            J = len(jobs)
            prof = profiles_from_lists(jobs, ready=rng.integers(0, 20, J), wait=rng.integers(0, 9000, J),
                                       prio=rng.integers(0, 3, J))
            lens = np.diff(prof.off).astype(np.int64)
            progress = np.array([rng.integers(0, n + 1) for n in lens], dtype=np.uint32)
            G = int(rng.integers(1, 90))
            gaps = gaps_from_lists([(int(rng.integers(0, 7)), int(rng.integers(0, 30)), int(rng.integers(0, 400)),
                                     int(rng.integers(0, 110))) for _ in range(G)])
            power = rng.integers(0, 500, prof.n_steps).astype(np.uint32)
            caps = rng.integers(0, 520, G).astype(np.uint32)
            caps[rng.random(G) < 0.2] = U32MAX
            _load(ctx, prof, progress)
            ctx.load_power(prof.off, power)
            ctx.advertise(gaps)
            plain = oracle_mod.select(prof, progress, prof.ready_ms, gaps, policy)
            _same(ctx.select(policy, out="host"), plain)                    # no caps yet: nothing changes
            ctx.advertise_power_caps(caps)
            want = oracle_mod.select(prof, progress, prof.ready_ms, gaps, policy, power_W=power, power_cap_W=caps)
            for flags in (0, 2, 4):                                         # the caps decide the kernel
                _same(ctx.select(policy, flags=flags, out="host"), want)
            ctx.advertise_power_caps(None)
            _same(ctx.select(policy, out="host"), plain)


@pytest.mark.parametrize("base,changes", [
    (1, dict(n_jobs=1500, fixed_len=500, n_gaps=300)),
    (3, dict(n_jobs=1200, zipf_max=2500, n_gaps=400)),
    (4, dict(n_jobs=2500, fixed_len=400, n_gaps=500)),
])
def test_power_caps_committed_rounds(oracle_mod, base, changes):
    """Committed rounds with a trace and caps: the running maximum of granted jobs has to follow their progress.
    The trace is loaded after two plain rounds, i.e. from progress points in the middle of the jobs."""
    from paper_2509_19086_b200 import binding
    spec = wl.scaled(wl.SPECS[base], **changes)
    prof = wl.make_profiles(spec, threads=2)
    rng = np.random.default_rng(90 + base)
    # power follows memory loosely: 50 W idle + up to 350 W
    power = (50 + prof.mem_MiB.astype(np.int64) * 350 // 81920 + rng.integers(0, 120, prof.n_steps)).astype(np.uint32)
    progress = np.zeros(prof.n_jobs, np.uint32)
    ready = prof.ready_ms.copy()
    shut_out = 0
    with binding.Sja() as ctx:
        _load(ctx, prof)
        for rnd in range(7):
            gaps = wl.make_gaps(spec, rnd)
            ctx.advertise(gaps)
            caps = None
            if rnd == 2:
                ctx.load_power(prof.off, power)
            if rnd >= 2:
                caps = rng.integers(60, 400, gaps.shape[0]).astype(np.uint32)
                caps[::7] = U32MAX
                ctx.advertise_power_caps(caps)
            want = oracle_mod.select(prof, progress, ready, gaps, spec.policy,
                                     power_W=power if rnd >= 2 else None, power_cap_W=caps)
            if rnd >= 2:
                free = oracle_mod.select(prof, progress, ready, gaps, spec.policy)
                shut_out += int((free["job"] != want["job"]).sum())
            _same(ctx.select(spec.policy, out="host"), want)
            assert ctx.commit() == oracle_mod.commit(progress, ready, gaps, want)
            _same(ctx.get_awards(), want, FIELDS + ("granted",))
            p, r = ctx.get_state()
            assert np.array_equal(p, progress) and np.array_equal(r, ready)
        assert shut_out > 0


def test_power_errors_and_lifetime(oracle_mod):
    from paper_2509_19086_b200 import binding
    spec = wl.scaled(wl.SPECS[1], n_jobs=900, fixed_len=300, n_gaps=200)
    prof = wl.make_profiles(spec, threads=2)
    gaps = wl.make_gaps(spec)
    power = np.full(prof.n_steps, 300, np.uint32)
    z = np.zeros(prof.n_jobs, np.uint32)
    with binding.Sja() as ctx:
        with pytest.raises(binding.SjaError) as e:
            ctx.load_power(prof.off, power)                     # before any load
        assert e.value.status == 4
        _load(ctx, prof)
        with pytest.raises(binding.SjaError) as e:
            ctx.advertise_power_caps(np.zeros(0, np.uint32))    # before advertise
        assert e.value.status == 4
        bad = prof.off.copy()
        bad[10] += 1                                            # job 9 one step longer, job 10 one shorter
        with pytest.raises(binding.SjaError) as e:
            ctx.load_power(bad, power)
        assert e.value.status == 2
        ctx.load_power(prof.off, power)
        ctx.advertise(gaps)
        ctx.advertise_power_caps(np.full(gaps.shape[0], 299, np.uint32))
        assert (ctx.select(spec.policy, out="host")["job"] == U32MAX).all()      # everything draws 300 W
        ctx.advertise_power_caps(np.full(gaps.shape[0], 300, np.uint32))
        _same(ctx.select(spec.policy, out="host"), oracle_mod.select(prof, z, prof.ready_ms, gaps, spec.policy))
        ctx.advertise(gaps)                                     # a new batch drops the caps
        ctx.select(spec.policy)
        ctx.advertise_power_caps(np.full(gaps.shape[0], 299, np.uint32))
        with pytest.raises(binding.SjaError) as e:
            ctx.commit()                                        # the pending select was discarded
        assert e.value.status == 4
        _load(ctx, prof)                                        # a new load drops the trace: caps have no effect
        ctx.advertise(gaps)
        ctx.advertise_power_caps(np.full(gaps.shape[0], 0, np.uint32))
        _same(ctx.select(spec.policy, out="host"), oracle_mod.select(prof, z, prof.ready_ms, gaps, spec.policy))


def test_power_trace_on_a_load_with_long_jobs(oracle_mod):
    """A load that lists long jobs (far more steps left than the mean, at least 8192) takes the power scan's other
    hand-out: warps draw jobs from counters, the long ones first.  Long windows and loose capacities, so that awards
    reach deep into the long jobs' rows; some jobs entered at a progress point."""
    from paper_2509_19086_b200 import binding
    rng = np.random.default_rng(1400)
    lens = [int(x) for x in rng.integers(1, 700, 300)]
    for pos, n in ((0, 20_000), (7, 9_500), (8, 33_000), (150, 8_700), (299, 12_000)):
        lens[pos] = n
    N = int(np.sum(lens))
    off = np.zeros(len(lens) + 1, np.uint64)
    off[1:] = np.cumsum(lens)
    safe = (rng.random(N) < 0.1).astype(np.uint8)
    prof = wl.Profiles(off, rng.integers(1, 50, N).astype(np.uint32), rng.integers(1, 81920, N).astype(np.uint32),
                       wl.pack_safe_bits(safe), rng.integers(0, 100, len(lens)).astype(np.uint32), None, None)
    progress = np.zeros(len(lens), np.uint32)
    for pos, p in ((0, 10_001), (8, 7), (150, 8_000), (20, 100)):
        progress[pos] = min(p, lens[pos])
    power = rng.integers(50, 400, N).astype(np.uint32)
    G = 160
    gaps = gaps_from_lists([(int(rng.integers(0, 7)), int(rng.integers(100, 2000)),
                             int(rng.choice([500, 5_000, 100_000, 1_000_000])), int(rng.choice([40960, 81920])))
                            for _ in range(G)])
    caps = rng.integers(300, 420, G).astype(np.uint32)
    caps[rng.random(G) < 0.3] = U32MAX
    with binding.Sja() as ctx:
        _load(ctx, prof, progress)
        ctx.load_power(prof.off, power)
        ctx.advertise(gaps)
        ctx.advertise_power_caps(caps)
        want = oracle_mod.select(prof, progress, prof.ready_ms, gaps, 0, power_W=power, power_cap_W=caps)
        got = ctx.select(0, out="host")
        _same(got, want)
        assert (want["job"] != U32MAX).sum() > G // 4
        assert want["end_step"].max() > 1000      # some award runs far into a long job
