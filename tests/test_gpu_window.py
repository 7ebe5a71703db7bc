"""GPU parity for the window options (late start inside a gap, per-job deadlines): every select and
commit through the C ABI against the oracle, bit for bit."""
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
def test_window_options_tiny_random(oracle_mod, policy):
    from paper_2509_19086_b200 import binding
    rng = np.random.default_rng(900 + policy)
    with binding.Sja() as ctx:
        for trial in range(10):
            jobs = random_small_profiles(rng, int(rng.integers(1, 80)), 40, p_safe=float(rng.uniform(0.05, 0.9)),
                                         dmax=30, mmax=100, allow_zero=(trial % 4 == 0))
            J = len(jobs)
            prof = profiles_from_lists(jobs, ready=rng.integers(0, 400, J), wait=rng.integers(0, 9000, J),
                                       prio=rng.integers(0, 3, J))
            lens = np.diff(prof.off).astype(np.int64)
            progress = np.array([rng.integers(0, n + 1) for n in lens], dtype=np.uint32)
            G = int(rng.integers(1, 90))
            gaps = gaps_from_lists([(int(rng.integers(0, 7)), int(rng.integers(0, 300)), int(rng.integers(0, 400)),
                                     int(rng.integers(0, 110))) for _ in range(G)])
            deadline = rng.integers(0, 900, J).astype(np.uint32)
            deadline[rng.random(J) < 0.3] = U32MAX
            _load(ctx, prof, progress)
            for late, dl in ((True, None), (False, deadline), (True, deadline)):
                ctx.set_window_options(late, dl)
                ctx.advertise(gaps)
                want = oracle_mod.select(prof, progress, prof.ready_ms, gaps, policy, late_start=late, deadline_ms=dl)
                # the option decides the kernel: the flags below must not change anything
                for flags in (0, 2, 4):
                    _same(ctx.select(policy, flags=flags, out="host"), want)
            ctx.set_window_options(False, None)
            ctx.advertise(gaps)
            _same(ctx.select(policy, out="host"), oracle_mod.select(prof, progress, prof.ready_ms, gaps, policy))


@pytest.mark.parametrize("base,changes", [
    (1, dict(n_jobs=1500, fixed_len=500, n_gaps=300)),
    (2, dict(n_jobs=2500, fixed_len=400, n_gaps=500)),
    (3, dict(n_jobs=1200, zipf_max=2500, n_gaps=400)),
])
def test_window_options_streaming_rounds(oracle_mod, base, changes):
    """Several committed rounds with both options on: awards, grants and job state after every round."""
    from paper_2509_19086_b200 import binding
    spec = wl.scaled(wl.SPECS[base], **changes)
    prof = wl.make_profiles(spec, threads=2)
    J = prof.n_jobs
    rng = np.random.default_rng(70 + base)
    deadline = rng.integers(500, 9000, J).astype(np.uint32)
    deadline[rng.random(J) < 0.4] = U32MAX
    progress = np.zeros(J, np.uint32)
    ready = prof.ready_ms.copy()
    ready[::3] += 1500                      # many jobs turn ready inside the first windows
    late_wins = 0
    with binding.Sja() as ctx:
        ctx.load_profiles(prof.off, prof.dur_ms, prof.mem_MiB, prof.safe_bits, ready,
                          wait_ms=prof.wait_ms, prio=prof.prio)
        ctx.set_window_options(True, deadline)
        for rnd in range(6):
            gaps = wl.make_gaps(spec, rnd)
            ctx.advertise(gaps)
            got = ctx.select(spec.policy, out="host")
            want = oracle_mod.select(prof, progress, ready, gaps, spec.policy, late_start=True, deadline_ms=deadline)
            _same(got, want)
            win = want["job"] != U32MAX
            late_wins += int((ready[want["job"][win]] > gaps["start_ms"][win]).sum())
            n_gpu = ctx.commit()
            n_cpu = oracle_mod.commit(progress, ready, gaps, want, late_start=True)
            assert n_gpu == n_cpu
            _same(ctx.get_awards(), want, FIELDS + ("granted",))
            p, r = ctx.get_state()
            assert np.array_equal(p, progress) and np.array_equal(r, ready)
        assert late_wins > 0
        # finished-by-deadline holds for every grant of the last round
        g = np.nonzero(want["granted"] == 1)[0]
        j = want["job"][g]
        dl = deadline[j].astype(np.int64)
        assert (r[j].astype(np.int64) <= np.where(dl == U32MAX, 2**32, dl)).all()


def test_window_options_reauction_and_errors(oracle_mod):
    from paper_2509_19086_b200 import binding
    spec = wl.scaled(wl.SPECS[1], n_jobs=900, fixed_len=300, n_gaps=200)
    prof = wl.make_profiles(spec, threads=2)
    gaps = wl.make_gaps(spec)
    with binding.Sja() as ctx:
        with pytest.raises(binding.SjaError) as e:
            ctx.set_window_options(True, None)           # before any load
        assert e.value.status == 4
        _load(ctx, prof)
        ctx.set_window_options(True, None)
        ctx.advertise(gaps)
        ctx.select(spec.policy)
        ctx.set_window_options(False, None)              # discards the pending select
        with pytest.raises(binding.SjaError) as e:
            ctx.commit()
        assert e.value.status == 4
        ctx.select(spec.policy)
        ctx.commit()
        # re-auction under late start: every grant is the job's longest subjob in what is left of its gap
        _load(ctx, prof)
        ctx.set_window_options(True, None)
        ctx.advertise(gaps)
        n, passes = ctx.round_reauction(spec.policy)
        aw = ctx.get_awards()
        g = np.nonzero(aw["granted"] == 1)[0]
        assert n == g.size > 0 and passes >= 1
        assert np.unique(aw["job"][g]).size == g.size
        for gi in g[:60]:
            j = int(aw["job"][gi])
            want = oracle_mod.pair(prof, j, 0, int(prof.ready_ms[j]), int(gaps["start_ms"][gi]),
                                   int(gaps["T_ms"][gi]), int(gaps["C_MiB"][gi]), late_start=True)
            assert want is not None and want[0] == int(aw["end_step"][gi]) and want[1] == int(aw["dur_ms"][gi])
        # a new load keeps late_start and drops the deadlines
        dl = np.zeros(prof.n_jobs, np.uint32)            # everything overdue
        ctx.set_window_options(False, dl)
        ctx.advertise(gaps)
        assert (ctx.select(spec.policy, out="host")["job"] == U32MAX).all()
        _load(ctx, prof)
        ctx.advertise(gaps)
        _same(ctx.select(spec.policy, out="host"),
              oracle_mod.select(prof, np.zeros(prof.n_jobs, np.uint32), prof.ready_ms, gaps, spec.policy))
