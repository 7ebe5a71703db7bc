"""GPU parity for sja_update_profile: after re-profiling some jobs (new durations and memory values for the
steps they have left, boundaries unchanged) every select and commit matches the oracle run on the edited
profile arrays, bit for bit; rejected updates leave the job as it was."""
import numpy as np
import pytest

from paper_2509_19086_b200 import workloads as wl
from tests.helpers import gaps_from_lists, profiles_from_lists

pytestmark = pytest.mark.gpu
FIELDS = ("job", "end_step", "dur_ms", "score")
U32MAX = 0xFFFFFFFF


def _same(got, want, fields=FIELDS):
    for f in fields:
        bad = np.nonzero(got[f] != want[f])[0]
        assert bad.size == 0, (f, bad[:5], got[bad[:5]], want[bad[:5]])


@pytest.mark.parametrize("base,changes", [
    (1, dict(n_jobs=1500, fixed_len=600, n_gaps=300)),
    (2, dict(n_jobs=2000, fixed_len=500, n_gaps=400)),
    (3, dict(n_jobs=1000, zipf_max=20000, n_gaps=400)),
])
def test_update_profile_rounds_match_oracle(oracle_mod, base, changes):
    from paper_2509_19086_b200 import binding
    spec = wl.scaled(wl.SPECS[base], **changes)
    prof = wl.make_profiles(spec, threads=2)
    J = prof.n_jobs
    rng = np.random.default_rng(500 + base)
    off = prof.off.astype(np.int64)
    progress = np.zeros(J, np.uint32)
    ready = prof.ready_ms.copy()
    with binding.Sja() as ctx:
        ctx.load_profiles(prof.off, prof.dur_ms, prof.mem_MiB, prof.safe_bits, prof.ready_ms,
                          wait_ms=prof.wait_ms, prio=prof.prio)
        for rnd in range(6):
            gaps = wl.make_gaps(spec, rnd)
            ctx.advertise(gaps)
            want = oracle_mod.select(prof, progress, ready, gaps, spec.policy)
            for flags in (0, 1, 2):
                _same(ctx.select(spec.policy, flags=flags, out="host"), want)
            assert ctx.commit() == oracle_mod.commit(progress, ready, gaps, want)
            p, r = ctx.get_state()
            assert np.array_equal(p, progress) and np.array_equal(r, ready)
            # re-profile: recent winners (their progress point moved), the longest job, random others
            winners = np.unique(want["job"][want["granted"] == 1])[:20]
            picks = np.unique(np.concatenate([winners, [int(np.argmax(np.diff(off)))], rng.integers(0, J, 30)]))
            for j in picks:
                a, b = int(off[j]) + int(progress[j]), int(off[j + 1])
                n = b - a
                new_d = rng.integers(1, 60, n).astype(np.uint32)
                new_m = np.clip(prof.mem_MiB[a:b].astype(np.int64) + rng.integers(-3000, 3000, n), 1, 81920).astype(np.uint32)
                if rnd % 2:                                   # device inputs every other round
                    import torch
                    td = torch.from_numpy(new_d.view(np.int32)).cuda()
                    tm = torch.from_numpy(new_m.view(np.int32)).cuda()
                    ctx.update_profile(int(j), td, tm)
                else:
                    ctx.update_profile(int(j), new_d, new_m)
                prof.dur_ms[a:b] = new_d
                prof.mem_MiB[a:b] = new_m
        # the table rows of an updated job against the oracle's dense prefix arrays of the edited profile
        sc = ctx.get_scan()
        j = int(picks[0])
        b0, b1 = int(sc["boff"][j]), int(sc["boff"][j + 1])
        a, b = int(off[j]), int(off[j + 1])
        pj = int(progress[j])
        live = sc["k"][b0:b1] > pj
        k = sc["k"][b0:b1][live].astype(np.int64)
        m = prof.mem_MiB[a:b].astype(np.int64)
        assert np.array_equal(sc["M"][b0:b1][live].astype(np.int64), np.array([m[pj:kk].max() for kk in k]))


def test_update_profile_rejections_leave_the_job_alone(oracle_mod):
    from paper_2509_19086_b200 import binding
    prof = profiles_from_lists([([4, 4, 4, 4], [9, 9, 9, 9], [1, 0, 1, 1]), ([5] * 6, [7] * 6, [1] * 6)],
                               wait=[0, 5000], prio=[0, 1])
    gaps = gaps_from_lists([(0, 0, 9, 100), (0, 0, 30, 100)])
    z = np.zeros(2, np.uint32)
    with binding.Sja() as ctx:
        with pytest.raises(binding.SjaError) as e:
            ctx.update_profile(0, np.ones(4, np.uint32), np.ones(4, np.uint32))        # before any load
        assert e.value.status == 4
        ctx.load_profiles(prof.off, prof.dur_ms, prof.mem_MiB, prof.safe_bits, prof.ready_ms,
                          wait_ms=prof.wait_ms, prio=prof.prio)
        ctx.advertise(gaps)
        before = ctx.select(0, out="host")
        for bad_n in (3, 5, 0):
            with pytest.raises(binding.SjaError) as e:
                ctx.update_profile(0, np.ones(bad_n, np.uint32), np.ones(bad_n, np.uint32))
            assert e.value.status == 2, bad_n                                          # not the steps it has left
        with pytest.raises(binding.SjaError) as e:
            ctx.update_profile(2, np.ones(4, np.uint32), np.ones(4, np.uint32))        # no such job
        assert e.value.status == 1
        with pytest.raises(binding.SjaError) as e:
            ctx.update_profile(0, np.full(4, 2**31, np.uint32), np.ones(4, np.uint32))  # total duration >= 2^32
        assert e.value.status == 3
        ctx.advertise(gaps)
        assert ctx.select(0, out="host").tobytes() == before.tobytes()
        # an accepted update discards the pending select; then the new values rule
        ctx.update_profile(0, np.array([2, 2, 2, 2], np.uint32), np.array([50, 60, 70, 80], np.uint32))
        with pytest.raises(binding.SjaError) as e:
            ctx.commit()
        assert e.value.status == 4
        prof.dur_ms[:4] = [2, 2, 2, 2]
        prof.mem_MiB[:4] = [50, 60, 70, 80]
        for policy in (0, 1, 2, 3):
            _same(ctx.select(policy, out="host"), oracle_mod.select(prof, z, prof.ready_ms, gaps, policy))
        # a work total that breaks the fairness score bound is reported at select, as after a load
        ctx.update_profile(1, np.full(6, 2**25, np.uint32), np.full(6, 2**32 - 1, np.uint32))
        ctx.advertise(gaps)
        ctx.select(0)
        ctx.select(1)          # work 6 * 2^25 * 2^32 = 2^59.6, times the factor 6: 2^62.2, below 2^63
        ctx.update_profile(1, np.full(6, 2**27, np.uint32), np.full(6, 2**32 - 1, np.uint32))
        ctx.select(0)          # the work itself, 2^61.6, still fits
        with pytest.raises(binding.SjaError) as e:
            ctx.select(1)      # times 6: 2^64.2
        assert e.value.status == 3
