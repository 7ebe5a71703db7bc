"""GPU parity of the subjob duration thresholds (sja_set_duration_bounds) against the oracle."""
import numpy as np
import pytest

from paper_2509_19086_b200 import workloads as wl

pytestmark = pytest.mark.gpu
U32MAX = 0xFFFFFFFF
FIELDS = ("job", "end_step", "dur_ms", "score", "granted")


def _load(ctx, prof):
    ctx.load_profiles(prof.off, prof.dur_ms, prof.mem_MiB, prof.safe_bits, prof.ready_ms,
                      wait_ms=prof.wait_ms, prio=prof.prio)


@pytest.mark.parametrize("base,changes", [
    (1, dict(n_jobs=1100, fixed_len=300, n_gaps=260)),
    (2, dict(n_jobs=1300, fixed_len=500, n_gaps=200)),
    (3, dict(n_jobs=1500, zipf_max=3000, n_gaps=190)),
])
def test_duration_bounds_match_oracle(oracle_mod, base, changes):
    from paper_2509_19086_b200 import binding
    spec = wl.scaled(wl.SPECS[base], **changes)
    prof = wl.make_profiles(spec, threads=2)
    gaps = wl.make_gaps(spec)
    with binding.Sja() as ctx:
        for lo, hi in ((0, U32MAX), (400, U32MAX), (0, 900), (300, 2500), (2000, 2000), (6000, U32MAX)):
            progress = np.zeros(prof.n_jobs, np.uint32)
            ready = prof.ready_ms.copy()
            _load(ctx, prof)
            ctx.set_duration_bounds(lo, hi)
            for rnd in range(2):                      # second round starts from committed state
                want = oracle_mod.select(prof, progress, ready, gaps, spec.policy, lo, hi)
                for flags in (0, 1, 2, 4):
                    ctx.advertise(gaps)
                    got = ctx.select(spec.policy, flags=flags, out="host")
                    for f in FIELDS[:4]:
                        assert np.array_equal(got[f], want[f]), (lo, hi, rnd, flags, f)
                n_gpu = ctx.commit()
                n_cpu = oracle_mod.commit(progress, ready, gaps, want)
                assert n_gpu == n_cpu
                assert np.array_equal(ctx.get_awards()["granted"], want["granted"])
            win = want["job"] != U32MAX
            if win.any():
                assert want["dur_ms"][win].min() >= lo and want["dur_ms"][win].max() <= hi
            if lo == 6000:
                assert not win.any()                  # no window is that long
        with pytest.raises(binding.SjaError) as e:
            ctx.set_duration_bounds(10, 9)
        assert e.value.status == 1


def test_masked_commit_matches_oracle(oracle_mod):
    """sja_commit_masked: grants that are not taken up leave their jobs where they were."""
    from paper_2509_19086_b200 import binding
    spec = wl.scaled(wl.SPECS[4], n_jobs=1400, fixed_len=260, n_gaps=220, n_rounds=12)
    prof = wl.make_profiles(spec, threads=2)
    progress = np.zeros(prof.n_jobs, np.uint32)
    ready = prof.ready_ms.copy()
    rng = np.random.default_rng(12)
    with binding.Sja() as ctx:
        _load(ctx, prof)
        for r in range(spec.n_rounds):
            gaps = wl.make_gaps(spec, r)
            accept = (rng.random(gaps.shape[0]) < 0.7).astype(np.uint8)
            want = oracle_mod.select(prof, progress, ready, gaps, spec.policy)
            n_cpu = oracle_mod.commit_masked(progress, ready, gaps, want, accept)
            ctx.advertise(gaps)
            ctx.select(spec.policy)
            if r % 2:
                import torch
                n_gpu = ctx.commit_masked(torch.from_numpy(accept).cuda())
            else:
                n_gpu = ctx.commit_masked(accept)
            got = ctx.get_awards()
            assert n_gpu == n_cpu
            for f in FIELDS:
                assert np.array_equal(got[f], want[f]), (r, f)
        p, rd = ctx.get_state()
        assert np.array_equal(p, progress) and np.array_equal(rd, ready)
