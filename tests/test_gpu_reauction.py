"""GPU parity of the round with re-auction (sja_round_reauction) against the oracle, bit-exact."""
import numpy as np
import pytest

from paper_2509_19086_b200 import workloads as wl

pytestmark = pytest.mark.gpu
FIELDS = ("job", "end_step", "dur_ms", "score", "granted")


def _load(ctx, prof):
    ctx.load_profiles(prof.off, prof.dur_ms, prof.mem_MiB, prof.safe_bits, prof.ready_ms,
                      wait_ms=prof.wait_ms, prio=prof.prio)


def _assert_equal(got, want):
    for f in FIELDS:
        bad = np.nonzero(got[f] != want[f])[0]
        assert bad.size == 0, (f, bad[:5], got[bad[:5]], want[bad[:5]])


@pytest.mark.parametrize("flags", [0, 1, 2, 4])
@pytest.mark.parametrize("base,changes", [
    (1, dict(n_jobs=900, fixed_len=300, n_gaps=300)),
    (2, dict(n_jobs=1500, fixed_len=400, n_gaps=257)),
    (3, dict(n_jobs=2000, zipf_max=2000, n_gaps=200)),
])
def test_reauction_matches_oracle(oracle_mod, base, changes, flags):
    from paper_2509_19086_b200 import binding
    spec = wl.scaled(wl.SPECS[base], **changes)
    prof = wl.make_profiles(spec, threads=2)
    gaps = wl.make_gaps(spec)
    for max_passes in (0, 1, 2):
        progress = np.zeros(prof.n_jobs, np.uint32)
        ready = prof.ready_ms.copy()
        want, n_cpu, k_cpu = oracle_mod.round_with_reauction(prof, progress, ready, gaps, spec.policy, max_passes)
        with binding.Sja() as ctx:
            _load(ctx, prof)
            ctx.advertise(gaps)
            n_gpu, k_gpu = ctx.round_reauction(spec.policy, flags=flags, max_passes=max_passes)
            assert (n_gpu, k_gpu) == (n_cpu, k_cpu)
            _assert_equal(ctx.get_awards(), want)
            p, r = ctx.get_state()
            assert np.array_equal(p, progress) and np.array_equal(r, ready)
        if max_passes == 0:
            assert k_cpu > 1          # the workload really orphans gaps


def test_reauction_streaming_rounds(oracle_mod):
    """Several consecutive rounds, each with re-auction: awards, grant counts and state stay bit-exact."""
    from paper_2509_19086_b200 import binding
    spec = wl.scaled(wl.SPECS[4], n_jobs=1200, fixed_len=250, n_gaps=160, n_rounds=25)
    prof = wl.make_profiles(spec, threads=2)
    progress = np.zeros(prof.n_jobs, np.uint32)
    ready = prof.ready_ms.copy()
    plain_total = reauction_total = 0
    with binding.Sja() as ctx:
        _load(ctx, prof)
        for r in range(spec.n_rounds):
            gaps = wl.make_gaps(spec, r)
            want, n_cpu, k_cpu = oracle_mod.round_with_reauction(prof, progress, ready, gaps, spec.policy)
            ctx.advertise(gaps)
            n_gpu, k_gpu = ctx.round_reauction(spec.policy)
            assert (n_gpu, k_gpu) == (n_cpu, k_cpu)
            _assert_equal(ctx.get_awards(), want)
            reauction_total += n_cpu
        p, rd = ctx.get_state()
        assert np.array_equal(p, progress) and np.array_equal(rd, ready)
    assert reauction_total > spec.n_rounds


def test_reauction_full_size_large_uniform(oracle_mod):
    """65 536 jobs x 4096 gaps (fairness): every pass of the round against the oracle."""
    from paper_2509_19086_b200 import binding
    spec = wl.SPECS[2]
    prof = wl.make_profiles(spec, threads=16)
    gaps = wl.make_gaps(spec)
    progress = np.zeros(prof.n_jobs, np.uint32)
    ready = prof.ready_ms.copy()
    want, n_cpu, k_cpu = oracle_mod.round_with_reauction(prof, progress, ready, gaps, spec.policy)
    with binding.Sja() as ctx:
        _load(ctx, prof)
        ctx.advertise(gaps)
        n_gpu, k_gpu = ctx.round_reauction(spec.policy)
        assert (n_gpu, k_gpu) == (n_cpu, k_cpu)
        _assert_equal(ctx.get_awards(), want)
        p, r = ctx.get_state()
        assert np.array_equal(p, progress) and np.array_equal(r, ready)
    print("re-auction cfg2: grants", n_cpu, "passes", k_cpu, "of", gaps.shape[0], "gaps")
