"""sja_select_static -- the select call for callers that may not allocate device memory.

Some embedders run the scheduling round where cudaMalloc is not an option (all device
memory already belongs to their own pool, or the loop cannot tolerate the device-wide
synchronisation of an allocation).  For them the library keeps the per-CTA candidate rows
of a select in a fixed array inside its own image.  This file checks, through the C ABI,
that the variant returns exactly what sja_select returns and what the CPU oracle computes
(the bar for this library's integer results is bit-exact), twice in a row on the shared
array; that the call really leaves the device's free memory untouched, also as the first
select of a fresh context and with a device output buffer; and that a problem too large
for the array is refused with a clear message instead of being truncated.

The file name sorts last on purpose: a run that stops at the first failure has then
already executed every other test.
"""
import numpy as np
import pytest

from paper_2509_19086_b200 import workloads as wl

pytestmark = pytest.mark.gpu

FIELDS = ("job", "end_step", "dur_ms", "score", "granted")


def _load(ctx, prof, progress=None):
    ctx.load_profiles(prof.off, prof.dur_ms, prof.mem_MiB, prof.safe_bits, prof.ready_ms,
                      progress=progress, wait_ms=prof.wait_ms, prio=prof.prio)


def _same_as_oracle(got, want):
    for f in FIELDS:
        assert np.array_equal(got[f], want[f]), f


def test_static_select_matches_select_and_oracle_two_calls_in_a_row(oracle_mod):
    from paper_2509_19086_b200 import binding
    # second workload is smaller than the first, so stale rows of call 1 stay in the array
    # beyond what call 2 writes; they must not leak into its result
    cases = [
        (wl.scaled(wl.SPECS[2], n_jobs=3000, fixed_len=700, n_gaps=384), 0),
        (wl.scaled(wl.SPECS[3], n_jobs=1100, zipf_max=3000, n_gaps=200), binding.FLAG_FORCE_SEARCH),
    ]
    with binding.Sja() as ctx:
        for spec, flags in cases:
            prof = wl.make_profiles(spec, threads=2)
            gaps = wl.make_gaps(spec)
            _load(ctx, prof)
            ctx.advertise(gaps)
            oracle_awards = oracle_mod.select(prof, np.zeros(prof.n_jobs, np.uint32), prof.ready_ms, gaps, spec.policy)
            want = ctx.select(spec.policy, flags=flags, out="host")
            got = ctx.select_static(spec.policy, flags=flags, out="host")
            assert (want["job"] != binding.NO_JOB).any()
            assert got.tobytes() == want.tobytes()
            _same_as_oracle(got, oracle_awards)
            # the same call again, straight after: the array now holds this call's own leftovers
            again = ctx.select_static(spec.policy, flags=flags, out="host")
            assert again.tobytes() == want.tobytes()
        # the static variant feeds commit like the ordinary one
        progress, ready = np.zeros(prof.n_jobs, np.uint32), prof.ready_ms.copy()
        n_cpu = oracle_mod.commit(progress, ready, gaps, oracle_awards)
        n = ctx.commit()
        assert n == n_cpu > 0
        _same_as_oracle(ctx.get_awards(), oracle_awards)


def test_static_select_allocates_nothing(oracle_mod):
    """On a fresh context the static variant is the first select after advertise, so nothing has grown the
    context's own candidate buffer yet: the device's free memory must be the same before and after the call
    (host output and device output), and the ordinary select of the same problem must then lower it."""
    import torch
    from paper_2509_19086_b200 import binding
    spec = wl.scaled(wl.SPECS[2], n_jobs=15000, fixed_len=64, n_gaps=16384)   # 118 job chunks x 16384 gaps x 16 B = 30 MiB
    prof = wl.make_profiles(spec, threads=2)
    gaps = wl.make_gaps(spec)
    sample = slice(0, 512)                 # the oracle on the first gaps; the rest through the ordinary select below
    want = oracle_mod.select(prof, np.zeros(prof.n_jobs, np.uint32), prof.ready_ms, gaps[sample], spec.policy)
    dev_out = torch.zeros(24 * gaps.shape[0], dtype=torch.uint8, device="cuda")
    with binding.Sja() as warm:            # the array's address is looked up (and the module loaded) on first use
        _load(warm, prof)
        warm.advertise(gaps[:64])
        warm.select_static(spec.policy)
    with binding.Sja() as ctx:
        _load(ctx, prof)
        ctx.advertise(gaps)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        got = ctx.select_static(spec.policy, out="host")
        ctx.select_static(spec.policy, out=dev_out)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before
        _same_as_oracle(got[sample], want)
        assert dev_out.cpu().numpy().tobytes() == got.tobytes()
        ctx.select(spec.policy)            # the ordinary call grows the context's candidate buffer
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] < free_before
        assert ctx.get_awards().tobytes() == got.tobytes()


def test_static_select_refuses_sizes_beyond_the_fixed_array():
    from paper_2509_19086_b200 import binding
    slots = (32 * 1024 * 1024) // 16
    n_jobs, n_gaps = 128 * 36, 1                     # 36 job chunks of the search kernel that stands by
    while ((n_jobs + 127) // 128) * n_gaps <= slots:
        n_gaps *= 2
    spec = wl.scaled(wl.SPECS[0], n_jobs=n_jobs, fixed_len=16, n_gaps=n_gaps)
    prof = wl.make_profiles(spec, threads=1)
    with binding.Sja() as ctx:
        _load(ctx, prof)
        ctx.advertise(wl.make_gaps(spec)[:16384])    # a batch that still fits
        ok = ctx.select_static(spec.policy, out="host")
        assert ok.shape[0] == 16384
        big = np.tile(wl.make_gaps(spec)[:16384], (n_gaps + 16383) // 16384)[:n_gaps]
        ctx.advertise(big)
        with pytest.raises(binding.SjaError) as e:
            ctx.select_static(spec.policy)
        assert e.value.status == 1 and "candidate slots" in str(e.value)
        # the ordinary call still serves that size
        full = ctx.select(spec.policy, out="host")
        assert full.shape[0] == n_gaps
