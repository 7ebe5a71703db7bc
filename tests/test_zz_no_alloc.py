"""sja_select_static -- the select call for callers that may not allocate device memory.

Some embedders run the scheduling round where cudaMalloc is not an option (all device
memory already belongs to their own pool, or the loop cannot tolerate the device-wide
synchronisation of an allocation).  For them the library keeps the per-CTA candidate rows
of a select in a fixed array inside its own image.  This file checks, through the C ABI,
that the variant returns exactly what sja_select returns (the bar for this library's
integer results is bit-exact), twice in a row on the shared array, and that a problem too
large for the array is refused with a clear message instead of being truncated.

The file name sorts last on purpose: a run that stops at the first failure has then
already executed every other test.
"""
import ctypes

import numpy as np
import pytest

from paper_2509_19086_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _load(ctx, prof, progress=None):
    ctx.load_profiles(prof.off, prof.dur_ms, prof.mem_MiB, prof.safe_bits, prof.ready_ms,
                      progress=progress, wait_ms=prof.wait_ms, prio=prof.prio)


def test_static_select_matches_select_two_calls_in_a_row():
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
            want = ctx.select(spec.policy, flags=flags, out="host")
            got = ctx.select_static(spec.policy, flags=flags, out="host")
            assert (want["job"] != binding.NO_JOB).any()
            assert got.tobytes() == want.tobytes()
            # the same call again, straight after: the array now holds this call's own leftovers
            again = ctx.select_static(spec.policy, flags=flags, out="host")
            assert again.tobytes() == want.tobytes()
        # the static variant feeds commit like the ordinary one
        n = ctx.commit()
        assert n == int((ctx.get_awards()["granted"] == 1).sum()) and n > 0


def test_static_select_refuses_sizes_beyond_the_fixed_array():
    from paper_2509_19086_b200 import binding
    slots = (32 * 1024 * 1024) // 16
    n_jobs, n_gaps = 512 * 9, 1                      # 9 job chunks of the merge kernel
    while ((n_jobs + 511) // 512) * n_gaps <= slots:
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
