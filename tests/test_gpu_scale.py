"""Full-size published configurations on the GPU, in the launch configuration bench.py times.

Where the oracle finishes in seconds it is run here in full.  For the two largest configurations every award
of every round is compared with results the CPU oracles computed beforehand (fingerprints stored under
tests/golden/, written by tests/golden/make_trajectories.py), and sampled gaps / rounds are recomputed by the
walk in the test itself.  No expected value comes from the CUDA path.
"""
import json
import os

import numpy as np
import pytest

from paper_2509_19086_b200 import workloads as wl

pytestmark = pytest.mark.gpu

U32MAX = 0xFFFFFFFF
GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
FIELDS = ("job", "end_step", "dur_ms", "score")


def _load(ctx, prof):
    ctx.load_profiles(prof.off, prof.dur_ms, prof.mem_MiB, prof.safe_bits, prof.ready_ms,
                      wait_ms=prof.wait_ms, prio=prof.prio)


def _assert_equal(got, want, fields=FIELDS):
    for f in fields:
        bad = np.nonzero(got[f] != want[f])[0]
        assert bad.size == 0, (f, bad[:5], got[bad[:5]], want[bad[:5]])


def test_cfg2_large_uniform_all_awards(oracle_mod):
    """65 536 jobs x 4096 steps, 4096 gaps, fairness: every award against the oracle."""
    from paper_2509_19086_b200 import binding
    spec = wl.SPECS[2]
    prof = wl.make_profiles(spec, threads=16)
    gaps = wl.make_gaps(spec)
    with binding.Sja() as ctx:
        _load(ctx, prof)
        safe = wl.unpack_safe_bits(prof.safe_bits, prof.n_steps)
        assert ctx.scan_size() == int(safe.sum())
        ctx.advertise(gaps)
        got = ctx.select(spec.policy, out="host")
        progress = np.zeros(prof.n_jobs, np.uint32)
        ready = prof.ready_ms.copy()
        want = oracle_mod.select(prof, progress, ready, gaps, spec.policy)
        _assert_equal(got, want)
        n_gpu = ctx.commit()
        n_cpu = oracle_mod.commit(progress, ready, gaps, want)
        assert n_gpu == n_cpu > 0
        _assert_equal(ctx.get_awards(), want, FIELDS + ("granted",))
        p, r = ctx.get_state()
        assert np.array_equal(p, progress) and np.array_equal(r, ready)
        # the per-pair search kernel on a sample of the gaps
        sub = gaps[::16]
        ctx.advertise(sub)
        want = oracle_mod.select(prof, progress, ready, sub, spec.policy)
        _assert_equal(ctx.select(spec.policy, flags=binding.FLAG_FORCE_SEARCH, out="host"), want)
        # and the per-gap merge kernel
        _assert_equal(ctx.select(spec.policy, flags=binding.FLAG_FORCE_MERGE, out="host"), want)


def _golden(name):
    with open(os.path.join(GOLDEN, name)) as f:
        return json.load(f)


def test_cfg3_heavy_tailed_every_gap(oracle_mod):
    """262 144 ragged jobs (about 1e9 steps), 16 384 gaps, SLA.  Every award, the grants and the state after the
    commit are compared with the stored results of the CPU oracles (tests/golden/trajectory_cfg3.json, written
    by tests/golden/make_trajectories.py: every gap computed by the step-by-step walk) through 64-bit
    fingerprints, per block of 256 gaps so that a mismatch is located; 1024 sampled gaps are also recomputed
    by the walk here, and every award is re-derived structurally from the raw arrays."""
    from oracle import trajectory
    from paper_2509_19086_b200 import binding
    gold = _golden("trajectory_cfg3.json")
    spec = wl.SPECS[3]
    prof = wl.make_profiles(spec, threads=16)
    gaps = wl.make_gaps(spec)
    assert (gold["seed"], gold["jobs"], gold["steps_total"]) == (spec.seed, prof.n_jobs, prof.n_steps)
    assert 0.8e9 < prof.n_steps < 1.2e9
    with binding.Sja() as ctx:
        _load(ctx, prof)
        ctx.advertise(gaps)
        got = ctx.select(spec.policy, out="host")
        block = gold["block"]
        blocks = [trajectory.digest(got[i:i + block]) for i in range(0, got.shape[0], block)]
        bad = [i for i, (a, b) in enumerate(zip(blocks, gold["select_blocks"])) if a != b]
        assert not bad and len(blocks) == len(gold["select_blocks"]), ("gap blocks that differ from the oracle", bad[:8])
        assert trajectory.digest(got) == gold["select"]
        assert int((got["job"] != U32MAX).sum()) == gold["winners"]
        progress = np.zeros(prof.n_jobs, np.uint32)
        rng = np.random.default_rng(33)
        sample = np.sort(rng.choice(gaps.shape[0], 1024, replace=False))
        want = oracle_mod.select(prof, progress, prof.ready_ms, gaps[sample], spec.policy)
        _assert_equal(got[sample], want)
        # the other select kernel agrees on every gap
        assert ctx.select(spec.policy, flags=binding.FLAG_FORCE_MERGE, out="host").tobytes() == got.tobytes()
        # every award: winner eligible, subjob inside the job, ends on a boundary, fits T
        win = got["job"] != U32MAX
        assert win.mean() > 0.9
        j = got["job"][win].astype(np.int64)
        k = got["end_step"][win].astype(np.int64)
        lens = np.diff(prof.off).astype(np.int64)
        assert (k >= 1).all() and (k <= lens[j]).all()
        last = prof.off[j].astype(np.int64) + k - 1
        bit = (prof.safe_bits[last >> 5] >> (last & 31).astype(np.uint32)) & 1
        assert ((bit == 1) | (k == lens[j])).all()
        assert (got["dur_ms"][win] <= gaps["T_ms"][win]).all()
        assert (gaps["start_ms"][win] >= prof.ready_ms[j]).all()
        n = ctx.commit()
        aw = ctx.get_awards()
        assert n == gold["grants"]
        assert trajectory.digest(aw) == gold["committed"]
        p, rd = ctx.get_state()
        assert trajectory.digest(p) == gold["final_progress"] and trajectory.digest(rd) == gold["final_ready"]


def test_cfg4_streaming_1000_rounds(oracle_mod):
    """100 000 jobs x 2048 steps, 1000 committed rounds of 8192 gaps.  Every round's awards (job, end step,
    duration, score, granted flag) and grant count, and the final progress pointers and ready times, are
    compared with the stored trajectory of the CPU oracles (tests/golden/trajectory_cfg4.json: all rounds by
    the prefix-array oracle, the first ten, every 50th and the last recomputed by the step-by-step walk from
    that state).  On top of that: rounds 0-2 in full and 256 gaps of sampled later rounds are recomputed by the
    walk right here from the library's own state, and every grant of every round is re-derived from the raw
    arrays (fits T and C, ends on a boundary, is maximal, starts at the job's progress point)."""
    from oracle import trajectory
    from paper_2509_19086_b200 import binding
    gold = _golden("trajectory_cfg4.json")
    spec = wl.SPECS[4]
    prof = wl.make_profiles(spec, threads=16)
    J = prof.n_jobs
    assert (gold["seed"], gold["jobs"], gold["n_rounds"]) == (spec.seed, J, spec.n_rounds)
    off = prof.off.astype(np.int64)
    cum_d = np.zeros(prof.n_steps + 1, dtype=np.int64)
    np.cumsum(prof.dur_ms, out=cum_d[1:])
    safe = wl.unpack_safe_bits(prof.safe_bits, prof.n_steps)
    # next safe end index at or after each step (within the concatenated arrays; the end of a job is one)
    nxt = np.where(safe == 1, np.arange(1, prof.n_steps + 1, dtype=np.int64), np.int64(1) << 62)
    nxt = np.minimum.accumulate(nxt[::-1])[::-1]
    o_progress = np.zeros(J, np.uint32)
    o_ready = prof.ready_ms.copy()
    replay_p = np.zeros(J, np.int64)
    replay_r = prof.ready_ms.astype(np.int64)
    total = 0
    mismatched = []
    rng = np.random.default_rng(44)
    with binding.Sja() as ctx:
        _load(ctx, prof)
        for r in range(spec.n_rounds):
            gaps = wl.make_gaps(spec, r)
            sampled = r == 10 or (r % 100 == 0 and r > 0) or r == spec.n_rounds - 1
            if sampled:
                state_p, state_r = ctx.get_state()
            ctx.advertise(gaps)
            ctx.select(spec.policy)
            if r % 100 == 50:
                # late rounds (jobs partly consumed, ready times spread out): both ordered-gap kernels agree
                a = ctx.select(spec.policy, flags=binding.FLAG_FORCE_MERGE, out="host")
                b = ctx.select(spec.policy, out="host")
                assert a.tobytes() == b.tobytes(), r
            n = ctx.commit()
            aw = ctx.get_awards()
            if (n, trajectory.digest(aw)) != (gold["rounds"][r][0], gold["rounds"][r][1]):
                mismatched.append(r)
            assert len(mismatched) == 0, ("first rounds that differ from the oracle trajectory", mismatched)
            if r < 3:
                want = oracle_mod.select(prof, o_progress, o_ready, gaps, spec.policy)
                n_cpu = oracle_mod.commit(o_progress, o_ready, gaps, want)
                _assert_equal(aw, want, FIELDS + ("granted",))
                assert n == n_cpu
                p, rd = ctx.get_state()
                assert np.array_equal(p, o_progress) and np.array_equal(rd, o_ready)
            if sampled:
                # the walk from the library's state before this round, on 256 of its gaps against all jobs
                pick = np.sort(rng.choice(gaps.shape[0], 256, replace=False))
                want = oracle_mod.select(prof, state_p, state_r, gaps[pick], spec.policy)
                _assert_equal(aw[pick], want)
            # every grant of the round, re-derived from the raw arrays
            g = np.nonzero(aw["granted"] == 1)[0]
            assert g.size == n
            j = aw["job"][g].astype(np.int64)
            k = aw["end_step"][g].astype(np.int64)
            assert np.unique(j).size == j.size                       # one grant per job and round
            assert (k > replay_p[j]).all() and (k <= 2048).all()     # progress moves forward
            dur = cum_d[off[j] + k] - cum_d[off[j] + replay_p[j]]
            assert (dur == aw["dur_ms"][g]).all()                    # subjob starts at the job's progress
            assert (dur <= gaps["T_ms"][g]).all()
            assert (gaps["start_ms"][g] >= replay_r[j]).all()
            last = off[j] + k - 1
            assert ((safe[last] == 1) | (k == 2048)).all()           # every cut is a safe boundary
            C = gaps["C_MiB"][g].astype(np.int64)
            T = gaps["T_ms"][g].astype(np.int64)
            for i in range(g.size):                                  # window maximum <= C, and the subjob is maximal
                a0, a1 = off[j[i]] + replay_p[j[i]], off[j[i]] + k[i]
                peak = int(prof.mem_MiB[a0:a1].max())
                assert peak <= C[i]
                if k[i] < 2048:
                    k2 = min(int(nxt[a1]), int(off[j[i] + 1]))       # the next boundary: breaks T or C
                    d2 = cum_d[k2] - cum_d[a0]
                    m2 = max(peak, int(prof.mem_MiB[a1:k2].max()))
                    assert d2 > T[i] or m2 > C[i], (r, int(g[i]))
            winners = np.unique(aw["job"][aw["job"] != U32MAX])
            assert np.array_equal(winners, np.sort(j))               # every winning job gets exactly one gap
            replay_p[j] = k
            replay_r[j] = gaps["start_ms"][g].astype(np.int64) + dur
            total += n
        p, rd = ctx.get_state()
        assert np.array_equal(p.astype(np.int64), replay_p)
        assert np.array_equal(rd.astype(np.int64), replay_r)
        assert trajectory.digest(p) == gold["final_progress"] and trajectory.digest(rd) == gold["final_ready"]
        assert total == gold["total_grants"]
        print("cfg4 grants over 1000 rounds:", total)
        assert total > 50_000


@pytest.mark.parametrize("case", ["many_classes", "equal_T", "equal_ready_and_start", "unbounded_T", "late_progress",
                                  "ragged_counts"])
def test_select_kernels_agree_on_structured_batches(oracle_mod, case):
    """Batches built to stress the ordered-gap kernels (runs of one gap, a single run, one eligibility prefix for
    everybody, windows longer than any job, cursors that start deep inside the jobs, counts that are not multiples
    of anything): tile, merge and search kernels give identical awards, and 200 sampled gaps match the oracle."""
    from paper_2509_19086_b200 import binding
    rng = np.random.default_rng(7000 + sum(map(ord, case)))
    n_jobs, n_gaps = (20011, 1999) if case == "ragged_counts" else (20000, 2000)
    spec = wl.scaled(wl.SPECS[3], n_jobs=n_jobs, zipf_max=4000, n_gaps=n_gaps)
    prof = wl.make_profiles(spec, threads=8)
    gaps = wl.make_gaps(spec)
    progress = np.zeros(prof.n_jobs, np.uint32)
    ready = prof.ready_ms.copy()
    if case == "many_classes":
        gaps["C_MiB"] = rng.choice(np.arange(2000, 82000, 700), n_gaps)          # 115 capacities, runs of ~17 gaps
    elif case == "equal_T":
        gaps["T_ms"] = 1234
    elif case == "equal_ready_and_start":
        ready[:] = 500
        gaps["start_ms"] = rng.choice([499, 500], n_gaps)
    elif case == "unbounded_T":
        gaps["T_ms"] = U32MAX
        gaps["start_ms"] = 1000
    elif case == "late_progress":
        lens = np.diff(prof.off).astype(np.int64)
        progress = (lens * rng.uniform(0.0, 1.0, prof.n_jobs)).astype(np.uint32)
    with binding.Sja() as ctx:
        ctx.load_profiles(prof.off, prof.dur_ms, prof.mem_MiB, prof.safe_bits, ready,
                          progress=progress, wait_ms=prof.wait_ms, prio=prof.prio)
        ctx.advertise(gaps)
        for policy in (0, 2, 3):
            tile = ctx.select(policy, flags=binding.FLAG_FORCE_TILE, out="host")
            assert ctx.select(policy, flags=binding.FLAG_FORCE_MERGE, out="host").tobytes() == tile.tobytes(), policy
            assert ctx.select(policy, flags=binding.FLAG_FORCE_SEARCH, out="host").tobytes() == tile.tobytes(), policy
            sample = np.sort(rng.choice(n_gaps, 200, replace=False))
            want = oracle_mod.select(prof, progress, ready, gaps[sample], policy)
            _assert_equal(tile[sample], want)
