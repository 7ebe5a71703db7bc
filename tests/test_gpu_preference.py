"""GPU parity for the hysteresis rule (Section 3.9) and the locality / checkpoint-size penalty (Section 4.4,
item 5; Preference signal of Section 3.5): the CUDA library through its C ABI against the CPU oracle, bit for bit,
on hand-computed examples, tiny random rounds, and committed rounds of scaled configurations (with the other
per-pair options mixed in)."""
import json
import os

import numpy as np
import pytest

from paper_2509_19086_b200 import workloads as wl
from tests.helpers import gaps_from_lists, profiles_from_lists, random_small_profiles

pytestmark = pytest.mark.gpu

U32MAX = 0xFFFFFFFF
FIELDS = ("job", "end_step", "dur_ms", "score")
GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "preference_examples.json")


def _load(ctx, prof, progress=None):
    ctx.load_profiles(prof.off, prof.dur_ms, prof.mem_MiB, prof.safe_bits, prof.ready_ms,
                      progress=progress, wait_ms=prof.wait_ms, prio=prof.prio)


def _same(got, want, fields=FIELDS, ctx=None):
    for f in fields:
        bad = np.nonzero(got[f] != want[f])[0]
        assert bad.size == 0, (ctx, f, bad[:5], got[bad[:5]], want[bad[:5]])


def test_golden_examples_on_the_gpu():
    from paper_2509_19086_b200 import binding
    with open(GOLDEN) as f:
        doc = json.load(f)
    with binding.Sja() as ctx:
        for ex in doc["examples"]:
            prof = profiles_from_lists([tuple(j) for j in ex["jobs"]], ready=ex.get("ready"), wait=ex.get("wait"),
                                       prio=ex.get("prio"))
            gaps = gaps_from_lists([tuple(g) for g in ex["gaps"]])
            _load(ctx, prof, np.array(ex.get("progress", [0] * prof.n_jobs), np.uint32))
            ctx.set_hysteresis(ex.get("min_slack_gain_MiB", 0))
            if "ckpt_MiB" in ex:
                ctx.set_locality(np.array(ex["ckpt_MiB"], np.uint32), np.array(ex["last_slice"], np.uint32),
                                 ex["locality_weight"])
            ctx.advertise(gaps)
            aw = ctx.select(ex["policy"], out="host")
            assert aw["job"].tolist() == ex["expect"]["job"], ex["name"]
            assert aw["end_step"].tolist() == ex["expect"]["end_step"], ex["name"]
            assert aw["score"].tolist() == ex["expect"]["score"], ex["name"]
            if "granted" in ex["expect"]:
                ctx.commit()
                assert ctx.get_awards()["granted"].tolist() == ex["expect"]["granted"], ex["name"]
                if "ckpt_MiB" in ex:
                    assert ctx.get_locality().tolist() == ex["expect"]["last_slice_after"], ex["name"]
        ctx.set_hysteresis(0)


def test_tiny_random_rounds(oracle_mod):
    from paper_2509_19086_b200 import binding
    rng = np.random.default_rng(2024)
    with binding.Sja() as ctx:
        for trial in range(40):
            jobs = random_small_profiles(rng, int(rng.integers(1, 40)), 30, p_safe=float(rng.uniform(0.1, 0.9)),
                                         mmax=40, allow_zero=(trial % 4 == 0))
            J = len(jobs)
            prof = profiles_from_lists(jobs, ready=rng.integers(0, 6, J), wait=rng.integers(0, 5000, J),
                                       prio=rng.integers(0, 3, J))
            lens = np.diff(prof.off).astype(np.int64)
            progress = np.array([rng.integers(0, n + 1) for n in lens], dtype=np.uint32)
            gaps = gaps_from_lists([(int(rng.integers(0, 3)), int(rng.integers(0, 8)), int(rng.integers(0, 90)),
                                     int(rng.integers(0, 45))) for _ in range(int(rng.integers(1, 70)))])
            delta = int(rng.integers(0, 25)) if trial % 3 else 0
            ckpt = rng.integers(0, 60, J).astype(np.uint32) if trial % 2 else None
            last = rng.choice(np.array([0, 1, 2, U32MAX], dtype=np.uint32), J) if trial % 4 != 3 else None
            weight = int(rng.integers(0, 9))
            late = trial % 5 == 0
            _load(ctx, prof, progress)
            ctx.set_hysteresis(delta)
            ctx.set_locality(ckpt, last, weight)
            ctx.set_window_options(late, None)
            ctx.advertise(gaps)
            for policy in (0, 1, 2, 3):
                got = ctx.select(policy, out="host")
                want = oracle_mod.select(prof, progress, prof.ready_ms, gaps, policy, late_start=late,
                                         min_slack_gain_MiB=delta, ckpt_MiB=ckpt,
                                         last_slice=last if ckpt is None or last is not None else np.full(J, U32MAX, np.uint32),
                                         locality_weight=weight)
                _same(got, want, ctx=(trial, policy))
        ctx.set_hysteresis(0)
        ctx.set_window_options(False, None)


@pytest.mark.parametrize("index,scale", [(2, dict(n_jobs=3000, fixed_len=700, n_gaps=384)),
                                         (3, dict(n_jobs=2500, zipf_max=3000, n_gaps=300)),
                                         (4, dict(n_jobs=2000, fixed_len=500, n_gaps=256, n_rounds=8))])
def test_committed_rounds_on_scaled_configs(oracle_mod, index, scale):
    """Eight committed rounds with both rules on: awards, grants, progress, ready times and last slices follow the
    oracle; the rules must also have changed something against the plain round (else the test proves nothing)."""
    from paper_2509_19086_b200 import binding
    spec = wl.scaled(wl.SPECS[index], **scale)
    prof = wl.make_profiles(spec, threads=2)
    J = prof.n_jobs
    rng = np.random.default_rng(7 + index)
    ckpt = rng.integers(0, 4000, J).astype(np.uint32)
    last = rng.choice(np.array([0, 1, 2, 3, 4, 5, 6, U32MAX], dtype=np.uint32), J).astype(np.uint32)
    weight, delta = 37, 6000
    progress = np.zeros(J, np.uint32)
    ready = prof.ready_ms.copy()
    differs = 0
    with binding.Sja() as ctx:
        _load(ctx, prof)
        ctx.set_hysteresis(delta)
        ctx.set_locality(ckpt, last, weight)
        for r in range(8):
            gaps = wl.make_gaps(spec, r)
            if spec.n_rounds == 1:
                gaps["start_ms"] += np.uint32(1500 * r)
            ctx.advertise(gaps)
            got = ctx.select(spec.policy, out="host")
            want = oracle_mod.select(prof, progress, ready, gaps, spec.policy, min_slack_gain_MiB=delta, ckpt_MiB=ckpt,
                                     last_slice=last, locality_weight=weight)
            _same(got, want, ctx=(spec.name, r))
            plain = oracle_mod.select(prof, progress, ready, gaps, spec.policy)
            differs += int((plain["job"] != want["job"]).sum() + (plain["end_step"] != want["end_step"]).sum())
            n_gpu = ctx.commit()
            n_cpu = oracle_mod.commit(progress, ready, gaps, want, last_slice=last)
            assert n_gpu == n_cpu
            _same(ctx.get_awards(), want, FIELDS + ("granted",), ctx=(spec.name, r, "commit"))
            p, rd = ctx.get_state()
            assert np.array_equal(p, progress) and np.array_equal(rd, ready)
            assert np.array_equal(ctx.get_locality(), last)
        assert differs > 0
        # re-auction takes the same kernels: one more round through it
        gaps = wl.make_gaps(spec, 9)
        gaps["start_ms"] += np.uint32(20000)
        ctx.advertise(gaps)
        n_gpu, passes = ctx.round_reauction(spec.policy)
        assert passes >= 1 and n_gpu == int((ctx.get_awards()["granted"] == 1).sum())


def test_rules_off_is_the_plain_round_and_state_rules(oracle_mod):
    """Threshold 0 and no checkpoint sizes give the plain round bit for bit (through the default kernel); a new
    load drops the locality arrays; get_locality without set_locality is a call-order error."""
    from paper_2509_19086_b200 import binding
    spec = wl.scaled(wl.SPECS[1], n_jobs=900, fixed_len=300, n_gaps=200)
    prof = wl.make_profiles(spec, threads=1)
    gaps = wl.make_gaps(spec)
    zero = np.zeros(prof.n_jobs, np.uint32)
    with binding.Sja() as ctx:
        _load(ctx, prof)
        with pytest.raises(binding.SjaError) as e:
            ctx.get_locality()
        assert e.value.status == 4
        ctx.set_hysteresis(0)
        ctx.set_locality(None, None, 5)
        ctx.advertise(gaps)
        want = oracle_mod.select(prof, zero, prof.ready_ms, gaps, spec.policy)
        _same(ctx.select(spec.policy, out="host"), want)
        ctx.set_locality(np.ones(prof.n_jobs, np.uint32), None, 5)
        assert (ctx.get_locality() == U32MAX).all()
        with pytest.raises(binding.SjaError) as e:
            ctx.commit()                       # the select was discarded by set_locality
        assert e.value.status == 4
        _load(ctx, prof)
        with pytest.raises(binding.SjaError):
            ctx.get_locality()
