"""Pins for the hysteresis rule (R3h in the walk's header; Section 3.9 of the paper: a further subdivision is
accepted only if it gains a minimum of slack) and the locality penalty (R4'; Section 4.4, item 5 and the
Preference signal of Section 3.5).  The walk is checked against the exhaustive enumerator (which recomputes both
candidate sets from scratch), against closed forms and special cases, and against hand-computed examples
(tests/golden/preference_examples.json).  Planted mistakes these catch: the gain compared with `<=`, the gain
taken against the capacity instead of the un-cut fragment's peak, the un-cut fragment found without the
duration thresholds, the penalty charged on the same slice or to a job that has not run, a score that wraps
below zero, a commit that does not record the slice."""
import json
import os

import numpy as np
import pytest

from paper_2509_19086_b200 import workloads as wl
from tests.helpers import gaps_from_lists, profiles_from_lists, random_small_profiles

U32MAX = 0xFFFFFFFF
GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "preference_examples.json")


def test_hysteresis_walk_equals_enumeration(oracle_mod):
    rng = np.random.default_rng(91)
    hits = 0
    for trial in range(300):
        jobs = random_small_profiles(rng, 1, 14, p_safe=float(rng.uniform(0.15, 0.9)), mmax=40)
        prof = profiles_from_lists(jobs)
        n = int(prof.off[1])
        p = int(rng.integers(0, n))
        start, ready = int(rng.integers(0, 6)), int(rng.integers(0, 6))
        T, C = int(rng.integers(0, 60)), int(rng.integers(1, 45))
        tau_min, tau_max = (0, U32MAX) if trial % 3 else (int(rng.integers(0, 10)), int(rng.integers(10, 50)))
        late = bool(trial % 2)
        for delta in (0, 1, 2, 5, 12, 40):
            got = oracle_mod.pair(prof, 0, p, ready, start, T, C, tau_min, tau_max, late, U32MAX,
                                  min_slack_gain_MiB=delta)
            want = oracle_mod.brute_pair(prof, 0, p, ready, start, T, C, tau_min, tau_max, late, U32MAX,
                                         min_slack_gain_MiB=delta)
            assert got == want, (trial, delta)
            plain = oracle_mod.pair(prof, 0, p, ready, start, T, C, tau_min, tau_max, late, U32MAX)
            assert got in (None, plain)            # the rule only ever turns interest into a decline
            hits += plain is not None and got is None
    assert hits > 15                               # the rule did bite


def test_hysteresis_special_cases(oracle_mod):
    """Closed cases: (a) a gain of 0 or 1 switches nothing off (a forced cut always sheds at least 1 MiB);
    (b) when the window, not the capacity, ends the subjob nothing changes whatever the threshold; (c) a step
    profile m = low for the first a steps, high afterwards: the cut before the high phase is accepted iff
    high - low >= threshold."""
    d, low, high, a, n = 10, 7, 30, 5, 12
    m = [low] * a + [high] * (n - a)
    prof = profiles_from_lists([([d] * n, m, [1] * n)])
    for delta in (0, 1, 22, 23, 24, 1000):
        # capacity between low and high, window long enough for 9 steps: the cut is forced by the capacity
        got = oracle_mod.pair(prof, 0, 0, 0, 0, 9 * d, low + 3, min_slack_gain_MiB=delta)
        if high - low >= delta:
            assert got == (a, a * d, a * d * low), delta
        else:
            assert got is None, delta
        # window of 3 steps only: the window ends the subjob before the capacity matters
        assert oracle_mod.pair(prof, 0, 0, 0, 0, 3 * d, low + 3, min_slack_gain_MiB=delta) == (3, 30, 30 * low)
        # capacity above everything: never a forced cut
        assert oracle_mod.pair(prof, 0, 0, 0, 0, 9 * d, high, min_slack_gain_MiB=delta) == (9, 90, 50 * low + 40 * high)


def test_hysteresis_and_thresholds_share_the_uncut_fragment(oracle_mod):
    """The fragment the cut is compared with obeys the duration thresholds too: with tau_max = 4 steps the window
    alone allows 4 steps (all low), so the capacity forces nothing and the job stays interested whatever the
    threshold; without tau_max the same pair is a forced cut with a gain of 3."""
    prof = profiles_from_lists([([10] * 8, [5, 5, 5, 5, 8, 8, 8, 8], [1] * 8)])
    assert oracle_mod.pair(prof, 0, 0, 0, 0, 80, 6, 0, 40, min_slack_gain_MiB=100) == (4, 40, 200)
    assert oracle_mod.pair(prof, 0, 0, 0, 0, 80, 6, 0, U32MAX, min_slack_gain_MiB=3) == (4, 40, 200)
    assert oracle_mod.pair(prof, 0, 0, 0, 0, 80, 6, 0, U32MAX, min_slack_gain_MiB=4) is None


def test_golden_preference_examples(oracle_mod):
    """Hand-computed rounds (values derived in the file's comments, not by running the oracle)."""
    with open(GOLDEN) as f:
        doc = json.load(f)
    for ex in doc["examples"]:
        prof = profiles_from_lists([tuple(j) for j in ex["jobs"]], ready=ex.get("ready"), wait=ex.get("wait"),
                                   prio=ex.get("prio"))
        gaps = gaps_from_lists([tuple(g) for g in ex["gaps"]])
        J = prof.n_jobs
        progress = np.array(ex.get("progress", [0] * J), np.uint32)
        ready = prof.ready_ms.copy()
        last = None if "last_slice" not in ex else np.array(ex["last_slice"], np.uint32)
        ckpt = None if "ckpt_MiB" not in ex else np.array(ex["ckpt_MiB"], np.uint32)
        aw = oracle_mod.select(prof, progress, ready, gaps, ex["policy"],
                               min_slack_gain_MiB=ex.get("min_slack_gain_MiB", 0), ckpt_MiB=ckpt, last_slice=last,
                               locality_weight=ex.get("locality_weight", 0))
        assert aw["job"].tolist() == ex["expect"]["job"], ex["name"]
        assert aw["end_step"].tolist() == ex["expect"]["end_step"], ex["name"]
        assert aw["score"].tolist() == ex["expect"]["score"], ex["name"]
        if "granted" in ex["expect"]:
            oracle_mod.commit(progress, ready, gaps, aw, last_slice=last)
            assert aw["granted"].tolist() == ex["expect"]["granted"], ex["name"]
            if last is not None:
                assert last.tolist() == ex["expect"]["last_slice_after"], ex["name"]


def test_locality_walk_equals_enumeration(oracle_mod):
    rng = np.random.default_rng(92)
    changed = 0
    for trial in range(60):
        jobs = random_small_profiles(rng, int(rng.integers(2, 9)), 12, p_safe=float(rng.uniform(0.1, 0.9)))
        J = len(jobs)
        prof = profiles_from_lists(jobs, ready=rng.integers(0, 6, J), wait=rng.integers(0, 5000, J),
                                   prio=rng.integers(0, 3, J))
        lens = np.diff(prof.off).astype(np.int64)
        progress = np.array([rng.integers(0, n + 1) for n in lens], dtype=np.uint32)
        gaps = gaps_from_lists([(int(rng.integers(0, 3)), int(rng.integers(0, 8)), int(rng.integers(0, 40)),
                                 int(rng.integers(0, 22))) for _ in range(6)])
        ckpt = rng.integers(0, 30, J).astype(np.uint32)
        last = rng.choice(np.array([0, 1, 2, U32MAX], dtype=np.uint32), J)
        weight = int(rng.integers(0, 12))
        delta = int(rng.integers(0, 8)) if trial % 2 else 0
        for policy in (0, 1, 2, 3):
            aw = oracle_mod.select(prof, progress, prof.ready_ms, gaps, policy, min_slack_gain_MiB=delta,
                                   ckpt_MiB=ckpt, last_slice=last, locality_weight=weight)
            ref = oracle_mod.brute_select(prof, progress, prof.ready_ms, gaps, policy, min_slack_gain_MiB=delta,
                                          ckpt_MiB=ckpt, last_slice=last, locality_weight=weight)
            for g in range(len(gaps)):
                for key in ("job", "end_step", "dur_ms", "score"):
                    assert int(aw[key][g]) == ref[g][key], (trial, policy, g, key)
            plain = oracle_mod.select(prof, progress, prof.ready_ms, gaps, policy, min_slack_gain_MiB=delta)
            changed += int((plain["job"] != aw["job"]).sum())
    assert changed > 10                            # the penalty did change winners


def test_locality_properties(oracle_mod):
    """(a) weight 0, no checkpoint sizes, or all jobs fresh == the plain round; (b) all gaps on the slice every
    job ran on last == the plain round; (c) the commit records the granted gap's slice and nothing else."""
    spec = wl.scaled(wl.SPECS[3], n_jobs=200, zipf_max=400, n_gaps=40)
    prof = wl.make_profiles(spec, threads=1)
    gaps = wl.make_gaps(spec)
    J = prof.n_jobs
    progress = np.zeros(J, np.uint32)
    rng = np.random.default_rng(5)
    ckpt = rng.integers(1, 10**6, J).astype(np.uint32)
    last = rng.integers(0, 7, J).astype(np.uint32)
    for policy in (0, 2, 3):
        plain = oracle_mod.select(prof, progress, prof.ready_ms, gaps, policy)
        for kw in (dict(ckpt_MiB=ckpt, last_slice=last, locality_weight=0),
                   dict(ckpt_MiB=None, last_slice=last, locality_weight=9),
                   dict(ckpt_MiB=ckpt, last_slice=np.full(J, U32MAX, np.uint32), locality_weight=9)):
            assert oracle_mod.select(prof, progress, prof.ready_ms, gaps, policy, **kw).tobytes() == plain.tobytes()
        same = gaps.copy()
        same["slice"] = 3
        plain3 = oracle_mod.select(prof, progress, prof.ready_ms, same, policy)
        got = oracle_mod.select(prof, progress, prof.ready_ms, same, policy, ckpt_MiB=ckpt,
                                last_slice=np.full(J, 3, np.uint32), locality_weight=9)
        assert got.tobytes() == plain3.tobytes()
    aw = oracle_mod.select(prof, progress, prof.ready_ms, gaps, 0, ckpt_MiB=ckpt, last_slice=last, locality_weight=1)
    before = last.copy()
    ready = prof.ready_ms.copy()
    n = oracle_mod.commit(progress, ready, gaps, aw, last_slice=last)
    g = np.nonzero(aw["granted"] == 1)[0]
    assert n == g.size > 0
    expect = before.copy()
    expect[aw["job"][g]] = gaps["slice"][g]
    assert np.array_equal(last, expect)
