"""Full-size trajectories of the published configurations, computed by the CPU oracles only.

TEST INFRASTRUCTURE ONLY.  The streaming configuration (100 000 jobs, 1000 committed rounds of 8192 gaps) is
far beyond what the step-by-step walk finishes in a test run, and the heavy-tailed configuration (16 384 gaps
x 262 144 jobs) takes it minutes.  This module runs them once on the CPU and reduces the results to small
fingerprints that are stored under tests/golden/ (written by tests/golden/make_trajectories.py); the GPU suite
recomputes the same fingerprints from the CUDA path's awards and compares every round.

Who computes what:
  * streaming configuration: the fast oracle (fast_oracle.c) carries all rounds; from its state the walk
    (sja_oracle.c) recomputes select + commit of the sampled rounds (the first ten, every 50th, the last) and
    must agree bit for bit, which also pins the state those rounds started from;
  * heavy-tailed configuration: the walk computes every gap itself; the fast oracle must agree.

A fingerprint is the 64-bit BLAKE2b digest of an array's bytes (awards: the 24-byte records job, end_step,
dur_ms, granted, score in the order the gaps were advertised).
"""
from __future__ import annotations

import hashlib
import time

import numpy as np

from . import api, fast

FORMAT = "blake2b-64 over the little-endian bytes of the array"


def digest(a: np.ndarray) -> str:
    return hashlib.blake2b(np.ascontiguousarray(a).tobytes(), digest_size=8).hexdigest()


def walk_rounds(n_rounds: int) -> list:
    """Rounds the walk recomputes from the fast oracle's state: the first ten, every 50th, the last."""
    return sorted(set(range(min(10, n_rounds))) | set(range(0, n_rounds, 50)) | {n_rounds - 1})


def streaming_trajectory(prof, make_gaps, n_rounds: int, policy: int, check_rounds=None, log=None) -> dict:
    """All ``n_rounds`` committed rounds from progress 0.  ``make_gaps(r)`` gives the batch of round r."""
    check_rounds = walk_rounds(n_rounds) if check_rounds is None else sorted(check_rounds)
    progress = np.zeros(prof.n_jobs, np.uint32)
    ready = prof.ready_ms.copy()
    rounds = []
    total = 0
    t0 = time.time()
    with fast.FastOracle(prof) as fo:
        for r in range(n_rounds):
            gaps = make_gaps(r)
            aw = fo.select(progress, ready, gaps, policy)
            if r in check_rounds:
                p_w, r_w = progress.copy(), ready.copy()
                want = api.select(prof, p_w, r_w, gaps, policy)
                n_w = api.commit(p_w, r_w, gaps, want)
            n = fast.commit(progress, ready, gaps, aw)
            if r in check_rounds:
                if aw.tobytes() != want.tobytes() or n != n_w or not np.array_equal(progress, p_w) \
                        or not np.array_equal(ready, r_w):
                    raise AssertionError(f"round {r}: the fast oracle and the walk disagree")
            rounds.append([int(n), digest(aw)])
            total += n
            if log and (r % 10 == 9 or r in check_rounds):
                log(f"round {r}: {n} grants, {total} so far, {time.time() - t0:.0f} s")
    return {
        "n_rounds": n_rounds, "policy": int(policy), "fingerprint": FORMAT,
        "rounds": rounds, "total_grants": int(total),
        "final_progress": digest(progress), "final_ready": digest(ready),
        "finished_jobs": int((progress.astype(np.int64) == np.diff(prof.off).astype(np.int64)).sum()),
        "walk_checked_rounds": check_rounds,
    }


def single_round(prof, gaps, policy: int, block: int = 256, log=None) -> dict:
    """One round from progress 0, every gap by the walk; the fast oracle has to agree."""
    progress = np.zeros(prof.n_jobs, np.uint32)
    ready = prof.ready_ms.copy()
    t0 = time.time()
    aw = api.select(prof, progress, ready, gaps, policy)
    if log:
        log(f"walk select: {time.time() - t0:.0f} s")
    with fast.FastOracle(prof) as fo:
        other = fo.select(progress, ready, gaps, policy)
    if aw.tobytes() != other.tobytes():
        raise AssertionError("the walk and the fast oracle disagree")
    select_blocks = [digest(aw[i:i + block]) for i in range(0, aw.shape[0], block)]
    select_all = digest(aw)
    n = api.commit(progress, ready, gaps, aw)
    return {
        "policy": int(policy), "fingerprint": FORMAT, "block": block,
        "select": select_all, "select_blocks": select_blocks,
        "winners": int((aw["job"] != api.NO_JOB).sum()),
        "grants": int(n), "committed": digest(aw),
        "final_progress": digest(progress), "final_ready": digest(ready),
    }
