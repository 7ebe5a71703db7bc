"""Exhaustive prefix enumeration for tiny inputs -- TEST INFRASTRUCTURE ONLY.

For one (gap, job) pair every end index k in (p, len] is tried; the window sum and the
window maximum are recomputed from scratch for each k (no running state), the candidate
set of Sections 3.1 / 3.8 / 3.9 is filtered literally, and the longest candidate is kept.
This is O(len^2) per pair and is only meant to check the step-by-step walk.
"""
from __future__ import annotations

NO_JOB = 0xFFFFFFFF
_MASK64 = (1 << 64) - 1


def _safe(bits, i: int) -> bool:
    return bool((int(bits[i >> 5]) >> (i & 31)) & 1)


def brute_pair(prof, j: int, p: int, ready_ms: int, start_ms: int, T_ms: int, C_MiB: int,
               tau_min_ms: int = 0, tau_max_ms: int = 0xFFFFFFFF, late_start: bool = False,
               deadline_ms: int = 0xFFFFFFFF, power_W=None, power_cap_W: int = 0xFFFFFFFF,
               min_slack_gain_MiB: int = 0):
    """``None`` (decline) or ``(k, dur, work)`` of the longest feasible subjob.

    Window options: with ``late_start`` the subjob occupies ``[begin, begin + dur)`` with
    ``begin = max(start, ready)`` and has to lie inside the gap ``[start, start + T]``; without it the
    job must be ready when the gap opens.  It has to be over by ``deadline_ms``.  With a per-step power trace
    and a cap, no step of the subjob may draw more than the cap (Section 4.4, item 1).  With
    ``min_slack_gain_MiB`` > 0 (hysteresis, Section 3.9) the job declines when the capacity forces a cut
    earlier than the window alone would allow and that cut sheds less than this much memory demand."""
    s, e = int(prof.off[j]), int(prof.off[j + 1])
    length = e - s
    if p >= length:
        return None
    if start_ms < ready_ms and not late_start:
        return None
    begin = max(start_ms, ready_ms)
    d = [int(x) for x in prof.dur_ms[s:e]]
    m = [int(x) for x in prof.mem_MiB[s:e]]
    candidates = []             # every rule
    window_only = []            # every rule but the memory capacity
    for k in range(p + 1, length + 1):
        ends_safe = _safe(prof.safe_bits, s + k - 1) or k == length
        if not ends_safe:
            continue
        if begin + sum(d[p:k]) > start_ms + T_ms:               # ends inside the gap
            continue
        if deadline_ms != 0xFFFFFFFF and begin + sum(d[p:k]) > deadline_ms:   # Section 4.4 (2): done by the deadline
            continue
        if not (tau_min_ms <= sum(d[p:k]) <= tau_max_ms):      # Section 4.3 (5) thresholds
            continue
        if power_W is not None and power_cap_W != 0xFFFFFFFF and \
                max(int(x) for x in power_W[s + p:s + k]) > power_cap_W:
            continue
        window_only.append(k)
        if max(m[p:k]) > C_MiB:
            continue
        candidates.append(k)
    if not candidates:
        return None
    k = max(candidates)
    if min_slack_gain_MiB > 0:
        k_window = max(window_only)
        if k_window > k and max(m[p:k_window]) - max(m[p:k]) < min_slack_gain_MiB:
            return None         # cutting at k instead of k_window gains too little slack
    dur = sum(d[p:k])
    work = sum(d[i] * m[i] for i in range(p, k))
    return k, dur, work


def brute_select(prof, progress, ready_ms, gaps, policy: int, min_slack_gain_MiB: int = 0, ckpt_MiB=None,
                 last_slice=None, locality_weight: int = 0):
    """Per-gap winner by sorting all interested jobs; returns a list of dicts.  ``ckpt_MiB`` / ``last_slice`` /
    ``locality_weight``: a job whose last fragment ran on another slice than the gap's loses
    ``locality_weight * ckpt_MiB[j]`` of its score, not below zero (Section 4.4, item 5)."""
    out = []
    n_jobs = len(prof.off) - 1
    for g in range(len(gaps)):
        start, T, C = int(gaps["start_ms"][g]), int(gaps["T_ms"][g]), int(gaps["C_MiB"][g])
        entries = []
        for j in range(n_jobs):
            r = brute_pair(prof, j, int(progress[j]), int(ready_ms[j]), start, T, C,
                           min_slack_gain_MiB=min_slack_gain_MiB)
            if r is None:
                continue
            k, dur, work = r
            cls = 0
            score = work
            if policy == 1:
                score = (work * (1 + int(prof.wait_ms[j]) // 1000)) & _MASK64
            elif policy == 2:
                cls = int(prof.prio[j])
            elif policy == 3:
                s0 = int(prof.off[j])
                score = max(int(x) for x in prof.mem_MiB[s0 + int(progress[j]):s0 + k])   # peak of the subjob
            if ckpt_MiB is not None and last_slice is not None and int(last_slice[j]) != 0xFFFFFFFF \
                    and int(last_slice[j]) != int(gaps["slice"][g]):
                score = max(0, score - locality_weight * int(ckpt_MiB[j]))
            # larger class, then larger score, then smaller job id
            entries.append((-cls, -score, j, k, dur, score))
        if not entries:
            out.append(dict(job=NO_JOB, end_step=0, dur_ms=0, score=0))
        else:
            _, _, j, k, dur, score = min(entries)
            out.append(dict(job=j, end_step=k, dur_ms=dur, score=score))
    return out
