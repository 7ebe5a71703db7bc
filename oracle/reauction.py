"""Round with re-auction of orphaned gaps -- TEST INFRASTRUCTURE ONLY.

Greedy slot filling is the intended design (Section 4.2): the scheduler does not look
ahead, it fills each advertised window with an interested job.  When one job wins several
gaps it can materialise only one subjob (one progress point, Sections 3.1 / 3.5), so the
other gaps it won are left without a job although further jobs had signalled interest.
Re-auction repeats the second and third protocol phase (Section 3.5) for exactly those
gaps until nothing changes:

  pass 0   select over all gaps and all jobs, commit (rule R6 of the walk's header);
  pass i   the gaps that had a winner but were not granted are advertised again; jobs that
           were granted a gap earlier in this round decline (one subjob per job and round);
           select, commit;
  stop     when a pass leaves no such gap, grants nothing, or max_passes is reached.

The award of a gap is the one of the last pass it took part in.  The walk itself
(``select`` / ``commit``) is reused as a step; nothing else is added.
"""
from __future__ import annotations

import numpy as np

from .api import AWARD_DTYPE, NO_JOB, commit, select


def round_with_reauction(prof, progress: np.ndarray, ready_ms: np.ndarray, gaps: np.ndarray,
                         policy: int, max_passes: int = 0):
    """Runs the round in place on ``progress`` / ``ready_ms``.

    Returns ``(awards[G], n_granted, n_passes)``.  ``max_passes = 0`` means "until stable".
    """
    n_gaps = gaps.shape[0]
    lens = np.diff(prof.off).astype(np.uint32)
    awards = np.zeros(n_gaps, dtype=AWARD_DTYPE)
    awards["job"] = NO_JOB
    blocked = np.zeros(prof.n_jobs, dtype=bool)
    active = np.arange(n_gaps)
    total = 0
    passes = 0
    while active.size and (max_passes == 0 or passes < max_passes):
        sub = np.ascontiguousarray(gaps[active])
        # a blocked job declines: present it to the walk as finished
        seen_progress = np.where(blocked, lens, progress).astype(np.uint32)
        aw = select(prof, seen_progress, ready_ms, sub, policy)
        n = commit(progress, ready_ms, sub, aw)
        awards[active] = aw
        passes += 1
        total += n
        blocked[aw["job"][aw["granted"] == 1]] = True
        orphan = (aw["job"] != NO_JOB) & (aw["granted"] == 0)
        if n == 0:
            break
        active = active[orphan]
    return awards, total, passes
