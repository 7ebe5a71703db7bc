"""Per-job prefix quantities of the scan step, written out -- TEST INFRASTRUCTURE ONLY.

For a job with steps d[0..len), m[0..len), safe bits s[0..len) and progress p, the scan
step of the round provides, for every end index k in [p, len]:

    D[k] = sum_{p <= i < k} d[i]            cumulative duration of the window [p, k)
    M[k] = max_{p <= i < k} m[i]            running maximum of the memory envelope U
                                            (the window-max test of Section 3.9)
    L[k] = largest safe end index <= k      (0 if there is none above p); a subjob may
                                            only end at such an index (Section 3.7)
    W[k] = sum_{p <= i < k} d[i] * m[i]     prefix work, the efficiency score

``dense_prefix`` returns these four arrays (library cumsum / maximum.accumulate serve as
steps).  ``boundary_table`` lists only the safe end indices above p, with the same
quantities and the maximum of m over the segment since the previous boundary; that is
the subset of the dense arrays a feasibility search can ever return.
"""
from __future__ import annotations

import numpy as np


def _job_slices(prof, j: int):
    s, e = int(prof.off[j]), int(prof.off[j + 1])
    d = prof.dur_ms[s:e].astype(np.uint64)
    m = prof.mem_MiB[s:e].astype(np.uint64)
    idx = np.arange(s, e, dtype=np.uint64)
    safe = ((prof.safe_bits[(idx >> np.uint64(5)).astype(np.int64)]
             >> (idx & np.uint64(31)).astype(np.uint32)) & 1).astype(bool)
    if e > s:
        safe[-1] = True     # the end of a job is always a boundary
    return d, m, safe


def dense_prefix(prof, j: int, p: int = 0):
    """D, M, L, W for k = p..len (arrays of length len - p + 1, entry 0 is k = p)."""
    d, m, safe = _job_slices(prof, j)
    d, m, safe = d[p:], m[p:], safe[p:]
    n = d.shape[0]
    D = np.zeros(n + 1, dtype=np.uint64)
    W = np.zeros(n + 1, dtype=np.uint64)
    M = np.zeros(n + 1, dtype=np.uint64)
    L = np.zeros(n + 1, dtype=np.uint64)
    if n:
        D[1:] = np.cumsum(d)
        W[1:] = np.cumsum(d * m)
        M[1:] = np.maximum.accumulate(m)
        ends = np.where(safe, np.arange(p + 1, p + n + 1, dtype=np.uint64), 0)
        L[1:] = np.maximum.accumulate(ends)
    return D, M, L, W


def boundary_table(prof, j: int, p: int = 0):
    """Rows (k, D[k], M[k], segmax, W[k]) for every safe end index k > p, ascending."""
    d, m, safe = _job_slices(prof, j)
    D, M, L, W = dense_prefix(prof, j, p)
    n = d.shape[0] - p
    ks = [p + i + 1 for i in range(n) if safe[p + i]]
    rows = []
    prev = p
    for k in ks:
        seg = int(m[prev:k].max())
        rows.append((k, int(D[k - p]), int(M[k - p]), seg, int(W[k - p])))
        prev = k
    return rows
