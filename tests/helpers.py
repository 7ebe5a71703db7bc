"""Small input builders shared by the tests (no method arithmetic here)."""
import numpy as np

from paper_2509_19086_b200 import workloads as wl


def profiles_from_lists(jobs, ready=None, wait=None, prio=None):
    """jobs: list of (d_list, m_list, safe_list) -> workloads.Profiles."""
    lens = [len(j[0]) for j in jobs]
    off = np.zeros(len(jobs) + 1, dtype=np.uint64)
    off[1:] = np.cumsum(lens)
    d = np.array([x for j in jobs for x in j[0]], dtype=np.uint32)
    m = np.array([x for j in jobs for x in j[1]], dtype=np.uint32)
    s = np.array([x for j in jobs for x in j[2]], dtype=np.uint8)
    bits = wl.pack_safe_bits(s) if s.size else np.zeros(0, dtype=np.uint32)
    n = len(jobs)
    ready = np.zeros(n, np.uint32) if ready is None else np.asarray(ready, np.uint32)
    wait = None if wait is None else np.asarray(wait, np.uint32)
    prio = None if prio is None else np.asarray(prio, np.uint8)
    return wl.Profiles(off, d, m, bits, ready, wait, prio)


def gaps_from_lists(rows):
    """rows: list of (slice, start, T, C)."""
    g = np.zeros(len(rows), dtype=wl.GAP_DTYPE)
    for i, (sl, st, T, C) in enumerate(rows):
        g[i] = (sl, st, T, C)
    return g


def random_small_profiles(rng, n_jobs, max_len, p_safe=0.3, dmax=9, mmax=20,
                          allow_zero=False, force_last=True):
    jobs = []
    for _ in range(n_jobs):
        n = int(rng.integers(0 if allow_zero else 1, max_len + 1))
        lo = 0 if allow_zero else 1
        d = rng.integers(lo, dmax + 1, size=n).tolist()
        m = rng.integers(lo, mmax + 1, size=n).tolist()
        s = (rng.random(n) < p_safe).astype(int).tolist()
        if n and force_last:
            s[-1] = 1
        jobs.append((d, m, s))
    return jobs
