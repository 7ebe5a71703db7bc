"""ctypes wrapper around ``sja_oracle.c`` (the naive walk).  Test infrastructure only."""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sja_oracle.c")
_LIB = os.path.join(_HERE, "libsja_oracle.so")

NO_JOB = 0xFFFFFFFF

GAP_DTYPE = np.dtype(
    [("slice", "<u4"), ("start_ms", "<u4"), ("T_ms", "<u4"), ("C_MiB", "<u4")]
)
AWARD_DTYPE = np.dtype(
    [("job", "<u4"), ("end_step", "<u4"), ("dur_ms", "<u4"), ("granted", "<u4"),
     ("score", "<u8")]
)

_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (-O2 -fopenmp) next to its source."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + f".tmp{os.getpid()}"
    cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-Wall", "-Wextra",
           "-o", tmp, _SRC]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    build()
    lib = ctypes.CDLL(_LIB)
    u32p = ctypes.POINTER(ctypes.c_uint32)
    u64p = ctypes.POINTER(ctypes.c_uint64)
    u8p = ctypes.POINTER(ctypes.c_uint8)
    vp = ctypes.c_void_p
    lib.orc_pair.restype = ctypes.c_int
    lib.orc_pair.argtypes = [vp, vp, vp, ctypes.c_uint64, ctypes.c_uint64, ctypes.c_uint32,
                             ctypes.c_uint32, ctypes.c_uint32, ctypes.c_uint32, ctypes.c_uint32,
                             ctypes.c_uint32, ctypes.c_uint32, ctypes.c_int, ctypes.c_uint32, vp, ctypes.c_uint32,
                             ctypes.c_uint32, u32p, u32p, u64p, u32p]
    lib.orc_select.restype = ctypes.c_int
    lib.orc_select.argtypes = [ctypes.c_uint32, vp, vp, vp, vp, vp, vp, vp, vp,
                               ctypes.c_uint32, vp, ctypes.c_uint32, ctypes.c_uint32, ctypes.c_uint32,
                               ctypes.c_int, vp, vp, vp, ctypes.c_uint32, vp, vp, ctypes.c_uint32, vp]
    lib.orc_commit.restype = ctypes.c_int64
    lib.orc_commit.argtypes = [ctypes.c_uint32, vp, vp, ctypes.c_uint32, vp, vp, ctypes.c_int, vp]
    lib.orc_num_threads.restype = ctypes.c_int
    lib.orc_num_threads.argtypes = []
    del u8p
    _lib = lib
    return lib


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data


def _as(a, dtype):
    if a is None:
        return None
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def num_threads() -> int:
    return int(_load().orc_num_threads())


U32MAX = 0xFFFFFFFF


def pair(prof, j: int, p: int, ready_ms: int, start_ms: int, T_ms: int, C_MiB: int,
         tau_min_ms: int = 0, tau_max_ms: int = U32MAX, late_start: bool = False, deadline_ms: int = U32MAX,
         want_peak: bool = False, power_W: Optional[np.ndarray] = None, power_cap_W: int = U32MAX,
         min_slack_gain_MiB: int = 0):
    """R1-R3 (with the duration thresholds of R2' and the window options of R1'') for one (gap, job)
    pair: ``None`` for decline, else ``(k, dur, work)`` (``(k, dur, work, peak)`` with ``want_peak``).
    ``power_W`` (u32 per step, aligned with the profile arrays) and ``power_cap_W`` switch on R2'';
    ``min_slack_gain_MiB`` > 0 switches on the hysteresis rule R3h."""
    lib = _load()
    k = ctypes.c_uint32()
    dur = ctypes.c_uint32()
    work = ctypes.c_uint64()
    peak = ctypes.c_uint32()
    ok = lib.orc_pair(prof.dur_ms.ctypes.data, prof.mem_MiB.ctypes.data,
                      prof.safe_bits.ctypes.data, int(prof.off[j]), int(prof.off[j + 1]),
                      int(p), int(ready_ms), int(start_ms), int(T_ms), int(C_MiB),
                      int(tau_min_ms), int(tau_max_ms), int(bool(late_start)), int(deadline_ms),
                      _ptr(_as(power_W, np.uint32)), int(power_cap_W), int(min_slack_gain_MiB),
                      ctypes.byref(k), ctypes.byref(dur), ctypes.byref(work), ctypes.byref(peak))
    if not ok:
        return None
    if want_peak:
        return int(k.value), int(dur.value), int(work.value), int(peak.value)
    return int(k.value), int(dur.value), int(work.value)


def select(prof, progress: np.ndarray, ready_ms: np.ndarray, gaps: np.ndarray,
           policy: int, tau_min_ms: int = 0, tau_max_ms: int = U32MAX, late_start: bool = False,
           deadline_ms: Optional[np.ndarray] = None, power_W: Optional[np.ndarray] = None,
           power_cap_W: Optional[np.ndarray] = None, min_slack_gain_MiB: int = 0,
           ckpt_MiB: Optional[np.ndarray] = None, last_slice: Optional[np.ndarray] = None,
           locality_weight: int = 0) -> np.ndarray:
    """R1-R5 for a batch of gaps; returns ``AWARD_DTYPE[G]`` (``granted`` all zero).
    ``late_start`` / ``deadline_ms`` (u32 per job) switch on the window options of R1''; ``power_W`` (u32 per
    step) with ``power_cap_W`` (u32 per gap) the power envelope of R2''; ``min_slack_gain_MiB`` the hysteresis
    rule R3h; ``ckpt_MiB`` / ``last_slice`` (u32 per job) with ``locality_weight`` the locality penalty R4'."""
    lib = _load()
    off = _as(prof.off, np.uint64)
    d = _as(prof.dur_ms, np.uint32)
    m = _as(prof.mem_MiB, np.uint32)
    s = _as(prof.safe_bits, np.uint32)
    progress = _as(progress, np.uint32)
    ready_ms = _as(ready_ms, np.uint32)
    wait = _as(prof.wait_ms, np.uint32)
    prio = _as(prof.prio, np.uint8)
    gaps = np.ascontiguousarray(gaps, dtype=GAP_DTYPE)
    awards = np.zeros(gaps.shape[0], dtype=AWARD_DTYPE)
    deadline = _as(deadline_ms, np.uint32)
    assert deadline is None or deadline.shape[0] == off.shape[0] - 1
    power = _as(power_W, np.uint32)
    caps = _as(power_cap_W, np.uint32)
    assert power is None or power.shape[0] == d.shape[0]
    assert caps is None or caps.shape[0] == gaps.shape[0]
    ckpt = _as(ckpt_MiB, np.uint32)
    last = _as(last_slice, np.uint32)
    assert ckpt is None or ckpt.shape[0] == off.shape[0] - 1
    assert last is None or last.shape[0] == off.shape[0] - 1
    rc = lib.orc_select(off.shape[0] - 1, _ptr(off), _ptr(d), _ptr(m), _ptr(s),
                        _ptr(progress), _ptr(ready_ms), _ptr(wait), _ptr(prio),
                        gaps.shape[0], _ptr(gaps), int(policy), int(tau_min_ms), int(tau_max_ms),
                        int(bool(late_start)), _ptr(deadline), _ptr(power), _ptr(caps), int(min_slack_gain_MiB),
                        _ptr(ckpt), _ptr(last), int(locality_weight), _ptr(awards))
    if rc != 0:
        raise ValueError("oracle select: unknown policy or missing attribute array")
    return awards


def commit(progress: np.ndarray, ready_ms: np.ndarray, gaps: np.ndarray,
           awards: np.ndarray, late_start: bool = False, last_slice: Optional[np.ndarray] = None) -> int:
    """R6, in place on ``progress``, ``ready_ms`` and ``awards['granted']``.  With ``late_start`` a granted
    subjob began at ``max(start, ready)`` (R1''), so that is what the new ready time counts from.  ``last_slice``
    (u32 per job, in place): the slice of the granted gap is recorded for every granted job (R4')."""
    lib = _load()
    assert progress.dtype == np.uint32 and progress.flags.c_contiguous
    assert ready_ms.dtype == np.uint32 and ready_ms.flags.c_contiguous
    assert awards.dtype == AWARD_DTYPE and awards.flags.c_contiguous
    gaps = np.ascontiguousarray(gaps, dtype=GAP_DTYPE)
    assert last_slice is None or (last_slice.dtype == np.uint32 and last_slice.flags.c_contiguous)
    n = lib.orc_commit(progress.shape[0], _ptr(progress), _ptr(ready_ms),
                       gaps.shape[0], _ptr(gaps), _ptr(awards), int(bool(late_start)), _ptr(last_slice))
    if n < 0:
        raise OverflowError("oracle commit: begin + dur does not fit in 32 bits")
    return int(n)


def commit_masked(progress: np.ndarray, ready_ms: np.ndarray, gaps: np.ndarray, awards: np.ndarray,
                  accept: np.ndarray, late_start: bool = False) -> int:
    """R6 restricted to the gaps with ``accept[g] != 0``.

    A subjob that failed or was never started leaves its parent job at the last completed
    fragment (Section 3.10): such a grant is simply not committed.  Gaps that are not accepted take
    no part in R6 (a job that also won an accepted gap is granted that one) and stay ungranted.
    """
    accept = np.asarray(accept).astype(bool)
    visible = awards.copy()
    visible["job"][~accept] = NO_JOB
    n = commit(progress, ready_ms, gaps, visible, late_start)
    awards["granted"] = visible["granted"]
    return n
