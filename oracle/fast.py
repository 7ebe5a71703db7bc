"""ctypes wrapper around ``fast_oracle.c`` (prefix arrays + binary search).  Test infrastructure only.

The second CPU oracle: same round as the walk (``api.py``), written separately, fast enough to carry the
1000-round streaming configuration.  It is pinned against the walk and the exhaustive enumerator in
``tests/test_oracle_fast_pins.py``; ``trajectory.py`` uses it to write the stored trajectories.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

from .api import AWARD_DTYPE, GAP_DTYPE

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fast_oracle.c")
_LIB = os.path.join(_HERE, "libsja_oracle_fast.so")

_lib = None


def build(force: bool = False) -> str:
    """Compile the fast oracle with gcc (-O2 -fopenmp) next to its source."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + f".tmp{os.getpid()}"
    cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-Wall", "-Wextra", "-o", tmp, _SRC]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    build()
    lib = ctypes.CDLL(_LIB)
    vp, u32 = ctypes.c_void_p, ctypes.c_uint32
    lib.o3_create.restype = vp
    lib.o3_create.argtypes = [u32, vp, vp, vp, vp]
    lib.o3_destroy.restype = None
    lib.o3_destroy.argtypes = [vp]
    lib.o3_select.restype = ctypes.c_int
    lib.o3_select.argtypes = [vp, vp, vp, vp, vp, u32, vp, u32, vp]
    lib.o3_commit.restype = ctypes.c_int64
    lib.o3_commit.argtypes = [u32, vp, vp, u32, vp, vp]
    lib.o3_num_threads.restype = ctypes.c_int
    lib.o3_num_threads.argtypes = []
    _lib = lib
    return lib


def num_threads() -> int:
    return int(_load().o3_num_threads())


class FastOracle:
    """Prefix arrays of one set of job profiles; ``select`` / ``commit`` as in ``oracle.api``."""

    def __init__(self, prof):
        self._lib = _load()
        # the C side keeps pointers to off and mem_MiB: hold the arrays
        self._off = np.ascontiguousarray(prof.off, dtype=np.uint64)
        self._d = np.ascontiguousarray(prof.dur_ms, dtype=np.uint32)
        self._m = np.ascontiguousarray(prof.mem_MiB, dtype=np.uint32)
        self._s = np.ascontiguousarray(prof.safe_bits, dtype=np.uint32)
        self._wait = None if prof.wait_ms is None else np.ascontiguousarray(prof.wait_ms, dtype=np.uint32)
        self._prio = None if prof.prio is None else np.ascontiguousarray(prof.prio, dtype=np.uint8)
        self.n_jobs = int(self._off.shape[0] - 1)
        self._h = self._lib.o3_create(self.n_jobs, self._off.ctypes.data, self._d.ctypes.data,
                                      self._m.ctypes.data, self._s.ctypes.data)
        if not self._h:
            raise MemoryError("fast oracle: could not allocate the prefix arrays")

    def close(self) -> None:
        if getattr(self, "_h", None):
            self._lib.o3_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def select(self, progress: np.ndarray, ready_ms: np.ndarray, gaps: np.ndarray, policy: int) -> np.ndarray:
        """R1-R5 for a batch of gaps; returns ``AWARD_DTYPE[G]`` (``granted`` all zero)."""
        progress = np.ascontiguousarray(progress, dtype=np.uint32)
        ready_ms = np.ascontiguousarray(ready_ms, dtype=np.uint32)
        gaps = np.ascontiguousarray(gaps, dtype=GAP_DTYPE)
        assert progress.shape[0] == self.n_jobs and ready_ms.shape[0] == self.n_jobs
        awards = np.zeros(gaps.shape[0], dtype=AWARD_DTYPE)
        rc = self._lib.o3_select(self._h, progress.ctypes.data, ready_ms.ctypes.data,
                                 None if self._wait is None else self._wait.ctypes.data,
                                 None if self._prio is None else self._prio.ctypes.data,
                                 gaps.shape[0], gaps.ctypes.data, int(policy), awards.ctypes.data)
        if rc == -1:
            raise ValueError("fast oracle select: unknown policy or missing attribute array")
        if rc != 0:
            raise MemoryError("fast oracle select: out of memory")
        return awards


def commit(progress: np.ndarray, ready_ms: np.ndarray, gaps: np.ndarray, awards: np.ndarray) -> int:
    """R6, in place on ``progress``, ``ready_ms`` and ``awards['granted']``."""
    lib = _load()
    assert progress.dtype == np.uint32 and progress.flags.c_contiguous
    assert ready_ms.dtype == np.uint32 and ready_ms.flags.c_contiguous
    assert awards.dtype == AWARD_DTYPE and awards.flags.c_contiguous
    gaps = np.ascontiguousarray(gaps, dtype=GAP_DTYPE)
    n = lib.o3_commit(progress.shape[0], progress.ctypes.data, ready_ms.ctypes.data, gaps.shape[0],
                      gaps.ctypes.data, awards.ctypes.data)
    if n == -1:
        raise OverflowError("fast oracle commit: start + dur does not fit in 32 bits")
    if n < 0:
        raise MemoryError("fast oracle commit: out of memory")
    return int(n)
