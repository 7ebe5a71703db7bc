"""ctypes binding of libsja.so.  Argument marshalling only: every step runs in the library.

Arrays may be numpy arrays (host memory) or torch CUDA tensors (device memory); the
memory space is inferred per call and all arrays of one call must agree.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import numpy as np

from .build import LIB_PATH

SJA_OK = 0
STATUS_NAMES = {
    0: "SJA_OK", 1: "SJA_ERR_INVALID_ARG", 2: "SJA_ERR_BAD_PROFILE", 3: "SJA_ERR_OVERFLOW",
    4: "SJA_ERR_STATE", 5: "SJA_ERR_OOM", 6: "SJA_ERR_CUDA", 7: "SJA_ERR_TIMEOUT",
}
MEM_HOST, MEM_DEVICE = 0, 1
POLICY_EFFICIENCY, POLICY_FAIRNESS, POLICY_SLA, POLICY_TIGHT_FIT = 0, 1, 2, 3
FLAG_FORCE_SEARCH = 1
FLAG_FORCE_MERGE = 2
FLAG_FORCE_TILE = 4
NO_JOB = 0xFFFFFFFF

GAP_DTYPE = np.dtype([("slice", "<u4"), ("start_ms", "<u4"), ("T_ms", "<u4"), ("C_MiB", "<u4")])
BID_DTYPE = np.dtype([("key", "<u8"), ("job", "<u4"), ("end_step", "<u4"), ("dur_ms", "<u4"), ("rank", "<u4"),
                      ("score", "<u8")])
AWARD_DTYPE = np.dtype([("job", "<u4"), ("end_step", "<u4"), ("dur_ms", "<u4"), ("granted", "<u4"),
                        ("score", "<u8")])

EXPORTS = [
    "sja_create", "sja_destroy", "sja_load_profiles", "sja_advertise", "sja_select", "sja_select_static", "sja_commit", "sja_commit_masked", "sja_round_reauction", "sja_set_duration_bounds", "sja_set_window_options", "sja_set_hysteresis", "sja_set_locality", "sja_get_locality", "sja_update_profile", "sja_load_power", "sja_advertise_power_caps", "sja_get_bids", "sja_reduce_bids",
    "sja_get_awards", "sja_get_state", "sja_scan_size", "sja_get_scan", "sja_profile_enable",
    "sja_profile_read", "sja_last_error", "sja_debug_fail_alloc",
]


class SjaPolicy(ctypes.Structure):
    _fields_ = [("kind", ctypes.c_uint32), ("flags", ctypes.c_uint32)]


class SjaTiming(ctypes.Structure):
    _fields_ = [("scan_ms", ctypes.c_float), ("prep_ms", ctypes.c_float),
                ("advertise_ms", ctypes.c_float), ("select_ms", ctypes.c_float),
                ("commit_ms", ctypes.c_float),
                ("scan_launches", ctypes.c_uint32), ("prep_launches", ctypes.c_uint32),
                ("advertise_launches", ctypes.c_uint32), ("select_launches", ctypes.c_uint32),
                ("commit_launches", ctypes.c_uint32)]


class SjaError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{STATUS_NAMES.get(status, status)}: {message}")
        self.status = status


_lib = None


def load_library() -> ctypes.CDLL:
    """dlopen libsja.so; raises if it has not been built (there is no fallback path)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2509_19086_b200.build` "
            "(needs nvcc); this package has no CPU fallback")
    lib = ctypes.CDLL(LIB_PATH)
    vp, u32, i32 = ctypes.c_void_p, ctypes.c_uint32, ctypes.c_int
    lib.sja_create.argtypes = [ctypes.POINTER(vp), i32, vp]
    lib.sja_destroy.argtypes = [vp]
    lib.sja_load_profiles.argtypes = [vp, u32, vp, vp, vp, vp, vp, vp, vp, vp, i32]
    lib.sja_advertise.argtypes = [vp, u32, vp, i32]
    lib.sja_select.argtypes = [vp, ctypes.POINTER(SjaPolicy), vp, i32]
    lib.sja_select_static.argtypes = [vp, ctypes.POINTER(SjaPolicy), vp, i32]
    lib.sja_commit.argtypes = [vp, ctypes.POINTER(u32)]
    lib.sja_round_reauction.argtypes = [vp, ctypes.POINTER(SjaPolicy), u32, ctypes.POINTER(u32), ctypes.POINTER(u32)]
    lib.sja_set_duration_bounds.argtypes = [vp, u32, u32]
    lib.sja_set_window_options.argtypes = [vp, u32, vp, i32]
    lib.sja_set_hysteresis.argtypes = [vp, u32]
    lib.sja_set_locality.argtypes = [vp, vp, vp, u32, i32]
    lib.sja_get_locality.argtypes = [vp, vp, i32]
    lib.sja_update_profile.argtypes = [vp, u32, u32, vp, vp, i32]
    lib.sja_load_power.argtypes = [vp, vp, vp, i32]
    lib.sja_get_bids.argtypes = [vp, u32, u32, vp, i32]
    lib.sja_reduce_bids.argtypes = [vp, u32, u32, vp, vp, vp, i32]
    lib.sja_advertise_power_caps.argtypes = [vp, vp, i32]
    lib.sja_commit_masked.argtypes = [vp, vp, i32, ctypes.POINTER(u32)]
    lib.sja_get_awards.argtypes = [vp, vp, i32]
    lib.sja_get_state.argtypes = [vp, vp, vp, i32]
    lib.sja_scan_size.argtypes = [vp, ctypes.POINTER(ctypes.c_uint64)]
    lib.sja_get_scan.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32]
    lib.sja_profile_enable.argtypes = [vp, i32]
    lib.sja_profile_read.argtypes = [vp, ctypes.POINTER(SjaTiming)]
    lib.sja_last_error.argtypes = [vp]
    lib.sja_debug_fail_alloc.argtypes = [vp, i32]
    lib.sja_last_error.restype = ctypes.c_char_p
    for name in EXPORTS:
        if name != "sja_last_error":
            getattr(lib, name).restype = i32
    _lib = lib
    return lib


def _is_torch(a) -> bool:
    return type(a).__module__.startswith("torch")


def _ptr_space(a, space: Optional[int], np_dtype=None):
    """(pointer, memspace, keepalive) of a numpy array or torch tensor."""
    if a is None:
        return None, space, None
    if _is_torch(a):
        if not a.is_cuda:
            raise TypeError("torch tensors passed to libsja must live on the CUDA device")
        if not a.is_contiguous():
            raise TypeError("tensor must be contiguous")
        sp = MEM_DEVICE
        ptr, keep = a.data_ptr(), a
    else:
        arr = np.ascontiguousarray(a) if np_dtype is None else np.ascontiguousarray(a, dtype=np_dtype)
        sp = MEM_HOST
        ptr, keep = arr.ctypes.data, arr
    if space is not None and space != sp:
        raise TypeError("all arrays of one call must be in the same memory space")
    return ptr, sp, keep


class Sja:
    """One scheduler context on one CUDA device (wraps ``sja_ctx``)."""

    def __init__(self, device: int = 0, stream: Optional[int] = None):
        self._lib = load_library()
        self._h = ctypes.c_void_p()
        st = self._lib.sja_create(ctypes.byref(self._h), int(device), ctypes.c_void_p(stream or 0))
        if st != SJA_OK:
            self._h = ctypes.c_void_p()
            raise SjaError(st, "sja_create failed (is a CUDA device present?)")
        self.n_jobs = 0
        self.n_gaps = 0

    def close(self) -> None:
        if getattr(self, "_h", None) is not None and self._h:
            self._lib.sja_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def _check(self, st: int) -> None:
        if st != SJA_OK:
            msg = self._lib.sja_last_error(self._h)
            raise SjaError(st, msg.decode() if msg else "")

    # -- sja_load_profiles
    def load_profiles(self, off, dur_ms, mem_MiB, safe_bits, ready_ms, progress=None, wait_ms=None,
                      prio=None) -> None:
        n_jobs = int(off.shape[0]) - 1
        keep = []
        space = None
        ptrs = []
        for a, dt in ((off, np.uint64), (dur_ms, np.uint32), (mem_MiB, np.uint32), (safe_bits, np.uint32),
                      (ready_ms, np.uint32), (progress, np.uint32), (wait_ms, np.uint32), (prio, np.uint8)):
            p, space, k = _ptr_space(a, space, dt)
            ptrs.append(p)
            keep.append(k)
        self._check(self._lib.sja_load_profiles(self._h, n_jobs, *ptrs, space))
        self.n_jobs = n_jobs

    # -- sja_advertise
    def advertise(self, gaps) -> None:
        if _is_torch(gaps):
            p, space, keep = _ptr_space(gaps, None)
            n = gaps.numel() * gaps.element_size() // GAP_DTYPE.itemsize
        else:
            gaps = np.ascontiguousarray(gaps, dtype=GAP_DTYPE)
            p, space, keep = _ptr_space(gaps, None)
            n = gaps.shape[0]
        self._check(self._lib.sja_advertise(self._h, int(n), p, space))
        self.n_gaps = int(n)

    # -- sja_select
    def select(self, policy: int, flags: int = 0, out=None):
        """Run signal + score + select.  ``out``: None (awards stay in the context), the string
        "host" (returns a numpy AWARD_DTYPE array), or a CUDA uint8 tensor of 24*G bytes."""
        pol = SjaPolicy(int(policy), int(flags))
        if out is None:
            self._check(self._lib.sja_select(self._h, ctypes.byref(pol), None, MEM_HOST))
            return None
        if isinstance(out, str):
            arr = np.empty(self.n_gaps, dtype=AWARD_DTYPE)
            self._check(self._lib.sja_select(self._h, ctypes.byref(pol), arr.ctypes.data, MEM_HOST))
            return arr
        p, space, _ = _ptr_space(out, None)
        self._check(self._lib.sja_select(self._h, ctypes.byref(pol), p, space))
        return out

    # -- sja_select_static
    def select_static(self, policy: int, flags: int = 0, out=None):
        """sja_select_static: same arguments and results as :meth:`select`, but the library
        allocates nothing on this path (fixed scratch; sizes beyond it raise SjaError)."""
        pol = SjaPolicy(int(policy), int(flags))
        if out is None:
            self._check(self._lib.sja_select_static(self._h, ctypes.byref(pol), None, MEM_HOST))
            return None
        if isinstance(out, str):
            arr = np.empty(self.n_gaps, dtype=AWARD_DTYPE)
            self._check(self._lib.sja_select_static(self._h, ctypes.byref(pol), arr.ctypes.data, MEM_HOST))
            return arr
        p, space, _ = _ptr_space(out, None)
        self._check(self._lib.sja_select_static(self._h, ctypes.byref(pol), p, space))
        return out

    # -- sja_commit
    def commit(self, want_count: bool = True) -> Optional[int]:
        if want_count:
            n = ctypes.c_uint32()
            self._check(self._lib.sja_commit(self._h, ctypes.byref(n)))
            return int(n.value)
        self._check(self._lib.sja_commit(self._h, None))
        return None

    # -- sja_commit_masked
    def commit_masked(self, accept, want_count: bool = True) -> Optional[int]:
        """sja_commit_masked: ``accept`` is a u8 array (numpy or CUDA tensor) with one entry per gap.
        Without ``want_count`` the call does not wait for the GPU and returns None."""
        p, space, _keep = _ptr_space(accept, None, np.uint8)
        if not want_count:
            self._check(self._lib.sja_commit_masked(self._h, p, space, None))
            return None
        n = ctypes.c_uint32()
        self._check(self._lib.sja_commit_masked(self._h, p, space, ctypes.byref(n)))
        return int(n.value)

    # -- sja_round_reauction
    def round_reauction(self, policy: int, flags: int = 0, max_passes: int = 0):
        """select + commit, repeated for gaps orphaned by multi-winners; returns (n_granted, n_passes)."""
        pol = SjaPolicy(int(policy), int(flags))
        n, k = ctypes.c_uint32(), ctypes.c_uint32()
        self._check(self._lib.sja_round_reauction(self._h, ctypes.byref(pol), int(max_passes),
                                                  ctypes.byref(n), ctypes.byref(k)))
        return int(n.value), int(k.value)

    # -- sja_set_duration_bounds
    def set_duration_bounds(self, tau_min_ms: int = 0, tau_max_ms: int = 0xFFFFFFFF) -> None:
        self._check(self._lib.sja_set_duration_bounds(self._h, int(tau_min_ms), int(tau_max_ms)))

    # -- sja_set_window_options
    def set_window_options(self, late_start: bool = False, deadline_ms=None) -> None:
        """``deadline_ms``: u32 per job (numpy or CUDA tensor) or None."""
        p, space, _keep = _ptr_space(deadline_ms, None, np.uint32)
        if deadline_ms is not None and int(_keep.shape[0]) != self.n_jobs:
            raise ValueError("deadline_ms needs one entry per loaded job")
        self._check(self._lib.sja_set_window_options(self._h, 1 if late_start else 0, p,
                                                     MEM_HOST if space is None else space))

    # -- sja_set_hysteresis
    def set_hysteresis(self, min_slack_gain_MiB: int = 0) -> None:
        self._check(self._lib.sja_set_hysteresis(self._h, int(min_slack_gain_MiB)))

    # -- sja_set_locality / sja_get_locality
    def set_locality(self, ckpt_MiB=None, last_slice=None, weight: int = 0) -> None:
        """``ckpt_MiB`` / ``last_slice``: u32 per job (numpy or CUDA tensors); ``ckpt_MiB=None`` switches it off."""
        pc, space, kc = _ptr_space(ckpt_MiB, None, np.uint32)
        pl, space, kl = _ptr_space(last_slice, space, np.uint32)
        for k in (kc, kl):
            if k is not None and int(k.shape[0]) != self.n_jobs:
                raise ValueError("locality arrays need one entry per loaded job")
        self._check(self._lib.sja_set_locality(self._h, pc, pl, int(weight), MEM_HOST if space is None else space))

    def get_locality(self) -> np.ndarray:
        out = np.empty(self.n_jobs, dtype=np.uint32)
        self._check(self._lib.sja_get_locality(self._h, out.ctypes.data, MEM_HOST))
        return out

    # -- sja_get_bids / sja_reduce_bids (one scheduler over several GPUs)
    def get_bids(self, job_base: int, rank: int, out=None):
        """Bids of this shard for the advertised gaps: a numpy BID_DTYPE array, or written to the CUDA uint8
        tensor ``out`` (32 * G bytes)."""
        if out is None:
            arr = np.empty(self.n_gaps, dtype=BID_DTYPE)
            self._check(self._lib.sja_get_bids(self._h, int(job_base), int(rank), arr.ctypes.data, MEM_HOST))
            return arr
        p, space, _ = _ptr_space(out, None)
        self._check(self._lib.sja_get_bids(self._h, int(job_base), int(rank), p, space))
        return out

    def reduce_bids(self, n_ranks: int, my_rank: int, all_bids, accept=None, global_awards=None):
        """Fold the gathered bids (rank r at ``all_bids[r * G]``).  Host arrays in: returns ``(accept u8[G],
        awards AWARD_DTYPE[G])``.  CUDA tensors in: ``accept`` (G bytes) and ``global_awards`` (24 * G bytes,
        may be None) are CUDA uint8 tensors that receive the result."""
        if _is_torch(all_bids):
            p, space, _ = _ptr_space(all_bids, None)
            pa, space, _ = _ptr_space(accept, space)
            pg, space, _ = _ptr_space(global_awards, space)
            self._check(self._lib.sja_reduce_bids(self._h, int(n_ranks), int(my_rank), p, pa, pg, space))
            return accept, global_awards
        all_bids = np.ascontiguousarray(all_bids, dtype=BID_DTYPE)
        acc = np.empty(self.n_gaps, dtype=np.uint8)
        aw = np.empty(self.n_gaps, dtype=AWARD_DTYPE)
        self._check(self._lib.sja_reduce_bids(self._h, int(n_ranks), int(my_rank), all_bids.ctypes.data,
                                              acc.ctypes.data, aw.ctypes.data, MEM_HOST))
        return acc, aw

    # -- sja_load_power / sja_advertise_power_caps
    def load_power(self, off, power_W) -> None:
        """Per-step power trace (u32, aligned with the loaded profile arrays) and the CSR offsets again."""
        po, space, _k0 = _ptr_space(off, None, np.uint64)
        pp, space, _k1 = _ptr_space(power_W, space, np.uint32)
        self._check(self._lib.sja_load_power(self._h, po, pp, space))

    def advertise_power_caps(self, cap_W) -> None:
        """One cap per gap of the advertised batch (u32, numpy or CUDA tensor), or None."""
        p, space, keep = _ptr_space(cap_W, None, np.uint32)
        if keep is not None and int(keep.shape[0]) != self.n_gaps:
            raise ValueError("cap_W needs one entry per advertised gap")
        self._check(self._lib.sja_advertise_power_caps(self._h, p, MEM_HOST if space is None else space))

    # -- sja_update_profile
    def update_profile(self, job: int, dur_ms, mem_MiB) -> None:
        """New durations / memory values (u32, numpy or CUDA tensors) for the steps ``job`` has left."""
        pd, space, keep_d = _ptr_space(dur_ms, None, np.uint32)
        pm, space, keep_m = _ptr_space(mem_MiB, space, np.uint32)
        n = int(keep_d.shape[0]) if keep_d is not None else 0
        if keep_m is not None and int(keep_m.shape[0]) != n:
            raise ValueError("dur_ms and mem_MiB must have the same length")
        self._check(self._lib.sja_update_profile(self._h, int(job), n, pd, pm, MEM_HOST if space is None else space))

    # -- sja_get_awards / sja_get_state
    def get_awards(self) -> np.ndarray:
        arr = np.empty(self.n_gaps, dtype=AWARD_DTYPE)
        self._check(self._lib.sja_get_awards(self._h, arr.ctypes.data, MEM_HOST))
        return arr

    def get_state(self):
        p = np.empty(self.n_jobs, dtype=np.uint32)
        r = np.empty(self.n_jobs, dtype=np.uint32)
        self._check(self._lib.sja_get_state(self._h, p.ctypes.data, r.ctypes.data, MEM_HOST))
        return p, r

    # -- sja_scan_size / sja_get_scan
    def scan_size(self) -> int:
        n = ctypes.c_uint64()
        self._check(self._lib.sja_scan_size(self._h, ctypes.byref(n)))
        return int(n.value)

    def get_scan(self):
        n = self.scan_size()
        boff = np.empty(self.n_jobs + 1, dtype=np.uint64)
        k = np.empty(n, np.uint32)
        D = np.empty(n, np.uint32)
        M = np.empty(n, np.uint32)
        S = np.empty(n, np.uint32)
        W = np.empty(n, np.uint64)
        self._check(self._lib.sja_get_scan(self._h, boff.ctypes.data, k.ctypes.data, D.ctypes.data,
                                           M.ctypes.data, S.ctypes.data, W.ctypes.data, MEM_HOST))
        return dict(boff=boff, k=k, D=D, M=M, S=S, W=W)

    # -- sja_debug_fail_alloc
    def debug_fail_alloc(self, nth: int) -> None:
        """Host-side fault injection: the nth growing allocation from now reports SJA_ERR_OOM (0 = off)."""
        self._check(self._lib.sja_debug_fail_alloc(self._h, int(nth)))

    # -- profiling
    def profile_enable(self, on=True) -> None:
        """``on``: False / 0 off, True / 1 every phase, 2 the scan kernel only."""
        self._check(self._lib.sja_profile_enable(self._h, int(on)))

    def profile_read(self) -> dict:
        t = SjaTiming()
        self._check(self._lib.sja_profile_read(self._h, ctypes.byref(t)))
        return {name: getattr(t, name) for name, _ in SjaTiming._fields_}
