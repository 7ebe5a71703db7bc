"""Host-side logic of one scheduler spread over several GPUs.

Jobs are sharded over the ranks in contiguous id ranges, every rank advertises the same gaps and selects among
its own jobs; one all-gather of a 32-byte bid per gap and rank is the only exchange of a round
(``sja_get_bids`` / ``sja_reduce_bids`` in include/sja.h do the arithmetic on the GPU).  This module holds the
partitioning and the collective call, so that both can be exercised with the ``gloo`` backend on CPU; it
contains none of the method's arithmetic.
"""
from __future__ import annotations

from typing import Tuple

import numpy as np

BID_BYTES = 32
AWARD_BYTES = 24


def shard_bounds(n_jobs: int, world: int, rank: int) -> Tuple[int, int]:
    """Jobs ``[lo, hi)`` of ``rank``: contiguous, in rank order, sizes differing by at most one."""
    if not 0 <= rank < world:
        raise ValueError("rank out of range")
    base, extra = divmod(int(n_jobs), int(world))
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def shard_profiles(prof, lo: int, hi: int):
    """The profile arrays of jobs ``[lo, hi)`` as a new Profiles object (offsets rebased to 0).  The safe bits
    are re-packed from bit ``off[lo]`` on."""
    from . import workloads as wl

    a, b = int(prof.off[lo]), int(prof.off[hi])
    off = (prof.off[lo:hi + 1] - prof.off[lo]).astype(np.uint64)
    safe = wl.unpack_safe_bits(prof.safe_bits, prof.n_steps)[a:b]
    return wl.Profiles(off, np.ascontiguousarray(prof.dur_ms[a:b]), np.ascontiguousarray(prof.mem_MiB[a:b]),
                       wl.pack_safe_bits(safe), np.ascontiguousarray(prof.ready_ms[lo:hi]),
                       None if prof.wait_ms is None else np.ascontiguousarray(prof.wait_ms[lo:hi]),
                       None if prof.prio is None else np.ascontiguousarray(prof.prio[lo:hi]))


def gather_bids(local_bids, dist=None):
    """All ranks' bids, rank r at row r.  ``local_bids`` is a uint8 tensor of ``32 * G`` bytes (CPU tensor with
    gloo, CUDA tensor with NCCL); returns a tensor of shape ``(world, 32 * G)`` on the same device."""
    import torch

    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return local_bids.reshape(1, -1)
    world = dist.get_world_size()
    n = local_bids.numel()
    out = torch.empty(world * n, dtype=torch.uint8, device=local_bids.device)
    dist.all_gather_into_tensor(out, local_bids.reshape(-1).contiguous())
    return out.reshape(world, n)


class ShardedScheduler:
    """One rank of a sharded scheduler: wraps a loaded ``binding.Sja`` context that holds jobs ``[lo, hi)``.

    The collective is issued on torch's current CUDA stream, the library works on the stream its context was
    created with: create the context on the stream that is current when :meth:`round` is called (or on the
    default stream), so that the bids are complete before they are gathered."""

    def __init__(self, ctx, lo: int, rank: int, world: int, dist=None, device=None):
        import torch

        self.ctx, self.lo, self.rank, self.world, self.dist = ctx, int(lo), int(rank), int(world), dist
        self.device = device if device is not None else torch.device("cuda", torch.cuda.current_device())
        self._bids = self._accept = self._global = None

    def _buffers(self, G: int):
        import torch

        if self._bids is None or self._bids.numel() != BID_BYTES * G:
            self._bids = torch.empty(BID_BYTES * G, dtype=torch.uint8, device=self.device)
            self._accept = torch.empty(G, dtype=torch.uint8, device=self.device)
            self._global = torch.empty(AWARD_BYTES * G, dtype=torch.uint8, device=self.device)

    def round(self, gaps, policy: int, flags: int = 0, want_count: bool = False):
        """advertise + select on this shard, exchange, commit what this shard won.  Returns
        ``(global_awards, n_granted_here)``: a CUDA uint8 tensor of ``24 * G`` bytes (the winning award of every
        gap with global job ids) and this rank's grant count (None unless ``want_count``)."""
        ctx = self.ctx
        ctx.advertise(gaps)
        G = ctx.n_gaps
        self._buffers(G)
        ctx.select(policy, flags=flags)
        ctx.get_bids(self.lo, self.rank, out=self._bids)
        all_bids = gather_bids(self._bids, self.dist)
        ctx.reduce_bids(self.world, self.rank, all_bids, self._accept, self._global)
        n = ctx.commit_masked(self._accept, want_count=want_count)
        return self._global, n
