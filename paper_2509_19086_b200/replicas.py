"""Host-side logic of multi-GPU runs: independent scheduler replicas, one per GPU.

The round has no exchange step when every GPU runs its own scheduler instance (its own
jobs and gaps), so ranks share nothing on the data path.  What they do share is the
measurement: whole-job throughput is the work of all ranks divided by the slowest rank's
device time.  This module holds that logic so that it can be tested with the ``gloo``
backend on CPU; it contains none of the method's arithmetic.
"""
from __future__ import annotations

from typing import Optional

from . import workloads as wl


def replica_spec(spec: wl.WorkloadSpec, rank: int) -> wl.WorkloadSpec:
    """The workload of replica ``rank``: same shape, its own seed (rank 0 keeps the published one)."""
    if rank == 0:
        return spec
    return wl.scaled(spec, index=spec.index + 1000 * rank)


def aggregate(local_units: float, local_ms: list, dist=None, device: Optional[object] = None):
    """Sum of ``local_units`` over ranks and element-wise maximum of ``local_ms`` over ranks.

    ``dist`` is an initialised ``torch.distributed`` module (or None for one process).
    Returns ``(total_units, max_ms_list)``.
    """
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(local_units), [float(x) for x in local_ms]
    import torch

    kw = {} if device is None else {"device": device}
    u = torch.tensor([float(local_units)], dtype=torch.float64, **kw)
    t = torch.tensor([float(x) for x in local_ms], dtype=torch.float64, **kw)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(u[0]), [float(x) for x in t]


def throughput(total_units: float, steps: int, max_ms: float) -> float:
    """Units per second for ``steps`` timed steps that took ``max_ms`` on the slowest rank."""
    return total_units * steps / (max_ms * 1e-3) if max_ms > 0 else 0.0
