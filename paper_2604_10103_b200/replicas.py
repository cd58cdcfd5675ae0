"""Host-side bookkeeping for running the path on several GPUs.

Every (batch, head) pair owns its own cache, selection and state, and the path has no exchange step, so N GPUs
run N independent replicas (one process per GPU).  The only cross-rank work is measurement: the slowest rank's
device time and the sum of the units all ranks processed.  This module holds that logic so that it can be
exercised on CPU with the gloo backend.
"""
from __future__ import annotations


def replica_seed(base_seed: int, rank: int) -> int:
    """Distinct, reproducible input seed per replica."""
    return int(base_seed) + 7919 * int(rank)


def aggregate(ms_local: float, units_local: float, device=None):
    """(max over ranks of ms_local, sum over ranks of units_local).  Without an initialised process group the
    local values are returned unchanged.  `device`: where the reduction tensors live ("cuda" for NCCL)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms_local), float(units_local)
    dev = device if device is not None else ("cuda" if dist.get_backend() == "nccl" else "cpu")
    t_ms = torch.tensor([float(ms_local)], dtype=torch.float64, device=dev)
    t_units = torch.tensor([float(units_local)], dtype=torch.float64, device=dev)
    dist.all_reduce(t_ms, op=dist.ReduceOp.MAX)
    dist.all_reduce(t_units, op=dist.ReduceOp.SUM)
    return float(t_ms.item()), float(t_units.item())


def throughput(units_total: float, ms_max: float) -> float:
    """Whole-job units per second."""
    return units_total / (ms_max * 1e-3)
