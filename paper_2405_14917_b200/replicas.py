"""Multi-GPU plumbing of the benchmark: independent replicas, one process per GPU.

The layer does not exchange data between GPUs: every rank runs the same workload on its own
device and only the timing is combined (slowest rank).  Works with any torch.distributed backend
(nccl on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations


def max_over_ranks(ms_local: float, device=None) -> float:
    """Largest value of `ms_local` over all ranks (identity without an initialised process group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms_local)
    t = torch.tensor([ms_local], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: float, ms_local: float, device=None) -> float:
    """Units per second of the whole job: every rank processed `units_per_rank`; time = slowest rank."""
    import torch.distributed as dist
    world = dist.get_world_size() if (dist.is_available() and dist.is_initialized()) else 1
    return world * units_per_rank / (max_over_ranks(ms_local, device) * 1e-3)
