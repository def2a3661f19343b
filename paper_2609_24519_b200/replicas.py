"""Host-side bookkeeping for running independent replicas of the workload on several GPUs.

The exact product has no exchange step, so N GPUs run N independent replicas; the only
communication is the timing protocol: a barrier before and after the timed region, the maximum
elapsed time over ranks, and the sum of the units every rank processed.  Works with any
torch.distributed backend (NCCL on GPUs, gloo on CPU for the tests)."""
from __future__ import annotations

from typing import Tuple


def world() -> Tuple[int, int]:
    """(rank, world_size) of the initialised process group, (0, 1) without one."""
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        return dist.get_rank(), dist.get_world_size()
    return 0, 1


def barrier(device=None) -> None:
    import torch
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.barrier()
    if device is not None and torch.cuda.is_available():
        torch.cuda.synchronize(device)


def aggregate(ms_local: float, units_local: float, device=None) -> Tuple[float, float]:
    """(max over ranks of the elapsed milliseconds, sum over ranks of the units processed)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms_local), float(units_local)
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    u = torch.tensor([units_local], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def throughput(ms_local: float, units_local: float, device=None) -> float:
    """Whole-job units per second: all ranks' units over the slowest rank's time."""
    ms, units = aggregate(ms_local, units_local, device)
    return units / (ms * 1e-3)
