"""Multi-GPU plumbing: the join has no exchange step, so N GPUs run N independent replicas (own store, own
batch).  The only cross-rank work is bookkeeping for the benchmark: a barrier, the maximum of the per-rank
device times and the sum of the per-rank candidate counts.  Works with any torch.distributed backend (nccl
on GPUs, gloo in the CPU tests); with no process group it is the identity."""
from __future__ import annotations

from typing import Optional

import torch
import torch.distributed as dist


def _world() -> int:
    return dist.get_world_size() if dist.is_available() and dist.is_initialized() else 1


def _reduce(x: float, op, device: Optional[torch.device]) -> float:
    if _world() == 1:
        return float(x)
    t = torch.tensor([float(x)], dtype=torch.float64, device=device or torch.device("cpu"))
    dist.all_reduce(t, op=op)
    return float(t.item())


def max_over_ranks(x: float, device: Optional[torch.device] = None) -> float:
    return _reduce(x, dist.ReduceOp.MAX, device)


def sum_over_ranks(x: float, device: Optional[torch.device] = None) -> float:
    return _reduce(x, dist.ReduceOp.SUM, device)


def barrier(device: Optional[torch.device] = None) -> None:
    if _world() > 1:
        dist.barrier()
    if device is not None and device.type == "cuda":
        torch.cuda.synchronize(device)


def job_throughput(local_units: float, local_ms_total: float, steps: int, device: Optional[torch.device] = None):
    """Whole-job units per second and ms per step for replicas that each processed `local_units` per step in
    `local_ms_total` over `steps` steps: sum of units over ranks / max of time over ranks."""
    ms_total = max_over_ranks(local_ms_total, device)
    units = sum_over_ranks(local_units, device)
    ms_per_step = ms_total / max(steps, 1)
    return units / (ms_per_step * 1e-3), ms_per_step


def rank_seed_offset(rank: int) -> int:
    """Replicas draw different batches: the workload seed is shifted by this much per rank."""
    return 17 * int(rank)
