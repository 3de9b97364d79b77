"""N independent replicas, one process per GPU: the hot path has no exchange step, so the only inter-process
traffic is the timing protocol of the benchmark - a barrier on both sides of the timed region and the maximum of the
per-rank device times.  Works with any torch.distributed backend (NCCL on GPUs, gloo on CPU for the tests)."""
from __future__ import annotations

import torch
import torch.distributed as dist


def world() -> int:
    return dist.get_world_size() if dist.is_available() and dist.is_initialized() else 1


def barrier(device: torch.device) -> None:
    if device.type == "cuda":
        torch.cuda.synchronize(device)
    if world() > 1:
        dist.barrier()
    if device.type == "cuda":
        torch.cuda.synchronize(device)


def max_over_ranks(x: float, device: torch.device) -> float:
    """The slowest rank's time: what the whole job waited for."""
    if world() == 1:
        return float(x)
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: float, ms_this_rank: float, device: torch.device) -> float:
    """Units per second of the whole job: every rank processed units_per_rank, the job took the slowest rank's time."""
    return world() * units_per_rank / (max_over_ranks(ms_this_rank, device) * 1e-3)
