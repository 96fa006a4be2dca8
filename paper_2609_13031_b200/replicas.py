"""Multi-GPU runs of the path are independent replicas: (b,h) pairs and query rows
never exchange data, so there is no collective on the data path.  The only
cross-rank step is the bookkeeping of a timed run: the slowest rank's time and the
whole-job throughput.  Works with any torch.distributed backend (NCCL on GPUs,
gloo on CPU)."""
from __future__ import annotations

import torch
import torch.distributed as dist


def max_over_ranks(value: float, device: str | torch.device = "cpu") -> float:
    """Largest ``value`` over all ranks (identity when not initialised / one rank)."""
    if not dist.is_available() or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: float, seconds_this_rank: float,
                   device: str | torch.device = "cpu") -> float:
    """Units all ranks processed divided by the slowest rank's time."""
    world = dist.get_world_size() if dist.is_available() and dist.is_initialized() else 1
    return world * units_per_rank / max_over_ranks(seconds_this_rank, device)


def barrier() -> None:
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()
