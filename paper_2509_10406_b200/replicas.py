"""Multi-GPU plumbing.  The layer has no exchange step: every (batch, kv-head group) is an
independent problem, so N GPUs run N independent replicas (or disjoint head ranges) and only
the timing is reduced.  torch.distributed is used for the barrier and the max over ranks."""
from __future__ import annotations

import torch
import torch.distributed as dist


def head_range(n_groups: int, rank: int, world: int):
    """Contiguous range of kv-head groups owned by `rank` (balanced to within one group)."""
    base, extra = divmod(n_groups, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def max_over_ranks(ms: float, device="cpu") -> float:
    """Slowest rank's time; identity when no process group is initialised."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(units_per_rank: float, ms: float, device="cpu") -> float:
    """Whole-job units per second: all ranks' units over the slowest rank's time."""
    world = dist.get_world_size() if dist.is_available() and dist.is_initialized() else 1
    return world * units_per_rank / (max_over_ranks(ms, device) * 1e-3)
