"""Multi-GPU plumbing for the benchmark: the path does not shard across GPUs in this build
("replicas only"), so N ranks run N independent copies of the workload.  The only exchange is
the barrier and the max-over-ranks of the measured time; no data-path collective exists."""
from __future__ import annotations


def max_over_ranks(seconds: float, device=None) -> float:
    """Slowest rank's time (all ranks get it).  No-op outside an initialised process group."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(seconds)
    t = torch.tensor([seconds], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank: float, seconds: float, device=None) -> float:
    """Whole-job throughput of N replicas: all ranks' units divided by the slowest rank's time."""
    import torch.distributed as dist
    world = dist.get_world_size() if dist.is_available() and dist.is_initialized() else 1
    return world * units_per_rank / max_over_ranks(seconds, device)
