"""Multi-GPU plumbing of the benchmark: the path shards over tenants with no data-path collective,
so N GPUs run N independent replicas.  The only cross-rank step is timing: barrier, then the MAX of
the per-rank device times; throughput is the units all ranks processed over that time."""
from __future__ import annotations


def max_over_ranks(value: float, dist, device="cpu") -> float:
    """MAX of a per-rank scalar over the process group (`dist` = torch.distributed, initialised)."""
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank: float, ms_per_rank: float, dist, device="cpu"):
    """(total units, max ms, units per second) for replicas that each processed `units_per_rank`."""
    world = dist.get_world_size()
    ms = max_over_ranks(ms_per_rank, dist, device)
    total = units_per_rank * world
    return total, ms, total / (ms / 1e3)
