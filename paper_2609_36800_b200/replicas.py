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


def shard_tenants(B: int, world: int, rank: int):
    """Tenants [start, start + count) that `rank` of `world` serves: a contiguous, even cut of the B tenants
    (the first B % world ranks take one more).  W_base is replicated, so a rank needs nothing from the others."""
    if B < 0 or world <= 0 or not 0 <= rank < world:
        raise ValueError("bad shard request")
    q, r = divmod(B, world)
    start = rank * q + min(rank, r)
    return start, q + (1 if rank < r else 0)


def tenant_shard(X, bits, alpha, world: int, rank: int):
    """This rank's slices of the per-tenant operands (X [B,m,K], bits [B,N,K/32], alpha [B]): views, no copies.
    The product of the shard is rows [start, start + count) of the full product."""
    start, count = shard_tenants(X.shape[0], world, rank)
    return X[start:start + count], bits[start:start + count], alpha[start:start + count], start
