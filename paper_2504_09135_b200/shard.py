"""Multi-GPU plumbing: the path shards by query with no exchange step.

Every GPU holds a replica of the constraint set and decodes its own contiguous block of queries
(all K candidates of a query stay on one GPU, because the K-way draw needs them together).  The
only communication is gathering the per-query results at the end, through torch.distributed
(NCCL on GPUs; gloo in the CPU tests).
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def shard_queries(B: int, world: int, rank: int) -> tuple[int, int]:
    """Contiguous, balanced split of B queries: (first query, number of queries) of `rank`."""
    if not (0 <= rank < world) or B < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(B, world)
    start = rank * base + min(rank, extra)
    return start, base + (1 if rank < extra else 0)


def gather_query_results(local: torch.Tensor, B: int) -> torch.Tensor:
    """All ranks' per-query rows ([b_local, ...] on each rank) -> [B, ...] on every rank, in
    query order.  Shards may differ in size by one row."""
    if not dist.is_initialized() or dist.get_world_size() == 1:
        return local
    world, rank = dist.get_world_size(), dist.get_rank()
    counts = [shard_queries(B, world, r)[1] for r in range(world)]
    if local.shape[0] != counts[rank]:
        raise ValueError("local shard has the wrong number of queries")
    pad = max(counts)
    buf = local.new_zeros((pad,) + tuple(local.shape[1:]))
    buf[:local.shape[0]] = local
    parts = [torch.empty_like(buf) for _ in range(world)]
    dist.all_gather(parts, buf)
    return torch.cat([p[:c] for p, c in zip(parts, counts)], dim=0)


def max_over_ranks(value: float, device="cpu") -> float:
    """Largest value of a per-rank timing (the job is as slow as its slowest rank)."""
    if not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device="cpu") -> float:
    """Sum of a per-rank count (the job's total when every rank reports its own share)."""
    if not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())
