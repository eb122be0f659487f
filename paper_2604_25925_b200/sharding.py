"""Data-parallel sharding of the verify step over ranks (one process per GPU).

Batch rows are independent units of the method (Algorithm 1 runs per prompt), so the path shards
by batch row with no collective in the data path: every rank verifies its own rows and keeps its
own outputs.  The only cross-rank traffic is measurement: timings are reduced with MAX.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def shard_rows(B: int, rank: int, world: int) -> tuple[int, int]:
    """Contiguous, balanced split of B batch rows: rows [start, stop) belong to `rank`.
    The first B % world ranks get one row more; every row belongs to exactly one rank."""
    if not (0 <= rank < world) or B < 0:
        raise ValueError("need 0 <= rank < world and B >= 0")
    base, extra = divmod(B, world)
    start = rank * base + min(rank, extra)
    return start, start + base + (1 if rank < extra else 0)


def max_over_ranks(value: float, device="cpu") -> float:
    """MAX of a scalar over all ranks (the time of a multi-rank step is its slowest rank's)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device="cpu") -> float:
    """SUM of a scalar over all ranks (units processed by the whole job)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())
