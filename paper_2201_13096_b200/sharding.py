"""Candidate sharding across ranks.  Candidates are independent problems against one timing table,
so the path shards with no data-path collective: each rank solves a contiguous slice.  The only
exchanges are control-plane: a barrier and a MAX reduction of timings."""
from __future__ import annotations

from typing import Tuple


def shard_range(n_total: int, rank: int, world: int) -> Tuple[int, int]:
    """Contiguous slice [start, start + count) of ``n_total`` candidates for ``rank``; the first
    ``n_total % world`` ranks take one extra candidate."""
    if world < 1 or not (0 <= rank < world) or n_total < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(n_total, world)
    count = base + (1 if rank < extra else 0)
    start = rank * base + min(rank, extra)
    return start, count


def max_over_ranks(value: float, device=None) -> float:
    """MAX all-reduce of a scalar (identity when torch.distributed is not initialised)."""
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: int, world: int, seconds_max: float) -> float:
    """Aggregate throughput when every rank processed ``units_per_rank`` units (weak scaling) and
    the slowest rank took ``seconds_max``."""
    return world * units_per_rank / seconds_max
