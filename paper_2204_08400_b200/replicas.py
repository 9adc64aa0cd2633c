"""Multi-GPU plumbing.  Queries are independent given replicated weights and
tables, so the path shards by query range with no exchange step: every rank runs
the single-GPU library on its own slice.  The only collective work is the
bookkeeping of a measurement (slowest rank's time, total queries)."""
from typing import Tuple

import torch
import torch.distributed as dist


def shard_range(n_queries: int, rank: int, world: int) -> Tuple[int, int]:
    """Contiguous slice [lo, hi) of the queries that `rank` serves; sizes differ by at most one."""
    base, extra = divmod(n_queries, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def slowest_rank_ms(ms: float, device=None) -> float:
    """Max of a per-rank time over all ranks (identity without a process group)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def total_units(units: int, device=None) -> int:
    """Sum of a per-rank count over all ranks."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return int(units)
    t = torch.tensor([units], dtype=torch.int64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return int(t.item())
