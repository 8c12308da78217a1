"""How the look-up path spreads over several GPUs: by requests, with no exchange on the data path.

The look-up of one request reads the caches and that request's activation only, so a batch can be cut into
contiguous shards, one per rank, each rank holding a replica of the caches.  The only collectives are a barrier
around timed regions and the reduction of the timing itself (max of the elapsed time, sum of the work).
"""
from __future__ import annotations

from typing import Tuple

import torch
import torch.distributed as dist


def shard_bounds(total: int, world: int, rank: int) -> Tuple[int, int]:
    """Contiguous shard [lo, hi) of `total` requests for `rank`; sizes differ by at most one."""
    if world < 1 or not 0 <= rank < world or total < 0:
        raise ValueError("need 0 <= rank < world and total >= 0")
    base, extra = divmod(total, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def reduce_timing(elapsed_ms: float, units: float, device=None) -> Tuple[float, float]:
    """Whole-job figures from per-rank ones: (max elapsed time over ranks, total units over ranks)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(elapsed_ms), float(units)
    t = torch.tensor([float(elapsed_ms)], dtype=torch.float64, device=device)
    u = torch.tensor([float(units)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())
