"""How the look-up path spreads over several GPUs: by requests, with no exchange on the data path.

The look-up of one request reads the caches and that request's activation only, so a batch can be cut into
contiguous shards, one per rank, each rank holding a replica of the caches.  The only collectives are a barrier
around timed regions and the reduction of the timing itself (max of the elapsed time, sum of the work).

A cache too large for one GPU can instead be split by rows: every rank looks the whole batch up in its rows, the
ranks exchange their k neighbour tuples per request in ONE all-gather (batch x k x 16 bytes per rank), and each
rank merges them with `fi_merge_shard_lookups` (`sharded_lookup` below).  The gathered tuples land in the rank's
own memory before the merge kernel reads them.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

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


def gather_shard_tuples(tensors: Sequence[torch.Tensor], group=None) -> List[torch.Tensor]:
    """One all-gather for several equally shaped tensors of 4-byte elements (a shard's neighbour distances, global
    indices, labels and weights): each comes back with a leading axis over the ranks, [world, *shape]."""
    shape = tuple(tensors[0].shape)
    if any(tuple(t.shape) != shape or t.element_size() != 4 for t in tensors):
        raise ValueError("tensors must share one shape and have 4-byte elements")
    packed = torch.stack([t.contiguous().view(torch.int32) for t in tensors])           # [fields, *shape]
    world = dist.get_world_size(group) if (dist.is_available() and dist.is_initialized()) else 1
    if world == 1:
        buf = packed.unsqueeze(0)
    else:
        flat = torch.empty((world * packed.shape[0],) + shape, dtype=torch.int32, device=packed.device)
        dist.all_gather_into_tensor(flat, packed, group=group)                          # ranks concatenated on axis 0
        buf = flat.view((world,) + tuple(packed.shape))
    return [buf[:, f].contiguous().view(t.dtype) for f, t in enumerate(tensors)]


def sharded_lookup(cache, queries: torch.Tensor, index_offset: int, *, group=None):
    """Look-up against a cache whose rows are split over the ranks of `group`; `cache` holds this rank's rows,
    whose global indices start at `index_offset`.  Returns the merged LookupOut (identical on every rank)."""
    from . import binding as fb
    out = cache.lookup_batch(queries)
    gi, lab, wgt = cache.neighbor_tuples(out.topk_idx, index_offset)
    parts = gather_shard_tuples([out.topk_dist, gi, lab, wgt], group)
    return fb.merge_shard_lookups(*parts, metric=cache.cfg.metric, rule=cache.cfg.rule, threshold=cache.cfg.threshold)
