"""Host-side plumbing for running the path on several GPUs (one process per GPU).

Tokens are independent units of the whole path, so a batch is cut into contiguous token ranges,
one per rank; every rank runs gate -> compaction -> head on its own range with replicated weights.
There is no collective on the data path. What ranks exchange afterwards, if the caller wants a
global view, is one survivor count per rank and, optionally, the survivor ids (made global by adding
the range start). Nothing here touches the method's arithmetic.
"""
from __future__ import annotations

from typing import List, Tuple


def token_range(n: int, world: int, rank: int) -> Tuple[int, int]:
    """[lo, hi) of rank `rank` when n tokens are cut into `world` contiguous, near-equal ranges."""
    assert world >= 1 and 0 <= rank < world and n >= 0
    base, rem = divmod(n, world)
    lo = rank * base + min(rank, rem)
    return lo, lo + base + (1 if rank < rem else 0)


def gather_counts(local_count: int, group=None) -> List[int]:
    """Survivor counts of all ranks (one small all-gather; off the hot path)."""
    import torch
    import torch.distributed as dist
    world = dist.get_world_size(group)
    mine = torch.tensor([int(local_count)], dtype=torch.int64)
    if dist.get_backend(group) == "nccl":
        mine = mine.cuda()
    parts = [torch.zeros_like(mine) for _ in range(world)]
    dist.all_gather(parts, mine, group=group)
    return [int(p.item()) for p in parts]


def gather_survivor_ids(local_idx, local_count: int, lo: int, group=None):
    """Global ascending survivor ids of the whole batch from every rank's local list.

    local_idx: 1-D int32 tensor whose first local_count entries are ascending local token ids.
    Returns (ids int64 tensor [total], counts list). Ranges are contiguous and ordered by rank, so
    concatenation in rank order is already ascending.
    """
    import torch
    import torch.distributed as dist
    world = dist.get_world_size(group)
    counts = gather_counts(local_count, group)
    cap = max(max(counts), 1)
    buf = torch.full((cap,), -1, dtype=torch.int64, device=local_idx.device)
    buf[:local_count] = local_idx[:local_count].to(torch.int64) + lo
    parts = [torch.empty_like(buf) for _ in range(world)]
    dist.all_gather(parts, buf, group=group)
    ids = torch.cat([p[:c] for p, c in zip(parts, counts)])
    return ids, counts


def max_over_ranks(value: float, device=None, group=None) -> float:
    """Max of a host scalar over all ranks (used for timing: the slowest rank sets the step time)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return float(t.item())
