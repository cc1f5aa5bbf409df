"""Row-block sharding of the join over ranks (one process per GPU).

Theorem 1's block decomposition makes the join of P against Q the union of the joins of
P's row blocks against Q, so ranks need no data-path collective: each rank joins its block
(with ``simjoin_set_offsets(start, 0)`` the emitted indices are already global) and only
the per-rank counts -- and, if wanted, the variable-length pair lists -- are exchanged.
This module holds that host logic; it runs on any torch.distributed backend.
"""
from __future__ import annotations

from typing import List, Tuple


def row_block(n: int, world: int, rank: int) -> Tuple[int, int]:
    """(first row, number of rows) of rank's contiguous block; blocks differ by at most one row."""
    if world <= 0 or not 0 <= rank < world or n < 0:
        raise ValueError("bad sharding arguments")
    base, extra = divmod(n, world)
    start = rank * base + min(rank, extra)
    return start, base + (1 if rank < extra else 0)


def exchange_counts(local_count: int, group=None) -> List[int]:
    """All ranks' pair counts, in rank order."""
    import torch
    import torch.distributed as dist
    world = dist.get_world_size(group)
    mine = torch.tensor([int(local_count)], dtype=torch.int64)
    out = [torch.zeros(1, dtype=torch.int64) for _ in range(world)]
    backend = dist.get_backend(group)
    if backend == "nccl":
        mine = mine.cuda()
        out = [t.cuda() for t in out]
    dist.all_gather(out, mine, group=group)
    return [int(t.item()) for t in out]


def gather_pairs(local_pairs, counts: List[int], group=None):
    """Concatenate every rank's (count_r, 2) int32 pair list on all ranks (rank order)."""
    import torch
    import torch.distributed as dist
    world = dist.get_world_size(group)
    cap = max(max(counts), 1)
    dev = local_pairs.device
    buf = torch.zeros((cap, 2), dtype=torch.int32, device=dev)
    buf[: local_pairs.shape[0]] = local_pairs
    out = [torch.zeros_like(buf) for _ in range(world)]
    dist.all_gather(out, buf, group=group)
    return torch.cat([o[:c] for o, c in zip(out, counts)], dim=0)
