"""Host-side helpers for spreading ONE search over several processes (one GPU each).

Candidates are independent, so a search shards by contiguous rank windows per size with no
exchange on the data path; the only communication is the merge of the per-rank results:
match counts add, the least solution is the smallest (size, rank) among the ranks that found
one.  The merge uses ``torch.distributed`` (NCCL between GPUs, gloo on CPU) on a handful of
int64 values.  Independent sketches need none of this: give each process its own.
"""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple


def shard_rank_windows(cand_count: Sequence[int], world: int, rank: int, hole: int = -1) -> List[Tuple[int, int, int, int]]:
    """Rank windows ``(hole, size, begin, end)`` of process ``rank`` out of ``world``: every size
    is cut into ``world`` contiguous pieces whose lengths differ by at most one.  Sizes whose
    piece is empty still get an (empty) window, so that the process searches nothing there."""
    out = []
    for size, n in enumerate(cand_count):
        if size == 0:
            continue
        base, extra = divmod(int(n), world)
        begin = rank * base + min(rank, extra)
        end = begin + base + (1 if rank < extra else 0)
        out.append((hole, size, begin, end))
    return out


def merge_results(match_count: Sequence[int], solved: bool, least_size: int, least_rank: int, group=None):
    """All-reduces one hole's windowed results over the process group.  Returns
    ``(match_count, solved, least_size, least_rank)`` of the whole search, the same on every rank."""
    import torch
    import torch.distributed as dist
    device = "cuda" if dist.get_backend(group) == "nccl" else "cpu"
    counts = torch.tensor([int(c) for c in match_count], dtype=torch.int64, device=device)
    dist.all_reduce(counts, op=dist.ReduceOp.SUM, group=group)
    world = dist.get_world_size(group)
    mine = torch.tensor([1 if solved else 0, int(least_size), int(least_rank)], dtype=torch.int64, device=device)
    every = [torch.zeros_like(mine) for _ in range(world)]
    dist.all_gather(every, mine, group=group)
    found = sorted((int(t[1]), int(t[2])) for t in every if int(t[0]))
    if not found:
        return [int(c) for c in counts.tolist()], False, 0, 0
    return [int(c) for c in counts.tolist()], True, found[0][0], found[0][1]
