"""Multi-GPU plumbing of the benchmark: trees are independent units, so a forest is sharded across
ranks with no data-path collective; only the timing and the counts are combined at the end.  Works
with any torch.distributed backend (NCCL on GPUs, gloo in the CPU tests)."""
from __future__ import annotations

from typing import List, Sequence, Tuple

import torch


def shard_trees(n_trees: int, rank: int, world: int) -> List[int]:
    """Tree ids of this rank: contiguous blocks whose sizes differ by at most one."""
    base, extra = divmod(n_trees, world)
    start = rank * base + min(rank, extra)
    return list(range(start, start + base + (1 if rank < extra else 0)))


def shard_trees_by_nodes(nodes_per_tree: Sequence[int], rank: int, world: int) -> List[int]:
    """Tree ids of this rank when the trees are dealt out by work: every tree, largest first (ties by
    tree id), goes to the rank with the fewest nodes so far (ties by rank).  Every rank computes the
    same assignment from the same sizes; the ids come back in ascending order.  The largest shard
    exceeds the mean by less than the largest tree."""
    sizes = [int(x) for x in nodes_per_tree]
    load = [0] * world
    mine: List[int] = []
    for t in sorted(range(len(sizes)), key=lambda i: (-sizes[i], i)):
        r = min(range(world), key=lambda q: (load[q], q))
        load[r] += sizes[t]
        if r == rank:
            mine.append(t)
    return sorted(mine)


def combine(times_ms: Sequence[float], counts: Sequence[int], device: str = "cpu") -> Tuple[List[float], List[int]]:
    """Max over ranks of every time, sum over ranks of every count (one all-reduce each)."""
    import torch.distributed as dist
    t = torch.tensor(list(times_ms), dtype=torch.float64, device=device)
    c = torch.tensor(list(counts), dtype=torch.int64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(c, op=dist.ReduceOp.SUM)
    return [float(x) for x in t.tolist()], [int(x) for x in c.tolist()]
