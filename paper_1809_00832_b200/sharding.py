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


def combine(times_ms: Sequence[float], counts: Sequence[int], device: str = "cpu") -> Tuple[List[float], List[int]]:
    """Max over ranks of every time, sum over ranks of every count (one all-reduce each)."""
    import torch.distributed as dist
    t = torch.tensor(list(times_ms), dtype=torch.float64, device=device)
    c = torch.tensor(list(counts), dtype=torch.int64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(c, op=dist.ReduceOp.SUM)
    return [float(x) for x in t.tolist()], [int(x) for x in c.tolist()]
