"""The N > 1 plumbing of the benchmark on CPU: two gloo ranks, each with its own forest shard."""
import os
import socket

import numpy as np
import torch
import torch.multiprocessing as mp

from paper_1809_00832_b200 import forests as fg, sharding


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out_dir):
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = fg.make_workload("tiny8", seed=rank)            # every rank draws its own forest
    mine = sharding.shard_trees(10, rank, world)
    times, counts = sharding.combine([1.0 + rank, 5.0 - rank], [w.forest.n_trees, w.forest.n_nodes, len(mine)])
    np.save(os.path.join(out_dir, f"r{rank}.npy"), np.array(times + counts, dtype=np.float64))
    dist.destroy_process_group()


def test_two_rank_combine(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    r0 = np.load(tmp_path / "r0.npy")
    r1 = np.load(tmp_path / "r1.npy")
    np.testing.assert_array_equal(r0, r1)               # every rank ends with the same aggregate
    assert r0[0] == 2.0 and r0[1] == 5.0                # max over ranks
    n0 = fg.make_workload("tiny8", 0).forest
    n1 = fg.make_workload("tiny8", 1).forest
    assert r0[2] == n0.n_trees + n1.n_trees and r0[3] == n0.n_nodes + n1.n_nodes
    assert r0[4] == 10                                  # the shards cover every tree once


def test_shards_partition_the_trees():
    for n, world in ((10, 3), (256, 8), (5, 8), (0, 2)):
        parts = [sharding.shard_trees(n, r, world) for r in range(world)]
        assert sorted(sum(parts, [])) == list(range(n))
        assert max(len(p) for p in parts) - min(len(p) for p in parts) <= 1


def test_shards_balanced_by_node_count():
    """trees dealt out by work: a partition, the same on every rank, and no shard above the mean by
    a whole largest tree (contiguous blocks of equal tree count can be far off on ragged batches)"""
    rng = np.random.default_rng(8)
    for world in (2, 3, 8):
        forest = fg.random_forest(rng, 57, 2, 56, 100)
        sizes = np.bincount(forest.tree_of, minlength=forest.n_trees)
        parts = [sharding.shard_trees_by_nodes(sizes, r, world) for r in range(world)]
        assert sorted(sum(parts, [])) == list(range(forest.n_trees))
        loads = [int(sizes[p].sum()) for p in parts]
        assert max(loads) - sum(loads) / world < sizes.max()
        assert max(loads) - min(loads) <= sizes.max()
    assert sharding.shard_trees_by_nodes([], 0, 2) == []
    assert sharding.shard_trees_by_nodes([5], 1, 2) == []
    # a skewed batch: one huge tree and many small ones
    sizes = [1000] + [10] * 100
    parts = [sharding.shard_trees_by_nodes(sizes, r, 2) for r in range(2)]
    assert parts[0] == [0] and len(parts[1]) == 100


def test_single_process_combine_is_identity():
    times, counts = sharding.combine([3.5], [7, 9])
    assert times == [3.5] and counts == [7, 9]
