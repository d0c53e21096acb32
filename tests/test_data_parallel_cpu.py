"""The gradient exchange of the data-parallel training step on CPU: two gloo ranks, each with its own
shard of a forest, per-rank gradients from the fp64 oracle (in place of the CUDA library); the
combined result must be the oracle's gradients on the whole forest."""
import os
import socket

import numpy as np
import torch
import torch.multiprocessing as mp

from oracle import treelstm_oracle as orc
from paper_1809_00832_b200 import data_parallel, forests as fg, sharding


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _problem():
    rng = np.random.default_rng(11)
    params = fg.draw_params(rng, 6, 5, 9, emb_dist="uniform", emb_scale=0.5, w_scale=0.5, n_classes=4)
    forest = fg.random_forest(rng, 7, 1, 9, 9)        # vocabulary of 9: tokens repeat within and across shards
    labels = rng.integers(0, 4, size=forest.n_nodes).astype(np.int32)
    return params, forest, labels


def _local_gradients(params, forest, labels, pad):
    g = orc.loss_and_gradients(forest.left, forest.right, forest.token, params.emb, params.W, params.b,
                               params.Wc, params.bc, labels)
    nt = len(g["touched_ids"])
    ids = np.full(nt + pad, -7, dtype=np.int32)       # rows past n_touched are unspecified in the library
    rows = np.full((nt + pad, params.E), 123.0)
    ids[:nt] = g["touched_ids"]
    rows[:nt] = g["dEmb_rows"]
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a))
    return dict(loss=t(np.array([g["loss"]])), dW=t(g["dW"]), db=t(g["db"]), dWc=t(g["dWc"]), dbc=t(g["dbc"]),
                touched_ids=t(ids), dEmb_rows=t(rows), n_touched=t(np.array([nt], dtype=np.int32)))


def _worker(rank, world, port, out_dir):
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    params, forest, labels = _problem()
    mine = sharding.shard_trees_by_nodes(np.bincount(forest.tree_of, minlength=forest.n_trees), rank, world)
    shard = fg.select_trees(forest, mine)
    shard_labels = labels[np.isin(forest.tree_of, mine)]
    local = _local_gradients(params, shard, shard_labels, pad=rank + 1)
    out = data_parallel.combine_gradients(local, shard.n_nodes)
    np.savez(os.path.join(out_dir, f"r{rank}.npz"), **{k: v.numpy() for k, v in out.items()})
    dist.destroy_process_group()


def test_two_rank_gradient_exchange(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    params, forest, labels = _problem()
    ref = orc.loss_and_gradients(forest.left, forest.right, forest.token, params.emb, params.W, params.b,
                                 params.Wc, params.bc, labels)
    for rank in range(world):
        got = np.load(tmp_path / f"r{rank}.npz")
        assert abs(float(got["loss"][0]) - ref["loss"]) < 1e-12
        for k in ("dW", "db", "dWc", "dbc"):
            assert np.max(np.abs(got[k] - ref[k])) < 1e-12, k
        assert int(got["n_touched"][0]) == len(ref["touched_ids"])
        np.testing.assert_array_equal(got["touched_ids"], ref["touched_ids"])
        assert np.max(np.abs(got["dEmb_rows"] - ref["dEmb_rows"])) < 1e-12


def test_single_process_is_identity_up_to_trimming():
    params, forest, labels = _problem()
    local = _local_gradients(params, forest, labels, pad=3)
    out = data_parallel.combine_gradients(local, forest.n_nodes)
    nt = int(local["n_touched"][0])
    assert out["touched_ids"].shape[0] == nt and out["dEmb_rows"].shape[0] == nt
    assert torch.equal(out["dW"], local["dW"]) and torch.equal(out["loss"], local["loss"])
