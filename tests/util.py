"""Shared helpers of the GPU parity tests: run the CUDA library and the CPU oracle on the same
seeded workload."""
import functools

import numpy as np
import torch

from oracle import treelstm_oracle as orc
from paper_1809_00832_b200 import binding, build, forests as fg

TOL = {"fp32": 1e-4, "bf16": 3e-2}     # max-abs tolerance on h, c and gradients


def lib_ready():
    build.build()
    binding.load_library()


def to_dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda()


def make_model(params: fg.Params, precision: str) -> binding.TreeLSTM:
    lib_ready()
    prec = binding.FP32 if precision == "fp32" else binding.BF16
    model = binding.TreeLSTM(params.H, params.E, params.vocab, to_dev(params.emb), to_dev(params.W),
                             to_dev(params.b), prec)
    if params.C:
        model.set_classifier(to_dev(params.Wc), to_dev(params.bc))
    return model


def gpu_forward(model, forest: fg.Forest, flags: int):
    out = model.forward(to_dev(forest.left), to_dev(forest.right), to_dev(forest.token), flags=flags)
    torch.cuda.synchronize()
    res = {k: v.cpu().numpy() for k, v in out.items()}
    res["n_levels"] = int(res["n_levels"][0])
    return res


@functools.lru_cache(maxsize=None)
def oracle_forward_cached(name: str, seed: int, n_trees=None):
    w = fg.make_workload(name, seed, n_trees)
    f, p = w.forest, w.params
    status, parent, level, order, off = orc.schedule(f.left, f.right, f.token, p.vocab)
    assert status == orc.OK
    h, c, _ = orc.forward_recursive(f.left, f.right, f.token, p.emb, p.W, p.b)
    return dict(parent=parent, level=level, order=order, level_offset=off, h=h, c=c)


def check_schedule(res, ref, n):
    """bit-exact: level of every node, ready order, wavefront boundaries"""
    n_levels = len(ref["level_offset"]) - 1
    assert res["n_levels"] == n_levels
    np.testing.assert_array_equal(res["level"][:n], ref["level"])
    np.testing.assert_array_equal(res["order"][:n], ref["order"])
    np.testing.assert_array_equal(res["level_offset"][:n_levels + 1], ref["level_offset"])


def max_abs(a, b):
    return float(np.max(np.abs(np.asarray(a, dtype=np.float64) - b))) if a.size else 0.0
