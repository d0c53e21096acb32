"""The checked build of the library (-DTREELSTM_CHECKED, a second shared object from the same
sources) on the parity workloads: every index a kernel reads from the caller's arrays or from the
schedule is range-checked before use, and every state row counts its writers - each node's h must
be written exactly once, each internal position's operand row exactly twice (one half per child),
a leaf position's never.  This is the stand-in for a memory checker: a value routed to the wrong
node instance (the failure the paper's Section 5 builds its lookup table against) shows up as a row
written twice and another never.  The runs must report TREELSTM_OK and still match the oracle."""
import numpy as np
import pytest
import torch

from oracle import recursive_cells_oracle as rc
from oracle import treelstm_oracle as orc
from paper_1809_00832_b200 import binding, build, forests as fg
from tests import util

pytestmark = pytest.mark.gpu
CHECKED = "checked"


@pytest.mark.parametrize("flags", [binding.PER_LEVEL, binding.PERSISTENT])
def test_checked_fp32_tiny_and_batch25(flags):
    for name in ("tiny8", "batch25_fp32"):
        w = fg.make_workload(name, 0)
        ref = util.oracle_forward_cached(name, 0)
        model = util.make_model(w.params, "fp32", variant=CHECKED)
        res = util.gpu_forward(model, w.forest, flags)          # raises on any recorded error, ERR_CHECK included
        assert model.status_sync() == binding.OK
        util.check_schedule(res, ref, w.forest.n_nodes)
        assert util.max_abs(res["h"], ref["h"]) < util.TOL["fp32"]
        assert util.max_abs(res["c"], ref["c"]) < util.TOL["fp32"]


@pytest.mark.parametrize("flags", [binding.PER_LEVEL, binding.PERSISTENT, binding.SUBFORESTS])
def test_checked_bf16_batch256(flags):
    w = fg.make_workload("batch256_bf16", 0)
    ref = util.oracle_forward_cached("batch256_bf16", 0)
    model = util.make_model(w.params, "bf16", variant=CHECKED)
    forest, new_of_old = fg.permute_node_ids(w.forest, np.random.default_rng(3))
    res = util.gpu_forward(model, forest, flags)
    assert model.status_sync() == binding.OK
    if flags == binding.SUBFORESTS:
        assert model.last_mode() == binding.SUBFORESTS
    assert util.max_abs(res["h"][new_of_old], ref["h"]) < util.TOL["bf16"]
    assert util.max_abs(res["c"][new_of_old], ref["c"]) < util.TOL["bf16"]


def test_checked_cluster_paths_chains_training_and_other_cells():
    rng = np.random.default_rng(5)
    # the narrow tail of a small forest and of a mixed one goes to the cluster kernel
    params = fg.draw_params(rng, 256, 300, 500, emb_dist="normal", emb_scale=0.3, w_scale=0.08)
    model = util.make_model(params, "bf16", variant=CHECKED)
    model.set_option(binding.OPT_TAIL_WIDTH, 64)
    model.set_option(binding.OPT_TAIL_MIN_LEVELS, 2)          # hand over whenever two narrow wavefronts remain
    small = fg.forest_from_shapes([fg.random_split_shape(rng, 40), None, fg.left_chain_shape(9)], rng, 500)
    util.gpu_forward(model, small, binding.PERSISTENT)
    assert model.status_sync() == binding.OK and model.last_launch_count() == 3
    mixed = fg.forest_from_shapes([fg.random_split_shape(rng, 40) for _ in range(30)] + [fg.left_chain_shape(50)] * 3, rng, 500)
    util.gpu_forward(model, mixed, binding.PERSISTENT)
    assert model.status_sync() == binding.OK and model.last_launch_count() == 3
    # 64 dependent wavefronts
    w = fg.make_workload("chains64_bf16", 0)
    model = util.make_model(w.params, "bf16", variant=CHECKED)
    util.gpu_forward(model, w.forest, binding.PERSISTENT)
    assert model.status_sync() == binding.OK
    # training step: the backward kernels read the same index arrays
    w = fg.make_workload("train25_fp32", 0, n_trees=8)
    ref = orc.loss_and_gradients(w.forest.left, w.forest.right, w.forest.token, w.params.emb, w.params.W, w.params.b,
                                 w.params.Wc, w.params.bc, w.labels)
    for flags in (binding.PER_LEVEL, binding.PERSISTENT):
        model = util.make_model(w.params, "fp32", variant=CHECKED)
        model.forward(*(util.to_dev(a) for a in (w.forest.left, w.forest.right, w.forest.token)),
                      flags=flags | binding.SAVE_FOR_BACKWARD)
        g = model.backward(util.to_dev(w.labels), w.forest.n_leaves)
        util.compare_training_step({k: v.cpu().numpy() for k, v in g.items()}, ref, util.TOL["fp32"], util.REL["fp32"])
    # TreeRNN and RNTN
    for cell, kind, tensor in ((binding.CELL_TREERNN, rc.TREERNN, False), (binding.CELL_RNTN, rc.RNTN, True)):
        p = fg.draw_recursive_params(rng, 20, 60, tensor=tensor, emb_scale=0.8, w_scale=0.2, v_scale=0.03)
        forest = fg.random_forest(rng, 9, 1, 20, 60)
        V = util.to_dev(p.V) if tensor else None
        build.build(variant=CHECKED)
        net = binding.TreeLSTM.recursive(cell, p.H, p.vocab, util.to_dev(p.emb), util.to_dev(p.W), util.to_dev(p.b), V,
                                         variant=CHECKED)
        for flags in (binding.PER_LEVEL, binding.PERSISTENT):
            res = util.gpu_forward(net, forest, flags)
            assert net.status_sync() == binding.OK
            h = rc.forward_recursive(kind, forest.left, forest.right, forest.token, p.emb, p.W, p.b, p.V)
            assert util.max_abs(res["h"], h) < util.TOL["fp32"]


def test_checked_build_reports_malformed_forests_as_before():
    """the scheduler's own validation still answers first: a malformed forest is INVALID_FOREST, not a
    check failure, and nothing is evaluated"""
    rng = np.random.default_rng(6)
    params = fg.draw_params(rng, 64, 64, 50, emb_dist="normal", emb_scale=0.3, w_scale=0.1)
    model = util.make_model(params, "bf16", variant=CHECKED)
    bad = [torch.tensor(x, dtype=torch.int32, device="cuda") for x in ([-1, -1, 0, 0], [-1, -1, 1, 1], [0, 1, 0, 0])]
    with pytest.raises(binding.TreeLSTMError) as err:
        model.forward(*bad, flags=binding.PERSISTENT)
    assert err.value.code == binding.ERR_INVALID_FOREST
