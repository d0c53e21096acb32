"""Parity of the CUDA training step (forward + backward through structure, via the C ABI) against
the fp64 oracle: loss and every gradient group within 1e-4 max-abs and within 2e-5 of the group's
own largest entry (several groups of the full-size workload lie below 1e-4 altogether)."""
import numpy as np
import pytest
import torch

from oracle import treelstm_oracle as orc
from paper_1809_00832_b200 import binding, forests as fg
from tests import util

pytestmark = pytest.mark.gpu


def _train_step(model, forest, labels, flags):
    out = model.forward(util.to_dev(forest.left), util.to_dev(forest.right), util.to_dev(forest.token),
                        flags=flags | binding.SAVE_FOR_BACKWARD)
    grads = model.backward(util.to_dev(labels), forest.n_leaves)
    torch.cuda.synchronize()
    res = {k: v.cpu().numpy() for k, v in grads.items()}
    res["h"] = out["h"].cpu().numpy()
    return res


def _compare(res, ref, tol):
    util.compare_training_step(res, ref, tol, util.REL["fp32"], loss_rel=1e-5)


@pytest.mark.parametrize("flags", [binding.PER_LEVEL, binding.PERSISTENT])
def test_training_step_matches_oracle(flags):
    w = fg.make_workload("train25_fp32", 0)
    f, p = w.forest, w.params
    ref = orc.loss_and_gradients(f.left, f.right, f.token, p.emb, p.W, p.b, p.Wc, p.bc, w.labels)
    model = util.make_model(p, "fp32")
    res = _train_step(model, f, w.labels, flags)
    assert util.max_abs(res["h"], ref["h"]) < util.TOL["fp32"]
    _compare(res, ref, util.TOL["fp32"])
    # gradients are overwritten, not accumulated: a second step gives the same numbers
    res2 = _train_step(model, f, w.labels, flags)
    _compare(res2, ref, util.TOL["fp32"])


@pytest.mark.parametrize("flags", [binding.PER_LEVEL, binding.PERSISTENT])
def test_training_step_full_size_with_large_gradients(flags):
    """the sizes of the training workload (H=150, E=300: 64 x 64 dW tiles, dIn chunks split over
    CTAs) with weights six times larger, so that every gradient group is far above the tolerance"""
    rng = np.random.default_rng(150)
    params = fg.draw_params(rng, 150, 300, 2000, emb_dist="normal", emb_scale=0.1, w_scale=0.3, n_classes=5)
    forest = fg.random_forest(rng, 25, 2, 56, 2000)
    forest, _ = fg.permute_node_ids(forest, rng)
    labels = rng.integers(0, 5, size=forest.n_nodes).astype(np.int32)
    ref = orc.loss_and_gradients(forest.left, forest.right, forest.token, params.emb, params.W, params.b,
                                 params.Wc, params.bc, labels)
    for k in util.GRAD_KEYS + ("dEmb_rows",):
        assert np.max(np.abs(ref[k])) > 5 * util.TOL["fp32"], k      # the case has signal in every group
    model = util.make_model(params, "fp32")
    res = _train_step(model, forest, labels, flags)
    assert util.max_abs(res["h"], ref["h"]) < util.TOL["fp32"]
    _compare(res, ref, util.TOL["fp32"])


def test_training_step_small_odd_sizes_and_duplicates():
    # larger gradients (weights +-0.5), sizes that match no tile, permuted ids, duplicated tokens and
    # duplicated subtrees: every node must receive its own forward values
    rng = np.random.default_rng(4)
    params = fg.draw_params(rng, 7, 5, 6, emb_dist="uniform", emb_scale=0.5, w_scale=0.5, n_classes=3)
    shape = fg.random_split_shape(rng, 9)
    forest = fg.forest_from_shapes([shape, shape, None, fg.left_chain_shape(12)], rng, 6)
    forest, _ = fg.permute_node_ids(forest, rng)
    labels = rng.integers(0, 3, size=forest.n_nodes).astype(np.int32)
    ref = orc.loss_and_gradients(forest.left, forest.right, forest.token, params.emb, params.W, params.b,
                                 params.Wc, params.bc, labels)
    model = util.make_model(params, "fp32")
    res = _train_step(model, forest, labels, binding.PERSISTENT)
    _compare(res, ref, util.TOL["fp32"])


def test_backward_errors():
    rng = np.random.default_rng(6)
    params = fg.draw_params(rng, 4, 4, 5, emb_dist="uniform", emb_scale=0.5, w_scale=0.5, n_classes=3)
    model = util.make_model(params, "fp32")
    forest = fg.forest_from_shapes([fg.random_split_shape(rng, 5)], rng, 5)
    arrs = [util.to_dev(a) for a in (forest.left, forest.right, forest.token)]
    labels = torch.zeros(forest.n_nodes, dtype=torch.int32, device="cuda")
    model.forward(*arrs, flags=binding.PERSISTENT)                  # nothing saved
    with pytest.raises(binding.TreeLSTMError) as err:
        model.backward(labels, forest.n_leaves)
    assert err.value.code == binding.ERR_STATE
    model.forward(*arrs, flags=binding.PERSISTENT | binding.SAVE_FOR_BACKWARD)
    labels[2] = 3
    with pytest.raises(binding.TreeLSTMError) as err:
        model.backward(labels, forest.n_leaves)
    assert err.value.code == binding.ERR_LABEL_OUT_OF_RANGE


def test_data_parallel_step_single_rank():
    """the data-parallel wrapper on one rank: same gradients, touched rows trimmed to their count"""
    from paper_1809_00832_b200 import data_parallel
    w = fg.make_workload("train25_fp32", 0, n_trees=6)
    f, p = w.forest, w.params
    ref = orc.loss_and_gradients(f.left, f.right, f.token, p.emb, p.W, p.b, p.Wc, p.bc, w.labels)
    model = util.make_model(p, "fp32")
    out = data_parallel.training_step(model, util.to_dev(f.left), util.to_dev(f.right), util.to_dev(f.token),
                                      util.to_dev(w.labels), f.n_leaves, binding.PERSISTENT)
    res = {k: v.cpu().numpy() for k, v in out.items()}
    assert res["touched_ids"].shape[0] == len(ref["touched_ids"])
    _compare(res, ref, util.TOL["fp32"])


@pytest.mark.parametrize("tensor_cores", [1, 0])
def test_weight_gradient_on_tensor_cores_and_on_fp32_units(tensor_cores):
    """dW and db of the one-launch backward, formed either by the split-bf16 tensor-core contraction
    (three bf16 pieces per fp32 value, six products per term) or by fp32 multiply-adds: both must meet
    the fp32 bounds against the oracle, on the full-size case with large gradients (several row tiles,
    a ragged last gate-column tile, several node runs) and on sizes that fill no tile"""
    rng = np.random.default_rng(151)
    cases = [(150, 300, 2000, fg.random_forest(rng, 25, 2, 56, 2000), 5, 0.3),
             (7, 5, 6, fg.forest_from_shapes([fg.random_split_shape(rng, 9), None, fg.left_chain_shape(70)], rng, 6), 3, 0.5)]
    for H, E, vocab, forest, n_classes, w_scale in cases:
        params = fg.draw_params(rng, H, E, vocab, emb_dist="normal", emb_scale=0.1, w_scale=w_scale, n_classes=n_classes)
        forest, _ = fg.permute_node_ids(forest, rng)
        labels = rng.integers(0, n_classes, size=forest.n_nodes).astype(np.int32)
        ref = orc.loss_and_gradients(forest.left, forest.right, forest.token, params.emb, params.W, params.b,
                                     params.Wc, params.bc, labels)
        model = util.make_model(params, "fp32")
        model.set_option(binding.OPT_DW_TENSOR_CORES, tensor_cores)
        res = _train_step(model, forest, labels, binding.PERSISTENT)
        _compare(res, ref, util.TOL["fp32"])


def test_training_step_on_forests_of_single_leaves_and_with_a_large_vocabulary():
    """no internal node at all (the weight gradient's second part is empty, W_h gets zeros), and a
    vocabulary beyond what the token scan keeps in shared memory (its ballots are then read again)"""
    rng = np.random.default_rng(152)
    vocab = 400_000
    params = fg.draw_params(rng, 6, 4, vocab, emb_dist="uniform", emb_scale=0.5, w_scale=0.5, n_classes=3)
    for shapes in ([None, None, None], [fg.random_split_shape(rng, 40), None, fg.left_chain_shape(5)]):
        forest = fg.forest_from_shapes(shapes, rng, vocab)
        forest.token[int(np.flatnonzero(forest.left < 0)[0])] = vocab - 1   # the last id of the table is in use
        labels = rng.integers(0, 3, size=forest.n_nodes).astype(np.int32)
        ref = orc.loss_and_gradients(forest.left, forest.right, forest.token, params.emb, params.W, params.b,
                                     params.Wc, params.bc, labels)
        model = util.make_model(params, "fp32")
        for flags in (binding.PERSISTENT, binding.PER_LEVEL):
            res = _train_step(model, forest, labels, flags)
            _compare(res, ref, util.TOL["fp32"])


@pytest.mark.parametrize("ctas", [1, 3, 40])
def test_training_step_on_small_grids(ctas):
    """the one-launch backward on a grid of one CTA (token scan and classifier in the same CTA), of a few
    CTAs (every CTA takes several blocks of a narrow wavefront, only the first of them fetched ahead of
    the grid barrier) and of fewer CTAs than a narrow wavefront has blocks"""
    rng = np.random.default_rng(160 + ctas)
    params = fg.draw_params(rng, 20, 12, 300, emb_dist="normal", emb_scale=0.3, w_scale=0.3, n_classes=4)
    forest = fg.random_forest(rng, 9, 2, 40, 300)
    forest, _ = fg.permute_node_ids(forest, rng)
    labels = rng.integers(0, 4, size=forest.n_nodes).astype(np.int32)
    ref = orc.loss_and_gradients(forest.left, forest.right, forest.token, params.emb, params.W, params.b,
                                 params.Wc, params.bc, labels)
    model = util.make_model(params, "fp32")
    model.set_option(binding.OPT_MAX_CTAS, ctas)
    res = _train_step(model, forest, labels, binding.PERSISTENT)
    _compare(res, ref, util.TOL["fp32"])
