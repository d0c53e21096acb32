"""Parity of the TreeRNN and RNTN forward (the paper's other two evaluation models, Section 6.1)
through the C ABI against their fp64 oracle: schedule bit-exact, states within 1e-4 max-abs (fp32
arithmetic) and within 1e-4 of the largest state."""
import numpy as np
import pytest
import torch

from oracle import recursive_cells_oracle as rc
from oracle import treelstm_oracle as orc
from paper_1809_00832_b200 import binding, forests as fg
from tests import util

pytestmark = pytest.mark.gpu

MODES = [binding.PER_LEVEL, binding.PERSISTENT]
KIND = {binding.CELL_TREERNN: rc.TREERNN, binding.CELL_RNTN: rc.RNTN}


def _model(cell, p):
    util.lib_ready()
    V = util.to_dev(p.V) if p.V is not None else None
    return binding.TreeLSTM.recursive(cell, p.H, p.vocab, util.to_dev(p.emb), util.to_dev(p.W), util.to_dev(p.b), V)


def _check(cell, p, forest, flags):
    model = _model(cell, p)
    res = util.gpu_forward(model, forest, flags)
    status, _, level, order, off = orc.schedule(forest.left, forest.right)
    util.check_schedule(res, dict(level=level, order=order, level_offset=off), forest.n_nodes)
    h = rc.forward_recursive(KIND[cell], forest.left, forest.right, forest.token, p.emb, p.W, p.b, p.V)
    err = util.max_abs(res["h"], h)
    assert err < util.TOL["fp32"], err
    assert err <= 1e-4 * np.max(np.abs(h))
    assert "c" not in res                               # these cells have no cell state
    np.testing.assert_array_equal(res["h"][forest.left < 0], p.emb[forest.token[forest.left < 0]])
    return model, res, h


@pytest.mark.parametrize("flags", MODES)
@pytest.mark.parametrize("H", [16, 50, 150])
def test_treernn_matches_oracle(H, flags):
    """sizes below, across and above one 64-unit tile; several row tiles and a ragged tail; permuted ids"""
    rng = np.random.default_rng(100 + H)
    p = fg.draw_recursive_params(rng, H, 300, tensor=False, emb_scale=0.8, w_scale=1.5 / np.sqrt(2 * H))
    forest = fg.random_forest(rng, 25, 2, 56, 300)
    forest, _ = fg.permute_node_ids(forest, rng)
    _check(binding.CELL_TREERNN, p, forest, flags)


@pytest.mark.parametrize("flags", MODES)
@pytest.mark.parametrize("H", [8, 25, 40])
def test_rntn_matches_oracle(H, flags):
    """the tensor term is a contraction over 4H^2 products per node; H = 25 (the size of the original
    model) and sizes that match no tile"""
    rng = np.random.default_rng(200 + H)
    p = fg.draw_recursive_params(rng, H, 200, tensor=True, emb_scale=0.8, w_scale=1.0 / np.sqrt(2 * H),
                                 v_scale=1.0 / (2 * H))
    forest = fg.random_forest(rng, 12, 1, 30, 200)
    forest, _ = fg.permute_node_ids(forest, rng)
    model, res, h = _check(binding.CELL_RNTN, p, forest, flags)
    # the tensor term matters at these scales: the same forest without it differs visibly
    h0 = rc.forward_recursive(rc.TREERNN, forest.left, forest.right, forest.token, p.emb, p.W, p.b)
    assert np.max(np.abs(h0 - h)) > 50 * util.TOL["fp32"]


@pytest.mark.parametrize("cell", [binding.CELL_TREERNN, binding.CELL_RNTN])
def test_shape_extremes_edge_cases_and_roots(cell):
    """left chains (one node per tree and wavefront), balanced trees, single leaves, the empty forest;
    roots come back with their states"""
    rng = np.random.default_rng(7)
    H = 24
    p = fg.draw_recursive_params(rng, H, 50, tensor=cell == binding.CELL_RNTN, emb_scale=0.8,
                                 w_scale=1.0 / np.sqrt(2 * H), v_scale=1.0 / (2 * H))
    shapes = [fg.left_chain_shape(40), fg.balanced_shape(64), None, None, fg.left_chain_shape(3)]
    forest = fg.forest_from_shapes(shapes, rng, 50)
    for flags in MODES:
        model, res, h = _check(cell, p, forest, flags)
        assert res["n_levels"] == 40
        roots = model.roots(forest.n_trees)
        torch.cuda.synchronize()
        ids = roots["root_ids"].cpu().numpy()
        np.testing.assert_array_equal(ids, np.sort(forest.roots))
        np.testing.assert_array_equal(roots["root_h"].cpu().numpy(), res["h"][ids])
    empty = fg.Forest(*(np.zeros(0, dtype=np.int32) for _ in range(5)))
    model = _model(cell, p)
    for flags in MODES:
        assert util.gpu_forward(model, empty, flags)["n_levels"] == 0
    # a malformed forest is still an error code; a backward without a classifier is refused
    bad = [torch.tensor(x, dtype=torch.int32, device="cuda") for x in ([-1, -1, 0], [-1, -1, 3], [0, 1, -1])]
    with pytest.raises(binding.TreeLSTMError) as err:
        model.forward(*bad, flags=binding.PERSISTENT)
    assert err.value.code == binding.ERR_INVALID_FOREST
    good = [util.to_dev(a) for a in (forest.left, forest.right, forest.token)]
    model.forward(*good, flags=binding.PERSISTENT | binding.SAVE_FOR_BACKWARD)
    with pytest.raises(binding.TreeLSTMError) as err:
        model.backward_recursive(util.to_dev(np.zeros(forest.n_nodes, np.int32)), forest.n_leaves)
    assert err.value.code in (binding.ERR_STATE, binding.ERR_INVALID_ARG)    # no classifier: empty gradient buffers


def test_treernn_large_hidden_size_and_host_entry_point():
    """H = 256 (four unit tiles, 64 KB of staged child states per tile) through the host-buffer call"""
    rng = np.random.default_rng(9)
    H = 256
    p = fg.draw_recursive_params(rng, H, 400, tensor=False, emb_scale=0.8, w_scale=1.5 / np.sqrt(2 * H))
    forest = fg.random_forest(rng, 30, 2, 56, 400)
    model = _model(binding.CELL_TREERNN, p)
    host = binding.pack_forest_host(forest.left, forest.right, forest.token)
    out = model.forward_host(*host, all_states=True, max_roots=forest.n_trees)
    h = rc.forward_recursive(rc.TREERNN, forest.left, forest.right, forest.token, p.emb, p.W, p.b)
    assert util.max_abs(out["h"].numpy(), h) < util.TOL["fp32"]
    roots = np.sort(forest.roots)
    np.testing.assert_array_equal(out["root_ids"].numpy(), roots)
    assert util.max_abs(out["root_h"].numpy(), h[roots]) < util.TOL["fp32"]


def _training_step(cell, p, forest, flags, n_classes=5, seed=7):
    rng = np.random.default_rng(seed)
    Wc = rng.uniform(-0.3, 0.3, size=(p.H, n_classes)).astype(np.float32)
    bc = rng.uniform(-0.1, 0.1, size=n_classes).astype(np.float32)
    labels = rng.integers(0, n_classes, size=forest.n_nodes).astype(np.int32)
    ref = rc.loss_and_gradients(KIND[cell], forest.left, forest.right, forest.token, p.emb, p.W, p.b, Wc, bc, labels, p.V)
    model = _model(cell, p)
    model.set_classifier(util.to_dev(Wc), util.to_dev(bc))
    model.forward(util.to_dev(forest.left), util.to_dev(forest.right), util.to_dev(forest.token),
                  flags=flags | binding.SAVE_FOR_BACKWARD)
    g = {k: v.cpu().numpy() for k, v in model.backward_recursive(util.to_dev(labels), forest.n_leaves).items()}
    util.compare_training_step(g, ref, util.TOL["fp32"], util.REL["fp32"], loss_rel=1e-5)
    if cell == binding.CELL_RNTN:
        err, scale = util.max_abs(g["dV"], ref["dV"]), float(np.max(np.abs(ref["dV"])))
        assert err < util.TOL["fp32"] and err <= util.REL["fp32"] * scale, (err, scale)
        assert scale > 0 or forest.n_nodes == forest.n_leaves
    model.close()
    return g, ref


@pytest.mark.parametrize("flags", MODES)
@pytest.mark.parametrize("H", [16, 50, 130])
def test_treernn_training_step_matches_oracle(H, flags):
    """loss and every gradient group (dW, db, dWc, dbc, touched embedding rows) of backpropagation
    through structure against the fp64 oracle: absolute 1e-4 and 2e-5 of each group's largest entry;
    duplicate tokens (vocabulary smaller than the number of leaves) accumulate into one row"""
    rng = np.random.default_rng(300 + H)
    p = fg.draw_recursive_params(rng, H, 40, tensor=False, emb_scale=0.8, w_scale=1.5 / np.sqrt(2 * H))
    forest = fg.random_forest(rng, 20, 1, 40, 40)
    forest, _ = fg.permute_node_ids(forest, rng)
    g, ref = _training_step(binding.CELL_TREERNN, p, forest, flags)
    assert len(ref["touched_ids"]) < forest.n_leaves          # duplicates were there
    assert float(np.max(np.abs(ref["dW"]))) > 100 * util.TOL["fp32"] * util.REL["fp32"]


@pytest.mark.parametrize("flags", MODES)
@pytest.mark.parametrize("H", [8, 25])
def test_rntn_training_step_matches_oracle(H, flags):
    """the same with the tensor term: dV [H][2H][2H] and the (V_j + V_j^T) x part of the children's gradient"""
    rng = np.random.default_rng(400 + H)
    p = fg.draw_recursive_params(rng, H, 60, tensor=True, emb_scale=0.8, w_scale=1.0 / np.sqrt(2 * H),
                                 v_scale=1.0 / (2 * H))
    forest = fg.random_forest(rng, 10, 1, 24, 60)
    forest, _ = fg.permute_node_ids(forest, rng)
    _training_step(binding.CELL_RNTN, p, forest, flags)


def test_recursive_training_edge_cases():
    """a forest of single-leaf trees only (no internal node: dW, db, dV are zero, the embedding rows carry
    the classifier's gradient), and the wrong backward call for the context kind is refused"""
    rng = np.random.default_rng(500)
    p = fg.draw_recursive_params(rng, 12, 30, tensor=True, emb_scale=0.8, w_scale=0.3, v_scale=0.05)
    forest = fg.random_forest(rng, 9, 1, 1, 30)
    g, ref = _training_step(binding.CELL_RNTN, p, forest, binding.PERSISTENT)
    assert not g["dW"].any() and not g["dV"].any() and not g["db"].any()
    model = _model(binding.CELL_TREERNN, p)
    model.set_classifier(util.to_dev(np.zeros((12, 3), np.float32)), util.to_dev(np.zeros(3, np.float32)))
    model.forward(util.to_dev(forest.left), util.to_dev(forest.right), util.to_dev(forest.token),
                  flags=binding.PERSISTENT | binding.SAVE_FOR_BACKWARD)
    with pytest.raises(binding.TreeLSTMError):
        model.backward(util.to_dev(np.zeros(forest.n_nodes, np.int32)), forest.n_leaves)
    model.close()
