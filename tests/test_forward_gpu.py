"""Parity of the CUDA forward path (through the C ABI) against the fp64 oracle on the same seeded
forests: schedule bit-exact, h and c within 1e-4 (fp32) / 3e-2 (bf16 operands)."""
import numpy as np
import pytest
import torch

from oracle import treelstm_oracle as orc
from paper_1809_00832_b200 import binding, forests as fg
from tests import util

pytestmark = pytest.mark.gpu

MODES = [binding.PER_LEVEL, binding.PERSISTENT]


@pytest.mark.parametrize("flags", MODES)
@pytest.mark.parametrize("name", ["tiny8", "batch25_fp32"])
def test_fp32_forward_matches_oracle(name, flags):
    w = fg.make_workload(name, 0)
    ref = util.oracle_forward_cached(name, 0)
    model = util.make_model(w.params, "fp32")
    res = util.gpu_forward(model, w.forest, flags)
    util.check_schedule(res, ref, w.forest.n_nodes)
    assert util.max_abs(res["h"], ref["h"]) < util.TOL["fp32"]
    assert util.max_abs(res["c"], ref["c"]) < util.TOL["fp32"]
    assert model.last_launch_count() >= 2


@pytest.mark.parametrize("single_cta", [True, False])
def test_schedule_paths_agree_with_oracle_on_permuted_ids(single_cta):
    rng = np.random.default_rng(11)
    w = fg.make_workload("batch25_fp32", 3)
    forest, new_of_old = fg.permute_node_ids(w.forest, rng)
    status, parent, level, order, off = orc.schedule(forest.left, forest.right)
    model = util.make_model(w.params, "fp32")
    if not single_cta:
        model.set_option(binding.OPT_SCHED_SINGLE_CTA_MAX, 0)
    res = util.gpu_forward(model, forest, binding.PERSISTENT)
    util.check_schedule(res, dict(level=level, order=order, level_offset=off), forest.n_nodes)
    # the recursive formulation does not depend on the numbering: same state per node
    href, cref, _ = orc.forward_recursive(forest.left, forest.right, forest.token, w.params.emb,
                                          w.params.W, w.params.b)
    assert util.max_abs(res["h"], href) < util.TOL["fp32"]
    assert util.max_abs(res["c"], cref) < util.TOL["fp32"]
    roots = model.roots(forest.n_trees + 3)
    torch.cuda.synchronize()
    n_roots = int(roots["n_roots"].item())
    assert n_roots == forest.n_trees
    ids = roots["root_ids"].cpu().numpy()[:n_roots]
    np.testing.assert_array_equal(ids, np.sort(forest.roots))
    np.testing.assert_array_equal(roots["root_h"].cpu().numpy()[:n_roots], res["h"][ids])
    np.testing.assert_array_equal(roots["root_c"].cpu().numpy()[:n_roots], res["c"][ids])
    res0 = util.gpu_forward(model, w.forest, binding.PERSISTENT)
    np.testing.assert_allclose(res["h"][new_of_old], res0["h"], atol=2e-6)


@pytest.mark.parametrize("single_cta", [True, False])
def test_deep_and_wide_schedules(single_cta):
    """closed-form shapes: chains (many levels, more than one radix digit) and balanced trees"""
    rng = np.random.default_rng(0)
    params = fg.draw_params(rng, 8, 8, 50, emb_dist="uniform", emb_scale=0.1, w_scale=0.1)
    model = util.make_model(params, "fp32")
    if not single_cta:
        model.set_option(binding.OPT_SCHED_SINGLE_CTA_MAX, 0)
    chain = fg.forest_from_shapes([fg.left_chain_shape(300), fg.left_chain_shape(5)], rng, 50)
    res = util.gpu_forward(model, chain, binding.PERSISTENT)
    status, _, level, order, off = orc.schedule(chain.left, chain.right)
    util.check_schedule(res, dict(level=level, order=order, level_offset=off), chain.n_nodes)
    assert res["n_levels"] == 300
    href, cref, _ = orc.forward_recursive(chain.left, chain.right, chain.token, params.emb, params.W, params.b)
    assert util.max_abs(res["h"], href) < util.TOL["fp32"]
    bal = fg.forest_from_shapes([fg.balanced_shape(256)] * 3, rng, 50)
    res = util.gpu_forward(model, bal, binding.PER_LEVEL)
    assert np.diff(res["level_offset"][:10]).tolist() == [3 * 256 >> k for k in range(9)]
    href, cref, _ = orc.forward_recursive(bal.left, bal.right, bal.token, params.emb, params.W, params.b)
    assert util.max_abs(res["h"], href) < util.TOL["fp32"]
    assert util.max_abs(res["c"], cref) < util.TOL["fp32"]


def test_large_forest_uses_multi_cta_schedule():
    """more nodes than the single-CTA scheduler takes (32768): properties that hold at any size plus
    sampled trees against the oracle"""
    rng = np.random.default_rng(5)
    params = fg.draw_params(rng, 16, 16, 100, emb_dist="uniform", emb_scale=0.1, w_scale=0.1)
    forest = fg.random_forest(rng, 2200, 2, 56, 100)
    assert forest.n_nodes > 32768
    model = util.make_model(params, "fp32")
    res = util.gpu_forward(model, forest, binding.PERSISTENT)
    status, _, level, order, off = orc.schedule(forest.left, forest.right)
    util.check_schedule(res, dict(level=level, order=order, level_offset=off), forest.n_nodes)
    sample = [0, 7, 1100, 2199]
    sub = fg.select_trees(forest, sample)
    href, cref, _ = orc.forward_recursive(sub.left, sub.right, sub.token, params.emb, params.W, params.b)
    ids = np.nonzero(np.isin(forest.tree_of, sample))[0]
    assert util.max_abs(res["h"][ids], href) < util.TOL["fp32"]
    assert util.max_abs(res["c"][ids], cref) < util.TOL["fp32"]


def test_edge_cases():
    rng = np.random.default_rng(1)
    params = fg.draw_params(rng, 5, 3, 9, emb_dist="uniform", emb_scale=0.5, w_scale=0.5)
    model = util.make_model(params, "fp32")
    # empty forest
    empty = fg.Forest(*(np.zeros(0, dtype=np.int32) for _ in range(5)))
    for flags in MODES:
        res = util.gpu_forward(model, empty, flags)
        assert res["n_levels"] == 0
    # single leaf, forest of leaves only, and H, E that are not multiples of any tile size
    for shapes in ([None], [None] * 70, [fg.random_split_shape(rng, 3), None]):
        forest = fg.forest_from_shapes(shapes, rng, 9)
        for flags in MODES:
            res = util.gpu_forward(model, forest, flags)
            href, cref, _ = orc.forward_recursive(forest.left, forest.right, forest.token, params.emb,
                                                  params.W, params.b)
            assert util.max_abs(res["h"], href) < util.TOL["fp32"]
            assert util.max_abs(res["c"], cref) < util.TOL["fp32"]


@pytest.mark.parametrize("single_cta", [True, False])
@pytest.mark.parametrize("flags", MODES)
def test_malformed_forests_return_errors(single_cta, flags):
    rng = np.random.default_rng(2)
    params = fg.draw_params(rng, 4, 4, 5, emb_dist="uniform", emb_scale=0.5, w_scale=0.5)
    model = util.make_model(params, "fp32")
    if not single_cta:
        model.set_option(binding.OPT_SCHED_SINGLE_CTA_MAX, 0)
    cases = [
        ([-1, -1, 0], [-1, -1, 3], [0, 1, -1], binding.ERR_INVALID_FOREST),       # child out of range
        ([-1, -1, 0], [-1, -1, -1], [0, 1, 2], binding.ERR_INVALID_FOREST),       # one child only
        ([-1, -1, 0, 0], [-1, -1, 1, 1], [0, 1, 0, 0], binding.ERR_INVALID_FOREST),  # two parents
        ([-1, -1, 0], [-1, -1, 0], [0, 1, 0], binding.ERR_INVALID_FOREST),        # same child twice
        ([-1, -1, 2], [-1, -1, 1], [0, 1, 0], binding.ERR_INVALID_FOREST),        # own child
        ([-1, 2, 1, -1], [-1, 0, 3, -1], [0, 0, 0, 0], binding.ERR_INVALID_FOREST),  # cycle
        ([-1, -1, 0], [-1, -1, 1], [5, 1, -1], binding.ERR_TOKEN_OUT_OF_RANGE),
        ([-1, -1, 0], [-1, -1, 1], [-2, 1, -1], binding.ERR_TOKEN_OUT_OF_RANGE),
    ]
    for l, r, t, code in cases:
        arrs = [torch.tensor(x, dtype=torch.int32, device="cuda") for x in (l, r, t)]
        assert orc.schedule(np.array(l, dtype=np.int32), np.array(r, dtype=np.int32), np.array(t, dtype=np.int32),
                            5)[0] == code
        with pytest.raises(binding.TreeLSTMError) as err:
            model.forward(*arrs, flags=flags)
        assert err.value.code == code
    # the context stays usable
    good = fg.forest_from_shapes([fg.random_split_shape(rng, 6)], rng, 5)
    res = util.gpu_forward(model, good, flags)
    href, _, _ = orc.forward_recursive(good.left, good.right, good.token, params.emb, params.W, params.b)
    assert util.max_abs(res["h"], href) < util.TOL["fp32"]


def test_argument_errors():
    rng = np.random.default_rng(3)
    params = fg.draw_params(rng, 4, 4, 5, emb_dist="uniform", emb_scale=0.5, w_scale=0.5)
    model = util.make_model(params, "fp32")
    lib = model.lib
    z = torch.zeros(8, dtype=torch.int32, device="cuda")
    f = torch.zeros(8, 4, device="cuda")
    ws = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    p = lambda t: None if t is None else __import__("ctypes").c_void_p(t.data_ptr())
    # workspace too small
    rc = lib.treelstm_forward(model.handle, 8, p(z), p(z), p(z), p(f), p(f), p(z), p(z), None, p(z), 0, p(ws), 16, None)
    assert rc == binding.ERR_INVALID_ARG
    rc = lib.treelstm_forward(model.handle, 8, None, p(z), p(z), p(f), p(f), p(z), p(z), None, p(z), 0, p(ws), 1 << 16, None)
    assert rc == binding.ERR_INVALID_ARG
    rc = lib.treelstm_forward(model.handle, 8, p(z), p(z), p(z), p(f), p(f), p(z), p(z), None, p(z), 64, p(ws), 1 << 16, None)
    assert rc == binding.ERR_INVALID_ARG
    assert lib.treelstm_backward(model.handle, p(z), p(f), p(f), p(f), p(f), p(f), p(z), p(f), p(z), None) == binding.ERR_STATE


def test_host_buffer_forward():
    w = fg.make_workload("tiny8", 0)
    ref = util.oracle_forward_cached("tiny8", 0)
    model = util.make_model(w.params, "fp32")
    f = w.forest
    host = [torch.from_numpy(a).pin_memory() for a in (f.left, f.right, f.token)]
    out = model.forward_host(*host, all_states=True, max_roots=f.n_trees)
    assert int(out["n_levels"][0]) == len(ref["level_offset"]) - 1
    assert int(out["n_roots"][0]) == f.n_trees
    np.testing.assert_array_equal(out["order"].numpy(), ref["order"])
    assert util.max_abs(out["h"].numpy(), ref["h"]) < util.TOL["fp32"]
    np.testing.assert_array_equal(out["root_ids"].numpy(), np.sort(f.roots))
    assert util.max_abs(out["root_h"].numpy(), ref["h"][np.sort(f.roots)]) < util.TOL["fp32"]
    assert util.max_abs(out["root_c"].numpy(), ref["c"][np.sort(f.roots)]) < util.TOL["fp32"]
    # roots only, second call reuses the library's staging buffers
    out2 = model.forward_host(*host, max_roots=f.n_trees)
    np.testing.assert_array_equal(out2["root_h"].numpy(), out["root_h"].numpy())


def test_bounded_waits_time_out_cleanly():
    """failure detection without a fault: a wait on a flag that nothing sets ends by its cycle limit,
    the status word says TIMEOUT, and the context keeps working afterwards"""
    w = fg.make_workload("tiny8", 0)
    ref = util.oracle_forward_cached("tiny8", 0)
    model = util.make_model(w.params, "fp32")
    model.set_option(binding.OPT_WAIT_LIMIT_CYCLES, 200)          # 200 * 1024 cycles, about 0.1 ms
    first_ok, status1, second_ok, status2 = model.selftest_waits()
    assert first_ok == 0 and status1 == binding.ERR_TIMEOUT
    assert second_ok == 0 and status2 == binding.ERR_TIMEOUT
    model.set_option(binding.OPT_WAIT_LIMIT_CYCLES, 1 << 20)
    res = util.gpu_forward(model, w.forest, binding.PERSISTENT)
    assert util.max_abs(res["h"], ref["h"]) < util.TOL["fp32"]


@pytest.mark.parametrize("H,E", [(33, 7), (170, 20), (200, 12), (96, 300)])
def test_fp32_persistent_odd_and_large_hidden_sizes(H, E):
    """hidden sizes that end in a partial 16-unit slice (33), odd sizes (scalar operand fetch), sizes
    whose weight slice still fits in shared memory (170) and sizes where it does not (200: the kernel
    streams the weights as in per-level mode); both modes against the oracle, and against each other"""
    rng = np.random.default_rng(H * 1000 + E)
    params = fg.draw_params(rng, H, E, 60, emb_dist="uniform", emb_scale=0.5, w_scale=0.3 / np.sqrt(H / 16))
    forest = fg.random_forest(rng, 40, 1, 30, 60)      # wide leaf wavefront (64-row tiles) and narrow ones
    forest, _ = fg.permute_node_ids(forest, rng)
    model = util.make_model(params, "fp32")
    h, c, _ = orc.forward_recursive(forest.left, forest.right, forest.token, params.emb, params.W, params.b)
    for flags in (binding.PER_LEVEL, binding.PERSISTENT):
        res = util.gpu_forward(model, forest, flags)
        assert util.max_abs(res["h"], h) < util.TOL["fp32"]
        assert util.max_abs(res["c"], c) < util.TOL["fp32"]
