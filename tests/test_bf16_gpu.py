"""Parity of the bf16 tensor-core forward (tcgen05 path, through the C ABI) against the fp64 oracle:
schedule bit-exact, h and c within 3e-2 max-abs; against the oracle with the same operands rounded
to bf16 the agreement must be much tighter (separates operand rounding from kernel mistakes)."""
import dataclasses

import numpy as np
import pytest

from oracle import treelstm_oracle as orc
from paper_1809_00832_b200 import binding, forests as fg
from tests import util

pytestmark = pytest.mark.gpu

MODES = [binding.PER_LEVEL, binding.PERSISTENT, binding.SUBFORESTS]
TIGHT = util.TIGHT   # vs. the oracle fed bf16-rounded operands: only accumulation order, fast
                     # activations and the bf16 rounding of h at slightly different values remain


def _subforests_apply(params, forest):
    """sub-forest mode exists for hidden sizes whose 64-padded value is 64, 128, 192 or 256 and
    forests the single-CTA scheduler can partition"""
    return -(-params.H // 64) * 64 <= 256 and forest.n_nodes <= 24576


def _check(params, forest, flags, full_ref=None, rounded_ref=None):
    model = util.make_model(params, "bf16")
    res = util.gpu_forward(model, forest, flags)
    res["mode_ran"] = model.last_mode()
    if flags == binding.SUBFORESTS and _subforests_apply(params, forest):
        assert model.last_mode() == binding.SUBFORESTS     # the cluster kernel ran, not its stand-in
    status, _, level, order, off = orc.schedule(forest.left, forest.right)
    util.check_schedule(res, dict(level=level, order=order, level_offset=off), forest.n_nodes)
    if full_ref is None:
        h, c, _ = orc.forward_recursive(forest.left, forest.right, forest.token, params.emb, params.W, params.b)
    else:
        h, c = full_ref["h"], full_ref["c"]
    assert util.max_abs(res["h"], h) < util.TOL["bf16"]
    assert util.max_abs(res["c"], c) < util.TOL["bf16"]
    if rounded_ref is not None:
        assert util.max_abs(res["h"], rounded_ref["h"]) < util.TIGHT_FULL_SIZE
        assert util.max_abs(res["c"], rounded_ref["c"]) < util.TIGHT_FULL_SIZE
    return res


@pytest.mark.parametrize("flags", MODES)
@pytest.mark.parametrize("H,E", [(64, 64), (32, 20), (150, 300), (72, 130)])
def test_bf16_small_matches_oracle_and_rounded_oracle(H, E, flags):
    rng = np.random.default_rng(H + E)
    params = fg.draw_params(rng, H, E, 500, emb_dist="normal", emb_scale=0.3, w_scale=0.2)
    forest = fg.random_forest(rng, 9, 1, 40, 500)          # > 128 leaves: several row tiles + ragged tail
    forest, _ = fg.permute_node_ids(forest, rng)
    res = _check(params, forest, flags)
    hr, cr, _ = orc.forward_recursive(forest.left, forest.right, forest.token, params.emb, params.W, params.b,
                                      operand_round=orc.round_to_bf16)
    assert util.max_abs(res["h"], hr) < TIGHT
    assert util.max_abs(res["c"], cr) < TIGHT


@pytest.mark.parametrize("flags", MODES)
def test_bf16_batch256_matches_oracle(flags):
    w = fg.make_workload("batch256_bf16", 0)
    ref = util.oracle_forward_cached("batch256_bf16", 0)
    _check(w.params, w.forest, flags, ref, util.oracle_forward_cached("batch256_bf16", 0, rounded=True))


@pytest.mark.parametrize("flags", MODES)
def test_bf16_chains_match_oracle(flags):
    """64 left chains of 64 leaves: 64 dependent wavefronts, error growth over depth stays bounded"""
    w = fg.make_workload("chains64_bf16", 0)
    ref = util.oracle_forward_cached("chains64_bf16", 0)
    res = _check(w.params, w.forest, flags, ref, util.oracle_forward_cached("chains64_bf16", 0, rounded=True))
    assert res["n_levels"] == 64


@pytest.mark.parametrize("flags", MODES)
def test_bf16_balanced_full_size_all_nodes(flags):
    """16 balanced trees of 1024 leaves in the benchmark's launch configuration: schedule exact and
    states of all 32752 nodes against the oracle and the rounded-operand oracle.  The forest is too
    large to be dealt out to sub-forests, so that flag must report the persistent kernel."""
    w = fg.make_workload("balanced1024_bf16", 0)
    ref = util.oracle_forward_cached("balanced1024_bf16", 0)
    res = _check(w.params, w.forest, flags, ref, util.oracle_forward_cached("balanced1024_bf16", 0, rounded=True))
    assert np.diff(ref["level_offset"]).tolist() == [16 * 1024 >> k for k in range(11)]
    assert res["n_levels"] == 11
    if flags == binding.SUBFORESTS:
        assert res["mode_ran"] == binding.PERSISTENT


def test_bf16_forward_then_fp32_backward():
    """a bf16 forward keeps the gates; backward (fp32 arithmetic) then matches the oracle's gradients
    to the accuracy the bf16 forward values allow"""
    rng = np.random.default_rng(12)
    params = fg.draw_params(rng, 64, 40, 300, emb_dist="normal", emb_scale=0.3, w_scale=0.1, n_classes=5)
    forest = fg.random_forest(rng, 6, 2, 30, 300)
    labels = rng.integers(0, 5, size=forest.n_nodes).astype(np.int32)
    ref = orc.loss_and_gradients(forest.left, forest.right, forest.token, params.emb, params.W, params.b,
                                 params.Wc, params.bc, labels)
    model = util.make_model(params, "bf16")
    model.forward(util.to_dev(forest.left), util.to_dev(forest.right), util.to_dev(forest.token),
                  flags=binding.PERSISTENT | binding.SAVE_FOR_BACKWARD)
    g = model.backward(util.to_dev(labels), forest.n_leaves)
    util.compare_training_step({k: v.cpu().numpy() for k, v in g.items()}, ref, util.TOL["bf16"], util.REL["bf16"])


def test_bf16_large_forest_multi_cta_schedule():
    """more nodes than the single-CTA scheduler takes: the multi-CTA scheduler feeds the tensor-core
    kernel; schedule exact on all nodes, states checked on sampled whole trees"""
    rng = np.random.default_rng(31)
    params = fg.draw_params(rng, 64, 48, 400, emb_dist="normal", emb_scale=0.3, w_scale=0.15)
    forest = fg.random_forest(rng, 1500, 2, 56, 400)
    assert forest.n_nodes > 32768
    model = util.make_model(params, "bf16")
    res = util.gpu_forward(model, forest, binding.PERSISTENT)
    status, _, level, order, off = orc.schedule(forest.left, forest.right)
    util.check_schedule(res, dict(level=level, order=order, level_offset=off), forest.n_nodes)
    sample = [3, 700, 1499]
    sub = fg.select_trees(forest, sample)
    h, c, _ = orc.forward_recursive(sub.left, sub.right, sub.token, params.emb, params.W, params.b)
    ids = np.nonzero(np.isin(forest.tree_of, sample))[0]
    assert util.max_abs(res["h"][ids], h) < util.TOL["bf16"]
    assert util.max_abs(res["c"][ids], c) < util.TOL["bf16"]
    assert np.all(np.isfinite(res["h"]))


def test_bf16_repeated_calls_and_changing_sizes():
    """the same context evaluates forests of different sizes back to back (operand maps are rebuilt,
    stale operand rows of an earlier, larger forest must not leak into a later one)"""
    rng = np.random.default_rng(32)
    params = fg.draw_params(rng, 64, 64, 300, emb_dist="normal", emb_scale=0.3, w_scale=0.2)
    model = util.make_model(params, "bf16")
    for n_trees in (40, 3, 17, 40):
        forest = fg.random_forest(rng, n_trees, 1, 30, 300)
        res = util.gpu_forward(model, forest, binding.PERSISTENT)
        h, c, _ = orc.forward_recursive(forest.left, forest.right, forest.token, params.emb, params.W, params.b)
        assert util.max_abs(res["h"], h) < util.TOL["bf16"]
        assert util.max_abs(res["c"], c) < util.TOL["bf16"]


def test_subforest_mode_single_tree_and_fewer_trees_than_clusters():
    """fewer trees than clusters: the spare clusters get empty sub-forests and leave at once"""
    rng = np.random.default_rng(41)
    params = fg.draw_params(rng, 128, 50, 300, emb_dist="normal", emb_scale=0.3, w_scale=0.15)
    for n_trees in (1, 2, 5):
        forest = fg.random_forest(rng, n_trees, 1, 56, 300)
        forest, _ = fg.permute_node_ids(forest, rng)
        _check(params, forest, binding.SUBFORESTS)


def test_subforest_mode_single_leaf_trees():
    """trees that are a single leaf: sub-forests with one wavefront only"""
    rng = np.random.default_rng(42)
    params = fg.draw_params(rng, 64, 64, 100, emb_dist="normal", emb_scale=0.3, w_scale=0.2)
    forest = fg.random_forest(rng, 20, 1, 1, 100)
    assert forest.n_nodes == 20
    _check(params, forest, binding.SUBFORESTS)


def test_subforest_mode_falls_back_when_it_does_not_apply():
    """H padded beyond 256: the call runs the grid-wide persistent kernel and says so"""
    rng = np.random.default_rng(43)
    params = fg.draw_params(rng, 264, 32, 100, emb_dist="normal", emb_scale=0.3, w_scale=0.05)
    forest = fg.random_forest(rng, 4, 2, 12, 100)
    model = util.make_model(params, "bf16")
    assert model.subforest_count() == 0
    res = util.gpu_forward(model, forest, binding.SUBFORESTS)
    assert model.last_mode() == binding.PERSISTENT
    h, c, _ = orc.forward_recursive(forest.left, forest.right, forest.token, params.emb, params.W, params.b)
    assert util.max_abs(res["h"], h) < util.TOL["bf16"]


def test_subforest_mode_repeated_calls():
    rng = np.random.default_rng(44)
    params = fg.draw_params(rng, 256, 64, 300, emb_dist="normal", emb_scale=0.3, w_scale=0.1)
    model = util.make_model(params, "bf16")
    assert model.subforest_count() >= 1
    for n_trees in (40, 3, 17, 40):
        forest = fg.random_forest(rng, n_trees, 1, 30, 300)
        res = util.gpu_forward(model, forest, binding.SUBFORESTS)
        assert model.last_mode() == binding.SUBFORESTS
        h, c, _ = orc.forward_recursive(forest.left, forest.right, forest.token, params.emb, params.W, params.b)
        assert util.max_abs(res["h"], h) < util.TOL["bf16"]
        assert util.max_abs(res["c"], c) < util.TOL["bf16"]


def test_subforest_forward_then_backward():
    """the sub-forest kernel keeps the gate activations too; the one-launch backward then matches the
    oracle's gradients to the accuracy the bf16 forward values allow"""
    rng = np.random.default_rng(45)
    params = fg.draw_params(rng, 64, 40, 300, emb_dist="normal", emb_scale=0.3, w_scale=0.1, n_classes=5)
    forest = fg.random_forest(rng, 11, 2, 30, 300)
    forest, _ = fg.permute_node_ids(forest, rng)
    labels = rng.integers(0, 5, size=forest.n_nodes).astype(np.int32)
    ref = orc.loss_and_gradients(forest.left, forest.right, forest.token, params.emb, params.W, params.b,
                                 params.Wc, params.bc, labels)
    model = util.make_model(params, "bf16")
    out = model.forward(util.to_dev(forest.left), util.to_dev(forest.right), util.to_dev(forest.token),
                        flags=binding.SUBFORESTS | binding.SAVE_FOR_BACKWARD)
    assert model.last_mode() == binding.SUBFORESTS
    assert util.max_abs(out["h"].cpu().numpy(), ref["h"]) < util.TOL["bf16"]
    g = model.backward(util.to_dev(labels), forest.n_leaves)
    util.compare_training_step({k: v.cpu().numpy() for k, v in g.items()}, ref, util.TOL["bf16"], util.REL["bf16"])


def test_subforest_mode_through_the_host_entry_point():
    """treelstm_forward_host with the sub-forest flag: roots and their states come back in node order"""
    import torch
    rng = np.random.default_rng(46)
    params = fg.draw_params(rng, 128, 64, 300, emb_dist="normal", emb_scale=0.3, w_scale=0.1)
    forest = fg.random_forest(rng, 9, 1, 40, 300)
    model = util.make_model(params, "bf16")
    host = binding.pack_forest_host(forest.left, forest.right, forest.token)   # adjacent arrays: single-copy path
    out = model.forward_host(*host, flags=binding.SUBFORESTS, all_states=True, max_roots=forest.n_trees)
    assert model.last_mode() == binding.SUBFORESTS
    h, c, _ = orc.forward_recursive(forest.left, forest.right, forest.token, params.emb, params.W, params.b)
    assert util.max_abs(out["h"].numpy(), h) < util.TOL["bf16"]
    assert int(out["n_roots"][0]) == forest.n_trees
    roots = np.sort(forest.roots)
    np.testing.assert_array_equal(out["root_ids"].numpy(), roots)
    assert util.max_abs(out["root_h"].numpy(), h[roots]) < util.TOL["bf16"]


def test_subforest_mode_large_forest_falls_back():
    """more nodes than the scheduler deals out to sub-forests: the persistent kernel runs instead"""
    rng = np.random.default_rng(47)
    params = fg.draw_params(rng, 64, 48, 400, emb_dist="normal", emb_scale=0.3, w_scale=0.15)
    forest = fg.random_forest(rng, 900, 10, 56, 400)
    assert 24576 < forest.n_nodes <= 32768 or forest.n_nodes > 32768
    model = util.make_model(params, "bf16")
    res = util.gpu_forward(model, forest, binding.SUBFORESTS)
    assert model.last_mode() == binding.PERSISTENT
    sample = [0, 450, 899]
    sub = fg.select_trees(forest, sample)
    h, c, _ = orc.forward_recursive(sub.left, sub.right, sub.token, params.emb, params.W, params.b)
    ids = np.nonzero(np.isin(forest.tree_of, sample))[0]
    assert util.max_abs(res["h"][ids], h) < util.TOL["bf16"]


def test_all_modes_give_identical_states():
    """how the ready nodes are grouped into launches, tiles or sub-forests must not change a single
    bit of the result (the paper's recursive and iterative executions are numerically identical,
    Section 6.2): every node's contraction runs over the same K blocks in the same order"""
    rng = np.random.default_rng(48)
    for H, E, n_trees, hi in ((256, 50, 120, 12), (150, 64, 300, 56), (64, 300, 30, 130), (192, 16, 2, 40)):
        params = fg.draw_params(rng, H, E, 500, emb_dist="normal", emb_scale=0.3, w_scale=0.1)
        forest = fg.random_forest(rng, n_trees, 1, hi, 500)
        forest, _ = fg.permute_node_ids(forest, rng)
        model = util.make_model(params, "bf16")
        ref = util.gpu_forward(model, forest, binding.PERSISTENT)
        for flags in (binding.PER_LEVEL, binding.SUBFORESTS, binding.PERSISTENT):
            res = util.gpu_forward(model, forest, flags)
            np.testing.assert_array_equal(res["h"], ref["h"])
            np.testing.assert_array_equal(res["c"], ref["c"])
            np.testing.assert_array_equal(res["order"], ref["order"])
        model.close()


def test_both_launch_forms_give_identical_states():
    """the persistent kernel launched as a programmatic dependent of the scheduler (it starts while
    the scheduler runs and waits for it on the device) and launched cooperatively in plain stream
    order: same bits, also when a malformed forest makes the scheduler report an error"""
    rng = np.random.default_rng(49)
    w = fg.make_workload("batch256_bf16", 0)
    model = util.make_model(w.params, "bf16")
    res = {}
    for form in (1, 0, 1):
        model.set_option(binding.OPT_OVERLAP_LAUNCH, form)
        for _ in range(3):                            # back to back: the next scheduler follows the kernel at once
            out = util.gpu_forward(model, w.forest, binding.PERSISTENT)
        res.setdefault(form, out)
        np.testing.assert_array_equal(out["h"], res[form]["h"])
    np.testing.assert_array_equal(res[0]["h"], res[1]["h"])
    np.testing.assert_array_equal(res[0]["c"], res[1]["c"])
    np.testing.assert_array_equal(res[0]["order"], res[1]["order"])
    bad = fg.random_forest(rng, 5, 2, 20, w.params.vocab)
    left = bad.left.copy()
    left[int(np.flatnonzero(bad.left >= 0)[0])] = bad.n_nodes + 7      # a child index out of range
    broken = dataclasses.replace(bad, left=left)
    for form in (1, 0):
        model.set_option(binding.OPT_OVERLAP_LAUNCH, form)
        with pytest.raises(binding.TreeLSTMError):
            util.gpu_forward(model, broken, binding.PERSISTENT)
        out = util.gpu_forward(model, w.forest, binding.PERSISTENT)     # the context keeps working
        np.testing.assert_array_equal(out["h"], res[0]["h"])
    model.close()


def test_leaves_taken_first_on_small_grids_and_leaf_only_forests():
    """the kernel started under the scheduler ranks the leaves itself (every CTA a share of the node
    ids): same bits as the run in plain stream order on grids of 1, 5 and 40 CTAs (several node ids
    per thread), on a forest of single-leaf trees only (one wavefront) and on a mixed one"""
    rng = np.random.default_rng(50)
    params = fg.draw_params(rng, 128, 72, 400, emb_dist="normal", emb_scale=0.3, w_scale=0.15)
    forests = [fg.random_forest(rng, 37, 1, 1, 400),        # leaves only
               fg.random_forest(rng, 60, 1, 24, 400)]
    forests[1], _ = fg.permute_node_ids(forests[1], rng)
    model = util.make_model(params, "bf16")
    for forest in forests:
        model.set_option(binding.OPT_MAX_CTAS, 0)
        model.set_option(binding.OPT_OVERLAP_LAUNCH, 0)
        ref = util.gpu_forward(model, forest, binding.PERSISTENT)
        h, c, _ = orc.forward_recursive(forest.left, forest.right, forest.token, params.emb, params.W, params.b)
        assert util.max_abs(ref["h"], h) < util.TOL["bf16"]
        model.set_option(binding.OPT_OVERLAP_LAUNCH, 1)
        model.set_option(binding.OPT_LEAVES_FIRST_MIN_NODES, 0)     # these forests are below the default threshold
        for ctas in (0, 1, 5, 40):
            model.set_option(binding.OPT_MAX_CTAS, ctas)
            res = util.gpu_forward(model, forest, binding.PERSISTENT)
            np.testing.assert_array_equal(res["h"], ref["h"])
            np.testing.assert_array_equal(res["c"], ref["c"])
            np.testing.assert_array_equal(res["order"], ref["order"])
    model.close()


def test_bf16_deeper_than_the_level_cache():
    """a left chain of 1100 leaves next to a few small trees: 1100 wavefronts, more than the kernels
    keep wavefront boundaries for in shared memory (the rest is read from global memory, and the
    sub-forest kernel spills its per-sub-forest table); all modes still agree bit for bit and stay
    within the bf16 tolerance of the oracle over that depth"""
    rng = np.random.default_rng(1100)
    params = fg.draw_params(rng, 64, 32, 200, emb_dist="normal", emb_scale=0.3, w_scale=0.1)
    shapes = [fg.left_chain_shape(1100), fg.balanced_shape(16), None, fg.left_chain_shape(7)]
    forest = fg.forest_from_shapes(shapes, rng, 200)
    forest, _ = fg.permute_node_ids(forest, rng)
    ref = None
    for flags in (binding.PERSISTENT, binding.SUBFORESTS, binding.PER_LEVEL):
        res = _check(params, forest, flags)
        assert res["n_levels"] == 1100
        if ref is None:
            ref = res
        np.testing.assert_array_equal(res["h"], ref["h"])
        np.testing.assert_array_equal(res["c"], ref["c"])


def test_narrow_tails_are_handed_to_one_cluster():
    """persistent mode: the last wavefronts of a forest, once they are all narrow, can be finished by one
    cluster that passes states from child to caller through distributed shared memory.  Whether that
    pays is decided on the device by a cost model (or forced with TAIL_MIN_LEVELS); either way it changes
    no bit of the result (every node's contraction runs over the same products in the same order),
    whatever the shape of the tail."""
    rng = np.random.default_rng(77)
    for H, E in ((256, 300), (150, 64), (128, 40), (64, 64)):
        params = fg.draw_params(rng, H, E, 500, emb_dist="normal", emb_scale=0.3, w_scale=0.08)
        model = util.make_model(params, "bf16")
        forced = util.make_model(params, "bf16")
        forced.set_option(binding.OPT_TAIL_WIDTH, 64)
        forced.set_option(binding.OPT_TAIL_MIN_LEVELS, 2)      # hand over whenever two narrow wavefronts remain
        plain = util.make_model(params, "bf16")
        plain.set_option(binding.OPT_TAIL_WIDTH, 0)            # every wavefront on the grid-wide kernel
        cases = [
            [fg.random_split_shape(rng, 56)],                                        # one tree
            [fg.random_split_shape(rng, 9) for _ in range(6)] + [None] * 3,          # a few small trees, single leaves
            [fg.left_chain_shape(60), fg.left_chain_shape(33)],                      # callers one wavefront up, leaves far below
            [fg.balanced_shape(64)],                                                 # both children always one wavefront below
            [fg.random_split_shape(rng, 40) for _ in range(30)] + [fg.left_chain_shape(50)] * 3,   # wide first, long narrow tail
            [fg.left_chain_shape(70)] * 64,                                          # exactly 64 nodes per wavefront
            [fg.random_split_shape(rng, 30) for _ in range(5)] + [fg.left_chain_shape(45)],   # callers one, two and more wavefronts up
        ]
        for shapes in cases:
            forest = fg.forest_from_shapes(shapes, rng, 500)
            forest, _ = fg.permute_node_ids(forest, rng)
            ref = util.gpu_forward(plain, forest, binding.PERSISTENT)
            assert plain.last_launch_count() == 2
            for m in (forced, model):
                res = util.gpu_forward(m, forest, binding.PERSISTENT)
                # (the model that decides for itself leaves the second launch out after forests without a tail)
                want = (3,) if m is forced else (2, 3)
                assert m.last_launch_count() in (want if forest.n_nodes <= 4096 else (2,)) and m.last_mode() == binding.PERSISTENT
                np.testing.assert_array_equal(res["order"], ref["order"])
                np.testing.assert_array_equal(res["h"], ref["h"])
                np.testing.assert_array_equal(res["c"], ref["c"])
            h, c, _ = orc.forward_recursive(forest.left, forest.right, forest.token, params.emb, params.W, params.b,
                                            operand_round=orc.round_to_bf16)
            assert util.max_abs(res["h"], h) < TIGHT and util.max_abs(res["c"], c) < TIGHT
        # a forest above the node limit only reaches the cluster kernel when the limit is raised
        forced.set_option(binding.OPT_TAIL_MAX_NODES, 1 << 20)
        wide = fg.forest_from_shapes(cases[5], rng, 500)            # 64 chains: 64 nodes in every wavefront above the leaves
        ref = util.gpu_forward(plain, wide, binding.PERSISTENT)
        res = util.gpu_forward(forced, wide, binding.PERSISTENT)
        assert forced.last_launch_count() == 3
        np.testing.assert_array_equal(res["h"], ref["h"])
        np.testing.assert_array_equal(res["c"], ref["c"])
        model = forced
        forest = fg.forest_from_shapes(cases[4], rng, 500)
        ref = util.gpu_forward(plain, forest, binding.PERSISTENT)
        # a forest without a narrow tail long enough stays on the grid-wide kernel (the cluster finds nothing to do)
        model.set_option(binding.OPT_TAIL_MIN_LEVELS, 1000)
        res = util.gpu_forward(model, forest, binding.PERSISTENT)
        np.testing.assert_array_equal(res["h"], ref["h"])
        model.set_option(binding.OPT_TAIL_MIN_LEVELS, 2)
        # saved gates for backward come out of the cluster kernel too
        small = fg.forest_from_shapes([fg.random_split_shape(rng, 30)], rng, 500)
        arrs = [util.to_dev(x) for x in (small.left, small.right, small.token)]
        labels = util.to_dev(rng.integers(0, 3, size=small.n_nodes).astype(np.int32))
        Wc, bc = util.to_dev(rng.uniform(-0.1, 0.1, (H, 3)).astype(np.float32)), util.to_dev(np.zeros(3, np.float32))
        grads = []
        for m in (model, plain):
            m.set_classifier(Wc, bc)
            m.forward(*arrs, flags=binding.PERSISTENT | binding.SAVE_FOR_BACKWARD)
            g = m.backward(labels, small.n_leaves)
            grads.append({k: v.cpu().numpy() for k, v in g.items()})
        np.testing.assert_allclose(grads[0]["dW"], grads[1]["dW"], rtol=0, atol=1e-7)
        np.testing.assert_allclose(grads[0]["loss"], grads[1]["loss"], rtol=0, atol=1e-6)
        model.close(); plain.close()


def test_cluster_launch_is_left_out_while_forests_have_no_tail():
    """the library reads the hand-over decision back with the control block: after a forest without a
    tail worth handing over the second launch is left out, after a deep narrow one it comes back; the
    results never change"""
    rng = np.random.default_rng(78)
    params = fg.draw_params(rng, 256, 300, 500, emb_dist="normal", emb_scale=0.3, w_scale=0.08)
    model = util.make_model(params, "bf16")
    plain = util.make_model(params, "bf16")
    plain.set_option(binding.OPT_TAIL_WIDTH, 0)
    bushy = fg.forest_from_shapes([fg.balanced_shape(32)] * 10, rng, 500)      # six wavefronts: nothing to gain
    chain = fg.forest_from_shapes([fg.left_chain_shape(40)] * 3, rng, 500)     # 39 wavefronts of 3 nodes
    seen = []
    for forest in (bushy, bushy, chain, chain, bushy, bushy):
        res = util.gpu_forward(model, forest, binding.PERSISTENT)              # reads the status back every time
        seen.append(model.last_launch_count())
        ref = util.gpu_forward(plain, forest, binding.PERSISTENT)
        np.testing.assert_array_equal(res["h"], ref["h"])
        np.testing.assert_array_equal(res["c"], ref["c"])
    assert seen == [3, 2, 2, 3, 3, 2]
