"""The comparison the GPU parity tests use must be able to fail: planted mistakes (in copies of the
oracle's own results, on the CPU) have to be rejected at the sizes of the full training workload,
where several gradient groups are smaller than the absolute tolerance altogether."""
import copy

import numpy as np
import pytest

from oracle import treelstm_oracle as orc
from paper_1809_00832_b200 import forests as fg
from tests import util


@pytest.fixture(scope="module")
def train_ref():
    w = fg.make_workload("train25_fp32", 0)
    f, p = w.forest, w.params
    ref = orc.loss_and_gradients(f.left, f.right, f.token, p.emb, p.W, p.b, p.Wc, p.bc, w.labels)
    ref["n_touched"] = np.asarray([len(ref["touched_ids"])])
    return ref


def _as_result(ref):
    res = copy.deepcopy(ref)
    res["loss"] = np.asarray([ref["loss"]])
    return res


def test_exact_copy_passes(train_ref):
    util.compare_training_step(_as_result(train_ref), train_ref, util.TOL["fp32"], util.REL["fp32"], loss_rel=1e-5)


@pytest.mark.parametrize("group", util.GRAD_KEYS + ("dEmb_rows",))
def test_zeroed_group_is_rejected(train_ref, group):
    res = _as_result(train_ref)
    res[group] = np.zeros_like(res[group])
    with pytest.raises(AssertionError):
        util.compare_training_step(res, train_ref, util.TOL["fp32"], util.REL["fp32"], loss_rel=1e-5)


def test_full_size_groups_below_the_absolute_tolerance_exist(train_ref):
    """why the relative bound is needed: dW and the embedding rows of this workload would pass the
    absolute tolerance as all zeros"""
    assert np.max(np.abs(train_ref["dW"])) < util.TOL["fp32"]
    assert np.max(np.abs(train_ref["dEmb_rows"])) < util.TOL["fp32"]


def test_dropped_leaf_rows_and_transposed_blocks_are_rejected(train_ref):
    res = _as_result(train_ref)
    E = 300
    res["dW"] = res["dW"].copy()
    res["dW"][:E] = 0.0                                   # the leaves' contribution dropped
    with pytest.raises(AssertionError):
        util.compare_training_step(res, train_ref, util.TOL["fp32"], util.REL["fp32"])
    res = _as_result(train_ref)
    H = train_ref["db"].shape[0] // 5
    db = res["db"].copy()
    db[H:2 * H], db[2 * H:3 * H] = res["db"][2 * H:3 * H], res["db"][H:2 * H]     # f_l and f_r swapped
    res["db"] = db
    with pytest.raises(AssertionError):
        util.compare_training_step(res, train_ref, util.TOL["fp32"], util.REL["fp32"])


def test_loss_relative_bound_is_tighter_than_the_absolute_one(train_ref):
    res = _as_result(train_ref)
    res["loss"] = res["loss"] * (1.0 + 3e-5)      # inside 1e-4 absolute, outside 1e-5 relative
    util.compare_training_step(res, train_ref, util.TOL["fp32"], util.REL["fp32"])
    with pytest.raises(AssertionError):
        util.compare_training_step(res, train_ref, util.TOL["fp32"], util.REL["fp32"], loss_rel=1e-5)
