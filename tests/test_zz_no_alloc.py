"""The allocation-free scheduling entry point (treelstm_schedule_static), called through the C ABI.

Some users of this library run where device allocations are forbidden: inside a framework whose
memory pool owns the whole GPU, in a service whose memory budget is fixed at start-up, or on a path
where the device-wide synchronisation an allocation can cause is not acceptable.  They can neither
create a context nor provide the workspace treelstm_forward asks for.  For them the library keeps
the scheduler's scratch in a fixed array of its own device image.  This test checks that the entry
point gives exactly what treelstm_forward reports for the same forest - and what the CPU oracle's
ready queue gives - on two calls in a row (the second on a smaller forest, so that anything left
over from the first call would show), at the largest size it takes, on a forest deep enough to need
two sorting passes and the large shared-memory opt-in, on the empty forest, that device memory in
use does not change across the calls, and that forests beyond the built-in limit are refused.  This file sorts last on purpose: a run that stops at
the first failure has then already run every other test."""
import numpy as np
import pytest
import torch

from oracle import treelstm_oracle as orc
from paper_1809_00832_b200 import binding, forests as fg
from tests import util

pytestmark = pytest.mark.gpu


def _static_schedule(forest, vocab, bufs):
    n = forest.n_nodes
    left, right, token = (util.to_dev(a) for a in (forest.left, forest.right, forest.token))
    rc = binding.schedule_static(left, right, token, vocab, bufs)
    assert rc == binding.OK
    torch.cuda.synchronize()
    assert int(bufs["status"].item()) == binding.OK
    n_levels = int(bufs["n_levels"].item())
    return dict(level=bufs["level"][:n].cpu().numpy(), order=bufs["order"][:n].cpu().numpy(),
                level_offset=bufs["level_offset"][:n_levels + 1].cpu().numpy(), n_levels=n_levels)


def test_static_schedule_matches_forward_twice_in_a_row():
    util.lib_ready()
    rng = np.random.default_rng(21)
    params = fg.draw_params(rng, 8, 8, 50, emb_dist="uniform", emb_scale=0.1, w_scale=0.1)
    model = util.make_model(params, "fp32")
    cap = 4096
    i32 = dict(dtype=torch.int32, device="cuda")
    # the caller's own buffers, made once up front: the calls under test allocate nothing
    bufs = dict(level=torch.empty(cap, **i32), order=torch.empty(cap, **i32),
                level_offset=torch.empty(cap + 2, **i32), n_levels=torch.zeros(1, **i32),
                status=torch.zeros(1, **i32))
    big = fg.random_forest(rng, 60, 2, 30, 50)
    big, _ = fg.permute_node_ids(big, rng)
    small = fg.forest_from_shapes([fg.left_chain_shape(9), fg.balanced_shape(8), None], rng, 50)
    assert small.n_nodes < big.n_nodes <= cap
    for forest in (big, small):
        got = _static_schedule(forest, 50, bufs)
        ref = util.gpu_forward(model, forest, binding.PERSISTENT)
        assert got["n_levels"] == ref["n_levels"]
        np.testing.assert_array_equal(got["level"], ref["level"])          # integer work: bit-exact
        np.testing.assert_array_equal(got["order"], ref["order"])
        np.testing.assert_array_equal(got["level_offset"], ref["level_offset"][:ref["n_levels"] + 1])
        _assert_matches_oracle(got, forest)


def _assert_matches_oracle(got, forest):
    status, _, level, order, off = orc.schedule(forest.left, forest.right)
    assert status == orc.OK
    assert got["n_levels"] == len(off) - 1
    np.testing.assert_array_equal(got["level"], level)
    np.testing.assert_array_equal(got["order"], order)
    np.testing.assert_array_equal(got["level_offset"], off)


def test_static_schedule_deep_full_and_empty_forests_allocate_nothing():
    """a left chain of 8191 leaves (16381 nodes, 8191 wavefronts: two sorting passes through the
    second sort buffer of the built-in array, and a launch above the default shared-memory limit),
    a forest of exactly the largest size, and the empty forest; twice each, with the free device
    memory unchanged from the first call to the last"""
    util.lib_ready()
    rng = np.random.default_rng(22)
    cap = binding.STATIC_MAX_NODES
    i32 = dict(dtype=torch.int32, device="cuda")
    bufs = dict(level=torch.empty(cap, **i32), order=torch.empty(cap, **i32),
                level_offset=torch.empty(cap + 2, **i32), n_levels=torch.zeros(1, **i32),
                status=torch.zeros(1, **i32))
    chain = fg.forest_from_shapes([fg.left_chain_shape(8191)], rng, 50)
    assert chain.n_nodes == 16381
    full = fg.forest_from_shapes([fg.random_split_shape(rng, 8192), None], rng, 50)
    full, _ = fg.permute_node_ids(full, rng)
    assert full.n_nodes == cap
    empty = fg.Forest(*(np.zeros(0, dtype=np.int32) for _ in range(5)))
    dev_forests = [(f, [util.to_dev(a) for a in (f.left, f.right, f.token)]) for f in (chain, full, empty)]
    # the first call on a device looks up the built-in array; allocations, if any, would show between
    # the calls that follow it
    assert binding.schedule_static(*dev_forests[2][1], 50, bufs) == binding.OK
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    results = []
    for _ in range(2):
        for forest, arrs in dev_forests:
            assert binding.schedule_static(*arrs, 50, bufs) == binding.OK
            torch.cuda.synchronize()
            free_now = torch.cuda.mem_get_info()[0]
            assert free_now == free_before
            assert int(bufs["status"].item()) == binding.OK
            n, n_levels = forest.n_nodes, int(bufs["n_levels"].item())
            results.append((forest, dict(level=bufs["level"][:n].cpu().numpy(), order=bufs["order"][:n].cpu().numpy(),
                                         level_offset=bufs["level_offset"][:n_levels + 1].cpu().numpy(),
                                         n_levels=n_levels)))
    for forest, got in results:
        if forest.n_nodes == 0:
            assert got["n_levels"] == 0 and got["level_offset"].tolist() == [0]
        else:
            _assert_matches_oracle(got, forest)
    assert results[0][1]["n_levels"] == 8191


def test_static_schedule_reports_errors_and_limit():
    util.lib_ready()
    i32 = dict(dtype=torch.int32, device="cuda")
    bufs = dict(level=torch.empty(8, **i32), order=torch.empty(8, **i32), level_offset=torch.empty(10, **i32),
                n_levels=torch.zeros(1, **i32), status=torch.zeros(1, **i32))
    bad = [torch.tensor(x, **i32) for x in ([-1, -1, 0, 0], [-1, -1, 1, 1], [0, 1, 0, 0])]   # two parents
    assert binding.schedule_static(*bad, 5, bufs) == binding.OK
    torch.cuda.synchronize()
    assert int(bufs["status"].item()) == binding.ERR_INVALID_FOREST
    good = [torch.tensor(x, **i32) for x in ([-1, -1, 0], [-1, -1, 1], [0, 1, -1])]
    assert binding.schedule_static(*good, 5, bufs) == binding.OK                      # status is cleared
    torch.cuda.synchronize()
    assert int(bufs["status"].item()) == binding.OK and int(bufs["n_levels"].item()) == 2
    lib = binding.load_library()
    too_many = binding.STATIC_MAX_NODES + 1
    rc = lib.treelstm_schedule_static(too_many, None, None, None, 5, None, None, None, None, None, None)
    assert rc in (binding.ERR_UNSUPPORTED, binding.ERR_INVALID_ARG)
    z = torch.zeros(too_many + 2, **i32)
    p = binding._ptr
    rc = lib.treelstm_schedule_static(too_many, p(z), p(z), p(z), 5, p(z), p(z), p(z), p(bufs["n_levels"]),
                                      p(bufs["status"]), None)
    assert rc == binding.ERR_UNSUPPORTED
