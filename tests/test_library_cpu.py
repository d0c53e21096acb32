"""Host-only checks of the C-ABI library: it builds, loads, and exports every symbol the public
header declares.  No kernel is launched here."""
import ctypes
import os
import re

import pytest

from paper_1809_00832_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load_library()


def _declared_symbols():
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in os.listdir(inc):
        if fn.endswith(".h"):
            text = open(os.path.join(inc, fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"TREELSTM_API[^;(]*?\b(treelstm_\w+)\s*\(", text))
    return names


def test_every_declared_symbol_is_exported(lib):
    declared = _declared_symbols()
    assert len(declared) >= 10
    for name in declared:
        assert hasattr(lib, name), f"{name} declared in include/ but not exported"
    assert declared == set(binding.SIGNATURES), "binding and header disagree on the call list"


def test_host_only_calls(lib):
    assert lib.treelstm_strerror(0) == b"ok"
    for code in range(-10, 0):
        assert lib.treelstm_strerror(code) not in (b"ok", b"unknown status")
    assert lib.treelstm_strerror(-100) == b"unknown status"
    assert lib.treelstm_destroy(None) == binding.OK
    assert lib.treelstm_workspace_bytes(None, 10, 0) == 0
    assert lib.treelstm_last_launch_count(None) == 0
    handle = ctypes.c_void_p()
    # argument errors are caught before any CUDA call
    rc = lib.treelstm_create(ctypes.byref(handle), 0, 4, 4, None, None, None, 0, None)
    assert rc == binding.ERR_INVALID_ARG and not handle.value
    rc = lib.treelstm_create(None, 4, 4, 4, None, None, None, 0, None)
    assert rc == binding.ERR_INVALID_ARG
    assert lib.treelstm_forward(None, 0, None, None, None, None, None, None, None, None, None, 0, None, 0,
                                None) == binding.ERR_INVALID_ARG
    assert lib.treelstm_status_sync(None) == binding.ERR_INVALID_ARG


def test_error_codes_match_header():
    text = open(os.path.join(ROOT, "include", "treelstm.h")).read()
    for name, value in re.findall(r"TREELSTM_(ERR_\w+|OK) = (-?\d+)", text):
        assert getattr(binding, name) == int(value)


def test_binding_refuses_without_cuda():
    import torch
    if torch.cuda.is_available():
        pytest.skip("CUDA present")
    with pytest.raises(RuntimeError):
        binding.TreeLSTM(4, 4, 4, torch.zeros(4, 4), torch.zeros(12, 20), torch.zeros(20))


def test_tile_plan_invariants(lib):
    """host-side view of the device's tile plan: whatever the wavefront, the tiles cover every node
    and every hidden unit exactly once, the operand boxes fit the shared-memory ring, and a split
    last round never has more pieces than CTAs"""
    for H, E in ((256, 300), (150, 300), (64, 64), (16, 16), (512, 100)):
        groups = -(-H // 64) * 64 // 8
        for n_ctas in (148, 37, 1):
            for leaf in (True, False):
                for rows in (1, 2, 31, 32, 33, 64, 100, 128, 129, 500, 954, 2397, 7240, 16384):
                    pl = binding.tile_plan(rows, H, E, n_ctas, leaf)
                    rt, g = pl["rows_per_tile"], pl["groups_per_tile"]
                    assert rt in (32, 64, 128) and g in (1, 2, 4) and groups % g == 0
                    if leaf:
                        assert rt == 128
                    fat = -(-rows // rt) * (groups // g)
                    pieces = 1 << pl["tail_log2_pieces"]
                    assert pieces <= g and 0 <= pl["tail_from"] <= fat
                    assert pl["tiles"] == pl["tail_from"] + (fat - pl["tail_from"]) * pieces
                    if pieces > 1:
                        assert pl["tail_from"] % n_ctas == 0            # whole rounds of fat tiles first
                        assert pl["tiles"] - pl["tail_from"] <= n_ctas  # the pieces fit one round
                    assert 1 <= pl["stages"] <= 8
                    assert pl["stages"] * pl["stage_bytes"] <= pl["ring_bytes"]
                    kblocks = (-(-E // 64)) if leaf else 2 * (-(-H // 64))
                    assert pl["boxes_per_tile"] * pl["kblocks_per_box"] >= kblocks
                    assert pl["stage_bytes"] % 1024 == 0               # every box lands on a swizzle boundary
    # a narrow wavefront gets small tiles (all SMs busy), a wide one fat tiles
    assert binding.tile_plan(123, 256, 300, 148, False)["rows_per_tile"] == 32
    assert binding.tile_plan(7240, 256, 300, 148, True)["groups_per_tile"] == 4
