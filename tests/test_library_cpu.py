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
    for code in range(-9, 0):
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
