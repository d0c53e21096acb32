"""ctypes binding of libtreelstm_b200.so: the same calls as include/treelstm.h, with torch tensors
standing in for the raw device pointers.  Argument marshalling only - every step of the path runs
inside the library's CUDA kernels.  There is no CPU fallback: without the built library or
without a CUDA device every call raises."""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_PKG_DIR = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG_DIR, "libtreelstm_b200.so")

OK = 0
ERR_INVALID_ARG = -1
ERR_INVALID_FOREST = -2
ERR_TOKEN_OUT_OF_RANGE = -3
ERR_LABEL_OUT_OF_RANGE = -4
ERR_TIMEOUT = -5
ERR_CUDA = -6
ERR_NO_DEVICE = -7
ERR_UNSUPPORTED = -8
ERR_STATE = -9
ERR_CHECK = -10

FP32 = 0
BF16 = 1
PER_LEVEL = 0
PERSISTENT = 1
SAVE_FOR_BACKWARD = 2
SUBFORESTS = 4
CELL_TREERNN = 1
CELL_RNTN = 2
OPT_SCHED_SINGLE_CTA_MAX = 1
OPT_WAIT_LIMIT_CYCLES = 2
OPT_MAX_CTAS = 3
OPT_TIME_WAVEFRONT_KERNEL = 4
OPT_TAIL_WIDTH = 5
OPT_TAIL_MIN_LEVELS = 6
OPT_TAIL_MAX_NODES = 7
OPT_OVERLAP_LAUNCH = 8
OPT_LEAVES_FIRST_MIN_NODES = 9
OPT_DW_TENSOR_CORES = 10

_vp = ctypes.c_void_p
_i = ctypes.c_int

# name -> (restype, argtypes); mirrors include/treelstm.h
SIGNATURES = {
    "treelstm_create": (_i, [ctypes.POINTER(_vp), _i, _i, _i, _vp, _vp, _vp, _i, _vp]),
    "treelstm_create_recursive": (_i, [ctypes.POINTER(_vp), _i, _i, _i, _vp, _vp, _vp, _vp, _vp]),
    "treelstm_update_weights": (_i, [_vp, _vp, _vp, _vp, _vp]),
    "treelstm_set_classifier": (_i, [_vp, _i, _vp, _vp, _vp]),
    "treelstm_set_option": (_i, [_vp, _i, ctypes.c_longlong]),
    "treelstm_workspace_bytes": (ctypes.c_size_t, [_vp, _i, _i]),
    "treelstm_forward": (_i, [_vp, _i, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i, _vp,
                              ctypes.c_size_t, _vp]),
    "treelstm_status_sync": (_i, [_vp]),
    "treelstm_roots": (_i, [_vp, _i, _vp, _vp, _vp, _vp, _vp]),
    "treelstm_backward": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "treelstm_backward_recursive": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "treelstm_forward_host": (_i, [_vp, _i, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i, _vp, _vp,
                                   _vp, _vp, _i, _vp]),
    "treelstm_host_staging_bytes": (ctypes.c_size_t, [_vp, _i]),
    "treelstm_set_host_staging": (_i, [_vp, _vp, ctypes.c_size_t]),
    "treelstm_schedule_static": (_i, [_i, _vp, _vp, _vp, _i, _vp, _vp, _vp, _vp, _vp, _vp]),
    "treelstm_selftest_waits": (_i, [_vp, _vp, ctypes.c_size_t, _vp, _vp]),
    "treelstm_last_kernel_ms": (_i, [_vp, ctypes.POINTER(ctypes.c_float)]),
    "treelstm_last_launch_count": (_i, [_vp]),
    "treelstm_last_mode": (_i, [_vp]),
    "treelstm_subforest_count": (_i, [_vp]),
    "treelstm_tile_plan": (_i, [_i, _i, _i, _i, _i, _vp]),
    "treelstm_last_cuda_error": (_i, [_vp]),
    "treelstm_destroy": (_i, [_vp]),
    "treelstm_strerror": (ctypes.c_char_p, [_i]),
}

_libs = {}
# which build of the library the handles use unless told otherwise: "" (the library itself),
# "checked" or "trace" (see build.py); the environment variable switches a whole run over
DEFAULT_VARIANT = os.environ.get("TREELSTM_LIB_VARIANT", "")


class TreeLSTMError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = load_library().treelstm_strerror(code).decode()
        super().__init__(f"{where}: {msg} ({code})")


def load_library(variant: Optional[str] = None) -> ctypes.CDLL:
    """dlopen the in-tree shared library and declare every prototype.  Raises if it is not built."""
    variant = DEFAULT_VARIANT if variant is None else variant
    if variant in _libs:
        return _libs[variant]
    path = LIB_PATH if not variant else os.path.join(_PKG_DIR, f"libtreelstm_b200_{variant}.so")
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing: build it with `python -m paper_1809_00832_b200.build`")
    lib = ctypes.CDLL(path)
    for name, (res, args) in SIGNATURES.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    _libs[variant] = lib
    return lib


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _dev(t: torch.Tensor, dtype, name: str) -> torch.Tensor:
    if not t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise ValueError(f"{name} must be a contiguous CUDA tensor of dtype {dtype}")
    return t


def _stream() -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


STATIC_MAX_NODES = 16384


def schedule_static(left: torch.Tensor, right: torch.Tensor, token: torch.Tensor, vocab: int, out: dict) -> int:
    """treelstm_schedule_static: ready-set construction for callers that may not allocate device
    memory.  Everything, outputs included, is passed in: `out` holds the caller's int32 CUDA tensors
    level [n], order [n], level_offset [n + 2], n_levels [1] and status [1].  Neither this wrapper
    nor the library allocates; the kernel's scratch is a fixed array inside the library.  Returns
    the host-side return code (the device-side status lands in out["status"])."""
    lib = load_library()
    n = int(left.shape[0])
    return int(lib.treelstm_schedule_static(n, _ptr(left), _ptr(right), _ptr(token), vocab, _ptr(out["level"]),
                                            _ptr(out["order"]), _ptr(out["level_offset"]), _ptr(out["n_levels"]),
                                            _ptr(out["status"]), _stream()))


TILE_PLAN_FIELDS = ("rows_per_tile", "groups_per_tile", "tiles", "tail_from", "tail_log2_pieces", "kblocks_per_box",
                    "boxes_per_tile", "stages", "stage_bytes", "ring_bytes")


def tile_plan(rows: int, H: int, E: int, n_ctas: int, leaf: bool) -> dict:
    """treelstm_tile_plan: the tile shape the bf16 kernel picks for a wavefront (host-side, no CUDA)."""
    out = (ctypes.c_int32 * 10)()
    rc = load_library().treelstm_tile_plan(rows, H, E, n_ctas, int(leaf), ctypes.cast(out, ctypes.c_void_p))
    if rc != OK:
        raise TreeLSTMError(rc, "treelstm_tile_plan")
    return dict(zip(TILE_PLAN_FIELDS, [int(v) for v in out]))


def pack_forest_host(left, right, token):
    """The three forest arrays (numpy or CPU tensors) as rows of one pinned int32 tensor; returns the
    three row views.  treelstm_forward_host copies arrays that are adjacent like this in one piece."""
    rows = [torch.as_tensor(a, dtype=torch.int32) for a in (left, right, token)]
    pack = torch.empty((3, rows[0].shape[0]), dtype=torch.int32, pin_memory=torch.cuda.is_available())
    for i, r in enumerate(rows):
        pack[i].copy_(r)
    return pack[0], pack[1], pack[2]


class TreeLSTM:
    """Thin handle around a treelstm_t*.  Tensors are the caller's; the handle only keeps the
    workspace it allocates through torch (device memory is PyTorch's job here)."""

    def __init__(self, H: int, E: int, vocab: int, emb: torch.Tensor, W: torch.Tensor, b: torch.Tensor,
                 precision: int = FP32, variant: Optional[str] = None):
        if not torch.cuda.is_available():
            raise RuntimeError("no CUDA device: the TreeLSTM library has no CPU path")
        self.lib = load_library(variant)
        self.H, self.E, self.vocab, self.precision = H, E, vocab, precision
        self.C = 0
        self.cell = 0
        _dev(emb, torch.float32, "emb"); _dev(W, torch.float32, "W"); _dev(b, torch.float32, "b")
        assert emb.shape == (vocab, E) and W.shape == (E + 2 * H, 5 * H) and b.shape == (5 * H,)
        handle = ctypes.c_void_p()
        rc = self.lib.treelstm_create(ctypes.byref(handle), H, E, vocab, _ptr(emb), _ptr(W), _ptr(b),
                                      precision, _stream())
        if rc != OK:
            raise TreeLSTMError(rc, "treelstm_create")
        self.handle = handle
        self._ws: Optional[torch.Tensor] = None
        self._host_staging: Optional[torch.Tensor] = None
        self._keep = None

    @classmethod
    def recursive(cls, cell: int, H: int, vocab: int, emb: torch.Tensor, W: torch.Tensor, b: torch.Tensor,
                  V: Optional[torch.Tensor] = None, variant: Optional[str] = None) -> "TreeLSTM":
        """treelstm_create_recursive: a TreeRNN (CELL_TREERNN) or RNTN (CELL_RNTN) context.  forward()
        then returns h only (no cell state)."""
        if not torch.cuda.is_available():
            raise RuntimeError("no CUDA device: the library has no CPU path")
        self = cls.__new__(cls)
        self.lib = load_library(variant)
        self.H, self.E, self.vocab, self.precision, self.C, self.cell = H, H, vocab, FP32, 0, cell
        for name, t in (("emb", emb), ("W", W), ("b", b)) + ((("V", V),) if V is not None else ()):
            _dev(t, torch.float32, name)
        assert emb.shape == (vocab, H) and W.shape == (2 * H, H) and b.shape == (H,)
        assert V is None or V.shape == (H, 2 * H, 2 * H)
        handle = ctypes.c_void_p()
        rc = self.lib.treelstm_create_recursive(ctypes.byref(handle), cell, H, vocab, _ptr(emb), _ptr(W), _ptr(b),
                                                _ptr(V), _stream())
        if rc != OK:
            raise TreeLSTMError(rc, "treelstm_create_recursive")
        self.handle = handle
        self._ws = None
        self._host_staging = None
        self._keep = None
        return self

    def close(self):
        if getattr(self, "handle", None):
            self.lib.treelstm_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- parameters ---------------------------------------------------------------------------
    def update_weights(self, emb, W, b):
        rc = self.lib.treelstm_update_weights(self.handle, _ptr(emb), _ptr(W), _ptr(b), _stream())
        if rc != OK:
            raise TreeLSTMError(rc, "treelstm_update_weights")

    def set_classifier(self, Wc: torch.Tensor, bc: torch.Tensor):
        _dev(Wc, torch.float32, "Wc"); _dev(bc, torch.float32, "bc")
        C = int(bc.shape[0])
        assert Wc.shape == (self.H, C)
        rc = self.lib.treelstm_set_classifier(self.handle, C, _ptr(Wc), _ptr(bc), _stream())
        if rc != OK:
            raise TreeLSTMError(rc, "treelstm_set_classifier")
        self.C = C

    def set_option(self, key: int, value: int):
        rc = self.lib.treelstm_set_option(self.handle, key, value)
        if rc != OK:
            raise TreeLSTMError(rc, "treelstm_set_option")

    def workspace_bytes(self, max_nodes: int, with_backward: bool) -> int:
        return int(self.lib.treelstm_workspace_bytes(self.handle, max_nodes, int(with_backward)))

    def _workspace(self, n: int, with_backward: bool) -> torch.Tensor:
        need = self.workspace_bytes(n, with_backward)
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty(need + 256, dtype=torch.uint8, device="cuda")
        return self._ws

    # -- forward ------------------------------------------------------------------------------
    def forward(self, left: torch.Tensor, right: torch.Tensor, token: torch.Tensor, flags: int = PERSISTENT,
                out: Optional[dict] = None, check: bool = True) -> dict:
        """treelstm_forward.  Returns a dict of device tensors h, c, level, order, level_offset,
        n_levels.  `out` lets the caller reuse the output tensors of an earlier call.  With
        check=False the call stays asynchronous in persistent mode (status is not read)."""
        n = int(left.shape[0])
        for name, t in (("left", left), ("right", right), ("token", token)):
            _dev(t, torch.int32, name)
        if out is None:
            out = dict(
                h=torch.empty((n, self.H), dtype=torch.float32, device="cuda"),
                c=torch.empty((n, self.H), dtype=torch.float32, device="cuda") if self.cell == 0 else None,
                level=torch.empty(n, dtype=torch.int32, device="cuda"),
                order=torch.empty(n, dtype=torch.int32, device="cuda"),
                level_offset=torch.empty(n + 2, dtype=torch.int32, device="cuda"),
                n_levels=torch.zeros(1, dtype=torch.int32, device="cuda"),
            )
        ws = self._workspace(n, bool(flags & SAVE_FOR_BACKWARD))
        base = ws.data_ptr()
        aligned = (base + 255) // 256 * 256
        rc = self.lib.treelstm_forward(self.handle, n, _ptr(left), _ptr(right), _ptr(token), _ptr(out["h"]),
                                       _ptr(out.get("c")), _ptr(out["level"]), _ptr(out["order"]),
                                       _ptr(out["level_offset"]), _ptr(out["n_levels"]), flags,
                                       ctypes.c_void_p(aligned), ws.numel() - (aligned - base), _stream())
        if rc != OK:
            raise TreeLSTMError(rc, "treelstm_forward")
        self._keep = (left, right, token, out)
        if check:
            rc = self.lib.treelstm_status_sync(self.handle)
            if rc != OK:
                raise TreeLSTMError(rc, "treelstm_forward (device status)")
        return out

    def status_sync(self) -> int:
        return int(self.lib.treelstm_status_sync(self.handle))

    def roots(self, max_roots: int) -> dict:
        out = dict(
            root_ids=torch.empty(max_roots, dtype=torch.int32, device="cuda"),
            root_h=torch.empty((max_roots, self.H), dtype=torch.float32, device="cuda"),
            root_c=torch.empty((max_roots, self.H), dtype=torch.float32, device="cuda"),
            n_roots=torch.zeros(1, dtype=torch.int32, device="cuda"),
        )
        rc = self.lib.treelstm_roots(self.handle, max_roots, _ptr(out["root_ids"]), _ptr(out["root_h"]),
                                     _ptr(out["root_c"]), _ptr(out["n_roots"]), _stream())
        if rc != OK:
            raise TreeLSTMError(rc, "treelstm_roots")
        return out

    # -- backward -----------------------------------------------------------------------------
    def backward(self, labels: torch.Tensor, n_leaves: int) -> dict:
        """treelstm_backward after forward(..., flags | SAVE_FOR_BACKWARD)."""
        _dev(labels, torch.int32, "labels")
        H, E, C = self.H, self.E, self.C
        f32 = dict(dtype=torch.float32, device="cuda")
        out = dict(
            loss=torch.zeros(1, **f32), dW=torch.empty((E + 2 * H, 5 * H), **f32), db=torch.empty(5 * H, **f32),
            dWc=torch.empty((H, C), **f32), dbc=torch.empty(C, **f32),
            touched_ids=torch.empty(max(n_leaves, 1), dtype=torch.int32, device="cuda"),
            dEmb_rows=torch.empty((max(n_leaves, 1), E), **f32),
            n_touched=torch.zeros(1, dtype=torch.int32, device="cuda"),
        )
        rc = self.lib.treelstm_backward(self.handle, _ptr(labels), _ptr(out["loss"]), _ptr(out["dW"]),
                                        _ptr(out["db"]), _ptr(out["dWc"]), _ptr(out["dbc"]),
                                        _ptr(out["touched_ids"]), _ptr(out["dEmb_rows"]),
                                        _ptr(out["n_touched"]), _stream())
        if rc != OK:
            raise TreeLSTMError(rc, "treelstm_backward")
        rc = self.lib.treelstm_status_sync(self.handle)
        if rc != OK:
            raise TreeLSTMError(rc, "treelstm_backward (device status)")
        return out

    def backward_recursive(self, labels: torch.Tensor, n_leaves: int) -> dict:
        """treelstm_backward_recursive (TreeRNN / RNTN contexts) after forward(..., flags | SAVE_FOR_BACKWARD)."""
        _dev(labels, torch.int32, "labels")
        H, C = self.H, self.C
        f32 = dict(dtype=torch.float32, device="cuda")
        out = dict(
            loss=torch.zeros(1, **f32), dW=torch.empty((2 * H, H), **f32), db=torch.empty(H, **f32),
            dWc=torch.empty((H, C), **f32), dbc=torch.empty(C, **f32),
            touched_ids=torch.empty(max(n_leaves, 1), dtype=torch.int32, device="cuda"),
            dEmb_rows=torch.empty((max(n_leaves, 1), H), **f32),
            n_touched=torch.zeros(1, dtype=torch.int32, device="cuda"),
        )
        if self.cell == CELL_RNTN:
            out["dV"] = torch.empty((H, 2 * H, 2 * H), **f32)
        rc = self.lib.treelstm_backward_recursive(
            self.handle, _ptr(labels), _ptr(out["loss"]), _ptr(out["dW"]), _ptr(out["db"]), _ptr(out.get("dV")),
            _ptr(out["dWc"]), _ptr(out["dbc"]), _ptr(out["touched_ids"]), _ptr(out["dEmb_rows"]),
            _ptr(out["n_touched"]), _stream())
        if rc != OK:
            raise TreeLSTMError(rc, "treelstm_backward_recursive")
        rc = self.lib.treelstm_status_sync(self.handle)
        if rc != OK:
            raise TreeLSTMError(rc, "treelstm_backward_recursive (device status)")
        return out

    # -- host-buffer forward ------------------------------------------------------------------
    def forward_host(self, left: torch.Tensor, right: torch.Tensor, token: torch.Tensor, *, flags: int = PERSISTENT,
                     all_states: bool = False, max_roots: int = 0, out: Optional[dict] = None) -> dict:
        """treelstm_forward_host: host (ideally pinned) int32 tensors in, host tensors out."""
        n = int(left.shape[0])
        for t in (left, right, token):
            if t.is_cuda or t.dtype != torch.int32 or not t.is_contiguous():
                raise ValueError("forest arrays must be contiguous CPU int32 tensors")
        # device staging is torch's memory too: hand the library a buffer large enough for this forest
        need = int(self.lib.treelstm_host_staging_bytes(self.handle, n))
        if self._host_staging is None or self._host_staging.numel() < need + 256:
            grown = torch.empty(need + need // 4 + 256, dtype=torch.uint8, device="cuda")
            base = grown.data_ptr()
            aligned = (base + 255) // 256 * 256
            rc = self.lib.treelstm_set_host_staging(self.handle, ctypes.c_void_p(aligned),
                                                    grown.numel() - (aligned - base))
            if rc != OK:
                raise TreeLSTMError(rc, "treelstm_set_host_staging")
            self._host_staging = grown
        if out is None:
            pin = dict(pin_memory=True)
            out = dict(n_levels=torch.zeros(1, dtype=torch.int32, **pin),
                       n_roots=torch.zeros(1, dtype=torch.int32, **pin))
            if all_states:
                out["h"] = torch.empty((n, self.H), dtype=torch.float32, **pin)
                out["c"] = torch.empty((n, self.H), dtype=torch.float32, **pin)
                out["level"] = torch.empty(n, dtype=torch.int32, **pin)
                out["order"] = torch.empty(n, dtype=torch.int32, **pin)
            if max_roots > 0:
                # one pinned buffer [ids | h | c]: the library then brings the roots back in one copy
                m, H = max_roots, self.H
                pack = torch.empty(4 * m * (1 + 2 * H), dtype=torch.uint8, **pin)
                out["root_ids"] = pack[:4 * m].view(torch.int32)
                out["root_h"] = pack[4 * m:4 * m * (1 + H)].view(torch.float32).view(m, H)
                out["root_c"] = pack[4 * m * (1 + H):].view(torch.float32).view(m, H)
                out["_roots_pack"] = pack
        g = out.get
        rc = self.lib.treelstm_forward_host(self.handle, n, _ptr(left), _ptr(right), _ptr(token), _ptr(g("h")),
                                            _ptr(g("c")), _ptr(g("level")), _ptr(g("order")), _ptr(g("n_levels")),
                                            max_roots, _ptr(g("root_ids")), _ptr(g("root_h")), _ptr(g("root_c")),
                                            _ptr(g("n_roots")), flags, _stream())
        if rc != OK:
            raise TreeLSTMError(rc, "treelstm_forward_host")
        return out

    def selftest_waits(self) -> list:
        """treelstm_selftest_waits; returns the four result words."""
        ws = torch.zeros(1024, dtype=torch.uint8, device="cuda")
        base = ws.data_ptr()
        aligned = (base + 255) // 256 * 256
        res = torch.full((4,), 99, dtype=torch.int32, device="cuda")
        rc = self.lib.treelstm_selftest_waits(self.handle, ctypes.c_void_p(aligned), 256, _ptr(res), _stream())
        if rc != OK:
            raise TreeLSTMError(rc, "treelstm_selftest_waits")
        torch.cuda.synchronize()
        return res.cpu().tolist()

    def last_kernel_ms(self) -> float:
        ms = ctypes.c_float()
        rc = self.lib.treelstm_last_kernel_ms(self.handle, ctypes.byref(ms))
        if rc != OK:
            raise TreeLSTMError(rc, "treelstm_last_kernel_ms")
        return float(ms.value)

    def last_launch_count(self) -> int:
        return int(self.lib.treelstm_last_launch_count(self.handle))

    def last_mode(self) -> int:
        """PER_LEVEL, PERSISTENT or SUBFORESTS: the evaluation the last forward actually ran."""
        return int(self.lib.treelstm_last_mode(self.handle))

    def subforest_count(self) -> int:
        return int(self.lib.treelstm_subforest_count(self.handle))
