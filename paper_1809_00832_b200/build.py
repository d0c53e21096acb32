"""Builds libtreelstm_b200.so (sm_100a) in-tree with nvcc.  `python -m paper_1809_00832_b200.build`.

Variants (same sources, one more preprocessor symbol, their own file name):
  ""         the library
  "checked"  -DTREELSTM_CHECKED: every index read from the caller's arrays or from the schedule is
             bounds-checked before use and every state row counts its writers (libtreelstm_b200_checked.so)
  "trace"    -DTREELSTM_TRACE: the wavefront kernels record cycle stamps per wavefront
             (libtreelstm_b200_trace.so; read with paper_1809_00832_b200.trace)
"""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(PKG_DIR, "csrc")
LIB_PATH = os.path.join(PKG_DIR, "libtreelstm_b200.so")
VARIANT_FLAGS = {"": [], "checked": ["-DTREELSTM_CHECKED"], "trace": ["-DTREELSTM_TRACE"]}


def lib_path(variant: str = "") -> str:
    if variant not in VARIANT_FLAGS:
        raise ValueError(f"unknown library variant {variant!r}")
    return os.path.join(PKG_DIR, f"libtreelstm_b200_{variant}.so" if variant else "libtreelstm_b200.so")
SOURCES = ("api.cu", "schedule.cu", "cell_fp32.cu", "cell_rec.cu", "gemm_tc.cu", "subforest_tc.cu", "tail_tc.cu", "backward.cu", "dweight_tc.cu")
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden"]


def _nvcc() -> str:
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(nvcc):
        raise RuntimeError("nvcc not found; the library can only be built with the CUDA toolkit")
    return nvcc


def _stale(path: str) -> bool:
    if not os.path.exists(path):
        return True
    built = os.path.getmtime(path)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)]
    deps.append(os.path.join(os.path.dirname(PKG_DIR), "include", "treelstm.h"))
    return any(os.path.getmtime(d) > built for d in deps)


def build(force: bool = False, verbose: bool = False, variant: str = "") -> str:
    """Compile every CUDA source for sm_100a and link the shared library.  Returns its path."""
    out_path = lib_path(variant)
    if not force and not _stale(out_path):
        return out_path
    nvcc = _nvcc()
    obj_dir = os.path.join(PKG_DIR, "_build", variant or "default")
    os.makedirs(obj_dir, exist_ok=True)
    objs = []
    procs = []
    for src in SOURCES:
        obj = os.path.join(obj_dir, src.replace(".cu", ".o"))
        cmd = [nvcc, *NVCC_FLAGS, *VARIANT_FLAGS[variant], "-c", os.path.join(CSRC, src), "-o", obj]
        if verbose:
            cmd.insert(1, "-Xptxas=-v")
        procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
        objs.append(obj)
    failed = False
    for src, proc in procs:
        out, _ = proc.communicate()
        if verbose or proc.returncode != 0:
            sys.stderr.write(f"--- {src}\n{out}\n")
        failed |= proc.returncode != 0
    if failed:
        raise RuntimeError("nvcc failed")
    link = [nvcc, "-shared", "-o", out_path, *objs, "-lcudart"]
    subprocess.run(link, check=True)
    return out_path


if __name__ == "__main__":
    chosen = [a.split("=", 1)[1] for a in sys.argv if a.startswith("--variant=")]
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, variant=chosen[0] if chosen else ""))
