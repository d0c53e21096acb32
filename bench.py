#!/usr/bin/env python
"""Benchmark of the TreeLSTM forward hot path (schedule + all wavefronts) on synthetic forests.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

One step = one treelstm_forward call (on-device ready-set construction + every wavefront) over one
forest.  Prints ONE JSON line (rank 0).  Under torchrun every rank evaluates its own forest (seed =
rank): trees are independent, so there is no data-path collective ("scaling": "weak").
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_1809_00832_b200 import forests as fg  # noqa: E402

METRIC = "treelstm_forward_trees_per_sec"
UNIT = "trees/s"
L2_FLUSH_BYTES = 256 << 20          # larger than the 126 MB L2
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the wavefront kernel, from the
# committed ncu capture named beside it (a constant copied from that capture, not measured by this
# run); None for workloads without a capture of the current kernel.
NCU_TRAFFIC = {
    "batch256_bf16": (6305536 + 8880896, "profiles/k_fwd_tc_batch256_bf16.md (static: ncu capture of one launch, not measured by this run)"),
    "balanced1024_bf16": (10304000 + 77163520, "profiles/k_fwd_tc_balanced1024_bf16.md (static: ncu capture of one launch, not measured by this run)"),
}
MODES = ("persistent", "per_level", "subforests")
TIMINGS = {}   # side results of the last time_forward call


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d["bf16_tflops"]),
                    bf16_tflops_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


def algorithmic_work(forest: fg.Forest, H: int, E: int, weight_bytes_per_elem: int):
    """Work the method must do for this forest: per leaf 2*E*3H flop and a 4E-byte embedding row; per
    internal node 2*2H*5H flop; per node 8H bytes of (h, c) written and, for non-roots, 8H read by the
    parent; the weights once; 20 bytes of indices and schedule per node."""
    n, nl, t = forest.n_nodes, forest.n_leaves, forest.n_trees
    ni = n - nl
    flops = nl * 2 * E * 3 * H + ni * 2 * (2 * H) * (5 * H)
    bytes_ = nl * 4 * E + n * 8 * H + (n - t) * 8 * H + (3 * H * E + 10 * H * H) * weight_bytes_per_elem + 20 * n
    return flops, bytes_


def roofline_block(forest, p, precision: str, kernel_ms: float, step_ms: float, peaks, workload: str):
    """Achieved fraction of the slower of the two ceilings: algorithmic bytes at the measured HBM copy
    bandwidth, gate flops at the measured tensor peak (bf16 path; the fp32 path runs on the FP32
    pipes and is reported against HBM only).  `frac` uses the wavefront kernel's own duration,
    `frac_of_step` the whole forward call (scheduler included)."""
    flops, abytes = algorithmic_work(forest, p.H, p.E, 2 if precision == "bf16" else 4)
    t_hbm = abytes / (peaks["hbm_gbs"] * 1e9)
    t_tensor = flops / (peaks["bf16_tflops_sustained"] * 1e12) if precision == "bf16" else 0.0
    gbs = abytes / (kernel_ms * 1e-3) / 1e9
    tfl = flops / (kernel_ms * 1e-3) / 1e12
    traffic, source = NCU_TRAFFIC.get(workload, (None, None))
    if t_tensor > t_hbm:
        head = {"bound": "tensor", "achieved": tfl, "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
                "frac": tfl / peaks["bf16_tflops_sustained"]}
    else:
        head = {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"]}
    head.update({
        "traffic": traffic, "traffic_source": source, "peak_source": peaks["source"],
        "kernel": "k_fwd_tc (persistent wavefront kernel)" if precision == "bf16" else "k_fwd_fp32_persistent",
        "kernel_timing": "the kernel of the timed steps run alone, between the library's event pair (the event keeps it "
                         "from starting under the scheduler as it does in the steps)",
        "kernel_ms_plain_order": TIMINGS.get("kernel_ms_plain_order"),
        "kernel_ms": kernel_ms, "algorithmic_bytes": abytes, "algorithmic_flops": flops,
        "frac_of_step": head["frac"] * kernel_ms / step_ms,
        "hbm_gbs": gbs, "hbm_frac": gbs / peaks["hbm_gbs"],
        "tensor_tflops": tfl, "tensor_frac_of_sustained": tfl / peaks["bf16_tflops_sustained"],
        "ceiling_ms": {"hbm": t_hbm * 1e3, "tensor": t_tensor * 1e3},
    })
    return head


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs (read-only)."""

    def __init__(self, index: int, period_s: float = 0.02):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._halt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.dev = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.dev, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        while not self._halt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.dev, nv.NVML_CLOCK_SM))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.dev)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.dev)
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._halt.set()
        self.join(timeout=2)
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ---- the CPU oracle as a timed baseline -------------------------------------------------------- #
_WORKER_WEIGHTS = {}


def _oracle_init(W, b):
    """Pool initializer: the gate weights travel to every worker once, outside the timed region."""
    _WORKER_WEIGHTS["W"], _WORKER_WEIGHTS["b"] = W, b


def _compact_embedding(token, emb):
    """The rows of the embedding table a forest touches, and its tokens renumbered to index them
    (an input-side gather: the oracle's arithmetic sees the same vectors)."""
    ids, inverse = np.unique(token[token >= 0], return_inverse=True)
    tok = token.copy()
    tok[token >= 0] = inverse.astype(token.dtype)
    return tok, np.ascontiguousarray(emb[ids]) if ids.size else emb[:1]


def _oracle_pass(args):
    """One worker's share: whole passes of the oracle (schedule + recursive evaluation) over its
    trees.  Runs in a spawned process, or in this one for the single-thread figure."""
    left, right, token, emb, W, b, passes = args
    if W is None:
        W, b = _WORKER_WEIGHTS["W"], _WORKER_WEIGHTS["b"]
    from oracle import treelstm_oracle as orc
    t0 = time.perf_counter()
    for _ in range(passes):
        orc.schedule(left, right)
        orc.forward_recursive(left, right, token, emb, W, b)
    return time.perf_counter() - t0


def oracle_baselines(w: fg.Workload, budget_s: float = 8.0):
    """The fp64 oracle, as it stands, on whole trees of the workload: (i) one thread, (ii) all host
    cores with the trees dealt out to one single-threaded process per core (the paper's own
    inter-instance parallelism, Section 6.3).  Each figure takes about budget_s seconds."""
    import multiprocessing as mp
    from threadpoolctl import threadpool_limits
    from paper_1809_00832_b200 import sharding
    p, forest = w.params, w.forest
    cores = os.cpu_count() or 1
    sizes = np.bincount(forest.tree_of, minlength=forest.n_trees)
    with threadpool_limits(limits=1):
        probe = fg.select_trees(forest, list(range(min(8, forest.n_trees))))
        per_node = _oracle_pass((probe.left, probe.right, probe.token, p.emb, p.W, p.b, 1)) / max(probe.n_nodes, 1)
        avg_nodes = forest.n_nodes / forest.n_trees
        want = int(max(1, min(forest.n_trees, budget_s / max(per_node * avg_nodes, 1e-9))))
        sample = fg.select_trees(forest, list(range(want)))
        passes1 = int(max(1, min(200, round(budget_s / max(per_node * sample.n_nodes, 1e-9)))))
        secs1 = _oracle_pass((sample.left, sample.right, sample.token, p.emb, p.W, p.b, passes1))
    one = {"value": sample.n_trees * passes1 / secs1, "unit": UNIT, "cores": 1, "kind": "oracle",
           "sample": f"{passes1} pass(es) over the first {sample.n_trees} of {forest.n_trees} trees "
                     f"({sample.n_nodes} nodes), {secs1:.1f} s, BLAS limited to one thread",
           "nodes_per_sec": sample.n_nodes * passes1 / secs1}
    # all cores: every worker gets a node-balanced share of the whole forest and repeats it
    workers = max(1, min(cores, forest.n_trees))
    passes = int(max(1, min(200, round(budget_s / max(per_node * forest.n_nodes / workers, 1e-9)))))
    jobs = []
    for r in range(workers):
        part = fg.select_trees(forest, sharding.shard_trees_by_nodes(sizes, r, workers))
        tok, emb_rows = _compact_embedding(part.token, p.emb)
        jobs.append((part.left, part.right, tok, emb_rows, None, None, passes))
    env_old = {k: os.environ.get(k) for k in ("OMP_NUM_THREADS", "OPENBLAS_NUM_THREADS", "MKL_NUM_THREADS")}
    for k in env_old:
        os.environ[k] = "1"                     # inherited by the spawned workers: one thread each
    try:
        ctx = mp.get_context("spawn")           # never fork a process that has touched the GPU
        with ctx.Pool(workers, initializer=_oracle_init, initargs=(p.W, p.b)) as pool:
            pool.map(_oracle_pass, [(j[0][:0], j[1][:0], j[2][:0], j[3][:1], None, None, 1) for j in jobs],
                     chunksize=1)               # start-up and imports, untimed
            t0 = time.perf_counter()
            pool.map(_oracle_pass, jobs, chunksize=1)
            secs = time.perf_counter() - t0
    finally:
        for k, v in env_old.items():
            if v is None:
                os.environ.pop(k, None)
            else:
                os.environ[k] = v
    many = {"value": forest.n_trees * passes / secs, "unit": UNIT, "cores": workers, "kind": "oracle",
            "sample": f"{passes} pass(es) over all {forest.n_trees} trees ({forest.n_nodes} nodes) dealt out by node count "
                      f"to {workers} single-threaded processes (host has {cores} cores), {secs:.1f} s wall",
            "nodes_per_sec": forest.n_nodes * passes / secs}
    return one, many


# ---- timing helpers ------------------------------------------------------------------------------ #
def _dev(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def time_forward(model, forest, flags, steps, warmup, flush, kernel_every=16, overlap_launch=None):
    """`steps` forward calls on a device-resident forest, L2 flushed before each (untimed), CUDA events
    on the launching stream around every call.  The wavefront kernel's own device time is taken in a
    second pass (same flushing, read on every kernel_every-th call): the library's event pair around
    that kernel sits between the scheduler and the wavefront kernel on the stream and keeps the
    latter from starting under the former, so it stays out of the timed steps.
    Returns (per-step ms list, mean kernel ms, launches, outputs)."""
    import torch
    from paper_1809_00832_b200 import binding
    left, right, token = _dev(forest.left), _dev(forest.right), _dev(forest.token)
    model.set_option(binding.OPT_TIME_WAVEFRONT_KERNEL, 0)
    out = model.forward(left, right, token, flags=flags)          # allocates outputs, checks status
    for _ in range(warmup):
        flush.fill_(1)
        model.forward(left, right, token, flags=flags, out=out, check=False)
    torch.cuda.synchronize()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    launches = 0
    for i in range(steps):
        flush.fill_(i & 0xFF)                       # evict the previous step's data from L2 (untimed)
        ev[i][0].record()
        model.forward(left, right, token, flags=flags, out=out, check=False)
        ev[i][1].record()
        launches += model.last_launch_count()
    torch.cuda.synchronize()
    status = model.status_sync()
    if status != 0:
        raise RuntimeError(f"device status {status} after the timed region")
    model.set_option(binding.OPT_TIME_WAVEFRONT_KERNEL, 1)

    def kernel_pass():
        ms = []
        for i in range(max(8 * kernel_every, min(steps, 512))):  # live device time of the wavefront kernel
            flush.fill_(i & 0xFF)
            model.forward(left, right, token, flags=flags, out=out, check=False)
            if i % kernel_every == kernel_every - 1:    # reading it waits for the device: not after every call
                ms.append(model.last_kernel_ms())
        return statistics.mean(ms)

    # the kernel of the timed steps, alone: the event in front of it makes it start when the scheduler has
    # ended, its code and order of work (large bf16 forests: leaves first) stay those of the steps
    k_ms = kernel_pass()
    TIMINGS["kernel_ms_plain_order"] = None
    if overlap_launch is None or overlap_launch:
        # for the record: the form the library uses in plain stream order (cooperative launch)
        model.set_option(binding.OPT_OVERLAP_LAUNCH, 0)
        TIMINGS["kernel_ms_plain_order"] = kernel_pass()
    model.set_option(binding.OPT_TIME_WAVEFRONT_KERNEL, 0)
    model.set_option(binding.OPT_OVERLAP_LAUNCH, 1 if overlap_launch is None else overlap_launch)
    return [a.elapsed_time(b) for a, b in ev], k_ms, launches, out


def extra_forward(name, n_trees, peaks, flush, steps=200, warmup=5):
    """One more workload for the record (not the headline): whole-call and kernel time, roofline."""
    from paper_1809_00832_b200 import binding
    w = fg.make_workload(name, 0, n_trees)
    f, p = w.forest, w.params
    prec = binding.BF16 if w.precision == "bf16" else binding.FP32
    model = binding.TreeLSTM(p.H, p.E, p.vocab, _dev(p.emb), _dev(p.W), _dev(p.b), prec)
    step_ms, k_ms, launches, out = time_forward(model, f, binding.PERSISTENT, steps, warmup, flush, kernel_every=4)
    mean = sum(step_ms) / len(step_ms)
    roof = roofline_block(f, p, w.precision, k_ms, mean, peaks, name if n_trees is None else f"{name}[{n_trees}]")
    res = {"workload": name if n_trees is None else f"{name}, {n_trees} tree(s)", "trees": f.n_trees, "nodes": f.n_nodes,
           "levels": int(out["n_levels"].item()), "dtype": "bf16" if w.precision == "bf16" else "f32",
           "ms_per_step": mean, "kernel_ms": k_ms, "trees_per_sec": f.n_trees / (mean * 1e-3),
           "nodes_per_sec": f.n_nodes / (mean * 1e-3), "steps": steps, "gpu_launches_per_step": launches // steps,
           "roofline": {k: roof[k] for k in ("bound", "achieved", "peak", "unit", "frac", "frac_of_step", "hbm_frac",
                                             "tensor_frac_of_sustained")}}
    model.close()
    return res


def wavefront_latency_floor(peaks, flush, levels_of_headline, steps=100, warmup=5):
    """Third, non-judged line: what the dependency depth alone costs.  A single left chain of 64
    leaves has 64 wavefronts of one or two nodes each: its kernel time / 64 is the latency of an
    (almost) empty wavefront; times the headline workload's level count = the floor no amount of
    bandwidth or tensor throughput removes."""
    import torch
    from paper_1809_00832_b200 import binding
    rng = np.random.default_rng(0)
    p = fg.draw_params(rng, 256, 300, 20000, emb_dist="normal", emb_scale=0.1, w_scale=0.05)
    forest = fg.forest_from_shapes([fg.left_chain_shape(64)], rng, p.vocab)
    model = binding.TreeLSTM(p.H, p.E, p.vocab, _dev(p.emb), _dev(p.W), _dev(p.b), binding.BF16)
    step_ms, k_ms, _, out = time_forward(model, forest, binding.PERSISTENT, steps, warmup, flush, kernel_every=4)
    levels = int(out["n_levels"].item())
    per = k_ms / levels
    model.close()
    return {"probe": "one left chain of 64 leaves, H=256, E=300, bf16", "probe_levels": levels, "probe_kernel_ms": k_ms,
            "ms_per_empty_wavefront": per, "levels": levels_of_headline, "floor_ms": per * levels_of_headline}


def train_step_time(peaks, flush, steps: int = 200, warmup: int = 5):
    """Extra figure: the training step (forward keeping activations + backward through structure) on
    the 25-tree fp32 workload, timed with CUDA events, L2 flushed between steps."""
    import torch
    from paper_1809_00832_b200 import binding
    w = fg.make_workload("train25_fp32", 0)
    f, p = w.forest, w.params
    model = binding.TreeLSTM(p.H, p.E, p.vocab, _dev(p.emb), _dev(p.W), _dev(p.b), binding.FP32)
    model.set_classifier(_dev(p.Wc), _dev(p.bc))
    left, right, token, labels = _dev(f.left), _dev(f.right), _dev(f.token), _dev(w.labels)
    flags = binding.PERSISTENT | binding.SAVE_FOR_BACKWARD
    out = model.forward(left, right, token, flags=flags)
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    launches = 0
    for i in range(-warmup, steps):
        flush.fill_(i & 0xFF)
        if i >= 0:
            ev[i][0].record()
        model.forward(left, right, token, flags=flags, out=out, check=False)
        launches = model.last_launch_count()
        model.backward(labels, f.n_leaves)
        launches += model.last_launch_count()
        if i >= 0:
            ev[i][1].record()
    torch.cuda.synchronize()
    ms = [a.elapsed_time(b) for a, b in ev]
    mean = sum(ms) / len(ms)
    # training step: forward flops + backward (dIn and dW: twice the forward contraction) and, beside the
    # forward's bytes, the saved gates written and read (5H floats per node), dz written and read twice,
    # dh/dc written and read, the gradients written once
    fl, by = algorithmic_work(f, p.H, p.E, 4)
    n, H, E, C = f.n_nodes, p.H, p.E, p.C
    flops = 3 * fl + 4 * n * H * C
    bytes_ = by + n * 5 * H * 4 * 2 + n * 5 * H * 4 * 3 + n * 2 * H * 4 * 2 + ((E + 2 * H) * 5 * H + 5 * H + H * C + C) * 4 + f.n_leaves * E * 4
    gbs = bytes_ / (mean * 1e-3) / 1e9
    return {"workload": "train25_fp32", "trees": f.n_trees, "nodes": f.n_nodes, "ms_per_step": mean,
            "trees_per_sec": f.n_trees / (mean * 1e-3), "nodes_per_sec": f.n_nodes / (mean * 1e-3),
            "steps": steps, "gpu_launches_per_step": launches, "dtype": "f32",
            "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": gbs / peaks["hbm_gbs"], "algorithmic_bytes": bytes_, "algorithmic_flops": flops,
                         "fp32_tflops": flops / (mean * 1e-3) / 1e12,
                         "note": "whole step (forward + backward launches together); fp32 FMA pipes except the "
                                 "weight gradient, a split-bf16 tensor-core contraction"},
            "note": "persistent forward + one-launch backward (wavefronts) + tensor-core dW/db kernel; the binding "
                    "reads the status word back after each"}


def run_sweeps(args):
    """Extra benchmark lines on synthetic trees, after the paper's shape study (Section 6.3, Table 1:
    balanced / moderate / linear trees at batch 1, 10, 25) and its time-per-instance-vs-length plot
    (Figure 11, batch 1).  One JSON line per point; not the headline metric."""
    import torch
    from paper_1809_00832_b200 import binding, build
    build.build()
    rng = np.random.default_rng(0)
    if args.cell == "treelstm":
        p = fg.draw_params(rng, 256, 300, 20000, emb_dist="normal", emb_scale=0.1, w_scale=0.05)
        model = binding.TreeLSTM(p.H, p.E, p.vocab, _dev(p.emb), _dev(p.W), _dev(p.b), binding.BF16)
    else:
        # the paper's Table 1 is measured on TreeRNN; the other cells run fp32 kernels on the same scheduler
        tensor = args.cell == "rntn"
        H = 32 if tensor else 128
        p = fg.draw_recursive_params(rng, H, 20000, tensor=tensor, emb_scale=0.5, w_scale=1.0 / np.sqrt(2 * H),
                                     v_scale=1.0 / (2 * H))
        model = binding.TreeLSTM.recursive(binding.CELL_RNTN if tensor else binding.CELL_TREERNN, H, p.vocab,
                                           _dev(p.emb), _dev(p.W), _dev(p.b), _dev(p.V) if tensor else None)
    if args.tail_width is not None and args.cell == "treelstm":
        model.set_option(binding.OPT_TAIL_WIDTH, args.tail_width)
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device="cuda")

    flags = {"persistent": binding.PERSISTENT, "per_level": binding.PER_LEVEL, "subforests": binding.SUBFORESTS}[args.mode]

    def time_forest(forest, steps=100, warmup=5):
        left, right, token = _dev(forest.left), _dev(forest.right), _dev(forest.token)
        out = model.forward(left, right, token, flags=flags)
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for i in range(-warmup, steps):
            flush.fill_(i & 0xFF)
            if i >= 0:
                ev[i][0].record()
            model.forward(left, right, token, flags=flags, out=out, check=False)
            if i >= 0:
                ev[i][1].record()
        torch.cuda.synchronize()
        return sum(a.elapsed_time(b) for a, b in ev) / steps, int(out["n_levels"].item())

    shapes = {"balanced": lambda: fg.balanced_shape(32), "moderate": lambda: fg.random_split_shape(rng, 32),
              "linear": lambda: fg.left_chain_shape(32)}
    if args.sweep in ("shapes", "all"):
        for name, make in shapes.items():
            for batch in (1, 10, 25):
                forest = fg.forest_from_shapes([make() for _ in range(batch)], rng, p.vocab)
                ms, levels = time_forest(forest)
                print(json.dumps({"sweep": "shape", "cell": args.cell, "mode": args.mode, "tail_width": args.tail_width, "shape": name, "leaves_per_tree": 32, "batch": batch,
                                  "levels": levels, "ms_per_step": ms, "trees_per_sec": batch / (ms * 1e-3)}))
    if args.sweep in ("length", "all"):
        for leaves in (2, 4, 8, 16, 24, 32, 40, 48, 56):
            forest = fg.forest_from_shapes([fg.random_split_shape(rng, leaves)], rng, p.vocab)
            ms, levels = time_forest(forest)
            print(json.dumps({"sweep": "length", "cell": args.cell, "mode": args.mode, "tail_width": args.tail_width, "leaves": leaves, "batch": 1, "levels": levels,
                              "ms_per_instance": ms}))
    return 0


def run_reference(args):
    """The reference arm of this build is the CPU oracle: one step = the oracle on a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    from oracle import treelstm_oracle as orc
    w = fg.make_workload(args.workload, 0, args.trees)
    p = w.params
    steps, warmup = args.steps, args.warmup
    # bound the sample so that steps + warmup oracle passes finish in a couple of minutes
    probe = fg.select_trees(w.forest, [0, 1, 2, 3])
    t0 = time.perf_counter()
    orc.forward_recursive(probe.left, probe.right, probe.token, p.emb, p.W, p.b)
    per_node = (time.perf_counter() - t0) / probe.n_nodes
    budget = 100.0 / max(steps + warmup, 1)
    avg_nodes = w.forest.n_nodes / w.forest.n_trees
    n_sample = int(max(1, min(w.forest.n_trees, budget / (per_node * avg_nodes))))
    sample = fg.select_trees(w.forest, list(range(n_sample)))
    times = []
    for it in range(warmup + steps):
        t0 = time.perf_counter()
        orc.schedule(sample.left, sample.right)
        orc.forward_recursive(sample.left, sample.right, sample.token, p.emb, p.W, p.b)
        if it >= warmup:
            times.append(time.perf_counter() - t0)
    total = sum(times)
    value = sample.n_trees * steps / total
    threads = 1
    try:
        from threadpoolctl import threadpool_info
        threads = max([q.get("num_threads", 1) for q in threadpool_info()] + [1])
    except Exception:
        pass
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": warmup, "ms_per_step": 1e3 * total / steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "trees_per_step": sample.n_trees, "nodes_per_step": sample.n_nodes,
                   "note": "CPU oracle on the first trees of the workload"},
        "nodes_per_sec": sample.n_nodes * steps / total,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                         "sample": f"first {sample.n_trees} of {w.forest.n_trees} trees ({sample.n_nodes} nodes) per step; one "
                                   f"process, NumPy's BLAS pool of {threads} thread(s) (host has {os.cpu_count()} cores)"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


def main() -> int:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--workload", default="batch256_bf16", choices=fg.WORKLOADS)
    ap.add_argument("--trees", type=int, default=None, help="number of trees of the workload (default: its own batch size)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--mode", default="persistent", choices=MODES)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-train", action="store_true", help="skip the extra training-step figure")
    ap.add_argument("--no-extra", action="store_true", help="skip the extra workloads and the latency-floor probe")
    ap.add_argument("--cell", default="treelstm", choices=["treelstm", "treernn", "rntn"],
                    help="cell of the sweeps (the benchmark line itself is always TreeLSTM)")
    ap.add_argument("--tail-width", type=int, default=None,
                    help="sweeps only: widest wavefront handed to the one-cluster kernel (0 = never hand over)")
    ap.add_argument("--leaves-first-min-nodes", type=int, default=None,
                    help="headline run only: smallest forest whose leaf wavefront runs before the wait for the schedule")
    ap.add_argument("--overlap-launch", type=int, default=None, choices=[0, 1],
                    help="headline run only: 0 = plain stream order between the scheduler and the wavefront kernel")
    ap.add_argument("--sweep", default=None, choices=["shapes", "length", "all"],
                    help="print the tree-shape / sentence-length sweeps instead of the benchmark line")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        return run_reference(args)
    if args.sweep:
        return run_sweeps(args)

    import torch
    from paper_1809_00832_b200 import binding, build

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the TreeLSTM library has no CPU path")

    w = fg.make_workload(args.workload, seed=rank, n_trees=args.trees)
    f, p = w.forest, w.params
    cpu_one = cpu_many = None
    if world == 1 and not args.no_cpu_baseline:
        cpu_one, cpu_many = oracle_baselines(w)      # before the first GPU call: it starts worker processes

    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    if rank == 0:
        build.build()
    if dist is not None:
        dist.barrier()
    prec = binding.BF16 if w.precision == "bf16" else binding.FP32
    model = binding.TreeLSTM(p.H, p.E, p.vocab, _dev(p.emb), _dev(p.W), _dev(p.b), prec)
    if args.overlap_launch is not None:
        model.set_option(binding.OPT_OVERLAP_LAUNCH, args.overlap_launch)
    if args.leaves_first_min_nodes is not None:
        model.set_option(binding.OPT_LEAVES_FIRST_MIN_NODES, args.leaves_first_min_nodes)
    flags = {"persistent": binding.PERSISTENT, "per_level": binding.PER_LEVEL, "subforests": binding.SUBFORESTS}[args.mode]
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device="cuda")

    sampler = ClockSampler(local_rank)
    sampler.start()
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    step_ms, k_ms, launches, out = time_forward(model, f, flags, args.steps, args.warmup, flush, overlap_launch=args.overlap_launch)
    if dist is not None:
        dist.barrier()
    ran = {binding.PERSISTENT: "persistent", binding.PER_LEVEL: "per_level", binding.SUBFORESTS: "subforests"}[model.last_mode()]
    total_ms = sum(step_ms)
    clocks = sampler.stop()

    # ---- end to end through the host-buffer entry point (pinned host arrays in, root states out) ----
    hl, hr, ht = binding.pack_forest_host(f.left, f.right, f.token)   # one pinned buffer: one host-to-device copy
    host_out = model.forward_host(hl, hr, ht, flags=flags, max_roots=f.n_trees)
    e2e_steps = max(20, min(args.steps, 200))
    for _ in range(3):
        model.forward_host(hl, hr, ht, flags=flags, max_roots=f.n_trees, out=host_out)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(e2e_steps):
        model.forward_host(hl, hr, ht, flags=flags, max_roots=f.n_trees, out=host_out)
    e1.record()
    torch.cuda.synchronize()
    e2e_ms = e0.elapsed_time(e1)
    e2e_wall_ms = 1e3 * (time.perf_counter() - t0)
    h2d = 3 * 4 * f.n_nodes
    d2h = f.n_trees * (2 * 4 * p.H + 4) + 8

    # ---- max over ranks, aggregate ----
    from paper_1809_00832_b200 import sharding
    (total_ms, e2e_ms), (agg_trees, agg_nodes) = sharding.combine([total_ms, e2e_ms], [f.n_trees, f.n_nodes],
                                                                  device="cuda")
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return 0

    peaks = measured_peaks()
    levels = int(out["n_levels"].item())
    value = agg_trees * args.steps / (total_ms * 1e-3)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if w.precision == "bf16" else "f32", "data": "synthetic",
        "config": {"workload": args.workload, "trees": f.n_trees, "nodes": f.n_nodes, "leaves": f.n_leaves,
                   "levels": levels, "H": p.H, "E": p.E, "vocab": p.vocab, "mode": ran,
                   "l2": "flushed between timed steps (256 MB write, untimed)", "seed": "rank"},
        "nodes_per_sec": agg_nodes * args.steps / (total_ms * 1e-3),
        "step_ms_p10_p50_p90": [float(np.percentile(step_ms, q)) for q in (10, 50, 90)],
        "clocks": clocks,
        "e2e": {"value": agg_trees * e2e_steps / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "steps": e2e_steps, "wall_ms_per_step": e2e_wall_ms / e2e_steps,
                "returns": "root ids and root (h, c) of every tree",
                "device_staging": "caller-provided (torch) through treelstm_set_host_staging"},
        "gpu_launches": launches,
        "roofline": roofline_block(f, p, w.precision, k_ms, total_ms / args.steps, peaks, args.workload),
    }
    if world == 1 and not args.no_extra:
        line["latency_floor"] = wavefront_latency_floor(peaks, flush, levels)
        extra = []
        for name, nt in (("batch25_fp32", None), ("chains64_bf16", None), ("balanced1024_bf16", None),
                         ("batch256_bf16", 1), ("batch256_bf16", 10), ("batch256_bf16", 25)):
            if name == args.workload and nt is None:
                continue
            extra.append(extra_forward(name, nt, peaks, flush))
        line["extra"] = extra
    if world == 1 and not args.no_train:
        line["train_step"] = train_step_time(peaks, flush)
    if cpu_many is not None:
        line["cpu_baseline"] = cpu_many
        line["cpu_baseline_1thread"] = cpu_one
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
