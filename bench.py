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
# dram__bytes_read.sum + dram__bytes_write.sum of one k_fwd_tc launch from the committed ncu capture
# (profiles/k_fwd_tc_batch256_bf16.md); None for workloads without a capture of the current kernel.
NCU_TRAFFIC_BYTES = {"batch256_bf16": 11202048}


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


def oracle_sample_time(w: fg.Workload, budget_s: float = 15.0):
    """Times the CPU oracle (fp64 recursive evaluation, as it stands) on whole trees of the workload,
    as many as fit in about `budget_s` seconds.  Returns (trees, nodes, seconds, threads)."""
    from oracle import treelstm_oracle as orc
    threads = 1
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        pass
    p = w.params
    probe = fg.select_trees(w.forest, list(range(min(8, w.forest.n_trees))))
    t0 = time.perf_counter()
    orc.schedule(probe.left, probe.right)
    orc.forward_recursive(probe.left, probe.right, probe.token, p.emb, p.W, p.b)
    dt = time.perf_counter() - t0
    per_node = dt / max(probe.n_nodes, 1)
    avg_nodes = w.forest.n_nodes / w.forest.n_trees
    want = int(max(8, min(w.forest.n_trees, budget_s / max(per_node * avg_nodes, 1e-9))))
    sample = fg.select_trees(w.forest, list(range(want)))
    # whole passes over the sample until about budget_s seconds of CPU work are done
    passes = int(max(1, min(200, round(budget_s / max(per_node * sample.n_nodes, 1e-9)))))
    t0 = time.perf_counter()
    for _ in range(passes):
        orc.schedule(sample.left, sample.right)
        orc.forward_recursive(sample.left, sample.right, sample.token, p.emb, p.W, p.b)
    dt = time.perf_counter() - t0
    return sample.n_trees * passes, sample.n_nodes * passes, dt, threads


def train_step_time(steps: int = 200, warmup: int = 5):
    """Extra figure: the training step (forward keeping activations + backward through structure) on
    the 25-tree fp32 workload, timed with CUDA events, L2 flushed between steps."""
    import torch
    from paper_1809_00832_b200 import binding
    w = fg.make_workload("train25_fp32", 0)
    f, p = w.forest, w.params
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    model = binding.TreeLSTM(p.H, p.E, p.vocab, dev(p.emb), dev(p.W), dev(p.b), binding.FP32)
    model.set_classifier(dev(p.Wc), dev(p.bc))
    left, right, token, labels = dev(f.left), dev(f.right), dev(f.token), dev(w.labels)
    flags = binding.PERSISTENT | binding.SAVE_FOR_BACKWARD
    out = model.forward(left, right, token, flags=flags)
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device="cuda")
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
    return {"workload": "train25_fp32", "trees": f.n_trees, "nodes": f.n_nodes, "ms_per_step": mean,
            "trees_per_sec": f.n_trees / (mean * 1e-3), "nodes_per_sec": f.n_nodes / (mean * 1e-3),
            "steps": steps, "gpu_launches_per_step": launches, "dtype": "f32",
            "note": "persistent forward + one-launch backward; the binding reads the status word back after each"}


def run_sweeps(args):
    """Extra benchmark lines on synthetic trees, after the paper's shape study (Section 6.3, Table 1:
    balanced / moderate / linear trees at batch 1, 10, 25) and its time-per-instance-vs-length plot
    (Figure 11, batch 1).  One JSON line per point; not the headline metric."""
    import torch
    from paper_1809_00832_b200 import binding, build
    build.build()
    rng = np.random.default_rng(0)
    p = fg.draw_params(rng, 256, 300, 20000, emb_dist="normal", emb_scale=0.1, w_scale=0.05)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    model = binding.TreeLSTM(p.H, p.E, p.vocab, dev(p.emb), dev(p.W), dev(p.b), binding.BF16)
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device="cuda")

    flags = {"persistent": binding.PERSISTENT, "per_level": binding.PER_LEVEL, "subforests": binding.SUBFORESTS}[args.mode]

    def time_forest(forest, steps=100, warmup=5):
        left, right, token = dev(forest.left), dev(forest.right), dev(forest.token)
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
                print(json.dumps({"sweep": "shape", "mode": args.mode, "shape": name, "leaves_per_tree": 32, "batch": batch,
                                  "levels": levels, "ms_per_step": ms, "trees_per_sec": batch / (ms * 1e-3)}))
    if args.sweep in ("length", "all"):
        for leaves in (2, 4, 8, 16, 24, 32, 40, 48, 56):
            forest = fg.forest_from_shapes([fg.random_split_shape(rng, leaves)], rng, p.vocab)
            ms, levels = time_forest(forest)
            print(json.dumps({"sweep": "length", "mode": args.mode, "leaves": leaves, "batch": 1, "levels": levels,
                              "ms_per_instance": ms}))
    return 0


def run_reference(args):
    """The reference arm of this build is the CPU oracle: one step = the oracle on a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    from oracle import treelstm_oracle as orc
    w = fg.make_workload(args.workload, 0)
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
                         "sample": f"first {sample.n_trees} of {w.forest.n_trees} trees ({sample.n_nodes} nodes) per step"},
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
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--mode", default="persistent", choices=["persistent", "per_level", "subforests"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-train", action="store_true", help="skip the extra training-step figure")
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
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    if rank == 0:
        build.build()
    if dist is not None:
        dist.barrier()
    w = fg.make_workload(args.workload, seed=rank)
    f, p = w.forest, w.params
    prec = binding.BF16 if w.precision == "bf16" else binding.FP32
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    model = binding.TreeLSTM(p.H, p.E, p.vocab, dev(p.emb), dev(p.W), dev(p.b), prec)
    model.set_option(binding.OPT_TIME_WAVEFRONT_KERNEL, 1)
    left, right, token = dev(f.left), dev(f.right), dev(f.token)
    flags = {"persistent": binding.PERSISTENT, "per_level": binding.PER_LEVEL, "subforests": binding.SUBFORESTS}[args.mode]
    out = model.forward(left, right, token, flags=flags)          # allocates outputs, checks status
    ran = {binding.PERSISTENT: "persistent", binding.PER_LEVEL: "per_level", binding.SUBFORESTS: "subforests"}[model.last_mode()]
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device="cuda")

    sampler = ClockSampler(local_rank)
    sampler.start()
    for _ in range(args.warmup):
        flush.fill_(1)
        model.forward(left, right, token, flags=flags, out=out, check=False)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    kernel_ms = []
    launches = 0
    torch.cuda.synchronize()
    for i in range(args.steps):
        flush.fill_(i & 0xFF)                       # evict the previous step's data from L2 (untimed)
        ev[i][0].record()
        model.forward(left, right, token, flags=flags, out=out, check=False)
        ev[i][1].record()
        launches += model.last_launch_count()
        if i % 16 == 0:                             # live device time of the wavefront kernel
            kernel_ms.append(model.last_kernel_ms())
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    status = model.status_sync()
    if status != 0:
        raise RuntimeError(f"device status {status} after the timed region")
    step_ms = [a.elapsed_time(b) for a, b in ev]
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
    flops, abytes = algorithmic_work(f, p.H, p.E, 2 if w.precision == "bf16" else 4)
    k_ms = statistics.mean(kernel_ms)
    achieved_gbs = abytes / (k_ms * 1e-3) / 1e9
    achieved_tflops = flops / (k_ms * 1e-3) / 1e12
    value = agg_trees * args.steps / (total_ms * 1e-3)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if w.precision == "bf16" else "f32", "data": "synthetic",
        "config": {"workload": args.workload, "trees": f.n_trees, "nodes": f.n_nodes, "leaves": f.n_leaves,
                   "levels": int(out["n_levels"].item()), "H": p.H, "E": p.E, "vocab": p.vocab, "mode": ran,
                   "l2": "flushed between timed steps (256 MB write, untimed)", "seed": "rank"},
        "nodes_per_sec": agg_nodes * args.steps / (total_ms * 1e-3),
        "step_ms_p10_p50_p90": [float(np.percentile(step_ms, q)) for q in (10, 50, 90)],
        "clocks": clocks,
        "e2e": {"value": agg_trees * e2e_steps / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "steps": e2e_steps, "wall_ms_per_step": e2e_wall_ms / e2e_steps,
                "returns": "root ids and root (h, c) of every tree"},
        "gpu_launches": launches,
        "roofline": {"bound": "hbm", "achieved": achieved_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": achieved_gbs / peaks["hbm_gbs"], "traffic": NCU_TRAFFIC_BYTES.get(args.workload), "peak_source": peaks["source"],
                     "kernel": "k_fwd_tc (persistent wavefront kernel)" if w.precision == "bf16" else "k_fwd_fp32_persistent",
                     "kernel_ms": k_ms, "algorithmic_bytes": abytes, "algorithmic_flops": flops,
                     "tensor_tflops": achieved_tflops,
                     "tensor_frac_of_sustained": achieved_tflops / peaks["bf16_tflops_sustained"]},
    }
    if world == 1 and not args.no_train:
        line["train_step"] = train_step_time()
    if world == 1 and not args.no_cpu_baseline:
        trees, nodes, secs, threads = oracle_sample_time(w)
        line["cpu_baseline"] = {"value": trees / secs, "unit": UNIT, "cores": threads, "kind": "oracle",
                                "sample": f"{trees} trees ({nodes} nodes) = whole passes over the first trees of the workload, {secs:.1f} s",
                                "nodes_per_sec": nodes / secs}
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
