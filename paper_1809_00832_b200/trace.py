"""Per-wavefront cycle tables of the bf16 wavefront kernels, from the trace build of the library.

    python -m paper_1809_00832_b200.trace --workload chains64_bf16 [--mode persistent|subforests]
                                          [--tail-width N] [--tail-min-levels M] [--trees T] [--levels A:B]

The trace build (-DTREELSTM_TRACE, libtreelstm_b200_trace.so) makes the first CTA of each kernel write
clock64 stamps for the first 256 wavefronts; the table prints them in cycles since the wavefront's
first stamp (s0), 0 where a stamp was not taken.

Grid-wide kernel (k_fwd_tc): s0 start of the wavefront, s6 its tiles are done in this CTA, s7 the grid
barrier has opened; first epilogue thread, the CTA's first tile of the wavefront: s1 accumulator
complete, s2 cell updates done, s3 tile left (outputs copied); s8, s9, s10 the same for the CTA's
second tile; operand producer: s14 / s15 first / last box of the first tile requested, s11 / s12 the
same for the second tile; MMA issuer: s4 first box of the first tile has landed, s13 first box of the
second tile has landed, s5 last MMAs of the (second, if any) tile issued.

Cluster kernel of the narrow tail (k_fwd_tc_tail), stamps of different warps of one CTA:
  s0  the CTA's per-wavefront barrier has opened (all warps but the MMA issuer)
  s14 epilogue: copies of the previous wavefront to global memory are out
  s12 / s13 fetching warps: tables of the next wavefront read / its older child cell states read
  s1 / s7 producer: prefetch of the next wavefront's operand rows requested / landed
  s2 / s3 MMA issuer: operands complete (prefetch and pushes) / last MMA committed
  s4  epilogue: accumulator complete      s8  gate values in shared memory
  s9  older child cell states are in      s5  cell updates done
  s10 new h complete in shared memory     s11 every peer's prefetch has landed (pushes may go)
  s6  pushes issued
One-launch backward (--train: train25_fp32, fp32 forward + k_bwd_persistent), first CTA, per wavefront in
reverse: s0 start, s1 gate gradients done, s2 barrier, s3 input gradients done, s4 barrier; and the
phases of the kernel.
The sub-forest kernel (--mode subforests) uses s0 start, s1 first operand request, s2 first box seen by
the MMA issuer, s3 last MMAs committed, s4 epilogue starts waiting, s5 last tile stored, s6 arrival at
the cluster barrier, s7 barrier left.  The stamps cost a few cycles each; the normal build is a little
faster.
"""
from __future__ import annotations

import argparse
import ctypes

import numpy as np
import torch

from . import binding, build, forests as fg

SLOTS, LEVELS = 16, 256


def read_trace(model: binding.TreeLSTM, which: int) -> np.ndarray:
    buf = (ctypes.c_longlong * (SLOTS * LEVELS))()
    fn = model.lib.treelstm_trace_read
    fn.restype = ctypes.c_int
    fn.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p, ctypes.c_int]
    got = fn(model.handle, which, ctypes.cast(buf, ctypes.c_void_p), SLOTS * LEVELS)
    if got < 0:
        raise binding.TreeLSTMError(got, "treelstm_trace_read")
    return np.frombuffer(buf, dtype=np.int64).reshape(LEVELS, SLOTS).copy()


def trace_training_step() -> int:
    w = fg.make_workload("train25_fp32", 0)
    f, p = w.forest, w.params
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    model = binding.TreeLSTM(p.H, p.E, p.vocab, dev(p.emb), dev(p.W), dev(p.b), binding.FP32, variant="trace")
    model.set_classifier(dev(p.Wc), dev(p.bc))
    left, right, token, labels = dev(f.left), dev(f.right), dev(f.token), dev(w.labels)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    for i in range(4):
        flush.fill_(i)
        out = model.forward(left, right, token, flags=binding.PERSISTENT | binding.SAVE_FOR_BACKWARD)
        model.backward(labels, f.n_leaves)
    torch.cuda.synchronize()
    widths = np.diff(out["level_offset"].cpu().numpy()[:int(out["n_levels"].item()) + 1])
    tf = read_trace(model, 1)
    phf = tf[LEVELS - 1]
    print(f"# fp32 persistent forward, first CTA, cycles since its start: weight slice fetched {int(phf[1] - phf[0])}, "
          f"schedule there {int(phf[2] - phf[0])}, last stamp {int(tf[:LEVELS - 1].max() - phf[0])}")
    print("level width tiles_done barrier_passed ids_resolved first_chunk contracted   (cycles since the wavefront's start; the last three: streaming tiles only)")
    for l in range(len(widths)):
        if tf[l, 0]:
            print(f"{l:<5d} {int(widths[l]):<5d} " + " ".join(f"{(tf[l, k] - tf[l, 0]) if tf[l, k] else 0:<10d}" for k in (1, 2, 3, 4, 5)))
    t = read_trace(model, 0)
    ph = t[LEVELS - 1]
    names = ("outputs and scratch cleared", "tokens marked", "own part of token scan / classifier done",
             "classifier, loss, token scan done everywhere", "all wavefronts done", "dW from the leaves (own blocks)",
             "dW from the internal nodes (own blocks)", "db done", "token scan: first warp has read its flags",
             "token scan: all warps have", "classifier (second CTA): starts", "classifier: first warp's node done",
             "classifier: all warps' nodes done", "classifier: partial sums sent")
    print("# one-launch backward, first CTA, cycles since its start: " +
          ", ".join(f"{nm} {int(ph[i + 1] - ph[0])}" for i, nm in enumerate(names) if ph[i + 1]))
    print("level width gates_done barrier dinput_done barrier first_dz contracted own_blocks operands_landed request_begin indices_requested weights_requested   (cycles since the wavefront's start; "
          "wavefronts run in reverse; the last three only where the gate gradients are formed inside the contraction)")
    for l in range(len(widths) - 1, -1, -1):
        if t[l, 0] == 0:
            continue
        print(f"{l:<5d} {int(widths[l]):<5d} " + " ".join(f"{(t[l, k] - t[l, 0]) if t[l, k] else 0:<10d}" for k in range(1, 12)))
    return 0


def main() -> int:
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="batch256_bf16", choices=[w for w in fg.WORKLOADS if w.endswith("bf16")])
    ap.add_argument("--mode", default="persistent", choices=["persistent", "subforests"])
    ap.add_argument("--tail-width", type=int, default=None)
    ap.add_argument("--tail-min-levels", type=int, default=None)
    ap.add_argument("--trees", type=int, default=None)
    ap.add_argument("--levels", default=None, help="A:B - print only wavefronts A..B-1")
    ap.add_argument("--train", action="store_true", help="trace the one-launch backward of a training step on train25_fp32")
    ap.add_argument("--plain-order", action="store_true",
                    help="launch the grid-wide kernel cooperatively behind the scheduler instead of under it")
    args = ap.parse_args()
    build.build(variant="trace")
    if args.train:
        return trace_training_step()
    w = fg.make_workload(args.workload, 0, args.trees)
    f, p = w.forest, w.params
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    model = binding.TreeLSTM(p.H, p.E, p.vocab, dev(p.emb), dev(p.W), dev(p.b), binding.BF16, variant="trace")
    if args.tail_width is not None:
        model.set_option(binding.OPT_TAIL_WIDTH, args.tail_width)
    if args.tail_min_levels is not None:
        model.set_option(binding.OPT_TAIL_MIN_LEVELS, args.tail_min_levels)
    flags = binding.PERSISTENT if args.mode == "persistent" else binding.SUBFORESTS
    left, right, token = dev(f.left), dev(f.right), dev(f.token)
    # the first call in plain stream order: it clears the stamp table (a call started under the scheduler
    # keeps the stamps of the call before)
    model.set_option(binding.OPT_OVERLAP_LAUNCH, 0)
    out = model.forward(left, right, token, flags=flags)
    model.set_option(binding.OPT_OVERLAP_LAUNCH, 0 if args.plain_order else 1)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    for i in range(4):                                   # the last call is the one read back, caches as in the bench
        flush.fill_(i)
        model.forward(left, right, token, flags=flags, out=out, check=False)
    torch.cuda.synchronize()
    widths = np.diff(out["level_offset"].cpu().numpy()[:int(out["n_levels"].item()) + 1])
    lo, hi = 0, len(widths)
    if args.levels:
        a, b = args.levels.split(":")
        lo, hi = int(a or 0), int(b or hi)
    buf = (ctypes.c_longlong * 16)()
    fn = model.lib.treelstm_trace_read
    fn.restype = ctypes.c_int
    fn.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p, ctypes.c_int]
    if fn(model.handle, 2, ctypes.cast(buf, ctypes.c_void_p), 16) > 0:
        names = ("cleared", "validated+linked", "links checked, leaves reported", "climbed", "levels written", "ordered")
        print("# single-CTA scheduler, thread 0, cycles since its start: " +
              ", ".join(f"{nm} {int(buf[i])}" for i, nm in enumerate(names)))
        print("#   inside the few-levels placement (cycles since its start): counts cleared, counted, rows scanned, "
              "starts known, placed = " + ", ".join(str(int(buf[8 + i])) for i in range(5)))
    for which, name in ((0, "grid-wide kernel"), (1, "cluster kernel")):
        t = read_trace(model, which)
        if which == 0 and t[LEVELS - 1, 4] != 0:
            ph = t[LEVELS - 1]
            names = ("set up, own node ids read", "leaf counts of all CTAs known", "own leaves ranked, embedding rows copied",
                     "all rows in place (leaf wavefront starts)", "leaf wavefront done everywhere", "scheduler ended, schedule read",
                     "slots written, leaf states handed over", "first internal wavefront may start")
            print("# grid-wide kernel started under the scheduler, first CTA, cycles since its start: " +
                  ", ".join(f"{nm} {int(ph[i + 1] - ph[0])}" for i, nm in enumerate(names)))
            t[LEVELS - 1] = 0
        rows = [l for l in range(min(len(widths), LEVELS)) if t[l, 0] != 0]
        if not rows:
            continue
        print(f"# {name}: wavefronts {rows[0]}..{rows[-1]}; cycles since the wavefront's start")
        print("level width " + " ".join(f"s{k:<6d}" for k in range(1, SLOTS)) + " total(to next start)")
        for l in rows:
            if not lo <= l < hi:
                continue
            base = t[l, 0]
            cells = " ".join(f"{(t[l, k] - base) if t[l, k] else 0:<7d}" for k in range(1, SLOTS))
            nxt = t[l + 1, 0] - base if l + 1 < LEVELS and t[l + 1, 0] else 0
            print(f"{l:<5d} {int(widths[l]):<5d} {cells} {nxt}")
        print(f"# first stamp to last stamp: {int(t[rows].max() - t[rows[0], 0])} cycles")
    return 0


if __name__ == "__main__":
    raise SystemExit(main())
