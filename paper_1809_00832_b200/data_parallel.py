"""Data-parallel training step across ranks (one process per GPU).

The paper scales training by data parallelism over machines (Section 6.2); here the trees of a
batch are independent units, so every rank runs forward + backward through structure on its own
shard of the forest and the gradients are then combined.  The exchange is the only collective on
the path:

  * the loss of the library is a mean over the nodes it was given, so a rank's loss and gradients
    are weighted by its share of the nodes, n_r / N, and summed (one all-reduce for the dense
    gradients dW, db, dWc, dbc and the loss);
  * the gradient of the embedding table is sparse: every rank has its own sorted list of touched
    token ids and one gradient row per id.  The lists are gathered, merged into one sorted list of
    distinct ids, and rows of the same id are added.

Works with any torch.distributed backend: NCCL over NVLink on GPUs, gloo in the CPU tests.  With a
single process (or without an initialised process group) every function returns its input
unchanged.
"""
from __future__ import annotations

from typing import Dict

import torch

DENSE_KEYS = ("dW", "db", "dWc", "dbc")


def _world() -> int:
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        return dist.get_world_size()
    return 1


def combine_gradients(local: Dict[str, torch.Tensor], n_local_nodes: int) -> Dict[str, torch.Tensor]:
    """Gradients of the mean loss over the WHOLE forest from the per-rank results.

    `local` is what treelstm_backward produced on this rank's shard: loss [1], dW, db, dWc, dbc,
    touched_ids [>= n_touched] (sorted, distinct), dEmb_rows [>= n_touched][E], n_touched [1]; all on
    one device.  Returns a dict with the same keys; touched_ids / dEmb_rows hold exactly n_touched
    entries, the same on every rank."""
    world = _world()
    nt = int(local["n_touched"].reshape(-1)[0].item())
    if world == 1:
        out = dict(local)
        out["touched_ids"] = local["touched_ids"][:nt]
        out["dEmb_rows"] = local["dEmb_rows"][:nt]
        return out
    import torch.distributed as dist
    dev = local["dW"].device
    ftype = local["dW"].dtype

    # share of the nodes: one small all-reduce gives N, the largest touched count and nothing else
    meta = torch.tensor([float(n_local_nodes)], dtype=torch.float64, device=dev)
    dist.all_reduce(meta, op=dist.ReduceOp.SUM)
    n_total = float(meta[0].item())
    weight = float(n_local_nodes) / n_total if n_total > 0 else 0.0

    # dense part: scale, flatten into one buffer, one all-reduce
    parts = [local["loss"].reshape(-1).to(ftype)] + [local[k].reshape(-1) for k in DENSE_KEYS]
    flat = torch.cat(parts) * weight
    dist.all_reduce(flat, op=dist.ReduceOp.SUM)
    out: Dict[str, torch.Tensor] = {}
    pos = 1
    out["loss"] = flat[:1].clone()
    for k in DENSE_KEYS:
        n = local[k].numel()
        out[k] = flat[pos:pos + n].reshape(local[k].shape).clone()
        pos += n

    # sparse part: gather (count, ids, rows) padded to the largest count, then merge
    E = local["dEmb_rows"].shape[1]
    cnt = torch.tensor([nt], dtype=torch.int64, device=dev)
    cmax = cnt.clone()
    dist.all_reduce(cmax, op=dist.ReduceOp.MAX)
    m = int(cmax.item())
    ids = torch.full((m,), -1, dtype=torch.int64, device=dev)
    rows = torch.zeros((m, E), dtype=ftype, device=dev)
    ids[:nt] = local["touched_ids"][:nt].to(torch.int64)
    rows[:nt] = local["dEmb_rows"][:nt] * weight
    all_ids = [torch.empty_like(ids) for _ in range(world)]
    all_rows = [torch.empty_like(rows) for _ in range(world)]
    dist.all_gather(all_ids, ids)
    dist.all_gather(all_rows, rows)
    cat_ids = torch.cat(all_ids)
    cat_rows = torch.cat(all_rows)
    keep = cat_ids >= 0
    cat_ids, cat_rows = cat_ids[keep], cat_rows[keep]
    uniq, inverse = torch.unique(cat_ids, sorted=True, return_inverse=True)
    merged = torch.zeros((uniq.numel(), E), dtype=ftype, device=dev)
    merged.index_add_(0, inverse, cat_rows)
    out["touched_ids"] = uniq.to(local["touched_ids"].dtype)
    out["dEmb_rows"] = merged
    out["n_touched"] = torch.tensor([uniq.numel()], dtype=local["n_touched"].dtype, device=dev)
    return out


def training_step(model, left: torch.Tensor, right: torch.Tensor, token: torch.Tensor, labels: torch.Tensor,
                  n_leaves: int, flags: int) -> Dict[str, torch.Tensor]:
    """One data-parallel training step on this rank's shard (device tensors): forward keeping the
    gate activations, backward through structure, then the gradient exchange.  `model` is a
    binding.TreeLSTM with a classifier; `flags` selects the forward mode."""
    from . import binding
    model.forward(left, right, token, flags=flags | binding.SAVE_FOR_BACKWARD, check=False)
    grads = model.backward(labels, n_leaves)
    return combine_gradients(grads, int(left.shape[0]))
