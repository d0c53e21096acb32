"""Seeded synthetic forests and parameter draws for the binary TreeLSTM path.

This module only *draws inputs*: tree shapes as child-index arrays, leaf token
ids, labels, and random parameter tensors.  It contains none of the TreeLSTM
arithmetic, so the CPU oracle and the CUDA path can both be fed from it without
sharing any of the method's code.

A forest of T trees with N nodes in total is three int32 arrays of length N:
``left[n]``, ``right[n]`` (both -1 for a leaf, both valid node ids for an
internal node) and ``token[n]`` (vocabulary id for a leaf, -1 for an internal
node).  This is the array form of ``tree.leaves[idx]`` / ``tree.children[idx]``
used by the paper's TreeLSTM pseudocode (Section 2.2, Figures 1 and 2).

The paper evaluates on binary parse trees of movie-review sentences (Section
6.1) at batch sizes 1, 10 and 25, and on balanced / moderate / linear tree
shapes (Section 6.3, Table 1).  That dataset is not reproduced here; the
generators below draw random shapes with the same structure: a uniform split
point at every internal node ("moderate"), fully left-branching chains
("linear") and perfectly balanced trees ("balanced").
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional

import numpy as np


@dataclass
class Forest:
    """Child-index arrays of a batch of binary trees plus leaf tokens."""

    left: np.ndarray          # int32[N], -1 for leaves
    right: np.ndarray         # int32[N], -1 for leaves
    token: np.ndarray         # int32[N], -1 for internal nodes
    roots: np.ndarray         # int32[T], node id of each tree's root
    tree_of: np.ndarray       # int32[N], which tree a node belongs to

    @property
    def n_nodes(self) -> int:
        return int(self.left.shape[0])

    @property
    def n_trees(self) -> int:
        return int(self.roots.shape[0])

    @property
    def n_leaves(self) -> int:
        return int((self.left < 0).sum())


@dataclass
class Params:
    """Model parameters (float32, the precision the C-ABI takes them in)."""

    H: int
    E: int
    vocab: int
    emb: np.ndarray           # [vocab][E]
    W: np.ndarray             # [E + 2H][5H], column blocks i, f_l, f_r, o, u
    b: np.ndarray             # [5H]
    C: int = 0
    Wc: Optional[np.ndarray] = None   # [H][C]
    bc: Optional[np.ndarray] = None   # [C]


@dataclass
class Workload:
    name: str
    forest: Forest
    params: Params
    precision: str                      # "fp32" or "bf16"
    labels: Optional[np.ndarray] = None  # int32[N]
    meta: Dict[str, object] = field(default_factory=dict)


# --------------------------------------------------------------------------- #
# tree shapes
# --------------------------------------------------------------------------- #

def _emit_postorder(shape, left, right, is_leaf):
    """shape is a nested tuple ((l, r)) or None for a leaf; appends nodes in
    post-order (children before parents) and returns the id of the subtree root.
    Iterative, so that chains of any depth do not hit the recursion limit."""
    # stack entries: (shape, state, left_id) with state 0=enter, 1=after left, 2=after right
    result = None
    stack = [[shape, 0, -1, -1]]
    while stack:
        top = stack[-1]
        node, state = top[0], top[1]
        if node is None:
            left.append(-1)
            right.append(-1)
            is_leaf.append(True)
            result = len(left) - 1
            stack.pop()
            continue
        if state == 0:
            top[1] = 1
            stack.append([node[0], 0, -1, -1])
        elif state == 1:
            top[2] = result
            top[1] = 2
            stack.append([node[1], 0, -1, -1])
        else:
            top[3] = result
            left.append(top[2])
            right.append(top[3])
            is_leaf.append(False)
            result = len(left) - 1
            stack.pop()
    return result


def random_split_shape(rng: np.random.Generator, n_leaves: int):
    """Random binary tree over ``n_leaves`` leaves: the left subtree of every
    internal node gets k leaves, k uniform in 1..n-1, recursively."""
    if n_leaves == 1:
        return None
    k = int(rng.integers(1, n_leaves))
    return (random_split_shape(rng, k), random_split_shape(rng, n_leaves - k))


def left_chain_shape(n_leaves: int):
    """Fully left-branching chain: ((((w0 w1) w2) w3) ...)."""
    shape = None
    for _ in range(n_leaves - 1):
        shape = (shape, None)
    return shape


def balanced_shape(n_leaves: int):
    """Perfectly balanced tree; ``n_leaves`` must be a power of two."""
    assert n_leaves >= 1 and (n_leaves & (n_leaves - 1)) == 0
    if n_leaves == 1:
        return None
    half = balanced_shape(n_leaves // 2)
    return (half, half)


def forest_from_shapes(shapes: List[object], rng: np.random.Generator, vocab: int) -> Forest:
    left: List[int] = []
    right: List[int] = []
    is_leaf: List[bool] = []
    roots: List[int] = []
    tree_of: List[int] = []
    for t, shape in enumerate(shapes):
        before = len(left)
        roots.append(_emit_postorder(shape, left, right, is_leaf))
        tree_of.extend([t] * (len(left) - before))
    leaf_mask = np.asarray(is_leaf, dtype=bool)
    token = np.full(len(left), -1, dtype=np.int32)
    token[leaf_mask] = rng.integers(0, vocab, size=int(leaf_mask.sum()), dtype=np.int64).astype(np.int32)
    return Forest(
        left=np.asarray(left, dtype=np.int32),
        right=np.asarray(right, dtype=np.int32),
        token=token,
        roots=np.asarray(roots, dtype=np.int32),
        tree_of=np.asarray(tree_of, dtype=np.int32),
    )


def random_forest(rng: np.random.Generator, n_trees: int, min_leaves: int, max_leaves: int,
                  vocab: int) -> Forest:
    """``n_trees`` random-split trees with leaf counts uniform in [min, max] (inclusive)."""
    shapes = []
    for _ in range(n_trees):
        n_leaves = int(rng.integers(min_leaves, max_leaves + 1))
        shapes.append(random_split_shape(rng, n_leaves))
    return forest_from_shapes(shapes, rng, vocab)


def permute_node_ids(forest: Forest, rng: np.random.Generator):
    """Renumber the nodes at random.  Returns (new_forest, new_id_of_old) so that
    per-node results of the permuted forest at ``new_id_of_old[n]`` must equal the
    results of the original forest at ``n``.  The recursive formulation does not
    need topologically sorted ids (Section 2.2), the iterative one does."""
    n = forest.n_nodes
    new_id_of_old = rng.permutation(n).astype(np.int32)
    left = np.full(n, -1, dtype=np.int32)
    right = np.full(n, -1, dtype=np.int32)
    token = np.full(n, -1, dtype=np.int32)
    tree_of = np.zeros(n, dtype=np.int32)
    for old in range(n):
        new = new_id_of_old[old]
        if forest.left[old] >= 0:
            left[new] = new_id_of_old[forest.left[old]]
            right[new] = new_id_of_old[forest.right[old]]
        token[new] = forest.token[old]
        tree_of[new] = forest.tree_of[old]
    roots = new_id_of_old[forest.roots]
    return Forest(left, right, token, roots.astype(np.int32), tree_of), new_id_of_old


def concat_forests(forests: List[Forest]) -> Forest:
    """Concatenate forests, shifting node ids and tree ids."""
    lefts, rights, tokens, roots, tree_of = [], [], [], [], []
    node_base = 0
    tree_base = 0
    for f in forests:
        shift_l = np.where(f.left >= 0, f.left + node_base, -1)
        shift_r = np.where(f.right >= 0, f.right + node_base, -1)
        lefts.append(shift_l.astype(np.int32))
        rights.append(shift_r.astype(np.int32))
        tokens.append(f.token)
        roots.append((f.roots + node_base).astype(np.int32))
        tree_of.append((f.tree_of + tree_base).astype(np.int32))
        node_base += f.n_nodes
        tree_base += f.n_trees
    return Forest(np.concatenate(lefts), np.concatenate(rights), np.concatenate(tokens),
                  np.concatenate(roots), np.concatenate(tree_of))


def select_trees(forest: Forest, tree_ids) -> Forest:
    """Sub-forest made of the given trees (node ids renumbered, order kept)."""
    keep = np.isin(forest.tree_of, np.asarray(tree_ids))
    old_ids = np.nonzero(keep)[0]
    new_of_old = np.full(forest.n_nodes, -1, dtype=np.int64)
    new_of_old[old_ids] = np.arange(old_ids.shape[0])
    left = np.where(forest.left[old_ids] >= 0, new_of_old[forest.left[old_ids]], -1).astype(np.int32)
    right = np.where(forest.right[old_ids] >= 0, new_of_old[forest.right[old_ids]], -1).astype(np.int32)
    tree_map = {int(t): i for i, t in enumerate(tree_ids)}
    tree_of = np.asarray([tree_map[int(t)] for t in forest.tree_of[old_ids]], dtype=np.int32)
    roots = new_of_old[forest.roots[np.asarray(tree_ids)]].astype(np.int32)
    return Forest(left, right, forest.token[old_ids].copy(), roots, tree_of)


# --------------------------------------------------------------------------- #
# parameters
# --------------------------------------------------------------------------- #

def draw_params(rng: np.random.Generator, H: int, E: int, vocab: int, *, emb_dist: str,
                emb_scale: float, w_scale: float, n_classes: int = 0) -> Params:
    """emb_dist: "normal" (std emb_scale) or "uniform" (in +-emb_scale).  W, b and the
    classifier are uniform in +-w_scale (non-zero biases so that bias paths are exercised)."""
    if emb_dist == "normal":
        emb = rng.normal(0.0, emb_scale, size=(vocab, E))
    else:
        emb = rng.uniform(-emb_scale, emb_scale, size=(vocab, E))
    W = rng.uniform(-w_scale, w_scale, size=(E + 2 * H, 5 * H))
    b = rng.uniform(-w_scale, w_scale, size=(5 * H,))
    p = Params(H=H, E=E, vocab=vocab, emb=emb.astype(np.float32), W=W.astype(np.float32),
               b=b.astype(np.float32))
    if n_classes > 0:
        p.C = n_classes
        p.Wc = rng.uniform(-w_scale, w_scale, size=(H, n_classes)).astype(np.float32)
        p.bc = rng.uniform(-w_scale, w_scale, size=(n_classes,)).astype(np.float32)
    return p


@dataclass
class RecursiveParams:
    """Parameters of a TreeRNN / RNTN model (float32): word vectors double as leaf states."""

    H: int
    vocab: int
    emb: np.ndarray           # [vocab][H]
    W: np.ndarray             # [2H][H]
    b: np.ndarray             # [H]
    V: Optional[np.ndarray] = None    # [H][2H][2H], RNTN only


def draw_recursive_params(rng: np.random.Generator, H: int, vocab: int, *, tensor: bool, emb_scale: float,
                          w_scale: float, v_scale: float = 0.0) -> RecursiveParams:
    """Word vectors uniform in +-emb_scale, W and b uniform in +-w_scale, the tensor slices (RNTN,
    tensor=True) uniform in +-v_scale."""
    emb = rng.uniform(-emb_scale, emb_scale, size=(vocab, H)).astype(np.float32)
    W = rng.uniform(-w_scale, w_scale, size=(2 * H, H)).astype(np.float32)
    b = rng.uniform(-w_scale, w_scale, size=(H,)).astype(np.float32)
    V = rng.uniform(-v_scale, v_scale, size=(H, 2 * H, 2 * H)).astype(np.float32) if tensor else None
    return RecursiveParams(H=H, vocab=vocab, emb=emb, W=W, b=b, V=V)


# --------------------------------------------------------------------------- #
# named workloads
# --------------------------------------------------------------------------- #

WORKLOADS = ("tiny8", "batch25_fp32", "batch256_bf16", "chains64_bf16", "balanced1024_bf16",
             "train25_fp32")


def make_workload(name: str, seed: int = 0, n_trees: Optional[int] = None) -> Workload:
    """The synthetic workloads the tests and the benchmark run.

    tiny8             8 random trees of exactly 8 leaves, H=E=16, vocab 100, all U(-0.1, 0.1), fp32
    batch25_fp32      25 random trees, 2..56 leaves, H=150, E=300, vocab 20000, emb N(0, 0.1),
                      W U(-0.05, 0.05), fp32 (batch 25 is the paper's largest batch, Section 6.2)
    batch256_bf16     256 such trees, H=256, E=300, bf16 operands (throughput mode)
    chains64_bf16     64 left chains of 64 leaves ("linear" shape of Table 1), H=256, E=300, bf16
    balanced1024_bf16 16 balanced trees of 1024 leaves ("balanced" shape of Table 1), same sizes
    train25_fp32      batch25_fp32 plus a 5-class classifier and uniform labels on every node
    ``n_trees`` overrides the batch size (the paper also runs batch 1 and 10).
    """
    rng = np.random.default_rng(seed)
    if name == "tiny8":
        T = n_trees or 8
        shapes = [random_split_shape(rng, 8) for _ in range(T)]
        forest = forest_from_shapes(shapes, rng, 100)
        params = draw_params(rng, 16, 16, 100, emb_dist="uniform", emb_scale=0.1, w_scale=0.1)
        return Workload(name, forest, params, "fp32")
    if name in ("batch25_fp32", "train25_fp32"):
        T = n_trees or 25
        forest = random_forest(rng, T, 2, 56, 20000)
        ncls = 5 if name == "train25_fp32" else 0
        params = draw_params(rng, 150, 300, 20000, emb_dist="normal", emb_scale=0.1,
                             w_scale=0.05, n_classes=ncls)
        labels = None
        if ncls:
            labels = rng.integers(0, ncls, size=forest.n_nodes, dtype=np.int64).astype(np.int32)
        return Workload(name, forest, params, "fp32", labels=labels)
    if name == "batch256_bf16":
        T = n_trees or 256
        forest = random_forest(rng, T, 2, 56, 20000)
        params = draw_params(rng, 256, 300, 20000, emb_dist="normal", emb_scale=0.1, w_scale=0.05)
        return Workload(name, forest, params, "bf16")
    if name == "chains64_bf16":
        T = n_trees or 64
        forest = forest_from_shapes([left_chain_shape(64) for _ in range(T)], rng, 20000)
        params = draw_params(rng, 256, 300, 20000, emb_dist="normal", emb_scale=0.1, w_scale=0.05)
        return Workload(name, forest, params, "bf16")
    if name == "balanced1024_bf16":
        T = n_trees or 16
        forest = forest_from_shapes([balanced_shape(1024) for _ in range(T)], rng, 20000)
        params = draw_params(rng, 256, 300, 20000, emb_dist="normal", emb_scale=0.1, w_scale=0.05)
        return Workload(name, forest, params, "bf16")
    raise ValueError(f"unknown workload {name!r}; known: {WORKLOADS}")
