"""CPU oracle for the two other recursive models of the paper's evaluation.  TEST INFRASTRUCTURE ONLY.

The paper evaluates three recursive neural networks (Section 6.1): TreeLSTM (see
``treelstm_oracle.py``), TreeRNN and RNTN; Table 1 (Section 6.3) is measured on TreeRNN.  It
prints the equations of none of them and takes the models "as suggested in the original papers",
so the cells stated here are the published ones:

    TreeRNN  (recursive neural network):   p = tanh(W^T [h_l ; h_r] + b)
    RNTN     (recursive neural tensor network):
             p_j = tanh([h_l ; h_r]^T V_j [h_l ; h_r] + (W^T [h_l ; h_r])_j + b_j),  j = 0 .. H-1

with W of shape [2H][H], b of shape [H] and V of shape [H][2H][2H] (one 2H x 2H slice per
output unit).  A leaf's state is its word vector, h = emb[token], so the embedding width equals
H; a node has no cell state.  Evaluation follows Figure 2 (Section 3.1): a node calls itself on
both children, the leaves are the base case; ``forward_iterative`` is the Figure 1 form over any
dependency-respecting order (Section 6.2: both are numerically identical).

Training as for the TreeLSTM workload (Section 6.1: every node carries a label): a softmax
classifier on every node's state, mean cross-entropy over all nodes, gradients by the recursion of
Section 4.2.2 run from the parents to the children.  Leaves are labelled too; their classifier
gradient flows into the embedding row.

Plain NumPy fp64, no blocking or fusion; shares no code with the CUDA path and imports nothing
from it.  Pins: tests/test_oracle_cells_pins.py (exact values from tanh(atanh 1/2), hand-unrolled
scalar chains, torch.nn.RNNCell on a left chain, torch.nn.Bilinear for the tensor term, an explicit
triple loop, V = 0 and antisymmetric V reducing to TreeRNN, swap symmetry, recursive == iterative,
central finite differences and torch autograd for the gradients).  No function is unpinned.
"""
from __future__ import annotations

import sys
from typing import Dict, Optional

import numpy as np

TREERNN = "treernn"
RNTN = "rntn"


def cell(kind: str, W: np.ndarray, b: np.ndarray, V: Optional[np.ndarray], h_l: np.ndarray,
         h_r: np.ndarray, round_in=None) -> np.ndarray:
    """State of an internal node from its two children's states."""
    x = np.concatenate([h_l, h_r])
    if round_in is not None:
        x = round_in(x)
    z = W.T @ x + b
    if kind == RNTN:
        z = z + np.array([x @ V[j] @ x for j in range(V.shape[0])])
    elif kind != TREERNN:
        raise ValueError(kind)
    return np.tanh(z)


def _find_roots(left, right):
    n = left.shape[0]
    has_parent = np.zeros(n, dtype=bool)
    for k in range(n):
        if left[k] >= 0:
            has_parent[left[k]] = True
            has_parent[right[k]] = True
    return np.nonzero(~has_parent)[0]


def forward_recursive(kind, left, right, token, emb, W, b, V=None, operand_round=None) -> np.ndarray:
    """Figure 2: state(idx) = word vector at a leaf, cell(state(left), state(right)) otherwise.
    Node ids may be in any order.  Returns h as fp64 [N][H]."""
    emb, W, b = (np.asarray(a, dtype=np.float64) for a in (emb, W, b))
    V = None if V is None else np.asarray(V, dtype=np.float64)
    n, H = left.shape[0], b.shape[0]
    assert emb.shape[1] == H and W.shape == (2 * H, H)
    if operand_round is not None:
        W = operand_round(W)
        V = None if V is None else operand_round(V)
    h = np.zeros((n, H))

    def state(idx: int) -> np.ndarray:
        if left[idx] < 0:
            h[idx] = emb[token[idx]]
        else:
            h_l = state(int(left[idx]))
            h_r = state(int(right[idx]))
            h[idx] = cell(kind, W, b, V, h_l, h_r, round_in=operand_round)
        return h[idx]

    old = sys.getrecursionlimit()
    sys.setrecursionlimit(max(old, 4 * n + 1000))
    try:
        for root in _find_roots(left, right):
            state(int(root))
    finally:
        sys.setrecursionlimit(old)
    return h


def forward_iterative(kind, left, right, token, emb, W, b, order, V=None) -> np.ndarray:
    """Figure 1: the same cell over a dependency-respecting node order, states in an indexed array."""
    emb, W, b = (np.asarray(a, dtype=np.float64) for a in (emb, W, b))
    V = None if V is None else np.asarray(V, dtype=np.float64)
    n, H = left.shape[0], b.shape[0]
    h = np.zeros((n, H))
    for idx in order:
        idx = int(idx)
        if left[idx] < 0:
            h[idx] = emb[token[idx]]
        else:
            h[idx] = cell(kind, W, b, V, h[int(left[idx])], h[int(right[idx])])
    return h


def classifier_loss(h, Wc, bc, labels):
    """Mean softmax cross-entropy over all nodes; returns (loss, probabilities [N][C])."""
    Wc, bc = np.asarray(Wc, dtype=np.float64), np.asarray(bc, dtype=np.float64)
    logits = h @ Wc + bc
    m = logits.max(axis=1, keepdims=True)
    lse = m[:, 0] + np.log(np.exp(logits - m).sum(axis=1))
    n = h.shape[0]
    loss = float(np.mean(lse - logits[np.arange(n), labels]))
    return loss, np.exp(logits - lse[:, None])


def _topological_order(left, right) -> np.ndarray:
    """Children before parents (post-order from every root), written without recursion."""
    order = []
    for root in _find_roots(left, right):
        stack = [(int(root), False)]
        while stack:
            idx, expanded = stack.pop()
            if left[idx] < 0 or expanded:
                order.append(idx)
            else:
                stack.append((idx, True))
                stack.append((int(right[idx]), False))
                stack.append((int(left[idx]), False))
    return np.asarray(order, dtype=np.int64)


def loss_and_gradients(kind, left, right, token, emb, W, b, Wc, bc, labels, V=None) -> Dict[str, object]:
    """Training step: forward, mean cross-entropy on every node's state, backpropagation through
    structure with parents before children (Section 4.2.2), every node using its own forward
    state (Sections 4.2.1 and 5).

        dh_n   = Wc (p_n - e_y)/N + [what the caller passes down]
        dz_n   = dh_n * (1 - h_n^2)                       (internal nodes)
        dW    += x_n (x) dz_n,  db += dz_n,  dV_j += dz_n[j] * x_n (x) x_n
        dx_n   = W dz_n + sum_j dz_n[j] (V_j + V_j^T) x_n   -> dh of the two children
        leaf:  dEmb[token] += dh_n

    Returns loss, dW, db, dWc, dbc, dV (RNTN), touched_ids (sorted unique leaf tokens), dEmb_rows
    (one summed row per touched id) and h."""
    emb64, W64, b64, Wc64, bc64 = (np.asarray(a, dtype=np.float64) for a in (emb, W, b, Wc, bc))
    V64 = None if V is None else np.asarray(V, dtype=np.float64)
    n, H = left.shape[0], b64.shape[0]
    h = forward_recursive(kind, left, right, token, emb64, W64, b64, V64)
    loss, probs = classifier_loss(h, Wc64, bc64, labels)
    dlogits = probs.copy()
    dlogits[np.arange(n), labels] -= 1.0
    dlogits /= n
    dWc = h.T @ dlogits
    dbc = dlogits.sum(axis=0)
    dh = dlogits @ Wc64.T
    dW = np.zeros_like(W64)
    db = np.zeros_like(b64)
    dV = None if V64 is None else np.zeros_like(V64)
    dEmb = {}
    for idx in _topological_order(left, right)[::-1]:      # parents before children
        idx = int(idx)
        if left[idx] < 0:
            t = int(token[idx])
            dEmb[t] = dEmb.get(t, np.zeros(H)) + dh[idx]
            continue
        l, r = int(left[idx]), int(right[idx])
        x = np.concatenate([h[l], h[r]])
        dz = dh[idx] * (1.0 - h[idx] * h[idx])
        dW += np.outer(x, dz)
        db += dz
        dx = W64 @ dz
        if kind == RNTN:
            for j in range(H):
                dV[j] += dz[j] * np.outer(x, x)
                dx += dz[j] * ((V64[j] + V64[j].T) @ x)
        dh[l] += dx[:H]
        dh[r] += dx[H:]
    touched = np.asarray(sorted(dEmb), dtype=np.int32)
    rows = np.stack([dEmb[int(t)] for t in touched]) if len(touched) else np.zeros((0, H))
    out = dict(loss=loss, dW=dW, db=db, dWc=dWc, dbc=dbc, touched_ids=touched, dEmb_rows=rows, h=h)
    if dV is not None:
        out["dV"] = dV
    return out


def loss_only(kind, left, right, token, emb, W, b, Wc, bc, labels, V=None) -> float:
    h = forward_recursive(kind, left, right, token, emb, W, b, V)
    return classifier_loss(h, Wc, bc, labels)[0]
