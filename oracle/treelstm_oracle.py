"""CPU oracle for the binary TreeLSTM hot path.  TEST INFRASTRUCTURE ONLY.

A plain, slow, fp64 NumPy statement of what the path computes.  It exists to
check the CUDA library and to be timed as a CPU baseline; the product never
calls it.  It shares no code with the CUDA path and imports nothing from it.

What follows which passage of the paper (arXiv 1809.00832):

* ``forward_recursive``  - the recursive TreeLSTM of Figure 2 (Section 3.1): a
  node's state is ``LSTM(embed(word))`` at a leaf and ``LSTM(left_state,
  right_state)`` at an internal node, the two child states coming from two
  recursive calls that do not depend on each other.
* ``forward_iterative``  - the iterative TreeLSTM of Figure 1 (Section 2.2):
  the same cell applied over topologically ordered node indices with the states
  kept in an indexed array.  Section 6.2 ("Convergence") states that both give
  numerically identical results.
* ``schedule``           - the dependency-driven execution of Section 4.1.1: a
  node is ready once all its inputs are resolved; the set of nodes that become
  ready together is a wavefront ("level").  Each node also records its caller
  (``parent``), the return location of Section 4.1.2 ("graph execution stack").
* ``loss_and_gradients`` - backpropagation through the recursion (Section
  4.2.2): gradient computation recurses at the same positions as the forward
  pass, parents before children, and every node instance uses its own retained
  forward values (Section 4.2.1, Section 5 "backpropagation cache").

The paper names the cell only as ``LSTM(...)``; the equations used here are the
standard binary (N-ary, N=2) TreeLSTM cell:

    in  = [x ; h_l ; h_r]                      (x = 0 at internal nodes,
                                                h_l = h_r = c_l = c_r = 0 at leaves)
    z   = W^T in + b,   W is [(E+2H)][5H],  z split into (z_i, z_fl, z_fr, z_o, z_u)
    i, f_l, f_r, o = sigmoid(.),  u = tanh(z_u)
    c   = i*u + f_l*c_l + f_r*c_r
    h   = o * tanh(c)

Training: logits_n = Wc^T h_n + bc on every node, loss = mean over all nodes of
the softmax cross-entropy against labels y_n.

Pins (tests/test_oracle_pins.py): exact leaf values from known function values,
a hand-unrolled scalar left chain, torch.nn.LSTMCell on the chain special case,
closed forms for W_h = 0 and saturated gates, duplicated-subtree identity, child
swap symmetry, recursive == iterative, brute-force tree heights, closed-form
level widths for chains and balanced trees, loss = ln C for uniform logits,
central finite differences for every gradient group.  No function is unpinned.
"""
from __future__ import annotations

import sys
from typing import Dict, Optional, Tuple

import numpy as np

# error codes of schedule() -- the numeric values mirror the library's public
# error enumeration (an interface, restated here, not shared code).
OK = 0
ERR_INVALID_FOREST = -2
ERR_TOKEN_OUT_OF_RANGE = -3


def sigmoid(z: np.ndarray) -> np.ndarray:
    return 1.0 / (1.0 + np.exp(-z))


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round fp64/fp32 values to the nearest bfloat16 (ties to even), returned as fp64.
    Diagnostic only: lets a test separate operand-rounding error from a bug."""
    f = np.asarray(a, dtype=np.float32)
    bits = f.view(np.uint32).astype(np.uint64)
    lsb = (bits >> np.uint64(16)) & np.uint64(1)
    rounded = (bits + np.uint64(0x7FFF) + lsb) & np.uint64(0xFFFF0000)
    return rounded.astype(np.uint32).view(np.float32).astype(np.float64).reshape(f.shape)


def cell(W: np.ndarray, b: np.ndarray, H: int, x: np.ndarray, h_l: np.ndarray, c_l: np.ndarray,
         h_r: np.ndarray, c_r: np.ndarray, round_in=None):
    """One TreeLSTM cell.  Returns (h, c, gates) with gates = (i, f_l, f_r, o, u).
    ``round_in`` (diagnostic) rounds the input vector before the contraction; the caller
    rounds W itself when it wants rounded weights."""
    inp = np.concatenate([x, h_l, h_r])
    if round_in is not None:
        inp = round_in(inp)
    z = W.T @ inp + b
    i = sigmoid(z[0 * H:1 * H])
    f_l = sigmoid(z[1 * H:2 * H])
    f_r = sigmoid(z[2 * H:3 * H])
    o = sigmoid(z[3 * H:4 * H])
    u = np.tanh(z[4 * H:5 * H])
    c = i * u + f_l * c_l + f_r * c_r
    h = o * np.tanh(c)
    return h, c, (i, f_l, f_r, o, u)


def _as64(*arrays):
    return [np.asarray(a, dtype=np.float64) for a in arrays]


def find_roots(left: np.ndarray, right: np.ndarray) -> np.ndarray:
    n = left.shape[0]
    has_parent = np.zeros(n, dtype=bool)
    for k in range(n):
        if left[k] >= 0:
            has_parent[left[k]] = True
            has_parent[right[k]] = True
    return np.nonzero(~has_parent)[0]


def forward_recursive(left, right, token, emb, W, b, operand_round=None):
    """Figure 2: TreeLSTM(idx) calls itself on both children; leaves are the base case.
    Node ids may be in any order.  Returns h, c as fp64 [N][H] and the gate tuple per node."""
    emb, W, b = _as64(emb, W, b)
    n = left.shape[0]
    H = b.shape[0] // 5
    E = emb.shape[1]
    h = np.zeros((n, H))
    c = np.zeros((n, H))
    gates = np.zeros((n, 5, H))
    zeros_h = np.zeros(H)
    zeros_x = np.zeros(E)
    if operand_round is not None:
        W = operand_round(W)

    def tree_lstm(idx: int):
        if left[idx] < 0:               # is_leaf_node(idx)
            x = emb[token[idx]]
            state = cell(W, b, H, x, zeros_h, zeros_h, zeros_h, zeros_h, round_in=operand_round)
        else:
            h_l, c_l = tree_lstm(int(left[idx]))
            h_r, c_r = tree_lstm(int(right[idx]))
            state = cell(W, b, H, zeros_x, h_l, c_l, h_r, c_r, round_in=operand_round)
        h[idx], c[idx] = state[0], state[1]
        gates[idx] = np.stack(state[2])
        return state[0], state[1]

    old = sys.getrecursionlimit()
    sys.setrecursionlimit(max(old, 4 * n + 1000))
    try:
        for root in find_roots(left, right):
            tree_lstm(int(root))
    finally:
        sys.setrecursionlimit(old)
    return h, c, gates


def schedule(left, right, token=None, vocab: Optional[int] = None):
    """Dependency-driven ready sets (Section 4.1.1).

    A leaf has no unresolved input and is ready at once (level 0); an internal node becomes
    ready as soon as both children are done: level = 1 + max(level of children).  ``order`` lists
    the nodes by ascending (level, node id) - the canonical ready order - and
    ``level_offset[l] .. level_offset[l+1]`` delimits wavefront l in ``order``.  ``parent`` is the
    caller of each node (-1 for roots).

    Returns (status, parent, level, order, level_offset).  status != OK for a forest that is not a
    set of disjoint binary trees (a child out of range, a node with exactly one child, a node that
    is its own child, a node with two parents, a cycle) or a leaf token outside [0, vocab)."""
    n = int(left.shape[0])
    parent = np.full(n, -1, dtype=np.int32)
    level = np.full(n, -1, dtype=np.int32)
    empty = np.zeros(0, dtype=np.int32)
    bad = (ERR_INVALID_FOREST, parent, level, empty, empty)
    for k in range(n):
        l, r = int(left[k]), int(right[k])
        if l < 0 and r < 0:
            if l != -1 or r != -1:
                return bad
            if token is not None and vocab is not None and not (0 <= int(token[k]) < vocab):
                return (ERR_TOKEN_OUT_OF_RANGE, parent, level, empty, empty)
            continue
        if l < 0 or r < 0 or l >= n or r >= n or l == r or l == k or r == k:
            return bad
        for ch in (l, r):
            if parent[ch] != -1:
                return bad
            parent[ch] = k
    # ready queue / waiting list: pending[k] = number of unresolved inputs
    pending = np.where(left < 0, 0, 2)
    ready = [k for k in range(n) if pending[k] == 0]
    for k in ready:
        level[k] = 0
    done = 0
    current = 0
    while ready:
        nxt = []
        for k in ready:
            done += 1
            p = int(parent[k])
            if p >= 0:
                pending[p] -= 1
                if pending[p] == 0:
                    level[p] = current + 1
                    nxt.append(p)
        ready = nxt
        current += 1
    if done != n:
        return bad                       # nodes on a cycle never become ready
    order = np.lexsort((np.arange(n), level)).astype(np.int32)
    n_levels = int(level.max()) + 1 if n else 0
    counts = np.bincount(level, minlength=n_levels) if n else np.zeros(0, dtype=np.int64)
    level_offset = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
    return OK, parent, level, order, level_offset


def forward_iterative(left, right, token, emb, W, b, order, operand_round=None):
    """Figure 1: walk the nodes in a dependency-respecting order, reading child states from the
    indexed state array.  ``order`` is any topological order (e.g. the one from ``schedule``)."""
    emb, W, b = _as64(emb, W, b)
    n = left.shape[0]
    H = b.shape[0] // 5
    E = emb.shape[1]
    h = np.zeros((n, H))
    c = np.zeros((n, H))
    gates = np.zeros((n, 5, H))
    zeros_h = np.zeros(H)
    zeros_x = np.zeros(E)
    if operand_round is not None:
        W = operand_round(W)
    for idx in order:
        idx = int(idx)
        if left[idx] < 0:
            state = cell(W, b, H, emb[token[idx]], zeros_h, zeros_h, zeros_h, zeros_h,
                         round_in=operand_round)
        else:
            l, r = int(left[idx]), int(right[idx])
            state = cell(W, b, H, zeros_x, h[l], c[l], h[r], c[r], round_in=operand_round)
        h[idx], c[idx] = state[0], state[1]
        gates[idx] = np.stack(state[2])
    return h, c, gates


def classifier_loss(h, Wc, bc, labels) -> Tuple[float, np.ndarray]:
    """Mean softmax cross-entropy over all nodes.  Returns (loss, probabilities [N][C])."""
    Wc, bc = _as64(Wc, bc)
    logits = h @ Wc + bc
    m = logits.max(axis=1, keepdims=True)
    lse = m[:, 0] + np.log(np.exp(logits - m).sum(axis=1))
    n = h.shape[0]
    loss = float(np.mean(lse - logits[np.arange(n), labels]))
    probs = np.exp(logits - lse[:, None])
    return loss, probs


def loss_and_gradients(left, right, token, emb, W, b, Wc, bc, labels) -> Dict[str, object]:
    """Training step: forward, mean cross-entropy on every node's h, and backpropagation
    through structure.  Gradients flow from parents to children (the gradient recursion visits
    the same positions as the forward recursion, Section 4.2.2), each node using its own saved
    gates and cell state (Section 5).

    Returns loss, dW, db, dWc, dbc, touched_ids (sorted unique leaf tokens) and dEmb_rows (one
    summed row per touched id), plus h, c for convenience."""
    emb64, W64, b64, Wc64, bc64 = _as64(emb, W, b, Wc, bc)
    n = left.shape[0]
    H = b64.shape[0] // 5
    E = emb64.shape[1]
    status, parent, level, order, _ = schedule(left, right)
    assert status == OK
    h, c, gates = forward_recursive(left, right, token, emb64, W64, b64)
    loss, probs = classifier_loss(h, Wc64, bc64, labels)

    dlogits = probs.copy()
    dlogits[np.arange(n), labels] -= 1.0
    dlogits /= n
    dWc = h.T @ dlogits
    dbc = dlogits.sum(axis=0)
    dh = dlogits @ Wc64.T                   # classifier contribution to every node's dh
    dc = np.zeros((n, H))
    dW = np.zeros_like(W64)
    db = np.zeros_like(b64)
    dEmb = {}

    for idx in order[::-1]:                 # parents before children
        idx = int(idx)
        i, f_l, f_r, o, u = gates[idx]
        tc = np.tanh(c[idx])
        dc_n = dc[idx] + dh[idx] * o * (1.0 - tc * tc)
        dz_o = dh[idx] * tc * o * (1.0 - o)
        dz_i = dc_n * u * i * (1.0 - i)
        dz_u = dc_n * i * (1.0 - u * u)
        if left[idx] < 0:
            x = emb64[token[idx]]
            inp = np.concatenate([x, np.zeros(2 * H)])
            dz_fl = np.zeros(H)
            dz_fr = np.zeros(H)
        else:
            l, r = int(left[idx]), int(right[idx])
            inp = np.concatenate([np.zeros(E), h[l], h[r]])
            dz_fl = dc_n * c[l] * f_l * (1.0 - f_l)
            dz_fr = dc_n * c[r] * f_r * (1.0 - f_r)
            dc[l] += dc_n * f_l
            dc[r] += dc_n * f_r
        dz = np.concatenate([dz_i, dz_fl, dz_fr, dz_o, dz_u])
        dW += np.outer(inp, dz)
        db += dz
        d_in = W64 @ dz
        if left[idx] < 0:
            t = int(token[idx])
            dEmb[t] = dEmb.get(t, np.zeros(E)) + d_in[:E]
        else:
            dh[l] += d_in[E:E + H]
            dh[r] += d_in[E + H:]
    touched = np.asarray(sorted(dEmb), dtype=np.int32)
    rows = np.stack([dEmb[int(t)] for t in touched]) if len(touched) else np.zeros((0, E))
    return dict(loss=loss, dW=dW, db=db, dWc=dWc, dbc=dbc, touched_ids=touched, dEmb_rows=rows,
                h=h, c=c)


def loss_only(left, right, token, emb, W, b, Wc, bc, labels) -> float:
    h, _, _ = forward_recursive(left, right, token, emb, W, b)
    return classifier_loss(h, Wc, bc, labels)[0]
