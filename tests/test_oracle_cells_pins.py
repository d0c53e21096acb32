"""Pins for oracle/recursive_cells_oracle.py (TreeRNN and RNTN, the paper's other two evaluation
models, Section 6.1): exact values from tanh(atanh 1/2), scalar hand-unrolling, torch.nn.RNNCell on
a left chain, torch.nn.Bilinear and an explicit triple loop for the tensor term, reductions of RNTN
to TreeRNN, symmetries, recursive == iterative, finite differences and torch autograd."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import recursive_cells_oracle as rc
from oracle import treelstm_oracle as orc
from paper_1809_00832_b200 import forests as fg

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
KINDS = (rc.TREERNN, rc.RNTN)


def _params(rng, H, vocab=7, scale=0.6, kind=rc.RNTN):
    emb = rng.uniform(-scale, scale, size=(vocab, H))
    W = rng.uniform(-scale, scale, size=(2 * H, H))
    b = rng.uniform(-scale, scale, size=H)
    V = rng.uniform(-scale, scale, size=(H, 2 * H, 2 * H)) if kind == rc.RNTN else None
    return emb, W, b, V


def _pair(tokens=(0, 1)):
    """two leaves (ids 0, 1) and their parent (id 2)"""
    left = np.array([-1, -1, 0], dtype=np.int32)
    right = np.array([-1, -1, 1], dtype=np.int32)
    token = np.array([tokens[0], tokens[1], -1], dtype=np.int32)
    return left, right, token


# --------------------------------------------------------------------------- #
# exact values: tanh(atanh(1/2)) = 1/2
# --------------------------------------------------------------------------- #
def test_pair_known_function_values():
    golden = np.loadtxt(os.path.join(GOLDEN, "recursive_cells_pair.txt"))
    left, right, token = _pair()
    emb = np.array([[1.0], [2.0]])                      # H = 1: leaf states 1 and 2
    a = math.atanh(0.5)
    # TreeRNN: z = w_l * 1 + w_r * 2 + b = atanh(1/2)
    W = np.array([[a], [-a]])
    b = np.array([2 * a])
    h = rc.forward_recursive(rc.TREERNN, left, right, token, emb, W, b)
    np.testing.assert_array_equal(h[:2, 0], [1.0, 2.0])  # a leaf's state is its word vector
    assert abs(h[2, 0] - golden[0]) < 1e-15 and golden[0] == 0.5
    # RNTN: x = (1, 2); x^T V x = v00 + 2 (v01 + v10) + 4 v11; linear part and bias zero
    V = np.array([[[a, 0.25], [-0.25, 0.0]]])           # a + 2 * 0 + 0 = atanh(1/2)
    h = rc.forward_recursive(rc.RNTN, left, right, token, emb, np.zeros((2, 1)), np.zeros(1), V)
    assert abs(h[2, 0] - golden[1]) < 1e-15 and golden[1] == 0.5
    # all three terms at once: 3 * atanh(1/2) = atanh(13/14)  (tanh addition theorem)
    V = np.array([[[0.0, 0.0], [0.0, a / 4]]])          # 4 * a / 4
    h = rc.forward_recursive(rc.RNTN, left, right, token, emb, np.array([[a], [0.0]]), np.array([a]), V)
    assert abs(h[2, 0] - golden[2]) < 1e-15 and abs(golden[2] - 13.0 / 14.0) < 1e-16


def test_scalar_hand_unrolled_chain():
    """H = 1, left chain of four leaves, every step written out in scalars"""
    rng = np.random.default_rng(3)
    f = fg.forest_from_shapes([fg.left_chain_shape(4)], rng, 4)
    token = f.token.copy()
    token[f.left < 0] = [0, 1, 2, 3]
    e = np.array([0.3, -0.7, 0.5, 0.9])
    wl, wr, bias = 0.8, -0.4, 0.1
    v = np.array([[0.2, -0.3], [0.5, 0.7]])
    emb = e[:, None]
    W = np.array([[wl], [wr]])
    b = np.array([bias])
    for kind in KINDS:
        def step(l, r):
            z = wl * l + wr * r + bias
            if kind == rc.RNTN:
                z += v[0, 0] * l * l + (v[0, 1] + v[1, 0]) * l * r + v[1, 1] * r * r
            return math.tanh(z)
        p1 = step(e[0], e[1])
        p2 = step(p1, e[2])
        p3 = step(p2, e[3])
        h = rc.forward_recursive(kind, f.left, f.right, token, emb, W, b, v[None] if kind == rc.RNTN else None)
        internal = np.nonzero(f.left >= 0)[0]            # post-order: the three internal nodes in chain order
        np.testing.assert_allclose(h[internal, 0], [p1, p2, p3], rtol=0, atol=1e-15)


# --------------------------------------------------------------------------- #
# library routines
# --------------------------------------------------------------------------- #
def test_left_chain_is_a_library_rnn_cell():
    """on a left chain the right child is always a word vector: the TreeRNN recurrence is an
    ordinary Elman cell with input = that word vector and hidden = the left state"""
    rng = np.random.default_rng(5)
    H, L = 5, 9
    emb, W, b, _ = _params(rng, H, vocab=11, kind=rc.TREERNN)
    f = fg.forest_from_shapes([fg.left_chain_shape(L)], rng, 11)
    h = rc.forward_recursive(rc.TREERNN, f.left, f.right, f.token, emb, W, b)
    cell = torch.nn.RNNCell(H, H, bias=True, nonlinearity="tanh").double()
    with torch.no_grad():
        cell.weight_hh.copy_(torch.from_numpy(W[:H].T))   # left state
        cell.weight_ih.copy_(torch.from_numpy(W[H:].T))   # right child = input
        cell.bias_ih.copy_(torch.from_numpy(b))
        cell.bias_hh.zero_()
        leaves = np.nonzero(f.left < 0)[0]
        state = torch.from_numpy(emb[f.token[leaves[0]]])[None]
        internal = np.nonzero(f.left >= 0)[0]
        for step, node in enumerate(internal):
            x = torch.from_numpy(emb[f.token[leaves[step + 1]]])[None]
            state = cell(x, state)
            assert np.max(np.abs(state[0].numpy() - h[node])) < 1e-14


def test_tensor_term_is_a_library_bilinear_form_and_a_triple_loop():
    rng = np.random.default_rng(6)
    H = 4
    emb, W, b, V = _params(rng, H)
    h_l, h_r = rng.uniform(-1, 1, H), rng.uniform(-1, 1, H)
    got = rc.cell(rc.RNTN, W, b, V, h_l, h_r)
    x = np.concatenate([h_l, h_r])
    # (i) torch.nn.Bilinear: y_j = x1^T A_j x2 + bias_j
    bil = torch.nn.Bilinear(2 * H, 2 * H, H, bias=True).double()
    with torch.no_grad():
        bil.weight.copy_(torch.from_numpy(V))
        bil.bias.copy_(torch.from_numpy(b))
        xt = torch.from_numpy(x)[None]
        z = bil(xt, xt)[0].numpy() + W.T @ x
    assert np.max(np.abs(np.tanh(z) - got)) < 1e-14
    # (ii) every product written out
    z2 = np.zeros(H)
    for j in range(H):
        acc = b[j]
        for a_ in range(2 * H):
            acc += W[a_, j] * x[a_]
            for b_ in range(2 * H):
                acc += x[a_] * V[j, a_, b_] * x[b_]
        z2[j] = acc
    assert np.max(np.abs(np.tanh(z2) - got)) < 1e-14


# --------------------------------------------------------------------------- #
# reductions and symmetries
# --------------------------------------------------------------------------- #
def test_rntn_reduces_to_treernn():
    rng = np.random.default_rng(7)
    H = 6
    emb, W, b, V = _params(rng, H, vocab=20)
    forest = fg.random_forest(rng, 5, 1, 12, 20)
    base = rc.forward_recursive(rc.TREERNN, forest.left, forest.right, forest.token, emb, W, b)
    zero = rc.forward_recursive(rc.RNTN, forest.left, forest.right, forest.token, emb, W, b, np.zeros_like(V))
    np.testing.assert_array_equal(zero, base)
    anti = V - np.transpose(V, (0, 2, 1))               # x^T A x = 0 for antisymmetric A
    same = rc.forward_recursive(rc.RNTN, forest.left, forest.right, forest.token, emb, W, b, anti)
    assert np.max(np.abs(same - base)) < 1e-14
    sym = 0.5 * (V + np.transpose(V, (0, 2, 1)))        # only the symmetric part of a slice matters
    full = rc.forward_recursive(rc.RNTN, forest.left, forest.right, forest.token, emb, W, b, V)
    half = rc.forward_recursive(rc.RNTN, forest.left, forest.right, forest.token, emb, W, b, sym)
    assert np.max(np.abs(full - half)) < 1e-14
    assert np.max(np.abs(full - base)) > 1e-3            # and the tensor term does something


@pytest.mark.parametrize("kind", KINDS)
def test_child_swap_symmetry_and_duplicated_subtrees(kind):
    rng = np.random.default_rng(8)
    H = 4
    emb, W, b, V = _params(rng, H, kind=kind)
    shape = fg.random_split_shape(rng, 6)
    forest = fg.forest_from_shapes([shape, shape], rng, 7)
    n1 = forest.n_nodes // 2
    token = forest.token.copy()
    token[n1:] = token[:n1]                               # second tree = copy of the first
    h = rc.forward_recursive(kind, forest.left, forest.right, token, emb, W, b, V)
    np.testing.assert_array_equal(h[:n1], h[n1:])
    # swapping the children of every node changes nothing when the parameters treat both sides alike
    Ws = np.concatenate([W[:H], W[:H]])
    Vs = None
    if V is not None:
        # x = [l ; r]: the diagonal blocks equal, the off-diagonal blocks one symmetric matrix
        blk = V[:, :H, :H]
        off = 0.5 * (V[:, :H, H:] + np.transpose(V[:, :H, H:], (0, 2, 1)))
        Vs = np.zeros_like(V)
        Vs[:, :H, :H] = blk
        Vs[:, H:, H:] = blk
        Vs[:, :H, H:] = off
        Vs[:, H:, :H] = off
    internal = forest.left >= 0
    sl, sr = forest.left.copy(), forest.right.copy()
    sl[internal], sr[internal] = forest.right[internal], forest.left[internal]
    a = rc.forward_recursive(kind, forest.left, forest.right, token, emb, Ws, b, Vs)
    bb = rc.forward_recursive(kind, sl, sr, token, emb, Ws, b, Vs)
    assert np.max(np.abs(a - bb)) < 1e-14
    c = rc.forward_recursive(kind, sl, sr, token, emb, W, b, V)     # negative control: asymmetric parameters
    assert np.max(np.abs(c - h)) > 1e-3


@pytest.mark.parametrize("kind", KINDS)
def test_recursive_equals_iterative_on_permuted_ids(kind):
    rng = np.random.default_rng(9)
    H = 5
    emb, W, b, V = _params(rng, H, vocab=30, kind=kind)
    forest = fg.random_forest(rng, 6, 1, 15, 30)
    perm, new_of_old = fg.permute_node_ids(forest, rng)
    h0 = rc.forward_recursive(kind, forest.left, forest.right, forest.token, emb, W, b, V)
    h1 = rc.forward_recursive(kind, perm.left, perm.right, perm.token, emb, W, b, V)
    np.testing.assert_array_equal(h1[new_of_old], h0)
    status, _, level, order, _ = orc.schedule(perm.left, perm.right)
    assert status == orc.OK
    h2 = rc.forward_iterative(kind, perm.left, perm.right, perm.token, emb, W, b, order, V)
    np.testing.assert_array_equal(h2, h1)
    assert np.all(np.abs(h1[perm.left >= 0]) < 1.0)


# --------------------------------------------------------------------------- #
# loss and gradients
# --------------------------------------------------------------------------- #
def test_uniform_logits_loss_is_log_classes():
    h = np.random.default_rng(0).uniform(-1, 1, size=(9, 3))
    loss, probs = rc.classifier_loss(h, np.zeros((3, 4)), np.zeros(4), np.arange(9) % 4)
    assert abs(loss - math.log(4.0)) < 1e-15
    assert np.max(np.abs(probs - 0.25)) < 1e-15


def _train_problem(kind, seed):
    rng = np.random.default_rng(seed)
    H, C, vocab = 3, 4, 6
    emb, W, b, V = _params(rng, H, vocab=vocab, kind=kind)
    Wc = rng.uniform(-0.6, 0.6, size=(H, C))
    bc = rng.uniform(-0.6, 0.6, size=C)
    forest = fg.random_forest(rng, 3, 1, 7, vocab)       # small vocabulary: tokens repeat
    forest, _ = fg.permute_node_ids(forest, rng)
    labels = rng.integers(0, C, size=forest.n_nodes).astype(np.int32)
    return forest, emb, W, b, V, Wc, bc, labels


@pytest.mark.parametrize("kind", KINDS)
@pytest.mark.parametrize("seed", [0, 1])
def test_gradients_match_central_finite_differences(kind, seed):
    forest, emb, W, b, V, Wc, bc, labels = _train_problem(kind, seed)
    g = rc.loss_and_gradients(kind, forest.left, forest.right, forest.token, emb, W, b, Wc, bc, labels, V)
    groups = {"W": (W, g["dW"]), "b": (b, g["db"]), "Wc": (Wc, g["dWc"]), "bc": (bc, g["dbc"])}
    if kind == rc.RNTN:
        groups["V"] = (V, g["dV"])
    dEmb = np.zeros_like(emb)
    dEmb[g["touched_ids"]] = g["dEmb_rows"]
    groups["emb"] = (emb, dEmb)
    eps = 1e-6
    for name, (arr, grad) in groups.items():
        flat = arr.reshape(-1)
        for i in range(flat.shape[0]):
            keep = flat[i]
            flat[i] = keep + eps
            up = rc.loss_only(kind, forest.left, forest.right, forest.token, emb, W, b, Wc, bc, labels, V)
            flat[i] = keep - eps
            dn = rc.loss_only(kind, forest.left, forest.right, forest.token, emb, W, b, Wc, bc, labels, V)
            flat[i] = keep
            fd = (up - dn) / (2 * eps)
            assert abs(fd - grad.reshape(-1)[i]) < 1e-8 + 1e-6 * abs(fd), (name, i)
    used = set(int(t) for t in forest.token[forest.left < 0])
    assert list(g["touched_ids"]) == sorted(used)


@pytest.mark.parametrize("kind", KINDS)
def test_backward_matches_torch_autograd(kind):
    forest, emb, W, b, V, Wc, bc, labels = _train_problem(kind, 5)
    g = rc.loss_and_gradients(kind, forest.left, forest.right, forest.token, emb, W, b, Wc, bc, labels, V)
    t = lambda a: torch.tensor(a, dtype=torch.float64, requires_grad=True)
    emb_t, W_t, b_t, Wc_t, bc_t = t(emb), t(W), t(b), t(Wc), t(bc)
    V_t = t(V) if V is not None else None
    status, _, _, order, _ = orc.schedule(forest.left, forest.right)
    states = [None] * forest.n_nodes
    for idx in order:
        idx = int(idx)
        if forest.left[idx] < 0:
            states[idx] = emb_t[int(forest.token[idx])]
        else:
            x = torch.cat([states[int(forest.left[idx])], states[int(forest.right[idx])]])
            z = W_t.T @ x + b_t
            if V_t is not None:
                z = z + torch.einsum("a,jab,b->j", x, V_t, x)
            states[idx] = torch.tanh(z)
    logits = torch.stack(states) @ Wc_t + bc_t
    loss = torch.nn.functional.cross_entropy(logits, torch.from_numpy(labels.astype(np.int64)))
    loss.backward()
    assert abs(loss.item() - g["loss"]) < 1e-14
    assert np.max(np.abs(W_t.grad.numpy() - g["dW"])) < 1e-14
    assert np.max(np.abs(b_t.grad.numpy() - g["db"])) < 1e-14
    assert np.max(np.abs(Wc_t.grad.numpy() - g["dWc"])) < 1e-14
    assert np.max(np.abs(bc_t.grad.numpy() - g["dbc"])) < 1e-14
    if V_t is not None:
        assert np.max(np.abs(V_t.grad.numpy() - g["dV"])) < 1e-14
    dEmb = np.zeros_like(emb)
    dEmb[g["touched_ids"]] = g["dEmb_rows"]
    assert np.max(np.abs(emb_t.grad.numpy() - dEmb)) < 1e-14
