"""Pins for the CPU oracle: each test ties one part of oracle/treelstm_oracle.py to something
other than the oracle itself - exact values that follow from known function values, scalar
hand-unrolling, a library LSTM cell, closed forms, brute force, finite differences."""
import itertools
import math
import os

import numpy as np
import pytest
import torch

from oracle import treelstm_oracle as orc
from paper_1809_00832_b200 import forests as fg

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _params(rng, H, E, vocab=7, scale=0.5):
    emb = rng.uniform(-scale, scale, size=(vocab, E))
    W = rng.uniform(-scale, scale, size=(E + 2 * H, 5 * H))
    b = rng.uniform(-scale, scale, size=5 * H)
    return emb, W, b


def _chain(n_leaves, tokens):
    """left chain ((w0 w1) w2) ... in post-order ids: leaves and internals interleaved."""
    f = fg.forest_from_shapes([fg.left_chain_shape(n_leaves)], np.random.default_rng(0), 5)
    tok = f.token.copy()
    tok[f.left < 0] = np.asarray(tokens, dtype=np.int32)
    return f.left, f.right, tok


# --------------------------------------------------------------------------- #
# leaf cell: exact values from sigma(0)=1/2, sigma(ln 3)=3/4, tanh(atanh(1/2))=1/2
# --------------------------------------------------------------------------- #
def test_single_leaf_known_function_values():
    # H = E = 1, x = 1.  Choose W_x so that z_i = 0, z_o = ln 3, z_u = atanh(1/2).  The forget
    # columns get large arbitrary values: a leaf has no child state, they must not matter.
    golden = np.loadtxt(os.path.join(GOLDEN, "single_leaf.txt"))
    c_expected, h_expected = golden          # 0.25, 0.75 * tanh(0.25)
    for f_junk in (-3.0, 0.0, 11.0):
        W = np.zeros((3, 5))
        W[0] = [0.0, f_junk, -f_junk, math.log(3.0), math.atanh(0.5)]
        b = np.zeros(5)
        emb = np.array([[1.0]])
        left = np.array([-1], dtype=np.int32)
        token = np.array([0], dtype=np.int32)
        h, c, _ = orc.forward_recursive(left, left, token, emb, W, b)
        assert abs(c[0, 0] - c_expected) < 1e-15
        assert abs(h[0, 0] - h_expected) < 1e-15
    # same value reached through the bias instead of the weights
    W = np.zeros((3, 5))
    b = np.array([0.0, 5.0, -5.0, math.log(3.0), math.atanh(0.5)])
    h, c, _ = orc.forward_recursive(left, left, token, emb, W, b)
    assert abs(c[0, 0] - 0.25) < 1e-15 and abs(h[0, 0] - h_expected) < 1e-15


def test_single_leaf_closed_form_vector():
    rng = np.random.default_rng(1)
    H, E = 3, 4
    emb, W, b = _params(rng, H, E)
    left = np.array([-1], dtype=np.int32)
    token = np.array([2], dtype=np.int32)
    h, c, _ = orc.forward_recursive(left, left, token, emb, W, b)
    for j in range(H):
        z = [sum(W[k, g * H + j] * emb[2, k] for k in range(E)) + b[g * H + j] for g in range(5)]
        i = 1 / (1 + math.exp(-z[0]))
        o = 1 / (1 + math.exp(-z[3]))
        u = math.tanh(z[4])
        assert abs(c[0, j] - i * u) < 1e-14
        assert abs(h[0, j] - o * math.tanh(i * u)) < 1e-14


# --------------------------------------------------------------------------- #
# recurrence: left chain unrolled by hand with scalars (H = E = 1)
# --------------------------------------------------------------------------- #
def _sig(x):
    return 1.0 / (1.0 + math.exp(-x))


def test_left_chain_hand_unrolled_scalar():
    rng = np.random.default_rng(2)
    emb, W, b = _params(rng, 1, 1, vocab=5, scale=0.9)
    wx = W[0]           # x  -> (i, fl, fr, o, u)
    wl = W[1]           # h_l -> ...
    wr = W[2]           # h_r -> ...
    tokens = [3, 1, 4, 0]
    left, right, tok = _chain(4, tokens)

    def leaf(t):
        x = emb[t, 0]
        i = _sig(wx[0] * x + b[0]); o = _sig(wx[3] * x + b[3]); u = math.tanh(wx[4] * x + b[4])
        c = i * u
        return o * math.tanh(c), c

    def node(hl, cl, hr, cr):
        z = [wl[g] * hl + wr[g] * hr + b[g] for g in range(5)]
        c = _sig(z[0]) * math.tanh(z[4]) + _sig(z[1]) * cl + _sig(z[2]) * cr
        return _sig(z[3]) * math.tanh(c), c

    h0, c0 = leaf(3); h1, c1 = leaf(1); h2, c2 = leaf(4); h3, c3 = leaf(0)
    ha, ca = node(h0, c0, h1, c1)          # (w0 w1)
    hb, cb = node(ha, ca, h2, c2)          # ((w0 w1) w2)
    hc, cc = node(hb, cb, h3, c3)          # (((w0 w1) w2) w3)
    h, c, _ = orc.forward_recursive(left, right, tok, emb, W, b)
    root = int(orc.find_roots(left, right)[0])
    assert abs(h[root, 0] - hc) < 1e-14 and abs(c[root, 0] - cc) < 1e-14
    # the intermediate states too: post-order ids are l0 l1 a l2 b l3 c
    np.testing.assert_allclose(h[:, 0], [h0, h1, ha, h2, hb, h3, hc], atol=1e-14)
    np.testing.assert_allclose(c[:, 0], [c0, c1, ca, c2, cb, c3, cc], atol=1e-14)


# --------------------------------------------------------------------------- #
# library pin: with f_r forced to 0 a left chain is an ordinary LSTM whose input at step t is
# the t-th leaf's h and whose recurrent state is the left child's (h, c).
# --------------------------------------------------------------------------- #
def test_left_chain_reduces_to_library_lstm_cell():
    rng = np.random.default_rng(3)
    H, E, L = 3, 2, 5
    emb, W, b = _params(rng, H, E, vocab=6)
    b[2 * H:3 * H] = -1e4                    # sigma(-1e4 + small) == 0 exactly in fp64
    tokens = [1, 5, 0, 2, 2]
    left, right, tok = _chain(L, tokens)
    h, c, _ = orc.forward_recursive(left, right, tok, emb, W, b)

    def torch_cell(n_in, w_in, w_rec):
        # torch gate order is (i, f, g, o); ours is (i, f_l, f_r, o, u)
        pick = np.concatenate([np.arange(0, H), np.arange(H, 2 * H), np.arange(4 * H, 5 * H),
                               np.arange(3 * H, 4 * H)])
        cell = torch.nn.LSTMCell(n_in, H, bias=True, dtype=torch.float64)
        with torch.no_grad():
            cell.weight_ih.copy_(torch.from_numpy(w_in[:, pick].T.copy()))
            cell.weight_hh.copy_(torch.from_numpy(w_rec[:, pick].T.copy()))
            cell.bias_ih.copy_(torch.from_numpy(b[pick].copy()))
            cell.bias_hh.zero_()
        return cell

    leaf_cell = torch_cell(E, W[:E], W[E:E + H])
    node_cell = torch_cell(H, W[E + H:], W[E:E + H])      # input = h_r, recurrent = h_l
    zero = torch.zeros(1, H, dtype=torch.float64)
    with torch.no_grad():
        leaf_states = [leaf_cell(torch.from_numpy(emb[t])[None], (zero, zero)) for t in tokens]
        hs, cs = leaf_states[0]
        for t in range(1, L):
            hs, cs = node_cell(leaf_states[t][0], (hs, cs))
    root = int(orc.find_roots(left, right)[0])
    np.testing.assert_allclose(h[root], hs[0].numpy(), atol=1e-14)
    np.testing.assert_allclose(c[root], cs[0].numpy(), atol=1e-14)


# --------------------------------------------------------------------------- #
# degenerate closed forms
# --------------------------------------------------------------------------- #
def test_zero_recurrent_weights_closed_form_root_cell():
    # W_h = 0: every internal gate is a constant (sigma(b), tanh(b)), so the root cell state is
    # sum over internal nodes of i*u times the product of forget gates on the path to the root,
    # plus the same for leaves with their own c.
    rng = np.random.default_rng(4)
    H, E = 2, 3
    emb, W, b = _params(rng, H, E)
    W[E:] = 0.0
    forest = fg.forest_from_shapes([fg.random_split_shape(rng, 9)], rng, 7)
    h, c, _ = orc.forward_recursive(forest.left, forest.right, forest.token, emb, W, b)
    si, sfl, sfr = (1 / (1 + np.exp(-b[g * H:(g + 1) * H])) for g in range(3))
    tu = np.tanh(b[4 * H:])
    status, parent, _, _, _ = orc.schedule(forest.left, forest.right)
    root = int(forest.roots[0])
    expected = np.zeros(H)
    for n in range(forest.n_nodes):
        own = c[n] if forest.left[n] < 0 else si * tu
        weight = np.ones(H)
        k = n
        while parent[k] >= 0:
            p = parent[k]
            weight = weight * (sfl if forest.left[p] == k else sfr)
            k = p
        expected += own * weight
    np.testing.assert_allclose(c[root], expected, atol=1e-13)


def test_saturated_gates():
    rng = np.random.default_rng(5)
    H, E = 2, 2
    emb, W, b = _params(rng, H, E)
    forest = fg.forest_from_shapes([fg.random_split_shape(rng, 6)], rng, 7)
    # forget gates shut: c of an internal node is i*u only, independent of the children's c
    b1 = b.copy(); b1[H:3 * H] = -1e4
    h, c, g = orc.forward_recursive(forest.left, forest.right, forest.token, emb, W, b1)
    internal = forest.left >= 0
    np.testing.assert_allclose(c[internal], (g[:, 0] * g[:, 4])[internal], atol=0)
    # output gate shut: h = 0 everywhere
    b2 = b.copy(); b2[3 * H:4 * H] = -1e4
    h, c, _ = orc.forward_recursive(forest.left, forest.right, forest.token, emb, W, b2)
    assert np.all(h == 0.0)
    # forget gates open, input gate shut: the root cell is the plain sum of... nothing (leaves have c = i*u = 0)
    b3 = b.copy(); b3[0:H] = -1e4; b3[H:3 * H] = 1e4
    h, c, _ = orc.forward_recursive(forest.left, forest.right, forest.token, emb, W, b3)
    assert np.all(c == 0.0)


# --------------------------------------------------------------------------- #
# structure handling
# --------------------------------------------------------------------------- #
def test_duplicated_subtrees_have_identical_states():
    rng = np.random.default_rng(6)
    H, E = 4, 3
    emb, W, b = _params(rng, H, E)
    shape = fg.random_split_shape(rng, 7)
    one = fg.forest_from_shapes([shape], np.random.default_rng(9), 7)
    # a tree whose two halves are copies of `one`, plus `one` again as a separate tree
    left = np.concatenate([one.left, np.where(one.left >= 0, one.left + one.n_nodes, -1),
                           [one.roots[0]], np.where(one.left >= 0, one.left + 2 * one.n_nodes + 1, -1)])
    right = np.concatenate([one.right, np.where(one.right >= 0, one.right + one.n_nodes, -1),
                            [one.roots[0] + one.n_nodes],
                            np.where(one.right >= 0, one.right + 2 * one.n_nodes + 1, -1)])
    token = np.concatenate([one.token, one.token, [-1], one.token])
    left = left.astype(np.int32); right = right.astype(np.int32); token = token.astype(np.int32)
    h, c, _ = orc.forward_recursive(left, right, token, emb, W, b)
    n1 = one.n_nodes
    np.testing.assert_array_equal(h[:n1], h[n1:2 * n1])
    np.testing.assert_array_equal(c[:n1], c[n1:2 * n1])
    np.testing.assert_array_equal(h[:n1], h[2 * n1 + 1:])
    assert not np.allclose(h[2 * n1], h[one.roots[0]])      # the joint root is a new state


def test_child_swap_symmetry():
    rng = np.random.default_rng(7)
    H, E = 3, 2
    emb, W, b = _params(rng, H, E)
    Wl = W[E:E + H].copy()
    Wr = W[E + H:]
    # symmetric parameters: the i, o, u columns treat both children alike; the two forget gates
    # are mirror images of each other.
    for g in (0, 3, 4):
        Wr[:, g * H:(g + 1) * H] = Wl[:, g * H:(g + 1) * H]
    Wr[:, 2 * H:3 * H] = Wl[:, 1 * H:2 * H]         # h_r -> f_r  ==  h_l -> f_l
    Wr[:, 1 * H:2 * H] = Wl[:, 2 * H:3 * H]         # h_r -> f_l  ==  h_l -> f_r
    b[2 * H:3 * H] = b[1 * H:2 * H]
    forest = fg.forest_from_shapes([fg.random_split_shape(rng, 8)], rng, 7)
    h, c, _ = orc.forward_recursive(forest.left, forest.right, forest.token, emb, W, b)
    h2, c2, _ = orc.forward_recursive(forest.right, forest.left, forest.token, emb, W, b)
    np.testing.assert_allclose(h, h2, atol=1e-15)
    np.testing.assert_allclose(c, c2, atol=1e-15)
    # and with asymmetric parameters the swap does change the root
    W[E + H:, :H] += 0.3
    h3, _, _ = orc.forward_recursive(forest.left, forest.right, forest.token, emb, W, b)
    h4, _, _ = orc.forward_recursive(forest.right, forest.left, forest.token, emb, W, b)
    root = int(forest.roots[0])
    assert np.abs(h3[root] - h4[root]).max() > 1e-6


# --------------------------------------------------------------------------- #
# evaluation order: recursive == iterative, also on permuted ids
# --------------------------------------------------------------------------- #
@pytest.mark.parametrize("seed", [0, 1, 2])
def test_recursive_equals_iterative(seed):
    rng = np.random.default_rng(seed)
    H, E = 5, 4
    emb, W, b = _params(rng, H, E, vocab=11)
    forest = fg.random_forest(rng, 6, 1, 9, 11)
    status, parent, level, order, off = orc.schedule(forest.left, forest.right)
    assert status == orc.OK
    hr, cr, _ = orc.forward_recursive(forest.left, forest.right, forest.token, emb, W, b)
    hi, ci, _ = orc.forward_iterative(forest.left, forest.right, forest.token, emb, W, b, order)
    np.testing.assert_array_equal(hr, hi)
    np.testing.assert_array_equal(cr, ci)
    # any other dependency-respecting order gives the same states
    hi2, _, _ = orc.forward_iterative(forest.left, forest.right, forest.token, emb, W, b,
                                      np.arange(forest.n_nodes))       # post-order ids
    np.testing.assert_array_equal(hr, hi2)
    perm, new_of_old = fg.permute_node_ids(forest, rng)
    hp, cp, _ = orc.forward_recursive(perm.left, perm.right, perm.token, emb, W, b)
    np.testing.assert_array_equal(hp[new_of_old], hr)
    s2, _, level_p, order_p, off_p = orc.schedule(perm.left, perm.right)
    np.testing.assert_array_equal(level_p[new_of_old], level)
    np.testing.assert_array_equal(off_p, off)


# --------------------------------------------------------------------------- #
# schedule
# --------------------------------------------------------------------------- #
def _brute_height(left, right, n):
    """longest downward path from n to a leaf, by enumerating all paths."""
    best = 0
    stack = [(n, 0)]
    while stack:
        k, d = stack.pop()
        if left[k] < 0:
            best = max(best, d)
        else:
            stack.append((int(left[k]), d + 1))
            stack.append((int(right[k]), d + 1))
    return best


def test_levels_are_brute_force_heights_and_order_is_canonical():
    rng = np.random.default_rng(8)
    forest = fg.random_forest(rng, 7, 1, 12, 5)
    forest, _ = fg.permute_node_ids(forest, rng)
    status, parent, level, order, off = orc.schedule(forest.left, forest.right)
    assert status == orc.OK
    n = forest.n_nodes
    for k in range(n):
        assert level[k] == _brute_height(forest.left, forest.right, k)
    keys = [(int(level[k]), k) for k in range(n)]
    assert [int(x) for x in order] == [k for _, k in sorted(keys)]
    assert off[0] == 0 and off[-1] == n
    for l in range(len(off) - 1):
        assert np.all(level[order[off[l]:off[l + 1]]] == l)
    for k in range(n):
        if forest.left[k] >= 0:
            assert parent[forest.left[k]] == k and parent[forest.right[k]] == k
    assert sorted(np.nonzero(parent < 0)[0].tolist()) == sorted(forest.roots.tolist())


def test_level_widths_closed_form():
    # Section 6.3: a full binary tree of N cells has (N+1)/2 independent leaves and log depth; a
    # linear tree allows one node at a time above the leaves.
    rng = np.random.default_rng(0)
    bal = fg.forest_from_shapes([fg.balanced_shape(64)] * 3, rng, 5)
    _, _, level, order, off = orc.schedule(bal.left, bal.right)
    assert np.diff(off).tolist() == [3 * 64 // (1 << k) for k in range(7)]
    ch = fg.forest_from_shapes([fg.left_chain_shape(10)] * 4, rng, 5)
    _, _, level, order, off = orc.schedule(ch.left, ch.right)
    assert np.diff(off).tolist() == [40] + [4] * 9


def test_schedule_rejects_malformed_forests():
    ok_left = np.array([-1, -1, 0], dtype=np.int32)
    ok_right = np.array([-1, -1, 1], dtype=np.int32)
    assert orc.schedule(ok_left, ok_right)[0] == orc.OK

    def status(l, r, tok=None, vocab=None):
        return orc.schedule(np.array(l, dtype=np.int32), np.array(r, dtype=np.int32),
                            None if tok is None else np.array(tok, dtype=np.int32), vocab)[0]

    assert status([-1, -1, 0], [-1, -1, 3]) == orc.ERR_INVALID_FOREST      # child out of range
    assert status([-1, -1, 0], [-1, -1, -1]) == orc.ERR_INVALID_FOREST     # one child only
    assert status([-1, -1, 0, 0], [-1, -1, 1, 1]) == orc.ERR_INVALID_FOREST  # two parents
    assert status([-1, -1, 0], [-1, -1, 0]) == orc.ERR_INVALID_FOREST      # same child twice
    assert status([-1, -1, 2], [-1, -1, 1]) == orc.ERR_INVALID_FOREST      # own child
    assert status([-1, 2, 1, -1], [-1, 0, 3, -1]) == orc.ERR_INVALID_FOREST  # 1 <-> 2 cycle
    assert status([-1, -1, 0], [-1, -1, 1], [5, 1, -1], 5) == orc.ERR_TOKEN_OUT_OF_RANGE
    assert status([-1, -1, 0], [-1, -1, 1], [4, 1, -1], 5) == orc.OK
    assert status([], []) == orc.OK


# --------------------------------------------------------------------------- #
# invariants
# --------------------------------------------------------------------------- #
def test_state_bounds():
    rng = np.random.default_rng(10)
    H, E = 6, 5
    emb, W, b = _params(rng, H, E, scale=2.0)
    forest = fg.random_forest(rng, 5, 1, 15, 7)
    h, c, _ = orc.forward_recursive(forest.left, forest.right, forest.token, emb, W, b)
    assert np.all(np.abs(h) < 1.0)
    size = np.ones(forest.n_nodes)
    for k in range(forest.n_nodes):        # post-order ids: children first
        if forest.left[k] >= 0:
            size[k] = 1 + size[forest.left[k]] + size[forest.right[k]]
    assert np.all(np.abs(c) < size[:, None])


def test_bf16_rounding_helper():
    # 1 + 2^-8 is a tie between 1 and 1 + 2^-7: ties to even gives 1; 1 + 3*2^-8 ties up to 1+2^-6
    vals = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -7, -0.1, 3.0e38])
    got = orc.round_to_bf16(vals)
    assert got[0] == 1.0 and got[1] == 1.0 and got[2] == 1.0 + 2.0 ** -6 and got[3] == 1.0 + 2.0 ** -7
    ref = torch.tensor(vals, dtype=torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    np.testing.assert_array_equal(got, ref)
    x = np.random.default_rng(0).normal(size=1000)
    ref = torch.tensor(x, dtype=torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    np.testing.assert_array_equal(orc.round_to_bf16(x), ref)


# --------------------------------------------------------------------------- #
# loss and backward
# --------------------------------------------------------------------------- #
def test_uniform_logits_loss_is_log_classes():
    h = np.random.default_rng(0).normal(size=(9, 4))
    loss, probs = orc.classifier_loss(h, np.zeros((4, 5)), np.full(5, 0.7), np.arange(9) % 5)
    assert abs(loss - math.log(5.0)) < 1e-15
    np.testing.assert_allclose(probs, 0.2, atol=1e-15)
    # one-hot certain prediction: loss -> 0 ; wrong certain prediction: loss -> margin
    Wc = np.zeros((4, 2)); bc = np.array([50.0, 0.0])
    assert orc.classifier_loss(h, Wc, bc, np.zeros(9, dtype=int))[0] < 1e-20
    assert abs(orc.classifier_loss(h, Wc, bc, np.ones(9, dtype=int))[0] - 50.0) < 1e-12


def _train_case(seed, H=3, E=2, C=4, vocab=6):
    rng = np.random.default_rng(seed)
    emb, W, b = _params(rng, H, E, vocab=vocab)
    Wc = rng.uniform(-0.5, 0.5, size=(H, C))
    bc = rng.uniform(-0.5, 0.5, size=C)
    forest = fg.random_forest(rng, 3, 1, 6, vocab)
    forest, _ = fg.permute_node_ids(forest, rng)
    labels = rng.integers(0, C, size=forest.n_nodes)
    return forest, emb, W, b, Wc, bc, labels


@pytest.mark.parametrize("seed", [0, 1])
def test_gradients_match_central_finite_differences(seed):
    forest, emb, W, b, Wc, bc, labels = _train_case(seed)
    args = (forest.left, forest.right, forest.token)
    out = orc.loss_and_gradients(*args, emb, W, b, Wc, bc, labels)
    eps = 1e-6

    def fd(arr, idx, fn):
        old = arr[idx]
        arr[idx] = old + eps; up = fn()
        arr[idx] = old - eps; dn = fn()
        arr[idx] = old
        return (up - dn) / (2 * eps)

    f = lambda: orc.loss_only(*args, emb, W, b, Wc, bc, labels)
    assert abs(out["loss"] - f()) < 1e-15
    for name, arr, grad in (("W", W, out["dW"]), ("b", b, out["db"]), ("Wc", Wc, out["dWc"]),
                            ("bc", bc, out["dbc"])):
        for idx in np.ndindex(arr.shape):
            g = fd(arr, idx, f)
            assert abs(g - grad[idx]) < 1e-8 + 1e-6 * abs(g), (name, idx, g, grad[idx])
    # embedding rows: touched ones match FD, untouched ones have zero FD gradient and are absent
    touched = out["touched_ids"].tolist()
    assert touched == sorted(set(forest.token[forest.left < 0].tolist()))
    for t in range(emb.shape[0]):
        for k in range(emb.shape[1]):
            g = fd(emb, (t, k), f)
            if t in touched:
                got = out["dEmb_rows"][touched.index(t), k]
                assert abs(g - got) < 1e-8 + 1e-6 * abs(g)
            else:
                assert g == 0.0


def test_gradient_structure():
    forest, emb, W, b, Wc, bc, labels = _train_case(3, H=3, E=2)
    E, H = 2, 3
    # a forest of leaves only: no gradient reaches the recurrent rows or the forget columns
    leaves = fg.forest_from_shapes([None, None, None], np.random.default_rng(0), 6)
    out = orc.loss_and_gradients(leaves.left, leaves.right, leaves.token, emb, W, b, Wc, bc,
                                 labels[:3])
    assert np.all(out["dW"][E:] == 0.0)
    assert np.all(out["dW"][:, H:3 * H] == 0.0) and np.all(out["db"][H:3 * H] == 0.0)
    assert np.any(out["dW"][:E] != 0.0)
    # classifier bias gradient sums to zero (softmax minus one-hot)
    assert abs(out["dbc"].sum()) < 1e-15
    # duplicate tokens accumulate into one row
    dup = fg.forest_from_shapes([fg.left_chain_shape(3)], np.random.default_rng(0), 6)
    tok = dup.token.copy(); tok[dup.left < 0] = 4
    out = orc.loss_and_gradients(dup.left, dup.right, tok, emb, W, b, Wc, bc, labels[:5])
    assert out["touched_ids"].tolist() == [4] and out["dEmb_rows"].shape == (1, E)


def test_backward_matches_torch_autograd():
    # an independent differentiation mechanism: the same forest written as torch ops, gradients
    # from reverse-mode autograd instead of the hand-derived recursion.
    forest, emb, W, b, Wc, bc, labels = _train_case(5, H=4, E=3, C=5, vocab=8)
    out = orc.loss_and_gradients(forest.left, forest.right, forest.token, emb, W, b, Wc, bc, labels)
    H, E = 4, 3
    t = {k: torch.tensor(v, dtype=torch.float64, requires_grad=True)
         for k, v in dict(emb=emb, W=W, b=b, Wc=Wc, bc=bc).items()}
    _, _, level, order, _ = orc.schedule(forest.left, forest.right)
    hs, cs = {}, {}
    zero = torch.zeros(H, dtype=torch.float64)
    for n in order.tolist():
        if forest.left[n] < 0:
            inp = torch.cat([t["emb"][int(forest.token[n])], zero, zero]); cl = cr = zero
        else:
            l, r = int(forest.left[n]), int(forest.right[n])
            inp = torch.cat([torch.zeros(E, dtype=torch.float64), hs[l], hs[r]]); cl, cr = cs[l], cs[r]
        z = inp @ t["W"] + t["b"]
        zi, zfl, zfr, zo, zu = z.split(H)
        cs[n] = torch.sigmoid(zi) * torch.tanh(zu) + torch.sigmoid(zfl) * cl + torch.sigmoid(zfr) * cr
        hs[n] = torch.sigmoid(zo) * torch.tanh(cs[n])
    hmat = torch.stack([hs[n] for n in range(forest.n_nodes)])
    loss = torch.nn.functional.cross_entropy(hmat @ t["Wc"] + t["bc"], torch.tensor(labels))
    loss.backward()
    assert abs(loss.item() - out["loss"]) < 1e-14
    np.testing.assert_allclose(out["dW"], t["W"].grad.numpy(), atol=1e-14)
    np.testing.assert_allclose(out["db"], t["b"].grad.numpy(), atol=1e-14)
    np.testing.assert_allclose(out["dWc"], t["Wc"].grad.numpy(), atol=1e-14)
    np.testing.assert_allclose(out["dbc"], t["bc"].grad.numpy(), atol=1e-14)
    np.testing.assert_allclose(out["dEmb_rows"], t["emb"].grad.numpy()[out["touched_ids"]], atol=1e-14)
