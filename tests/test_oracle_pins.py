"""Pins for the CPU oracle: closed forms, brute force, invariants, library
routines and finite differences.  None of these needs a GPU."""
import itertools
import math
import os

import numpy as np
import pytest
import torch
from scipy.special import softmax as scipy_softmax

from oracle import ec_oracle as O
from oracle.ref_einsum import layer_onehot
from paper_2202_09368_b200 import inputs as IN

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def mk(n, d, dff, E, seed=0, scale=1.0):
    li = IN.make_layer_inputs(n, d, dff, E, torch.float32, seed, scale)
    return [t.numpy().astype(np.float64) for t in (li.X, li.Wg, li.W1, li.W2, li.dX_out)]


# ---------------------------------------------------------------- Eq. 1
def test_capacity_eq1():
    assert O.capacity(256, 2, 4) == 128
    assert O.capacity(8192, 2, 32) == 512
    assert O.capacity(8192, 0.5, 64) == 64
    assert O.capacity(16384, 2, 64) == 512
    assert O.capacity(10, 1, 3) == 3          # floor
    assert O.capacity(8, 8, 8) == 8           # c = e: every expert takes every token
    with pytest.raises(ValueError):
        O.capacity(4, 0.1, 8)
    with pytest.raises(ValueError):
        O.capacity(4, 3, 2)


# ---------------------------------------------------------------- Eq. 2, worked example
def test_worked_example_closed_form():
    rows, rec = [], {}
    for line in open(os.path.join(GOLD, "softmax_topk_worked.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        p = line.split()
        if p[0][0].isalpha():
            rec[p[0]] = [float(v) for v in p[1:]]
        else:
            rows.append([float(v) for v in p])
    rows = np.array(rows)
    logits = np.log(rows[:, 1:3])
    # d = 2 with X = logits and Wg = identity gives exactly these logits
    r = O.route(logits, np.eye(2), c=1.0)
    assert r["k"] == 2
    np.testing.assert_allclose(r["S"], rows[:, 3:5], rtol=0, atol=1e-15)
    assert r["I"].tolist() == [[int(v) for v in rec["I0"]], [int(v) for v in rec["I1"]]]
    np.testing.assert_allclose(r["G"], [rec["G0"], rec["G1"]], atol=1e-15)
    assert r["row_ptr"].tolist() == [int(v) for v in rec["ROWPTR"]]
    assert r["slots"].tolist() == [int(v) for v in rec["SLOTS"]]


def test_gate_matches_library_softmax_and_is_distribution():
    X, Wg, *_ = mk(256, 64, 256, 4)
    S = O.gate(X, Wg)
    np.testing.assert_allclose(S, scipy_softmax(X @ Wg, axis=1), rtol=1e-13)
    np.testing.assert_allclose(S.sum(axis=1), 1.0, atol=1e-12)
    assert (S > 0).all() and (S <= 1).all()
    # softmax must run over experts, not tokens: column sums are not 1
    assert not np.allclose(S.sum(axis=0), 1.0)
    # shift invariance per token row
    np.testing.assert_allclose(O.gate(X, Wg), O.gate(np.hstack([X, np.ones((256, 1))]),
                                                     np.vstack([Wg, 3.0 * np.ones((1, 4))])), atol=1e-13)


# ---------------------------------------------------------------- TopK
def brute_topk(S, k):
    n, e = S.shape
    I = [[t for _, t in sorted((-S[t, i], t) for t in range(n))[:k]] for i in range(e)]
    return np.array(I)


@pytest.mark.parametrize("n,e,k,levels", [(16, 2, 4, 0), (33, 3, 7, 0), (40, 4, 10, 3), (12, 1, 12, 2), (9, 2, 1, 1)])
def test_topk_equals_bruteforce_sort(n, e, k, levels):
    rng = np.random.default_rng(n * 31 + e)
    S = rng.random((n, e))
    if levels:
        S = np.round(S * levels) / levels + 0.125      # heavy ties
    G, I = O.topk(S, k)
    assert np.array_equal(I, brute_topk(S, k))
    for i in range(e):
        assert np.array_equal(G[i], S[I[i], i])         # G is S at the chosen pairs, bit for bit
        sel = set(I[i].tolist())
        assert len(sel) == k                            # k distinct tokens
        rest = [t for t in range(n) if t not in sel]
        thr = G[i].min()
        if rest:
            assert thr >= max(S[t, i] for t in rest)    # threshold invariant
            # among scores equal to the threshold, the chosen tokens are the lowest ids
            eq_sel = [t for t in sel if S[t, i] == thr]
            eq_rest = [t for t in rest if S[t, i] == thr]
            if eq_rest:
                assert max(eq_sel) < min(eq_rest)
        # listed by descending score, equal scores by ascending token
        keys = [(-S[t, i], t) for t in I[i]]
        assert keys == sorted(keys)


def test_topk_all_equal_column_takes_lowest_tokens():
    S = np.full((10, 3), 1.0 / 3)
    G, I = O.topk(S, 4)
    assert I.tolist() == [[0, 1, 2, 3]] * 3


def test_load_balance_and_capacity_factor():
    X, Wg, *_ = mk(256, 64, 256, 4)
    for c in (0.5, 1, 2):
        r = O.route(X, Wg, c)
        k = r["k"]
        assert k == int(256 * c / 4)
        for i in range(4):
            assert len(set(r["I"][i].tolist())) == k and r["I"][i].min() >= 0 and r["I"][i].max() < 256
        cnt = O.experts_per_token(r["row_ptr"])
        assert cnt.sum() == 256 * c                     # c = average experts per token
        assert r["row_ptr"][-1] == 4 * k


def test_inverse_index_lists_exactly_the_slots_of_each_token():
    X, Wg, *_ = mk(64, 16, 32, 8)
    r = O.route(X, Wg, 2.0)
    I, k = r["I"], r["k"]
    for t in range(64):
        want = [i * k + j for i in range(8) for j in range(k) if I[i, j] == t]
        got = r["slots"][r["row_ptr"][t]:r["row_ptr"][t + 1]].tolist()
        assert got == want                              # ascending expert


# ---------------------------------------------------------------- GeLU
def test_gelu_against_math_erf_and_derivative():
    z = np.linspace(-6, 6, 241)
    ref = np.array([0.5 * v * (1 + math.erf(v / math.sqrt(2))) for v in z])
    np.testing.assert_allclose(O.gelu(z), ref, rtol=1e-14, atol=1e-16)
    assert O.gelu(0.0) == 0 and abs(O.gelu(10.0) - 10) < 1e-12 and abs(O.gelu(-10.0)) < 1e-12
    h = 1e-6
    for v in ("erf", "tanh"):
        fd = (O.gelu(z + h, v) - O.gelu(z - h, v)) / (2 * h)
        np.testing.assert_allclose(O.gelu_grad(z, v), fd, atol=1e-8)
    assert np.max(np.abs(O.gelu(z, "tanh") - O.gelu(z, "erf"))) < 1e-3   # the two forms are close, not equal
    assert np.max(np.abs(O.gelu(z, "tanh") - O.gelu(z, "erf"))) > 1e-5


# ---------------------------------------------------------------- whole forward
def dense_ffn(X, W1, W2):
    Z = X @ W1
    Phi = np.vectorize(lambda v: 0.5 * (1 + math.erf(v / math.sqrt(2))))(Z)
    return (Z * Phi) @ W2.T


def test_single_expert_degenerates_to_dense_ffn():
    # Section 4.1: with one expert per layer the model is a dense Transformer.
    X, Wg, W1, W2, dY = mk(32, 8, 24, 1)
    f = O.forward(X, Wg, W1, W2, c=1.0)
    assert f["k"] == 32 and np.all(f["S"] == 1.0)
    assert f["I"][0].tolist() == list(range(32))
    np.testing.assert_allclose(f["X_out"], dense_ffn(X, W1[0], W2[0]), rtol=1e-13, atol=1e-14)
    b = O.backward(X, Wg, W1, W2, dY, f)
    assert np.all(b["dWg"] == 0.0)                      # softmax over one expert is constant
    # dense FFN backward written out independently
    Z = X @ W1[0]
    H = O.gelu(Z)
    dH = dY @ W2[0]
    dZ = dH * O.gelu_grad(Z)
    np.testing.assert_allclose(b["dW2"][0], dY.T @ H, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(b["dW1"][0], X.T @ dZ, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(b["dX"], dZ @ W1[0].T, rtol=1e-12, atol=1e-13)


def test_full_capacity_is_soft_mixture():
    # c = e makes k = n: every expert processes every token and Eq. 4 is sum_i S[t,i] FFN_i(x_t).
    X, Wg, W1, W2, _ = mk(24, 8, 16, 3)
    f = O.forward(X, Wg, W1, W2, c=3.0)
    S = scipy_softmax(X @ Wg, axis=1)
    want = sum(S[:, [i]] * dense_ffn(X, W1[i], W2[i]) for i in range(3))
    np.testing.assert_allclose(f["X_out"], want, rtol=1e-12, atol=1e-13)


def test_unselected_tokens_get_zero_rows_and_selected_do_not():
    X, Wg, W1, W2, _ = mk(64, 8, 16, 4)
    f = O.forward(X, Wg, W1, W2, c=0.5)
    cnt = O.experts_per_token(f["row_ptr"])
    assert (cnt == 0).any()
    assert np.all(f["X_out"][cnt == 0] == 0.0)
    assert np.all(np.abs(f["X_out"][cnt > 0]).sum(axis=1) > 0)


def test_token_permutation_equivariance_and_expert_permutation_invariance():
    X, Wg, W1, W2, _ = mk(48, 8, 16, 4, seed=3)
    f = O.forward(X, Wg, W1, W2, c=2.0)
    perm = np.random.default_rng(0).permutation(48)
    fp = O.forward(X[perm], Wg, W1, W2, c=2.0)
    np.testing.assert_allclose(fp["X_out"], f["X_out"][perm], rtol=1e-12, atol=1e-13)
    ep = np.array([2, 0, 3, 1])
    fe = O.forward(X, Wg[:, ep], W1[ep], W2[ep], c=2.0)
    np.testing.assert_allclose(fe["X_out"], f["X_out"], rtol=1e-12, atol=1e-13)
    assert np.array_equal(fe["I"], f["I"][ep])


def test_matches_onehot_einsum_restatement():
    X, Wg, W1, W2, _ = mk(256, 64, 256, 4)            # the tiny configuration
    f = O.forward(X, Wg, W1, W2, c=2.0)
    g = layer_onehot(X, Wg, W1, W2, 2.0)
    np.testing.assert_allclose(f["S"], g["S"], atol=1e-14)
    P = np.zeros_like(g["P"])
    for i, j in itertools.product(range(4), range(f["k"])):
        P[i, j, f["I"][i, j]] = 1
    assert np.array_equal(P, g["P"])
    np.testing.assert_allclose(f["G"], g["G"], atol=1e-14)
    np.testing.assert_allclose(f["X_in"], g["X_in"], atol=0)
    np.testing.assert_allclose(f["X_e"], g["X_e"], rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(f["X_out"], g["X_out"], rtol=1e-12, atol=1e-12)


def test_overrides_reproduce_the_plain_forward():
    X, Wg, W1, W2, _ = mk(64, 8, 16, 4)
    f = O.forward(X, Wg, W1, W2, c=2.0)
    g = O.forward(X, Wg, W1, W2, c=2.0, S_override=f["S"], I_override=f["I"])
    for key in ("G", "X_out", "X_e"):
        assert np.array_equal(f[key], g[key])


# ---------------------------------------------------------------- backward: finite differences
@pytest.mark.parametrize("variant", ["erf", "tanh"])
@pytest.mark.parametrize("n,d,dff,E,c", [(32, 6, 10, 4, 2.0), (24, 5, 7, 3, 1.0)])
def test_backward_matches_finite_differences(n, d, dff, E, c, variant):
    X, Wg, W1, W2, R = mk(n, d, dff, E, seed=7)
    f = O.forward(X, Wg, W1, W2, c, variant)
    b = O.backward(X, Wg, W1, W2, R, f, variant)
    rng = np.random.default_rng(1)
    h = 1e-6

    def loss(Xp, Wgp, W1p, W2p):
        g = O.forward(Xp, Wgp, W1p, W2p, c, variant)
        assert np.array_equal(g["I"], f["I"])          # the routing did not flip at +-h
        return float((R * g["X_out"]).sum())

    for name, idx in (("dX", 0), ("dWg", 1), ("dW1", 2), ("dW2", 3)):
        base = [X, Wg, W1, W2]
        for _ in range(3):
            D = rng.standard_normal(base[idx].shape)
            plus = list(base); plus[idx] = base[idx] + h * D
            minus = list(base); minus[idx] = base[idx] - h * D
            fd = (loss(*plus) - loss(*minus)) / (2 * h)
            an = float((b[name] * D).sum())
            assert abs(fd - an) <= 1e-6 * max(1.0, abs(an)), (name, fd, an)


def test_backward_gate_gradient_is_orthogonal_to_constant_logit_shift():
    # adding a constant to all logits of a token leaves S unchanged, so dL rows sum to 0
    X, Wg, W1, W2, R = mk(32, 6, 10, 4, seed=2)
    f = O.forward(X, Wg, W1, W2, 2.0)
    b = O.backward(X, Wg, W1, W2, R, f)
    np.testing.assert_allclose(b["dL"].sum(axis=1), 0.0, atol=1e-12)


# ---------------------------------------------------------------- routing groups (Limitations section)
@pytest.mark.parametrize("groups,n,E,c", [(2, 24, 4, 2.0), (3, 16, 2, 1.0), (4, 10, 5, 1.5)])
def test_routing_groups_are_independent_layers_on_the_blocks(groups, n, E, c):
    """Experts act on rows independently, so routing g groups separately must give, on every block of n rows,
    exactly what the (already pinned) one-group layer gives on that block alone; the index lists are those of
    the blocks shifted to global row numbers, and every expert holds k tokens of every group."""
    d, dff = 6, 10
    X, Wg, W1, W2, R = mk(groups * n, d, dff, E, seed=11)
    f = O.forward(X, Wg, W1, W2, c, groups=groups)
    k = O.capacity(n, c, E)
    assert f["I"].shape == (E, groups * k) and f["k"] == groups * k
    for g in range(groups):
        blk = slice(g * n, (g + 1) * n)
        one = O.forward(X[blk], Wg, W1, W2, c)
        assert np.array_equal(f["I"][:, g * k:(g + 1) * k], one["I"] + g * n)
        assert np.array_equal(f["G"][:, g * k:(g + 1) * k], one["G"])
        np.testing.assert_allclose(f["X_out"][blk], one["X_out"], rtol=0, atol=1e-13)
        for i in range(E):                              # k distinct tokens of this group per expert
            own = f["I"][i, g * k:(g + 1) * k]
            assert len(set(own.tolist())) == k and own.min() >= g * n and own.max() < (g + 1) * n
    cnt = O.experts_per_token(f["row_ptr"])
    assert cnt.sum() == int(groups * n * c)
    assert np.array_equal(O.route(X, Wg, c, groups=1)["I"], O.route(X, Wg, c)["I"])     # one group: the paper's layer
    # the backward pass on grouped routing against finite differences (I frozen)
    b = O.backward(X, Wg, W1, W2, R, f)
    rng = np.random.default_rng(3)
    h = 1e-6

    def loss(Xp, Wgp, W1p, W2p):
        gq = O.forward(Xp, Wgp, W1p, W2p, c, groups=groups)
        assert np.array_equal(gq["I"], f["I"])
        return float((R * gq["X_out"]).sum())

    for name, idx in (("dX", 0), ("dWg", 1), ("dW1", 2), ("dW2", 3)):
        base = [X, Wg, W1, W2]
        D = rng.standard_normal(base[idx].shape)
        plus = list(base); plus[idx] = base[idx] + h * D
        minus = list(base); minus[idx] = base[idx] - h * D
        fd = (loss(*plus) - loss(*minus)) / (2 * h)
        an = float((b[name] * D).sum())
        assert abs(fd - an) <= 1e-6 * max(1.0, abs(an)), (name, fd, an)


# ---------------------------------------------------------------- the bias terms Eq. 3 omits
def test_biases_dense_closed_form_and_zero_bias_is_no_bias():
    """One expert that takes every token: the layer is a dense feed-forward block with biases, S = 1."""
    n, d, dff = 40, 6, 10
    X, Wg, W1, W2, dY = mk(n, d, dff, 1, seed=4)
    rng = np.random.default_rng(2)
    b1, b2 = rng.standard_normal((1, dff)), rng.standard_normal((1, d))
    f = O.forward(X, Wg, W1, W2, 1.0, b1=b1, b2=b2)
    z = X @ W1[0] + b1[0]
    want = (z * 0.5 * (1 + np.vectorize(math.erf)(z / math.sqrt(2)))) @ W2[0].T + b2[0]
    order = f["I"][0]
    np.testing.assert_allclose(f["X_out"], want, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(f["Z"][0], z[order], rtol=1e-13, atol=1e-14)
    # gradients of the dense block, written out independently
    b = O.backward(X, Wg, W1, W2, dY, f)
    Phi = 0.5 * (1 + np.vectorize(math.erf)(z / math.sqrt(2)))
    dz = (dY @ W2[0]) * (Phi + z * np.exp(-0.5 * z * z) / math.sqrt(2 * math.pi))
    np.testing.assert_allclose(b["db2"][0], dY.sum(axis=0), rtol=1e-12)
    np.testing.assert_allclose(b["db1"][0], dz.sum(axis=0), rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(b["dW1"][0], X.T @ dz, rtol=1e-11, atol=1e-13)
    # zero biases change nothing, bit for bit
    X, Wg, W1, W2, dY = mk(64, 8, 12, 4, seed=6)
    f0 = O.forward(X, Wg, W1, W2, 2.0)
    fz = O.forward(X, Wg, W1, W2, 2.0, b1=np.zeros((4, 12)), b2=np.zeros((4, 8)))
    assert np.array_equal(f0["X_out"], fz["X_out"]) and np.array_equal(f0["Z"], fz["Z"])


@pytest.mark.parametrize("router", ["expert", "token"])
def test_bias_gradients_match_finite_differences(router):
    n, d, dff, E, c = 40, 6, 10, 4, 1.9
    X, Wg, W1, W2, dY = mk(n, d, dff, E, seed=13)
    rng = np.random.default_rng(5)
    b1, b2 = 0.5 * rng.standard_normal((E, dff)), 0.5 * rng.standard_normal((E, d))
    f = O.forward(X, Wg, W1, W2, c, router=router, b1=b1, b2=b2)
    b = O.backward(X, Wg, W1, W2, dY, f)
    h = 1e-6
    for name, key in (("db1", "b1"), ("db2", "b2"), ("dW1", "W1"), ("dX", "X")):
        base = dict(X=X, W1=W1, b1=b1, b2=b2)
        D = rng.standard_normal(base[key].shape)
        vals = []
        for sgn in (+1, -1):
            a = dict(base); a[key] = base[key] + sgn * h * D
            g = O.forward(a["X"], Wg, a["W1"], W2, c, router=router, b1=a["b1"], b2=a["b2"])
            assert np.array_equal(g["I"], f["I"])
            vals.append(float((dY * g["X_out"]).sum()))
        fd, an = (vals[0] - vals[1]) / (2 * h), float((b[name] * D).sum())
        assert abs(fd - an) <= 1e-6 * max(1.0, abs(an)), (name, fd, an)
