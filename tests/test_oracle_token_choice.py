"""Pins for the token-choice contrast of the oracle (Section 3.1: every token picks its two best experts, experts
have a fixed buffer and drop what does not fit).  CPU only.  The routing is checked against an independent
formulation (positions as prefix counts over a one-hot request matrix instead of a sequential walk), against
brute force on tiny inputs and against the cases in which it must coincide with what is already pinned:
two experts with room for every token is expert choice at c = e, the soft mixture."""
import math

import numpy as np
import pytest
import torch

from oracle import ec_oracle as O
from paper_2202_09368_b200 import inputs as IN


def mk(n, d, dff, E, seed=0, scale=1.0):
    li = IN.make_layer_inputs(n, d, dff, E, torch.float32, seed, scale)
    return [t.numpy().astype(np.float64) for t in (li.X, li.Wg, li.W1, li.W2, li.dX_out)]


def requests_onehot(S, top=2):
    """R[t, i] = 1 if expert i is among the `top` best of token t (ties: lower expert), by a full Python sort."""
    n, e = S.shape
    R = np.zeros((n, e), np.int64)
    for t in range(n):
        for _, i in sorted((-S[t, i], i) for i in range(e))[:top]:
            R[t, i] = 1
    return R


@pytest.mark.parametrize("n,e,cap,levels", [(64, 4, 32, 0), (200, 8, 50, 0), (97, 5, 20, 0), (128, 4, 64, 3), (50, 6, 50, 0)])
def test_routing_equals_prefix_count_formulation(n, e, cap, levels):
    if levels:
        X, Wg = IN.quantised_gate_inputs(n, 8, e, levels)
        S = O.gate(X.numpy(), Wg.numpy())                  # many exactly equal scores: expert ties
    else:
        X, Wg, *_ = mk(n, 16, 8, e, seed=n)
        S = O.gate(X, Wg)
    G, I, load, requested = O.token_choice(S, cap)
    R = requests_onehot(S)
    assert (R.sum(axis=1) == 2).all()
    pos = np.cumsum(R, axis=0) - R                          # requests to expert i from earlier tokens
    assert np.array_equal(requested, R.sum(axis=0))
    assert np.array_equal(load, np.minimum(requested, cap))
    want = np.full((e, cap), -1, np.int64)
    for t in range(n):
        for i in range(e):
            if R[t, i] and pos[t, i] < cap:
                want[i, pos[t, i]] = t
    assert np.array_equal(I, want)
    for i in range(e):
        f = I[i] >= 0
        assert f.sum() == load[i] and f[:load[i]].all()     # filled slots come first
        assert np.array_equal(G[i][f], S[I[i][f], i]) and (G[i][~f] == 0).all()
        assert (np.diff(I[i][f]) > 0).all()                  # in order of arrival: ascending token


def test_room_for_everyone_means_two_experts_per_token_and_nothing_dropped():
    X, Wg, *_ = mk(256, 32, 16, 8, seed=3)
    r = O.route(X, Wg, c=8.0, router="token")                # k = n: every buffer could take every token
    per_token = O.experts_per_token(r["row_ptr"])
    assert (per_token == 2).all() and r["row_ptr"][-1] == 512 == len(r["slots"])
    assert np.array_equal(r["load"], r["requested"]) and r["load"].sum() == 512
    # with the usual buffers of 2n/e slots some experts overflow on these scores and tokens lose experts
    r2 = O.route(X, Wg, c=2.0, router="token")
    per2 = O.experts_per_token(r2["row_ptr"])
    assert per2.max() <= 2 and r2["requested"].max() > r2["k"] and per2.sum() == r2["load"].sum() < 512
    over = r2["requested"][0] > r2["k"]
    assert (r2["load"][0][over] == r2["k"]).all()


def test_inverse_index_skips_empty_slots():
    I = np.array([[3, 0, -1, -1], [0, 2, 3, -1]])
    row_ptr, slots = O.inverse_index(I, 5)
    assert row_ptr.tolist() == [0, 2, 2, 3, 5, 5]
    assert slots.tolist() == [1, 4, 5, 0, 6]


def test_two_experts_with_room_is_the_soft_mixture():
    """e = 2, two choices per token, buffers of n slots: every token reaches both experts, which is expert choice at
    c = e (already pinned against the closed form); only the order of an expert's slots differs."""
    X, Wg, W1, W2, dY = mk(48, 8, 16, 2, seed=5)
    tc = O.forward(X, Wg, W1, W2, 2.0, router="token")
    ec = O.forward(X, Wg, W1, W2, 2.0)
    np.testing.assert_allclose(tc["X_out"], ec["X_out"], rtol=1e-13, atol=1e-15)
    bt, be = O.backward(X, Wg, W1, W2, dY, tc), O.backward(X, Wg, W1, W2, dY, ec)
    for name in ("dX", "dWg", "dW1", "dW2"):
        np.testing.assert_allclose(bt[name], be[name], rtol=1e-11, atol=1e-13)


def test_dropped_tokens_get_what_their_surviving_experts_give_them():
    n, d, dff, E = 160, 12, 20, 4
    X, Wg, W1, W2, _ = mk(n, d, dff, E, seed=9, scale=3.0)    # sharper gates: uneven loads
    f = O.forward(X, Wg, W1, W2, 1.9, router="token")         # buffers of 76 slots for 72 to 85 requests: drops in three experts, empty slots in one
    S, R = f["S"], requests_onehot(f["S"])
    kept = np.zeros((n, E), bool)
    for i in range(E):
        kept[f["I"][i][f["I"][i] >= 0], i] = True
    assert (kept <= R.astype(bool)).all() and kept.sum() < R.sum()
    assert (kept.sum(axis=1) == 0).any() and (kept.sum(axis=1) == 1).any()
    for t in range(n):
        want = np.zeros(d)
        for i in range(E):
            if kept[t, i]:                                    # Eq. 3-4 for this token alone
                z = X[t] @ W1[i]
                want += S[t, i] * ((z * 0.5 * (1 + np.vectorize(math.erf)(z / math.sqrt(2)))) @ W2[i].T)
        np.testing.assert_allclose(f["X_out"][t], want, rtol=1e-12, atol=1e-14)
    # empty slots carry zero rows everywhere
    empty = f["I"] < 0
    assert empty.any() and not f["X_in"][empty].any() and not f["X_e"][empty].any()


@pytest.mark.parametrize("variant", ["erf", "tanh"])
def test_backward_matches_finite_differences_with_token_choice(variant):
    n, d, dff, E, c = 40, 6, 10, 4, 1.9      # buffers of 19 slots for 17 to 25 requests: drops and empty slots
    X, Wg, W1, W2, dY = mk(n, d, dff, E, seed=11)
    f = O.forward(X, Wg, W1, W2, c, variant, router="token")
    b = O.backward(X, Wg, W1, W2, dY, f, variant)
    assert (f["I"] < 0).any()
    rng = np.random.default_rng(0)
    h = 1e-6
    for name, P in (("dX", X), ("dWg", Wg), ("dW1", W1), ("dW2", W2)):
        D = rng.standard_normal(P.shape)
        args = dict(X=X, Wg=Wg, W1=W1, W2=W2)
        key = {"dX": "X", "dWg": "Wg", "dW1": "W1", "dW2": "W2"}[name]
        vals = []
        for sgn in (+1, -1):
            a = dict(args); a[key] = P + sgn * h * D
            g = O.forward(a["X"], a["Wg"], a["W1"], a["W2"], c, variant, router="token")
            assert np.array_equal(g["I"], f["I"])               # the routing did not move
            vals.append(float((dY * g["X_out"]).sum()))
        fd = (vals[0] - vals[1]) / (2 * h)
        an = float((b[name] * D).sum())
        assert abs(fd - an) <= 1e-6 * max(1.0, abs(an)), (name, fd, an)


def test_groups_are_routed_independently():
    X, Wg, W1, W2, _ = mk(96, 8, 12, 4, seed=2)
    many = O.route(X, Wg, 2.0, groups=3, router="token")
    k = many["k"] // 3
    for g in range(3):
        one = O.route(X[g * 32:(g + 1) * 32], Wg, 2.0, router="token")
        part = many["I"][:, g * k:(g + 1) * k]
        assert np.array_equal(part, np.where(one["I"] >= 0, one["I"] + g * 32, -1))
        assert np.array_equal(many["load"][g], one["load"][0]) and np.array_equal(many["requested"][g], one["requested"][0])
