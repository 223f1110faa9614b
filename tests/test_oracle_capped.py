"""Pins of the oracle's capped expert choice (Section 3.3) against things other than itself: brute force over all
0/1 assignments on tiny instances, a general-purpose constrained optimiser on the entropic programme, the closed
form of the first projection, the plain top-k when the cap cannot bind, and the invariants of every iterate."""
import itertools
import math

import numpy as np
import pytest
from scipy.optimize import minimize
from scipy.special import softmax

from oracle import ec_oracle as O


def _scores(n, e, seed):
    rng = np.random.default_rng(seed)
    return softmax(rng.standard_normal((n, e)), axis=1)


def _brute_force(S, k, b):
    """The 0/1 matrix A [e, n] with k ones per row and at most b per column that maximises <S^T, A>."""
    n, e = S.shape
    rows = [np.array(c) for c in itertools.combinations(range(n), k)]
    best, arg = -1.0, None
    for choice in itertools.product(range(len(rows)), repeat=e):
        A = np.zeros((e, n))
        for i, r in enumerate(choice):
            A[i, rows[r]] = 1.0
        if A.sum(axis=0).max() > b:
            continue
        v = float((S.T * A).sum())
        if v > best:
            best, arg = v, A
    return arg


@pytest.mark.parametrize("n,e,k,b,seed", [(7, 3, 2, 1, 0), (6, 3, 2, 1, 1), (6, 3, 3, 2, 2), (5, 4, 2, 2, 3), (6, 2, 3, 1, 4)])
def test_converges_to_the_best_capped_assignment(n, e, k, b, seed):
    """With a small entropy weight the solution is near-integer (as the section says) and equals the optimum of
    the linear programme, found here by enumeration."""
    S = _scores(n, e, seed)
    want = _brute_force(S, k, b)
    A = O.capped_assignment(S, k, b, lam=2e-3, iters=4000)
    assert np.array_equal(np.round(A), want) and np.abs(A - want).max() < 2e-2      # near-integer: gaps of ~lam remain
    assert np.allclose(A.sum(axis=1), k, atol=1e-3) and A.sum(axis=0).max() <= b + 1e-9     # still converging slowly


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_matches_a_general_optimiser_on_the_entropic_programme(seed):
    """Moderate entropy weight: the optimum is interior in places, so the entropy term and all three constraints
    shape it.  SLSQP maximises the section's objective directly."""
    n, e, k, b, lam = 7, 3, 2, 1, 0.05
    S = _scores(n, e, seed)
    A = O.capped_assignment(S, k, b, lam=lam, iters=20000)

    def neg_obj(a):
        a = np.clip(a, 1e-300, None)
        return -(float((S.T.reshape(-1) * a).sum()) - lam * float((a * np.log(a)).sum()))

    cons = [{"type": "eq", "fun": lambda a, i=i: a.reshape(e, n)[i].sum() - k} for i in range(e)]
    cons += [{"type": "ineq", "fun": lambda a, j=j: b - a.reshape(e, n)[:, j].sum()} for j in range(n)]
    best = None
    for start in (np.full(e * n, k / n), A.reshape(-1) * 0.9 + 0.04):
        r = minimize(neg_obj, start, method="SLSQP", bounds=[(1e-12, 1.0)] * (e * n), constraints=cons,
                     options={"maxiter": 2000, "ftol": 1e-15})
        if best is None or r.fun < best.fun:
            best = r
    assert -neg_obj(A.reshape(-1)) >= -best.fun - 1e-9          # at least as good as what SLSQP found
    assert np.abs(A - best.x.reshape(e, n)).max() < 2e-3


def test_first_projection_is_a_softmax_over_the_tokens():
    """k = 1 and b >= e: after one iteration no column and no entry is over its bound (a row of a softmax sums to
    one), so A = softmax of S^T / lam along each row, exactly."""
    S = _scores(40, 4, 5)
    A = O.capped_assignment(S, 1, 4, lam=0.01, iters=1)
    assert np.allclose(A, softmax(S.T / 0.01, axis=1), rtol=1e-12, atol=0)


def test_cap_that_cannot_bind_gives_plain_expert_choice():
    """b = e: column sums never exceed e, the programme separates into rows and its near-integer solution marks
    each expert's k best tokens: the same sets as Eq. 2's TopK."""
    n, e, k = 48, 4, 6
    S = _scores(n, e, 6)
    A = O.capped_assignment(S, k, e, lam=1e-3, iters=400)
    _, I_plain = O.topk(S, k)
    _, I_cap = O.topk(A.T, k)
    assert [sorted(r) for r in I_cap.tolist()] == [sorted(r) for r in I_plain.tolist()]
    r = O.route(np.zeros((n, 1)), np.zeros((1, e)), k * e / n, S_override=S, cap_b=e, cap_iters=400)
    assert np.array_equal(np.sort(r["I"], axis=1), np.sort(I_plain, axis=1))
    assert np.array_equal(r["G"], np.stack([S[r["I"][i], i] for i in range(e)]))


@pytest.mark.parametrize("iters", [1, 7, 100])
def test_invariants_of_every_iterate(iters):
    """Whatever the iteration count: entries in [0, 1] (the last projection of a round is the clip) and k distinct
    tokens per expert.  Row and column sums meet their bounds only in the limit: the correction factors put
    back, before each projection, what that projection removed the round before."""
    n, e, c, b = 512, 16, 2.0, 2
    S = _scores(n, e, 7)
    k = O.capacity(n, c, e)
    A = O.capped_assignment(S, k, b, iters=iters)
    assert A.min() >= 0 and A.max() <= 1
    r = O.route(np.zeros((n, 1)), np.zeros((1, e)), c, S_override=S, cap_b=b, cap_iters=iters)
    assert r["I"].shape == (e, k) and all(len(set(row)) == k for row in r["I"].tolist())


def test_capped_routing_limits_experts_per_token_once_converged():
    n, e, c, b = 64, 8, 2.0, 2                             # e*k = n*b: every token ends up with exactly b experts
    S = _scores(n, e, 12)
    k = O.capacity(n, c, e)
    plain = O.route(np.zeros((n, 1)), np.zeros((1, e)), c, S_override=S)
    capped = O.route(np.zeros((n, 1)), np.zeros((1, e)), c, S_override=S, cap_b=b, cap_iters=5000, cap_lambda=5e-3)
    per_token = lambda r: np.diff(r["row_ptr"])
    assert per_token(plain).max() > b                      # the instance needs the cap
    assert per_token(capped).max() <= b
    assert per_token(capped).sum() == e * k


def test_groups_are_capped_independently():
    n, e, c, b, groups = 32, 4, 2.0, 2, 3
    S = _scores(groups * n, e, 9)
    many = O.route(np.zeros((groups * n, 1)), np.zeros((1, e)), c, S_override=S, groups=groups, cap_b=b, cap_iters=50)
    k = O.capacity(n, c, e)
    for g in range(groups):
        one = O.route(np.zeros((n, 1)), np.zeros((1, e)), c, S_override=S[g * n:(g + 1) * n], cap_b=b, cap_iters=50)
        assert np.array_equal(many["I"][:, g * k:(g + 1) * k], one["I"] + g * n)
        assert np.array_equal(many["A"][g * n:(g + 1) * n], one["A"])


def test_forward_with_a_cap_routes_with_the_capped_indices():
    """oracle.forward(cap_b=...) is route(cap_b=...) followed by the uncapped Eq. 3-4 on those indices."""
    import torch
    from paper_2202_09368_b200 import inputs as IN
    li = IN.make_layer_inputs(96, 16, 24, 4, torch.float32, seed=2)
    X, Wg, W1, W2 = (t.numpy().astype(np.float64) for t in (li.X, li.Wg, li.W1, li.W2))
    cap = dict(cap_b=2, cap_lambda=5e-3, cap_iters=200)
    r = O.route(X, Wg, 2.0, **cap)
    f = O.forward(X, Wg, W1, W2, 2.0, **cap)
    plain = O.forward(X, Wg, W1, W2, 2.0)
    assert np.array_equal(f["I"], r["I"]) and np.array_equal(f["G"], r["G"]) and np.array_equal(f["A"], r["A"])
    assert not np.array_equal(f["I"], plain["I"])                    # the cap moved some tokens
    again = O.forward(X, Wg, W1, W2, 2.0, I_override=r["I"])         # same indices through the uncapped path
    assert np.array_equal(f["X_out"], again["X_out"])
    per_token = O.experts_per_token(f["row_ptr"])
    assert per_token.sum() == 96 * 2 and (per_token > 2).sum() < (O.experts_per_token(plain["row_ptr"]) > 2).sum()
