"""Plain fp64 CPU oracle of the expert-choice (EC) MoE feed-forward layer.

TEST INFRASTRUCTURE, NOT THE PRODUCT.  Slow and obvious on purpose: every
function is the paper's definition written out with numpy in float64 (inputs
are widened exactly; nothing is rounded in between), with no blocking, fusion
or reordering.  Library primitives used as steps: numpy matmul, numpy stable
argsort, scipy erf.

Notation (Section 3.2): n tokens, d model width, d' hidden width, e experts,
capacity factor c, k = n*c/e tokens per expert.  A "slot" is one (expert i,
position j) pair; its flat id is i*k + j.

Readings taken where the paper is silent (all listed in the design notes):
softmax runs over the experts of one token (Section 3.4 says the gate models a
distribution over experts); TopK breaks ties toward the lower token index and
lists each expert's tokens by descending score; GeLU is the exact erf form by
default (tanh form optional); no biases; G is used raw (no renormalisation);
a token chosen by no expert gets a zero output row; in the backward pass the
index matrix I is a constant, so the gate is trained through G only; the capped variant
of Section 3.3 is Dykstra's algorithm with Kullback-Leibler projections, one round = rows,
columns, box, on log A, and replaces only the indices (see capped_assignment).

Every function here is pinned by tests/test_oracle_*.py against closed forms,
brute force, invariants, library routines and finite differences, the `store=`
hook of forward() / backward() included (tests/test_oracle_store_hook.py: the
identity hook is bitwise the definition, the names it sees are fixed, and what a
bf16-rounding hook does to each output is bracketed by the single-rounding error
of that output and stored under tests/golden/); nothing in this file is
"parity unpinned".
"""
from __future__ import annotations

import math

import numpy as np
from scipy.special import erf as _erf

F64 = np.float64


def _keep(name, x):
    return x


def capacity(n: int, c: float, e: int) -> int:
    """Eq. 1: k = n*c/e.  Non-integer values are floored; k < 1 or k > n is an error."""
    k = int(math.floor(n * float(c) / e + 1e-9))
    if k < 1 or k > n:
        raise ValueError(f"capacity k={k} outside [1, n={n}]")
    return k


def gate(X, Wg):
    """Eq. 2, first line: S = Softmax(X . Wg), one distribution over the e experts per token."""
    L = np.asarray(X, F64) @ np.asarray(Wg, F64)
    L = L - L.max(axis=1, keepdims=True)
    P = np.exp(L)
    return P / P.sum(axis=1, keepdims=True)


def topk(S, k: int):
    """Eq. 2, second line: G, I = TopK(S^T, k).

    For expert i the tokens are ordered by score S[t, i] descending, equal
    scores by ascending t (a stable sort of the negated column); the first k
    are I[i, :], and G[i, j] = S[I[i, j], i].
    """
    S = np.asarray(S)
    n, e = S.shape
    I = np.empty((e, k), np.int64)
    G = np.empty((e, k), S.dtype)
    for i in range(e):
        order = np.argsort(-S[:, i], kind="stable")
        I[i] = order[:k]
        G[i] = S[I[i], i]
    return G, I


def inverse_index(I, n: int):
    """Index form of P = Onehot(I) (Eq. 2) read by token: for token t, the flat
    slot ids i*k+j with I[i, j] = t, in ascending order (hence ascending expert).
    Returns row_ptr [n+1] and slots [number of filled slots] (e*k with expert choice)."""
    I = np.asarray(I)
    e, k = I.shape
    flat = I.reshape(-1)
    filled = np.flatnonzero(flat >= 0)               # every slot with expert choice; token choice may leave slots empty (-1)
    order = filled[np.argsort(flat[filled], kind="stable")]      # ascending token, then ascending slot id
    counts = np.bincount(flat[filled], minlength=n)
    row_ptr = np.zeros(n + 1, np.int64)
    row_ptr[1:] = np.cumsum(counts)
    return row_ptr, order.astype(np.int64)


def gelu(z, variant: str = "erf"):
    """GeLU(z) = z * Phi(z) (erf form), or its tanh approximation."""
    z = np.asarray(z, F64)
    if variant == "erf":
        return 0.5 * z * (1.0 + _erf(z / math.sqrt(2.0)))
    if variant == "tanh":
        return 0.5 * z * (1.0 + np.tanh(math.sqrt(2.0 / math.pi) * (z + 0.044715 * z ** 3)))
    raise ValueError(variant)


def gelu_grad(z, variant: str = "erf"):
    """d GeLU / dz."""
    z = np.asarray(z, F64)
    if variant == "erf":
        Phi = 0.5 * (1.0 + _erf(z / math.sqrt(2.0)))
        phi = np.exp(-0.5 * z * z) / math.sqrt(2.0 * math.pi)
        return Phi + z * phi
    if variant == "tanh":
        a = math.sqrt(2.0 / math.pi)
        u = a * (z + 0.044715 * z ** 3)
        th = np.tanh(u)
        return 0.5 * (1.0 + th) + 0.5 * z * (1.0 - th * th) * a * (1.0 + 3 * 0.044715 * z * z)
    raise ValueError(variant)


def expert_ffn(X_in_i, W1_i, W2_i, gelu_variant: str = "erf", store=_keep, b1_i=None, b2_i=None):
    """Eq. 3 for one expert: Z = X_in[i] . W1[i], H = GeLU(Z), X_e[i] = H . W2[i]^T.
    The paper leaves the bias terms out of Eq. 3 "for brevity"; given b1[i] (d') and b2[i] (d) they are the usual ones
    of a feed-forward block, Z = X_in[i] . W1[i] + b1[i] and X_e[i] = H . W2[i]^T + b2[i].

    `store` (see forward()) is handed every tensor this function produces.  H is GeLU of the product
    itself, as Eq. 3 writes it, not of what `store` made of Z."""
    Z = X_in_i @ W1_i                                      # [k, d']
    if b1_i is not None:
        Z = Z + np.asarray(b1_i, F64)[None, :]
    H = store("H", gelu(Z, gelu_variant))
    Z = store("Z", Z)
    X_e = H @ W2_i.T                                       # [k, d]
    if b2_i is not None:
        X_e = X_e + np.asarray(b2_i, F64)[None, :]
    X_e = store("X_e", X_e)
    return Z, H, X_e


def expert_ffn_backward(dX_e_i, X_in_i, Z_i, H_i, W1_i, W2_i, gelu_variant: str = "erf", store=_keep):
    """Chain rule through Eq. 3 for one expert; returns dW1[i], dW2[i], dX_in[i], dH, dZ."""
    dH = dX_e_i @ W2_i                                     # [k, d']
    dW2 = store("dW2", dX_e_i.T @ H_i)                     # [d, d']
    dZ = store("dZ", dH * gelu_grad(Z_i, gelu_variant))    # dH is consumed here as computed; it is handed to `store` on return
    dW1 = store("dW1", X_in_i.T @ dZ)                      # [d, d']
    dX_in = store("dX_in", dZ @ W1_i.T)                    # [k, d]
    return dW1, dW2, dX_in, store("dH", dH), dZ


def combine(X_e, G, I, n: int):
    """Eq. 4: X_out[t, :] = sum over the slots (i, j) with I[i, j] = t of G[i, j] * X_e[i, j, :], experts in
    ascending order; rows of tokens that no expert chose stay zero."""
    e, k = I.shape
    X_out = np.zeros((n, X_e.shape[2]), F64)
    for i in range(e):
        for j in range(k):
            if I[i, j] >= 0:                               # empty slots (token choice only) hold no token
                X_out[I[i, j]] += G[i, j] * X_e[i, j]
    return X_out


def softmax_backward(S, I, dG, store=_keep):
    """Chain rule through Eq. 2 with I held constant: dS[t, i] = dG[i, j] where I[i, j] = t (else 0), and the
    softmax Jacobian per token row, dL = S * (dS - <dS, S>)."""
    n, e = S.shape
    dS = np.zeros((n, e), F64)
    for i in range(e):
        f = I[i] >= 0
        dS[I[i][f], i] = dG[i][f]                          # tokens of one expert are distinct
    dS = store("dS", dS)
    dL = store("dL", S * (dS - (dS * S).sum(axis=1, keepdims=True)))
    return dS, dL


def add_slot_rows(dX, I, dX_in):
    """Chain rule through Eq. 3's X_in = P . X: every slot's gradient row goes back to its token (in place)."""
    e, k = I.shape
    for i in range(e):
        for j in range(k):
            if I[i, j] >= 0:
                dX[I[i, j]] += dX_in[i, j]
    return dX


def capped_assignment(S, k: int, b: int, lam: float = 1e-3, iters: int = 100):
    """Section 3.3 (expert choice with at most b experts per token): the matrix A [e, n] of

        max <S^T, A> + lam * H(A)   s.t.  every row sums to k, every column sums to at most b, 0 <= A <= 1,

    by Dykstra's algorithm with I-projections (Kullback-Leibler projections): starting from exp(S^T / lam), the
    maximiser without constraints up to a constant factor, the iterate is projected in turn onto the three
    sets, each projection applied to the iterate times that set's correction factor, which then becomes
    (what was projected) / (its projection).  One iteration is one round over the three sets in the order
    the programme lists them.  The I-projections are: rows = k, rescale each row; columns <= b, rescale the
    columns whose sum exceeds b; entries <= 1, clip.  (The row set is affine: its correction factor is
    constant along a row and cancels in the rescaling, so none is kept.)  Everything is multiplicative, so
    the iteration runs on L = log A, where exp(S / lam) neither overflows nor underflows.
    Returns A after `iters` iterations; entries lie in [0, 1], rows sum to at most k, columns to at most b."""
    from scipy.special import logsumexp
    S = np.asarray(S, F64)
    n, e = S.shape
    L = S.T / lam                                          # [e, n], log of the starting point
    q_col = np.zeros(n)                                    # log correction factor of the column set (one per column)
    q_box = np.zeros((e, n))                               # log correction factor of the box set
    for _ in range(iters):
        L = L + (math.log(k) - logsumexp(L, axis=1))[:, None]          # rows sum to k
        B = L + q_col[None, :]
        m = np.minimum(0.0, math.log(b) - logsumexp(B, axis=0))        # columns above b are scaled down to b
        L = B + m[None, :]
        q_col = -m
        B = L + q_box
        L = np.minimum(B, 0.0)                                         # entries above 1 are clipped
        q_box = B - L
    return np.exp(L)


def token_choice(S, capacity: int, top: int = 2):
    """The conventional routing Section 3.1 contrasts expert choice with, on the same scores: every token
    independently picks its `top` highest-scoring experts (equal scores: the lower expert index), and an expert,
    whose buffer holds `capacity` tokens, takes the requests in token order and drops what no longer fits.
    Returns I [e, capacity] (token per slot in order of arrival, -1 = empty slot), G [e, capacity] (S at the
    filled slots, 0 at the empty ones), load [e] (slots filled) and requested [e] (requests before dropping)."""
    S = np.asarray(S)
    n, e = S.shape
    I = np.full((e, capacity), -1, np.int64)
    G = np.zeros((e, capacity), S.dtype)
    load = np.zeros(e, np.int64)
    requested = np.zeros(e, np.int64)
    for t in range(n):
        order = np.argsort(-S[t], kind="stable")           # descending score, equal scores by ascending expert
        for i in order[:top]:
            requested[i] += 1
            if load[i] < capacity:
                I[i, load[i]] = t
                G[i, load[i]] = S[t, i]
                load[i] += 1
    return G, I, load, requested


def route(X, Wg, c: float, S_override=None, groups: int = 1, cap_b: int = 0, cap_lambda: float = 1e-3,
          cap_iters: int = 100, router: str = "expert"):
    """Eq. 1-2: S, G, I and the token->slot inverse index.

    cap_b > 0 (Section 3.3): the indices are TopK(A, k) of the capped assignment A instead of TopK(S^T, k);
    the gate weights stay G[i, j] = S[I[i, j], i].  The result then also holds A as [n, e].

    router = "token": the token-choice contrast of token_choice() with two experts per token and buffers of
    k = n*c/e slots; I then holds -1 in empty slots, and the result also has load and requested, [groups, e].

    groups > 1 (the paper's Limitations section: route several groups of tokens independently):
    X holds `groups` blocks of n rows; Eq. 1-2 are applied to each block on its own with k = n*c/e,
    and expert i's row of I and G lists its k tokens of group 0, then of group 1, ...; token
    indices are row numbers of X.  k in the result is then groups * (n*c/e)."""
    N = np.asarray(X).shape[0]
    e = np.asarray(Wg).shape[1]
    if N % groups:
        raise ValueError("rows of X must divide into the groups")
    n = N // groups
    k = capacity(n, c, e)
    S = gate(X, Wg) if S_override is None else np.asarray(S_override, F64)
    if router == "token":
        parts = [token_choice(S[g * n:(g + 1) * n], k) for g in range(groups)]
        G = np.concatenate([p[0] for p in parts], axis=1)
        I = np.concatenate([np.where(p[1] >= 0, p[1] + g * n, -1) for g, p in enumerate(parts)], axis=1)
        row_ptr, slots = inverse_index(I, N)
        return dict(k=k * groups, S=S, G=G, I=I, row_ptr=row_ptr, slots=slots,
                    load=np.stack([p[2] for p in parts]), requested=np.stack([p[3] for p in parts]))
    if router != "expert":
        raise ValueError(router)
    if cap_b:
        A = np.concatenate([capped_assignment(S[g * n:(g + 1) * n], k, cap_b, cap_lambda, cap_iters).T
                            for g in range(groups)])
        I = np.concatenate([topk(A[g * n:(g + 1) * n], k)[1] + g * n for g in range(groups)], axis=1)
        G = np.stack([S[I[i], i] for i in range(e)])
        row_ptr, slots = inverse_index(I, N)
        return dict(k=k * groups, S=S, G=G, I=I, row_ptr=row_ptr, slots=slots, A=A)
    parts = [topk(S[g * n:(g + 1) * n], k) for g in range(groups)]
    G = np.concatenate([p[0] for p in parts], axis=1)
    I = np.concatenate([p[1] + g * n for g, p in enumerate(parts)], axis=1)
    row_ptr, slots = inverse_index(I, N)
    return dict(k=k * groups, S=S, G=G, I=I, row_ptr=row_ptr, slots=slots)


def forward(X, Wg, W1, W2, c: float, gelu_variant: str = "erf", S_override=None, I_override=None,
            store=_keep, groups: int = 1, cap_b: int = 0, cap_lambda: float = 1e-3, cap_iters: int = 100,
            router: str = "expert", b1=None, b2=None):
    """Eq. 1-4.  Returns every intermediate.

    S_override replaces the gate output (the routing is then taken from it);
    I_override additionally fixes the index matrix (G is read from S at I).
    Both exist so that later stages can be compared on identical routing.

    b1 [e, d'] and b2 [e, d] are the bias terms Eq. 3 omits (see expert_ffn); None = the equation as printed.
    With biases an empty slot (token choice only) no longer holds zeros in Z, H, X_e, but nothing reads them there.

    cap_b > 0 routes with the capped assignment of Section 3.3, router = "token" with the token-choice
    contrast of Section 3.1 (see route()); empty slots then hold zero rows throughout.

    `store(name, array)` is handed EVERY named tensor the layer produces after the routing
    (X_in, Z, H, X_e, X_out here; dX_e, dG, dH, dZ, dW1, dW2, dX_in, dS, dL, dWg, dX in backward()),
    once, at the point where the definition has finished computing it, and what it returns is
    what later steps read.  The default returns its argument, which is the definition in fp64.
    A test may pass a function that rounds the tensors of its choosing to a storage format, to
    measure how far that format alone moves the result; which tensors those are is the test's
    business, this file knows nothing of any implementation's storage.
    """
    X = np.asarray(X, F64); Wg = np.asarray(Wg, F64)
    W1 = np.asarray(W1, F64); W2 = np.asarray(W2, F64)
    n, d = X.shape
    e = Wg.shape[1]
    r = route(X, Wg, c, S_override, groups, cap_b, cap_lambda, cap_iters, router)
    k, S = r["k"], r["S"]
    if I_override is not None:
        I = np.asarray(I_override, np.int64)
        G = np.stack([np.where(I[i] >= 0, S[I[i], i], 0.0) for i in range(e)])
        row_ptr, slots = inverse_index(I, n)
        r.update(I=I, G=G, row_ptr=row_ptr, slots=slots)
    I, G = r["I"], r["G"]
    X_in = X[I]                                            # Eq. 3: X_in = P . X,  [e, k, d]
    if (I < 0).any():
        X_in[I < 0] = 0.0                                  # an empty slot (token choice only) holds a zero row
    X_in = store("X_in", X_in)
    per_expert = [expert_ffn(X_in[i], W1[i], W2[i], gelu_variant, store,
                             None if b1 is None else b1[i], None if b2 is None else b2[i]) for i in range(e)]
    Z = np.stack([p[0] for p in per_expert])               # [e, k, d']
    H = np.stack([p[1] for p in per_expert])               # [e, k, d']
    X_e = np.stack([p[2] for p in per_expert])             # [e, k, d]
    X_out = store("X_out", combine(X_e, G, I, n))          # Eq. 4
    r.update(X_in=X_in, Z=Z, H=H, X_e=X_e, X_out=X_out)
    return r


def backward(X, Wg, W1, W2, dX_out, fwd, gelu_variant: str = "erf", store=_keep):
    """Gradients of <dX_out, X_out> with respect to X, Wg, W1, W2 by the chain rule
    through Eq. 4, 3, 2 in that order, with I held constant.  `store` as in forward()."""
    X = np.asarray(X, F64); Wg = np.asarray(Wg, F64)
    W1 = np.asarray(W1, F64); W2 = np.asarray(W2, F64)
    dX_out = np.asarray(dX_out, F64)
    n, d = X.shape
    e = Wg.shape[1]
    S, G, I = fwd["S"], fwd["G"], fwd["I"]
    X_in, Z, H, X_e = fwd["X_in"], fwd["Z"], fwd["H"], fwd["X_e"]
    k = I.shape[1]
    dY = dX_out[I]                                         # [e, k, d] rows of dX_out seen by each slot
    if (I < 0).any():
        dY[I < 0] = 0.0                                    # empty slots see no token
    dX_e = store("dX_e", G[:, :, None] * dY)               # Eq. 4 w.r.t. X_e
    dG = store("dG", np.einsum("ijd,ijd->ij", dY, X_e))    # Eq. 4 w.r.t. G
    per_expert = [expert_ffn_backward(dX_e[i], X_in[i], Z[i], H[i], W1[i], W2[i], gelu_variant, store)
                  for i in range(e)]
    dW1 = np.stack([p[0] for p in per_expert])             # [e, d, d']
    dW2 = np.stack([p[1] for p in per_expert])             # [e, d, d']
    dX_in = np.stack([p[2] for p in per_expert])           # [e, k, d]
    dH = np.stack([p[3] for p in per_expert])
    dZ = np.stack([p[4] for p in per_expert])
    filled = (I >= 0)[:, :, None]                          # gradients of the bias terms Eq. 3 omits: sums over an expert's filled slots
    db1 = store("db1", (dZ * filled).sum(axis=1))          # [e, d']
    db2 = store("db2", (dX_e * filled).sum(axis=1))        # [e, d]
    dS, dL = softmax_backward(S, I, dG, store)
    dWg = store("dWg", X.T @ dL)
    dX = store("dX", add_slot_rows(dL @ Wg.T, I, dX_in))
    return dict(dX=dX, dWg=dWg, dW1=dW1, dW2=dW2, db1=db1, db2=db2, dX_e=dX_e, dG=dG, dH=dH, dZ=dZ,
                dX_in=dX_in, dS=dS, dL=dL)


def experts_per_token(row_ptr):
    """Number of experts that chose each token (the quantity of Fig. 3)."""
    row_ptr = np.asarray(row_ptr)
    return row_ptr[1:] - row_ptr[:-1]
