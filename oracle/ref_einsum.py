"""Second, independent restatement of Eq. 2-4 with the literal one-hot tensor P.

TEST INFRASTRUCTURE.  Used only to cross-check oracle/ec_oracle.py on tiny
inputs: here P = Onehot(I) in R^{e x k x n} is materialised and the shuffle and
unshuffle stages are the einsums the paper names, so the index-list form used
elsewhere is validated against the dense definition.  Top-k is a Python sort on
(-score, token) tuples rather than an argsort.
"""
import math

import numpy as np


def layer_onehot(X, Wg, W1, W2, c):
    X = np.asarray(X, np.float64); Wg = np.asarray(Wg, np.float64)
    W1 = np.asarray(W1, np.float64); W2 = np.asarray(W2, np.float64)
    n, d = X.shape
    e = Wg.shape[1]
    k = int(math.floor(n * c / e + 1e-9))              # Eq. 1, non-integer values floored
    logits = np.einsum("nd,de->ne", X, Wg)
    ex = np.exp(logits - logits.max(axis=1, keepdims=True))
    S = ex / ex.sum(axis=1, keepdims=True)
    P = np.zeros((e, k, n))
    G = np.zeros((e, k))
    for i in range(e):
        ranked = sorted(range(n), key=lambda t: (-S[t, i], t))
        for j, t in enumerate(ranked[:k]):
            P[i, j, t] = 1.0
            G[i, j] = S[t, i]
    X_in = np.einsum("ikn,nd->ikd", P, X)
    Z = np.einsum("ikd,idh->ikh", X_in, W1)
    Phi = np.vectorize(lambda v: 0.5 * (1.0 + math.erf(v / math.sqrt(2.0))))(Z)
    H = Z * Phi
    X_e = np.einsum("ikh,idh->ikd", H, W2)
    X_out = np.einsum("ikn,ik,ikd->nd", P, G, X_e)
    return dict(S=S, P=P, G=G, X_in=X_in, X_e=X_e, X_out=X_out)
