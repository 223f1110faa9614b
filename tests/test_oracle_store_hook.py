"""Pins for the `store=` hook of oracle.forward / oracle.backward (CPU only).

The GPU parity tests bound the bf16 path by what bf16 storage alone costs (the oracle re-evaluated with the
stored tensors rounded through the hook).  That floor must itself be tied to something other than the
oracle's own say-so:
  - with the identity hook the result is bit for bit the definition, and the hook sees a fixed list of names,
    each tensor exactly once, so nothing can be rounded twice or somewhere unexpected;
  - what a bf16-rounding hook does to each output is bracketed by the error of rounding the exact output
    once, which the format fixes (at most 2^-8 max|x| / RMS(x) in the tests' measure): at least 0.9 of it for
    the outputs that are themselves stored in bf16, at most 2.5 times it for any output;
  - the values on one seeded case are stored in tests/golden/store_floor.txt (written by make_store_floor.py,
    which calls only the oracle), so a later change to the hook's placement or to the set of rounded
    tensors shows up as a changed floor.
"""
import os
import sys

import numpy as np
import torch

from oracle import ec_oracle as O
from paper_2202_09368_b200 import inputs as IN

from _storage import BF16_STORED, bf16_store, round_bf16

GOLD = os.path.join(os.path.dirname(__file__), "golden")
sys.path.insert(0, GOLD)
import make_store_floor as MSF  # noqa: E402


def _inputs(n=96, d=24, dff=40, E=4, seed=3):
    li = IN.make_layer_inputs(n, d, dff, E, torch.bfloat16, seed)
    return [t.float().numpy().astype(np.float64) for t in (li.X, li.Wg, li.W1, li.W2, li.dX_out)]


def test_identity_hook_is_the_definition_and_sees_every_tensor_once():
    X, Wg, W1, W2, dY = _inputs()
    E = Wg.shape[1]
    seen = []

    def spy(name, x):
        seen.append(name)
        return x

    f0 = O.forward(X, Wg, W1, W2, 2.0)
    b0 = O.backward(X, Wg, W1, W2, dY, f0)
    f1 = O.forward(X, Wg, W1, W2, 2.0, store=spy)
    fwd_seen, seen[:] = list(seen), []
    b1 = O.backward(X, Wg, W1, W2, dY, f1, store=spy)
    for a, b in ((f0, f1), (b0, b1)):
        assert a.keys() == b.keys()
        for k_ in a:
            assert np.array_equal(np.asarray(a[k_]), np.asarray(b[k_])), k_
    per_expert_f, per_expert_b = ["H", "Z", "X_e"], ["dW2", "dZ", "dW1", "dX_in", "dH"]
    assert fwd_seen == ["X_in"] + per_expert_f * E + ["X_out"]
    assert seen == ["dX_e", "dG"] + per_expert_b * E + ["db1", "db2", "dS", "dL", "dWg", "dX"]
    assert BF16_STORED <= set(fwd_seen) | set(seen)          # every name the tests round is one the hook is given


def test_rounding_hook_rounds_what_it_is_told_and_nothing_else():
    X, Wg, W1, W2, dY = _inputs()
    ff = O.forward(X, Wg, W1, W2, 2.0, store=bf16_store)
    fb = O.backward(X, Wg, W1, W2, dY, ff, store=bf16_store)
    is_bf16 = lambda a: np.array_equal(round_bf16(a), a)
    for name in ("Z", "H", "X_out"):
        assert is_bf16(ff[name]), name
    for name in ("dX_e", "dZ", "dX_in", "dL", "dX", "dWg", "dW1", "dW2", "db1", "db2"):
        assert is_bf16(fb[name]), name
    for name, a in (("X_e", ff["X_e"]), ("dG", fb["dG"]), ("dH", fb["dH"])):
        assert not is_bf16(a), name                          # left in fp64
    # H is GeLU of the exact product (Eq. 3), not of the rounded Z
    f = O.forward(X, Wg, W1, W2, 2.0)
    assert np.array_equal(ff["H"], round_bf16(f["H"])) and np.array_equal(ff["Z"], round_bf16(f["Z"]))


def test_floor_is_bracketed_by_single_rounding_and_matches_the_stored_values():
    gold = {}
    for line in open(os.path.join(GOLD, "store_floor.txt")):
        if not line.startswith("#"):
            p = line.split()
            gold[p[0]] = [float(v) for v in p[1:]]
    rows = MSF.compute()
    assert [r[0] for r in rows] == list(gold)
    for name, floor, single, peak in rows:
        assert single <= 2.0 ** -8 * peak, name              # what the format allows one rounding to cost
        assert floor <= 2.5 * single, (name, floor, single)
        if name in BF16_STORED:
            assert floor >= 0.9 * single, (name, floor, single)
        else:
            assert floor <= single, (name, floor, single)     # X_e stays unrounded: cheaper than storing it in bf16 would be
        np.testing.assert_allclose([floor, single, peak], gold[name], rtol=1e-6)


def test_a_hook_that_rounds_too_much_is_caught_by_the_bracket():
    """Planted mistake: rounding X_e as well (or rounding twice to a coarser grid) lifts the floor of X_out
    beyond what the stored values allow."""
    X, Wg, W1, W2, dY = _inputs(192, 48, 64, 4, 5)
    f = O.forward(X, Wg, W1, W2, 2.0)
    coarse = lambda name, x: np.round(bf16_store(name, x) * 64) / 64 if name in ("H", "X_out") else bf16_store(name, x)
    good = MSF.rel_err(O.forward(X, Wg, W1, W2, 2.0, store=bf16_store)["X_out"], f["X_out"])
    bad = MSF.rel_err(O.forward(X, Wg, W1, W2, 2.0, store=coarse)["X_out"], f["X_out"])
    single = MSF.rel_err(round_bf16(f["X_out"]), f["X_out"])
    assert good <= 2.5 * single < bad
