"""Writes tests/golden/store_floor.txt: what bf16 storage alone costs each output of the layer on one fixed
seeded case, computed by the CPU oracle and nothing else.

    python tests/golden/make_store_floor.py

Per output tensor, in the measure of the parity tests (max |a - ref| / RMS(ref), ref = the plain fp64 oracle):
  single = the exact fp64 result rounded once to bf16;
  floor  = the oracle evaluated with every tensor of tests/_storage.BF16_STORED rounded to bf16 where it is kept
           (the `store=` hook of oracle.forward / oracle.backward).
tests/test_oracle_store_hook.py recomputes both and compares.  Nothing here touches the CUDA library.
"""
import os
import sys

import numpy as np
import torch

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(HERE))                  # tests/
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))  # repository root

from oracle import ec_oracle as O                          # noqa: E402
from paper_2202_09368_b200 import inputs as IN             # noqa: E402
from _storage import bf16_store, round_bf16                # noqa: E402

CASE = dict(n=384, d=96, dff=160, E=6, c=2.0, seed=21)
FWD, BWD = ("Z", "H", "X_e", "X_out"), ("dX", "dWg", "dW1", "dW2")


def rel_err(got, ref):
    return float(np.max(np.abs(got - ref)) / np.sqrt(np.mean(ref * ref)))


def compute():
    li = IN.make_layer_inputs(CASE["n"], CASE["d"], CASE["dff"], CASE["E"], torch.bfloat16, CASE["seed"])
    X, Wg, W1, W2, dY = (t.float().numpy().astype(np.float64) for t in (li.X, li.Wg, li.W1, li.W2, li.dX_out))
    f = O.forward(X, Wg, W1, W2, CASE["c"])
    b = O.backward(X, Wg, W1, W2, dY, f)
    ff = O.forward(X, Wg, W1, W2, CASE["c"], store=bf16_store)
    fb = O.backward(X, Wg, W1, W2, dY, ff, store=bf16_store)
    rows = []
    for name in FWD + BWD:
        ref = f[name] if name in FWD else b[name]
        low = ff[name] if name in FWD else fb[name]
        rows.append((name, rel_err(low, ref), rel_err(round_bf16(ref), ref),
                     float(np.max(np.abs(ref)) / np.sqrt(np.mean(ref * ref)))))
    return rows


if __name__ == "__main__":
    with open(os.path.join(HERE, "store_floor.txt"), "w") as out:
        out.write("# bf16 storage floor of the layer's outputs, written by tests/golden/make_store_floor.py (CPU oracle only)\n")
        out.write("# case: " + " ".join(f"{k}={v}" for k, v in CASE.items()) + ", bf16 inputs\n")
        out.write("# tensor  floor  single_rounding  max_over_rms\n")
        for name, floor, single, peak in compute():
            out.write(f"{name} {floor:.9e} {single:.9e} {peak:.6e}\n")
            print(name, f"floor {floor:.3e} single {single:.3e} ratio {floor / max(single, 1e-300):.2f} max/rms {peak:.2f}")
