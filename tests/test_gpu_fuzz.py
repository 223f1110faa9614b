"""Seeded random shapes through the whole layer (forward + backward, routing bit-exact, tensors within
tolerance): ragged tiles in every dimension, expert counts that do and do not allow the tensor-core and
vector-load paths, k from 1 to n, one or several routing groups."""
import numpy as np
import pytest
import torch

from paper_2202_09368_b200 import binding as B
from paper_2202_09368_b200 import inputs as IN

from _parity import run_and_check

pytestmark = pytest.mark.gpu


def _cases(count, seed):
    rng = np.random.default_rng(seed)
    out = []
    while len(out) < count:
        dtype = torch.bfloat16 if rng.random() < 0.6 else torch.float32
        mult = 8 if dtype == torch.bfloat16 else 4
        n = int(rng.integers(8, 700))
        d = int(rng.integers(1, 40)) * mult
        dff = int(rng.integers(1, 60)) * mult
        E = int(rng.choice([1, 2, 3, 4, 5, 7, 8, 12, 16, 24, 32, 40]))
        groups = int(rng.choice([1, 1, 1, 2, 3]))
        k = int(rng.integers(1, n + 1)) if rng.random() < 0.3 else max(1, int(n * rng.choice([0.5, 1, 2]) / E))
        k = min(k, n)
        c = (k + 0.25) * E / n                          # floor(n * c / E) == k
        cfg = B.make_config(n, d, dff, E, c, dtype, groups=groups)
        if B.ec_capacity(cfg) != k or B.ec_workspace_bytes(cfg) == 0:
            continue
        out.append((dtype, groups, n, d, dff, E, c, k))
    return out


@pytest.mark.parametrize("dtype,groups,n,d,dff,E,c,k", _cases(24, seed=2024))
def test_random_shapes(dtype, groups, n, d, dff, E, c, k):
    li = IN.make_layer_inputs(groups * n, d, dff, E, dtype, seed=n + E)
    gelu = "tanh" if (n + d) % 5 == 0 else "erf"
    run_and_check(n, d, dff, E, c, dtype, li, gelu=gelu, groups=groups)


@pytest.mark.parametrize("dtype,groups,n,d,dff,E,c,k", [t for t in _cases(40, seed=77) if t[5] >= 2][:16])
def test_random_shapes_token_choice_and_biases(dtype, groups, n, d, dff, E, c, k):
    """The same random shapes through the token-choice contrast routing (every second case) and with the bias terms of
    Eq. 3 (two cases in three): empty slots, dropped requests, skipped tiles and bias gradients at odd sizes."""
    token = (n + E) % 2 == 0
    li = IN.make_layer_inputs(groups * n, d, dff, E, dtype, seed=n + E + 1, expert_skew=0.5 if token else 0.0)
    biases = None
    if (n + d) % 3 != 0:
        biases = (IN.normal_tensor((E, dff), 0.5, n, IN.TID_AUX, dtype), IN.normal_tensor((E, d), 0.5, n + 1, IN.TID_AUX, dtype))
    run_and_check(n, d, dff, E, c, dtype, li, groups=groups, router="token" if token else "expert", biases=biases)
