"""The token-choice top-2 contrast workload (Section 3.1) through the C ABI on a B200: routing bit for bit against
the oracle's walk over the GPU's own S, then the whole layer forward and backward on the token-chosen slots, with
empty slots, dropped requests and the row tiles / k-blocks the tensor-core GEMMs skip."""
import numpy as np
import pytest
import torch

from oracle import ec_oracle as O
from paper_2202_09368_b200 import binding as B
from paper_2202_09368_b200 import inputs as IN

from _parity import TOL, check_token_choice, rel_err, run_and_check, to_np

pytestmark = pytest.mark.gpu
F32, BF16 = torch.float32, torch.bfloat16


@pytest.mark.parametrize("n,E,c,groups,dtype,skew", [
    (256, 4, 2.0, 1, F32, 0.0),
    (1000, 12, 1.5, 1, F32, 0.5),          # ragged, popular experts: some buffers overflow, others stay part empty
    (4096, 64, 2.0, 1, BF16, 0.1),
    (16384, 64, 2.0, 1, BF16, 0.05),       # the 8B/64E layer's routing shape
    (2048, 256, 2.0, 2, BF16, 0.3),        # eight experts per lane of the top-2 search, two groups
    (65536, 8, 2.0, 1, BF16, 0.2),         # 64 walks of 1024 tokens per expert
    (3000, 5, 5.0, 3, F32, 1.0),           # c = E: buffers of n slots, nothing can be dropped
])
def test_token_choice_routing(n, E, c, groups, dtype, skew):
    d = 64
    li = IN.make_layer_inputs(groups * n, d, 8, E, dtype, seed=17, expert_skew=skew, with_grad=False)
    cfg = B.make_config(n, d, 8, E, c, dtype, groups=groups, router="token")
    r = B.ec_route_token_choice(cfg, li.X.cuda(), li.Wg.cuda())
    assert rel_err(to_np(r.S), O.gate(to_np(li.X), to_np(li.Wg))) <= TOL[dtype]
    check_token_choice(cfg, r.S, r.I, r.G, r.row_ptr, r.slots, r.load, r.requested)
    per_token = (r.row_ptr[1:] - r.row_ptr[:-1]).cpu().numpy()
    assert per_token.max() <= 2 and int(r.requested.sum()) == 2 * groups * n
    if c >= E:
        assert (per_token == 2).all() and torch.equal(r.load, r.requested)


def test_token_choice_with_tied_scores():
    """Few distinct logits: whole runs of experts tie for a token; the lower expert index wins."""
    n, d, E = 2048, 16, 16
    X, Wg = IN.quantised_gate_inputs(n, d, E, 1, F32)
    cfg = B.make_config(n, d, 16, E, 2.0, F32, router="token")
    r = B.ec_route_token_choice(cfg, X.cuda(), Wg.cuda())
    check_token_choice(cfg, r.S, r.I, r.G, r.row_ptr, r.slots, r.load, r.requested)


@pytest.mark.parametrize("dtype,n,d,dff,E,c,groups,skew", [
    (F32, 300, 36, 100, 3, 1.9, 1, 0.0),
    (F32, 256, 64, 128, 8, 2.0, 2, 0.5),
    (BF16, 1024, 128, 256, 8, 2.0, 1, 0.5),       # k = 256: one expert gets 2.6 buffers' worth of requests, one a third of a buffer
    (BF16, 4096, 128, 384, 4, 2.6, 1, 1.0),       # k = 2662, eleven row tiles of 256 per expert, loads from 992 to 2662: whole
                                                  # tiles of empty slots are skipped, and the last k-blocks of dW1 and dW2
    (BF16, 6144, 256, 2304, 6, 2.5, 1, 1.0),      # long contraction over d': 256 x 512 tiles with skipped row tiles (loads 475 .. 2560)
    (BF16, 2048, 128, 256, 8, 2.0, 2, 0.7),       # two groups: nothing is skipped, empty slots are computed as zero rows
])
def test_token_choice_layer_forward_backward(dtype, n, d, dff, E, c, groups, skew):
    li = IN.make_layer_inputs(groups * n, d, dff, E, dtype, seed=19, expert_skew=skew)
    errs = run_and_check(n, d, dff, E, c, dtype, li, groups=groups, router="token")
    print({k_: f"{v_:.3e}" for k_, v_ in errs.items() if not k_.startswith("_")})


def test_expert_choice_entry_points_refuse_the_token_router():
    cfg = B.make_config(256, 64, 64, 4, 2.0, F32, router="token")
    li = IN.make_layer_inputs(256, 64, 64, 4, F32, with_grad=False)
    with pytest.raises(B.EcError) as e:
        B.ec_route(cfg, li.X.cuda(), li.Wg.cuda())
    assert e.value.code == B.EC_ERR_INVALID_ARG
    assert B.ec_workspace_bytes(B.make_config(256, 64, 64, 4, 2.0, F32, router="token", cap_b=2)) == 0
    assert B.ec_workspace_bytes(B.make_config(256, 64, 64, 1, 1.0, F32, router="token")) == 0
    torch.cuda.synchronize()
