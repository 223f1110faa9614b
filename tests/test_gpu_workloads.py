"""The two remaining workload families, through the C ABI on a B200:

  - routing-only stress (gate + softmax, column top-k, inverse index, shuffle, unshuffle with
    identity experts, X_e = X_in) at d = 1024, bf16, over a grid of group sizes and expert counts;
  - the capacity-factor sweep of the forward pass (E = 64, c in {0.5, 1, 2}, gate logits scaled
    x1 and x4 to vary the skew of the scores).

Routing and the index lists are compared bit for bit with the oracle evaluated on the GPU's own
S; the shuffle is a copy and must be exact; the unshuffle is compared with the fp64 sum of
Eq. 4 within the final bf16 rounding.
"""
import numpy as np
import pytest
import torch

from oracle import ec_oracle as O
from paper_2202_09368_b200 import binding as B
from paper_2202_09368_b200 import inputs as IN

from _parity import TOL, check_routing, rel_err, run_and_check, to_np

pytestmark = pytest.mark.gpu
BF16 = torch.bfloat16


@pytest.mark.parametrize("n,E", [(4096, 8), (4096, 32), (4096, 128), (4096, 256), (16384, 32), (16384, 256),
                                 (65536, 8), (65536, 128),
                                 # the largest groups of the stress grid: k = 65536 .. 2048, sixteen sort tiles and four
                                 # global bitonic levels at E = 8, eight expert chunks at E = 256
                                 (262144, 8), (262144, 32), (262144, 128), (262144, 256)])
def test_routing_only_chain_identity_experts(n, E):
    d, c = 1024, 2.0
    li = IN.make_layer_inputs(n, d, 8, E, BF16, seed=0, with_grad=False)
    cfg = B.make_config(n, d, 8, E, c, BF16)
    k = B.ec_capacity(cfg)
    X, Wg = li.X.cuda(), li.Wg.cuda()
    r = B.ec_route(cfg, X, Wg)
    Xn, Wgn = to_np(li.X), to_np(li.Wg)
    assert rel_err(to_np(r.S), O.gate(Xn, Wgn)) <= TOL[BF16]
    I = check_routing(cfg, r.S, r.I, r.G, r.row_ptr, r.slots)
    # perfect load balance: k distinct tokens per expert, n*c slots in all
    assert all(len(set(row)) == k for row in I[:: max(1, E // 8)])
    assert int(r.row_ptr[-1]) == E * k == int(n * c)
    # Eq. 3 with P as an index list: a copy
    X_in = B.ec_shuffle(cfg, X, r.I)
    assert torch.equal(X_in, X[r.I.long()])
    # Eq. 4 with identity experts
    X_e = X_in.float()
    X_out = B.ec_unshuffle(cfg, X_e, r.G, r.row_ptr, r.slots)
    G = to_np(r.G).reshape(-1)
    ref = np.zeros((n, d))
    for i in range(E):                                                     # fp64 sum over the slots of each token, Eq. 4;
        ref[I[i]] += G[i * k:(i + 1) * k, None] * Xn[I[i]]                 # an expert's tokens are distinct
    got = to_np(X_out)
    scale = np.sqrt(np.mean(ref ** 2))
    assert np.all(np.abs(got - ref) <= 2.0 ** -8 * np.abs(ref) + 1e-6 * scale)      # one bf16 rounding
    cnt = to_np(r.row_ptr)[1:] - to_np(r.row_ptr)[:-1]
    assert torch.all(X_out[torch.from_numpy(cnt == 0).cuda()] == 0)


@pytest.mark.parametrize("c", [0.5, 1.0, 2.0])
@pytest.mark.parametrize("scale", [1.0, 4.0])
def test_capacity_factor_sweep_forward(c, scale):
    n, d, dff, E = 8192, 768, 3072, 64
    li = IN.make_layer_inputs(n, d, dff, E, BF16, seed=0, logit_scale=scale, with_grad=False, device="cuda")
    errs = run_and_check(n, d, dff, E, c, BF16, li, backward=False)
    assert B.ec_capacity(B.make_config(n, d, dff, E, c, BF16)) == int(n * c / E)
    print(c, scale, {k_: (f"{v:.3e}" if not isinstance(v, dict) else v) for k_, v in errs.items()})


@pytest.mark.parametrize("dtype,groups,n,d,dff,E,c", [
    (torch.float32, 3, 100, 24, 40, 5, 1.5),       # ragged, E not a multiple of 4: scalar top-k path
    (torch.float32, 2, 256, 64, 128, 8, 2.0),
    (BF16, 4, 512, 128, 256, 16, 2.0),             # k = 64 per group, 256 slots per expert: two-CTA GEMMs
    (BF16, 8, 1024, 256, 512, 64, 1.0),            # 16 tokens per expert and group
])
def test_routing_groups_forward_backward(dtype, groups, n, d, dff, E, c):
    """Several routing groups per call (the Limitations section's suggestion): each block of n rows is routed
    on its own, experts serve groups * k slots."""
    li = IN.make_layer_inputs(groups * n, d, dff, E, dtype, seed=4)
    run_and_check(n, d, dff, E, c, dtype, li, groups=groups)


def test_routing_groups_match_separate_calls():
    """Routing g groups in one call selects, group by group, what g separate one-group calls select."""
    groups, n, d, E, c = 4, 2048, 128, 32, 2.0
    li = IN.make_layer_inputs(groups * n, d, 8, E, BF16, seed=6, with_grad=False)
    X, Wg = li.X.cuda(), li.Wg.cuda()
    many = B.ec_route(B.make_config(n, d, 8, E, c, BF16, groups=groups), X, Wg)
    one_cfg = B.make_config(n, d, 8, E, c, BF16)
    k = B.ec_capacity(one_cfg)
    for g in range(groups):
        one = B.ec_route(one_cfg, X[g * n:(g + 1) * n], Wg)
        assert torch.equal(many.S[g * n:(g + 1) * n], one.S)
        assert torch.equal(many.I[:, g * k:(g + 1) * k], one.I + g * n)
        assert torch.equal(many.G[:, g * k:(g + 1) * k], one.G)


@pytest.mark.parametrize("groups,n,E,c,dtype", [
    (2, 32768, 64, 2.0, BF16),                  # groups above the single-CTA size: histogram passes, k = 1024 per group
    (3, 20000, 8, 2.0, torch.float32),          # k = 5000 per group: candidates merged globally, multi-kernel sort
    (2, 17000, 12, 0.7, torch.float32),         # ragged k, E a multiple of 4 only
    # bf16: the gate's softmax epilogue counts the selection's first histogram; groups that do not end on a warp's
    # 32 rows, padded columns of a 64-wide tile, and the two-CTA tile whose warps split the columns of a row
    (3, 20000, 8, 2.0, BF16),
    (2, 17000, 40, 0.7, BF16),
    (2, 40000, 136, 1.5, BF16),
])
def test_routing_groups_large_groups(groups, n, E, c, dtype):
    """Routing groups on the multi-kernel top-k path (more than 16384 tokens per group)."""
    d = 32
    li = IN.make_layer_inputs(groups * n, d, 8, E, dtype, seed=8, with_grad=False)
    cfg = B.make_config(n, d, 8, E, c, dtype, groups=groups)
    r = B.ec_route(cfg, li.X.cuda(), li.Wg.cuda())
    assert rel_err(to_np(r.S), O.gate(to_np(li.X), to_np(li.Wg))) <= TOL[dtype]
    check_routing(cfg, r.S, r.I, r.G, r.row_ptr, r.slots)


def test_routing_groups_with_ties_on_the_multi_kernel_path():
    """Few distinct logits and large groups: thousands of exactly equal scores at the threshold of every expert
    and group, resolved toward the lower token by the walk in token order."""
    groups, n, d, E = 2, 20000, 16, 8
    for dtype in (torch.float32, BF16):           # bf16: first histogram counted by the gate's epilogue
        X, Wg = IN.quantised_gate_inputs(groups * n, d, E, 2, dtype)
        cfg = B.make_config(n, d, 16, E, 2.0, dtype, groups=groups)
        r = B.ec_route(cfg, X.cuda(), Wg.cuda())
        check_routing(cfg, r.S, r.I, r.G, r.row_ptr, r.slots)


@pytest.mark.parametrize("n,E,c,b,iters,lam,groups", [
    (512, 8, 2.0, 2, 100, 1e-3, 1),          # the paper's settings: lambda = 0.001, 100 rounds
    (1000, 12, 1.5, 2, 40, 1e-3, 1),         # E not a multiple of 32, ragged n
    (2048, 64, 2.0, 3, 100, 1e-3, 1),
    (4096, 256, 2.0, 4, 25, 1e-3, 1),        # eight experts per lane
    (300, 40, 2.0, 3, 300, 5e-3, 3),         # three groups, solved independently; close to converged
    (16384, 64, 2.0, 2, 100, 1e-3, 1),       # the 8B/64E layer's routing shape
    (40000, 64, 2.0, 2, 12, 1e-3, 1),        # too many tokens for the registers: state in shared memory
    (9000, 200, 2.0, 3, 7, 1e-3, 2),         # too much for shared memory too (seven experts per lane, two groups): one launch per round
])
def test_capped_routing(n, E, c, b, iters, lam, groups):
    """Section 3.3: A against the oracle's iterate, I = TopK(A, k) bit for bit on the GPU's own A, G = S at I."""
    d = 64
    li = IN.make_layer_inputs(groups * n, d, 8, E, BF16, seed=11, with_grad=False)
    cfg = B.make_config(n, d, 8, E, c, BF16, groups=groups, cap_b=b, cap_iters=iters, cap_lambda=lam)
    r = B.ec_route(cfg, li.X.cuda(), li.Wg.cuda())
    check_routing(cfg, r.S, r.I, r.G, r.row_ptr, r.slots)
    plain = B.ec_route(B.make_config(n, d, 8, E, c, BF16, groups=groups), li.X.cuda(), li.Wg.cuda())
    assert torch.equal(plain.S, r.S)


def test_capped_routing_converged_moves_tokens_under_the_cap():
    """Run to convergence, the solver leaves only the few tokens over the cap whose entries of A stay fractional
    (the solution is near-integer, not integer, and TopK rounds it)."""
    n, d, E, c, b = 1024, 64, 8, 2.0, 3
    li = IN.make_layer_inputs(n, d, 8, E, BF16, seed=12, with_grad=False)
    X, Wg = li.X.cuda(), li.Wg.cuda()
    over = lambda r: int(((r.row_ptr[1:] - r.row_ptr[:-1]) > b).sum())
    plain = B.ec_route(B.make_config(n, d, 8, E, c, BF16), X, Wg)
    capped = B.ec_route(B.make_config(n, d, 8, E, c, BF16, cap_b=b, cap_iters=500, cap_lambda=5e-3), X, Wg)
    assert over(plain) >= 10 and over(capped) <= over(plain) // 3
    assert int(capped.row_ptr[-1]) == n * 2


@pytest.mark.parametrize("dtype,groups", [(torch.float32, 1), (BF16, 2)])
def test_capped_layer_forward_backward(dtype, groups):
    """The whole layer with capped routing: everything after the routing is the uncapped path on other indices."""
    n, d, dff, E, c = 256, 64, 128, 8, 2.0
    li = IN.make_layer_inputs(groups * n, d, dff, E, dtype, seed=13)
    run_and_check(n, d, dff, E, c, dtype, li, groups=groups, cap_b=2, cap_iters=60)
