"""CUDA path against the CPU oracle, through the C ABI.  Needs a B200."""
import numpy as np
import pytest
import torch

from oracle import ec_oracle as O
from paper_2202_09368_b200 import binding as B
from paper_2202_09368_b200 import inputs as IN

from _parity import TOL, check_routing, rel_err, run_and_check, to_np

pytestmark = pytest.mark.gpu

F32, BF16 = torch.float32, torch.bfloat16


@pytest.mark.parametrize("n,d,dff,E,c", [
    (256, 64, 256, 4, 2.0),        # the tiny configuration
    (300, 36, 100, 3, 1.5),        # ragged everywhere: k = 150, tiles with tails
    (64, 16, 32, 1, 1.0),          # one expert: dense FFN
    (48, 8, 16, 4, 4.0),           # c = E: every expert takes every token
    (130, 12, 20, 8, 0.5),         # some tokens unselected; k = 8
    (97, 8, 8, 5, 0.06),           # k = 1
])
def test_fp32_forward_backward(n, d, dff, E, c):
    li = IN.make_layer_inputs(n, d, dff, E, F32, seed=0)
    run_and_check(n, d, dff, E, c, F32, li)


def test_fp32_tanh_gelu():
    li = IN.make_layer_inputs(128, 32, 64, 4, F32, seed=1)
    run_and_check(128, 32, 64, 4, 2.0, F32, li, gelu="tanh")


@pytest.mark.parametrize("n,d,dff,E,c", [
    (256, 64, 256, 4, 2.0),
    (512, 128, 384, 8, 2.0),       # k = 128: one full MMA tile per expert
    (1000, 200, 328, 16, 2.0),     # k = 125, ragged in every dimension
    (2048, 256, 512, 32, 2.0),
    (384, 64, 128, 3, 1.0),        # E not a multiple of 8
    (1024, 192, 448, 64, 0.5),     # k = 8
    (3040, 1000, 2072, 10, 1.0),   # k = 304, long contraction over d', 20 tile rows: GEMM-2 and dX_in take 512-column
                                   # tiles (one wave instead of two of 256-column ones), with tails in M, N and K
    (5120, 1024, 2048, 10, 1.0),   # k = 512: whole 256 x 512 tiles
    (8000, 512, 2056, 40, 1.0),    # k = 200, forty experts of one 256 x 512 tile each (d = 512), ragged K
])
def test_bf16_forward_backward(n, d, dff, E, c):
    li = IN.make_layer_inputs(n, d, dff, E, BF16, seed=0)
    run_and_check(n, d, dff, E, c, BF16, li)


def test_bf16_logit_scale_and_tanh():
    li = IN.make_layer_inputs(1024, 128, 256, 16, BF16, seed=2, logit_scale=4.0)
    run_and_check(1024, 128, 256, 16, 1.0, BF16, li, gelu="tanh")


@pytest.mark.parametrize("dtype", [F32, BF16])
@pytest.mark.parametrize("n,d,E,c,levels", [(512, 16, 4, 2.0, 2), (777, 8, 3, 1.0, 1), (4096, 64, 32, 2.0, 3)])
def test_routing_with_heavy_ties(n, d, E, c, levels, dtype):
    """Few distinct logits: columns of S are full of exact ties; the lower token must win."""
    X, Wg = IN.quantised_gate_inputs(n, d, E, levels, dtype)
    cfg = B.make_config(n, d, 16, E, c, dtype)
    r = B.ec_route(cfg, X.cuda(), Wg.cuda())
    assert len(np.unique(r.S.cpu().numpy()[:, 0])) <= d          # tokens t and t+d share a row of logits
    check_routing(cfg, r.S, r.I, r.G, r.row_ptr, r.slots)


def test_routing_all_equal_scores():
    n, d, E = 1500, 8, 6
    X = torch.zeros(n, d)
    Wg = torch.zeros(d, E)
    cfg = B.make_config(n, d, 16, E, 2.0, F32)
    r = B.ec_route(cfg, X.cuda(), Wg.cuda())
    k = B.ec_capacity(cfg)
    assert torch.equal(r.I.cpu(), torch.arange(k, dtype=torch.int32).repeat(E, 1))
    check_routing(cfg, r.S, r.I, r.G, r.row_ptr, r.slots)


@pytest.mark.parametrize("n,E,c", [(20000, 2, 2.0), (70000, 8, 2.0), (5000, 200, 2.0), (33000, 40, 0.7)])
def test_routing_large_k_and_many_experts(n, E, c):
    """k beyond one sort tile (multi-kernel bitonic path) and E beyond one column chunk."""
    d = 16
    li = IN.make_layer_inputs(n, d, 8, E, F32, seed=3, with_grad=False)
    cfg = B.make_config(n, d, 16, E, c, F32)
    r = B.ec_route(cfg, li.X.cuda(), li.Wg.cuda())
    assert rel_err(to_np(r.S), O.gate(to_np(li.X), to_np(li.Wg))) <= 1e-4
    check_routing(cfg, r.S, r.I, r.G, r.row_ptr, r.slots)


@pytest.mark.parametrize("n,E,groups", [(128, 256, 1), (64, 256, 2), (100, 200, 1), (128, 136, 1), (512, 256, 1)])
def test_gate_with_more_experts_than_one_column_tile_and_few_rows(n, E, groups):
    """E in (128, 256] with at most 128 token rows: the softmax of Eq. 2 still has to see all E logits of a row in one tile."""
    d = 64
    li = IN.make_layer_inputs(groups * n, d, 8, E, BF16, seed=7, with_grad=False)
    cfg = B.make_config(n, d, 8, E, 2.0 * E / 8, BF16, groups=groups)     # k = n / 4 tokens per expert and group
    r = B.ec_route(cfg, li.X.cuda(), li.Wg.cuda())
    S = to_np(r.S)
    assert rel_err(S, O.gate(to_np(li.X), to_np(li.Wg))) <= TOL[BF16]
    np.testing.assert_allclose(S.sum(axis=1), 1.0, atol=1e-5)
    check_routing(cfg, r.S, r.I, r.G, r.row_ptr, r.slots)


@pytest.mark.parametrize("dtype,n,d,dff,E", [(F32, 200, 24, 40, 4), (BF16, 1024, 128, 384, 4), (BF16, 2048, 256, 2304, 4)])
def test_expert_gemm_on_its_own(dtype, n, d, dff, E):
    """The three expert-batched products of Eq. 3 and its backward as calls of their own, against numpy in fp64."""
    cfg = B.make_config(n, d, dff, E, 2.0, dtype)
    k = B.ec_capacity(cfg)
    li = IN.make_layer_inputs(n, d, dff, E, dtype, seed=23)
    A = li.X[:E * k // 2].repeat(2, 1).view(E, k, d).contiguous().cuda()                  # [E, k, d]
    H = IN.normal_tensor((E, k, dff), 1.0, 23, IN.TID_AUX, dtype).cuda()                   # [E, k, d']
    W1, W2 = li.W1.cuda(), li.W2.cuda()
    tol = TOL[dtype]
    for kind, a, b_, ref in ((B.EC_GEMM_XW1, A, W1, np.einsum("ikd,idf->ikf", to_np(A), to_np(W1))),
                             (B.EC_GEMM_HW2T, H, W2, np.einsum("ikf,idf->ikd", to_np(H), to_np(W2))),
                             (B.EC_GEMM_ATB, A, H, np.einsum("ikd,ikf->idf", to_np(A), to_np(H)))):
        got = to_np(B.ec_expert_gemm(cfg, kind, a, b_))
        if dtype == BF16:                      # one rounding of the exact result to bf16
            assert np.all(np.abs(got - ref) <= 2.0 ** -8 * np.abs(ref) + 1e-5 * np.sqrt(np.mean(ref ** 2))), kind
        else:
            assert rel_err(got, ref) <= tol, kind


@pytest.mark.parametrize("dtype,n,d,dff,E,c,router,groups", [
    (F32, 300, 36, 100, 3, 1.5, "expert", 1),
    (F32, 256, 32, 64, 4, 1.9, "token", 1),
    (BF16, 1024, 128, 384, 8, 2.0, "expert", 1),
    (BF16, 2048, 256, 2304, 4, 2.0, "expert", 2),      # 256 x 512 tiles in the second product, whose epilogue adds b2
    (BF16, 4096, 128, 384, 4, 2.6, "token", 1),        # empty slots: their Z is b1, not zero, and must not reach any gradient
])
def test_bias_terms_forward_backward(dtype, n, d, dff, E, c, router, groups):
    """The bias terms Eq. 3 leaves out "for brevity": Z = X_in . W1 + b1, X_e = H . W2^T + b2, and db1, db2."""
    li = IN.make_layer_inputs(groups * n, d, dff, E, dtype, seed=29, expert_skew=1.0 if router == "token" else 0.0)
    b1 = IN.normal_tensor((E, dff), 0.5, 29, IN.TID_AUX, dtype)
    b2 = IN.normal_tensor((E, d), 0.5, 30, IN.TID_AUX, dtype)
    errs = run_and_check(n, d, dff, E, c, dtype, li, groups=groups, router=router, biases=(b1, b2))
    assert "db1" in errs and "db2" in errs
    # without biases the same call gives a different output (the terms are really there)
    cfg = B.make_config(n, d, dff, E, c, dtype, groups=groups, router=router)
    X, Wg, W1, W2 = (t.cuda() for t in (li.X, li.Wg, li.W1, li.W2))
    Y0, _ = B.ec_moe_forward(cfg, X, Wg, W1, W2, forward_only=True)
    Y1, _ = B.ec_moe_forward(cfg, X, Wg, W1, W2, forward_only=True, b1=b1.cuda(), b2=b2.cuda())
    assert not torch.equal(Y0, Y1)


def test_read_status_maps_the_status_word():
    """ec_read_status only reads the first word of the workspace: 0 is EC_OK, 5 a bounded wait that expired, anything
    else is reported as a CUDA error.  No kernel is involved."""
    ws = torch.zeros(1024, dtype=torch.int32, device="cuda")
    for word, want in ((0, B.EC_OK), (5, B.EC_ERR_TIMEOUT), (7, B.EC_ERR_CUDA), (4, B.EC_ERR_CUDA)):
        ws[0] = word
        assert B.ec_read_status(ws) == want
    assert B.lib().ec_read_status(None, None) == B.EC_ERR_INVALID_ARG


def test_run_to_run_determinism():
    n, d, dff, E = 1024, 128, 256, 8
    li = IN.make_layer_inputs(n, d, dff, E, BF16, seed=5)
    cfg = B.make_config(n, d, dff, E, 2.0, BF16)
    X, Wg, W1, W2, dY = (t.cuda() for t in (li.X, li.Wg, li.W1, li.W2, li.dX_out))
    outs = []
    for _ in range(2):
        Y, saved = B.ec_moe_forward(cfg, X, Wg, W1, W2)
        g = B.ec_moe_backward(cfg, X, Wg, W1, W2, dY, saved)
        outs.append([Y.clone()] + [t.clone() for t in g] + [t.clone() for t in B.saved_view(cfg, saved).values()])
    for a, b in zip(*outs):
        assert torch.equal(a.contiguous().view(torch.uint8), b.contiguous().view(torch.uint8))   # bitwise


def test_argument_errors_are_reported_before_any_launch():
    cfg = B.make_config(256, 64, 256, 4, 2.0, F32)
    li = IN.make_layer_inputs(256, 64, 256, 4, F32)
    X, Wg = li.X.cuda(), li.Wg.cuda()
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.EcError) as e:
        B.ec_route(cfg, X, Wg, ws=small)
    assert e.value.code == B.EC_ERR_WORKSPACE
    ws = B.alloc_workspace(cfg)
    with pytest.raises(B.EcError) as e:
        B.ec_route(cfg, X.view(-1)[1:], Wg, ws=ws)          # misaligned pointer
    assert e.value.code == B.EC_ERR_INVALID_ARG
    torch.cuda.synchronize()


@pytest.mark.parametrize("dtype,n,d,dff,E,c,groups", [(F32, 300, 36, 100, 3, 1.5, 1), (BF16, 2048, 256, 512, 32, 2.0, 1),
                                                      (BF16, 512, 128, 256, 16, 2.0, 4)])
def test_forward_only_gives_the_same_output_without_a_saved_blob(dtype, n, d, dff, E, c, groups):
    """saved = NULL: the intermediates live in the workspace, Z is never written, X_out is the same bits."""
    li = IN.make_layer_inputs(groups * n, d, dff, E, dtype, seed=9, with_grad=False)
    cfg = B.make_config(n, d, dff, E, c, dtype, groups=groups)
    X, Wg, W1, W2 = (t.cuda() for t in (li.X, li.Wg, li.W1, li.W2))
    Y_train, _ = B.ec_moe_forward(cfg, X, Wg, W1, W2)
    Y_inf, none = B.ec_moe_forward(cfg, X, Wg, W1, W2, forward_only=True)
    assert none is None
    assert torch.equal(Y_train.view(torch.uint8), Y_inf.view(torch.uint8))
    # a workspace that is too small for the intermediates is refused before anything is launched
    small = torch.empty(B.ec_workspace_bytes(cfg) // 2 if dff > d else 256, dtype=torch.uint8, device="cuda")
    code = B.lib().ec_moe_forward(__import__("ctypes").byref(cfg), X.data_ptr(), Wg.data_ptr(), W1.data_ptr(), W2.data_ptr(),
                                  None, None, Y_inf.data_ptr(), None, 0, small.data_ptr(), 256, None)
    assert code == B.EC_ERR_WORKSPACE
    torch.cuda.synchronize()


@pytest.mark.parametrize("cap", [{}, {"cap_b": 3, "cap_iters": 30}])
def test_a_step_can_be_captured_in_a_cuda_graph(cap):
    """Forward and backward only queue work on the caller's stream: a step captured once replays to the same bits
    (with the capped routing too, whose solver is a cooperative launch)."""
    n, d, dff, E = 1024, 128, 256, 8
    li = IN.make_layer_inputs(n, d, dff, E, BF16, seed=5)
    cfg = B.make_config(n, d, dff, E, 2.0, BF16, **cap)
    X, Wg, W1, W2, dY = (t.cuda() for t in (li.X, li.Wg, li.W1, li.W2, li.dX_out))
    ws, saved, Y = B.alloc_workspace(cfg), B.alloc_saved(cfg), torch.empty_like(X)
    grads = (torch.empty_like(X), torch.empty_like(Wg), torch.empty_like(W1), torch.empty_like(W2))

    def step():
        B.ec_moe_forward(cfg, X, Wg, W1, W2, Y, saved, ws)
        B.ec_moe_backward(cfg, X, Wg, W1, W2, dY, saved, grads, ws)

    step(); torch.cuda.synchronize()
    want = [t.clone() for t in (Y,) + grads]
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step()
    torch.cuda.current_stream().wait_stream(side)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    for t in (Y,) + grads:
        t.zero_()
    graph.replay(); torch.cuda.synchronize()
    for a, b in zip(want, (Y,) + grads):
        assert torch.equal(a.view(torch.uint8), b.view(torch.uint8))
