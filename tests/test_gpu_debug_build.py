"""ec_validate_routing, and the index-checking build of the library (-DEC_DEBUG), on a B200.

The debug build stands in for a memory checker: every index a kernel reads from I, row_ptr or slots is compared with
its range first, a bad one is recorded (EC_ERR_INDEX) and the access it would have addressed is skipped.  It must
give the same bits as the normal build on valid inputs, and survive corrupted index structures, which only it is given.
"""
import importlib.util
import os

import pytest
import torch

from paper_2202_09368_b200 import binding as B
from paper_2202_09368_b200 import build as BUILD
from paper_2202_09368_b200 import inputs as IN

pytestmark = pytest.mark.gpu
F32, BF16 = torch.float32, torch.bfloat16


@pytest.fixture(scope="module")
def D():
    """A second instance of the binding, loaded on libecmoe_debug.so."""
    path = os.path.join(os.path.dirname(B.__file__), "libecmoe_debug.so")
    if not os.path.exists(path):
        BUILD.build(debug=True)
    spec = importlib.util.spec_from_file_location("binding_debug", B.__file__)
    m = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(m)
    m._LIB_PATH = path
    assert m.ec_debug_build() and not B.ec_debug_build()
    return m


@pytest.mark.parametrize("router,groups,n,E,c", [("expert", 1, 2048, 16, 2.0), ("expert", 3, 1000, 12, 1.5), ("token", 1, 4096, 8, 2.0),
                                                ("token", 2, 1024, 8, 1.5), ("expert", 1, 40000, 8, 2.0)])
def test_validate_routing_accepts_what_the_router_makes_and_counts_what_is_wrong(router, groups, n, E, c):
    d = 32
    li = IN.make_layer_inputs(groups * n, d, 8, E, BF16, seed=31, with_grad=False, expert_skew=0.5 if router == "token" else 0.0)
    cfg = B.make_config(n, d, 8, E, c, BF16, groups=groups, router=router)
    X, Wg = li.X.cuda(), li.Wg.cuda()
    r = B.ec_route_token_choice(cfg, X, Wg) if router == "token" else B.ec_route(cfg, X, Wg)
    assert B.ec_validate_routing(cfg, r.I, r.row_ptr, r.slots) == 0
    k = B.ec_capacity(cfg) * groups
    filled = int(r.row_ptr[-1])

    def bad(I=None, row_ptr=None, slots=None):
        return B.ec_validate_routing(cfg, r.I if I is None else I, r.row_ptr if row_ptr is None else row_ptr,
                                     r.slots if slots is None else slots)

    I2 = r.I.clone(); I2[1, 3] = groups * n + 5                       # a token that does not exist
    assert bad(I=I2) >= 1
    I2 = r.I.clone(); I2[0, 0] = -7
    assert bad(I=I2) >= 1
    if router == "expert":
        I2 = r.I.clone(); I2[2, 1] = -1                               # empty slots exist only with the token-choice router
        assert bad(I=I2) >= 1
    if groups > 1:
        I2 = r.I.clone(); I2[0, 0] = I2[0, k - 1]                     # a token of the last group in a slot of the first
        assert bad(I=I2) >= 1
    rp = r.row_ptr.clone(); rp[5] = -3
    assert bad(row_ptr=rp) >= 1
    rp = r.row_ptr.clone(); rp[-1] += 1                               # one more slot listed than filled
    assert bad(row_ptr=rp) >= 1
    sl = r.slots.clone(); sl[2] = E * k + 9
    assert bad(slots=sl) >= 1
    if filled >= 4:
        sl = r.slots.clone(); sl[[0, filled - 1]] = sl[[filled - 1, 0]]   # two tokens' slots exchanged
        assert bad(slots=sl) >= 2


@pytest.mark.parametrize("dtype,n,d,dff,E,c,router", [(F32, 300, 36, 100, 3, 1.5, "expert"), (BF16, 1024, 128, 256, 8, 2.0, "expert"),
                                                      (BF16, 2048, 128, 384, 4, 2.6, "token"), (BF16, 1024, 128, 256, 8, 2.0, "capped"),
                                                      (BF16, 1024, 128, 256, 8, 2.0, "fused"), (F32, 300, 36, 100, 3, 1.5, "fused")])
def test_debug_build_gives_the_same_bits_and_reports_nothing_on_valid_inputs(D, dtype, n, d, dff, E, c, router):
    cap = dict(cap_b=3, cap_iters=20) if router == "capped" else dict(fuse_gather=True) if router == "fused" else {}
    rt = "token" if router == "token" else "expert"
    li = IN.make_layer_inputs(n, d, dff, E, dtype, seed=33, expert_skew=1.0 if rt == "token" else 0.0)
    X, Wg, W1, W2, dY = (t.cuda() for t in (li.X, li.Wg, li.W1, li.W2, li.dX_out))
    outs = []
    for lib in (B, D):
        cfg = lib.make_config(n, d, dff, E, c, dtype, router=rt, **cap)
        ws = lib.alloc_workspace(cfg)
        Y, saved = lib.ec_moe_forward(cfg, X, Wg, W1, W2, ws=ws)
        assert lib.ec_read_status(ws) == lib.EC_OK
        g = lib.ec_moe_backward(cfg, X, Wg, W1, W2, dY, saved, ws=ws)
        assert lib.ec_read_status(ws) == lib.EC_OK
        outs.append([Y] + list(g))
    for a, b in zip(*outs):
        assert torch.equal(a.view(torch.uint8), b.view(torch.uint8))


@pytest.mark.parametrize("fuse", [False, True])
@pytest.mark.parametrize("dtype", [F32, BF16])
def test_debug_build_survives_and_reports_corrupted_indices(D, dtype, fuse):
    """Only the debug library is given these: indices far outside their ranges in the saved blob between forward and
    backward, and in the arguments of the stand-alone shuffle and unshuffle.  Every bad access is skipped."""
    n, d, dff, E, c = 1024, 128, 256, 8, 2.0
    li = IN.make_layer_inputs(n, d, dff, E, dtype, seed=35)
    X, Wg, W1, W2, dY = (t.cuda() for t in (li.X, li.Wg, li.W1, li.W2, li.dX_out))
    cfg = D.make_config(n, d, dff, E, c, dtype, fuse_gather=fuse)    # fused: the dW1 product reads rows of X through the bad I
    k = D.ec_capacity(cfg)
    ws = D.alloc_workspace(cfg)
    Y, saved = D.ec_moe_forward(cfg, X, Wg, W1, W2, ws=ws)
    assert D.ec_read_status(ws) == D.EC_OK
    v = D.saved_view(cfg, saved)
    v["I"][0, 0] = n + 11; v["I"][3, 5] = -9
    v["slots"][3] = E * k + 5; v["slots"][100] = -2
    v["row_ptr"][7] = -3; v["row_ptr"][500] = E * k + 77
    g = D.ec_moe_backward(cfg, X, Wg, W1, W2, dY, saved, ws=ws)
    assert D.ec_read_status(ws) == D.EC_ERR_INDEX
    assert all(torch.isfinite(t.float()).all() for t in g)
    # the stand-alone calls have no workspace to report in; they must simply not touch memory they should not
    r = D.ec_route(cfg, X, Wg)
    I = r.I.clone(); I[0, :4] = torch.tensor([n, 2 * n, -5, 2 ** 30], dtype=torch.int32)
    X_in = D.ec_shuffle(cfg, X, I)
    assert torch.equal(X_in[0, 4:], X[r.I[0, 4:].long()]) and not X_in[0, :4].any()
    sl = r.slots.clone(); sl[:3] = torch.tensor([E * k, -1, 2 ** 30], dtype=torch.int32)
    rp = r.row_ptr.clone(); rp[9] = -4
    out = D.ec_unshuffle(cfg, X_in.float(), r.G, rp, sl)
    assert torch.isfinite(out.float()).all()
    torch.cuda.synchronize()
