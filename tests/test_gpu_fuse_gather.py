"""fuse_gather: Eq. 3's X_in = P . X read in place by GEMM-1 and by the dW1 product instead of being written.

The chosen rows of X reach the tensor cores through row-indexed TMA loads (or through the index list in the FMA
kernel), so every tensor must come out bit-identical to the default path, the saved blob must be smaller by the
E x k x d elements of X_in, and the layer must still agree with the oracle."""
import pytest
import torch

from paper_2202_09368_b200 import binding as B
from paper_2202_09368_b200 import inputs as IN

from _parity import run_and_check

pytestmark = pytest.mark.gpu
F32, BF16 = torch.float32, torch.bfloat16

# dtype, groups, n, d, d', E, c: tensor-core shapes with whole and ragged tiles in M (k), K (d) and N (d'), a one-CTA
# case (k <= 128), several tiles of k per expert, two routing groups, and the FMA path (fp32; bf16 rows that are no
# multiple of 16 bytes do not exist, so bf16 always takes the tensor cores)
SHAPES = [
    (BF16, 1, 1024, 128, 256, 8, 2.0),
    (BF16, 1, 1000, 72, 200, 5, 1.7),
    (BF16, 1, 512, 64, 128, 16, 2.0),
    (BF16, 1, 4096, 256, 512, 4, 1.0),
    (BF16, 1, 3000, 328, 520, 3, 0.9),
    (BF16, 2, 1024, 128, 384, 8, 2.0),
    (F32, 1, 300, 36, 100, 3, 1.5),
    (F32, 2, 256, 64, 128, 4, 2.0),
]


@pytest.mark.parametrize("dtype,groups,n,d,dff,E,c", SHAPES)
def test_fused_gather_matches_the_oracle(dtype, groups, n, d, dff, E, c):
    li = IN.make_layer_inputs(groups * n, d, dff, E, dtype, seed=51)
    run_and_check(n, d, dff, E, c, dtype, li, groups=groups, fuse_gather=True)


@pytest.mark.parametrize("dtype,groups,n,d,dff,E,c", SHAPES)
def test_fused_gather_gives_the_same_bits_with_a_smaller_blob(dtype, groups, n, d, dff, E, c):
    li = IN.make_layer_inputs(groups * n, d, dff, E, dtype, seed=52)
    X, Wg, W1, W2, dY = (t.cuda() for t in (li.X, li.Wg, li.W1, li.W2, li.dX_out))
    b1 = IN.normal_tensor((E, dff), 0.5, 5, IN.TID_AUX, dtype).cuda()
    b2 = IN.normal_tensor((E, d), 0.5, 6, IN.TID_AUX, dtype).cuda()
    outs, sizes = [], []
    for fuse in (False, True):
        cfg = B.make_config(n, d, dff, E, c, dtype, groups=groups, fuse_gather=fuse)
        sizes.append(B.ec_saved_bytes(cfg))
        ws = B.alloc_workspace(cfg)
        Y, saved = B.ec_moe_forward(cfg, X, Wg, W1, W2, ws=ws, b1=b1, b2=b2)
        assert B.ec_read_status(ws) == B.EC_OK
        v = B.saved_view(cfg, saved)
        assert (v["X_in"] is None) == fuse
        keep = [Y.clone(), v["Z"].clone(), v["H"].clone(), v["X_e"].clone()]
        db = (torch.empty_like(b1), torch.empty_like(b2))
        g = B.ec_moe_backward(cfg, X, Wg, W1, W2, dY, saved, ws=ws, bias_grads=db)
        assert B.ec_read_status(ws) == B.EC_OK
        outs.append(keep + list(g) + list(db))
        Yf, _ = B.ec_moe_forward(cfg, X, Wg, W1, W2, forward_only=True, b1=b1, b2=b2)
        assert torch.equal(Yf.view(torch.uint8), Y.view(torch.uint8))
    for a, b in zip(*outs):
        assert torch.equal(a.view(torch.uint8), b.view(torch.uint8))
    k = B.ec_capacity(B.make_config(n, d, dff, E, c, dtype, groups=groups)) * groups
    x_in_bytes = E * k * d * X.element_size()
    assert x_in_bytes <= sizes[0] - sizes[1] < x_in_bytes + 256          # exactly X_in, up to its alignment padding
