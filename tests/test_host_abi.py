"""Host-side behaviour of the C-ABI library: it loads without a GPU, exports every
symbol the header declares, and its size / validation functions follow Eq. 1."""
import ctypes
import os
import re

import pytest
import torch

from oracle import ec_oracle as O
from paper_2202_09368_b200 import binding as B
from paper_2202_09368_b200 import build as BUILD

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    BUILD.build()


def test_library_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "ecmoe.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    names = set(re.findall(r"\b(ec_[a-z_]+)\s*\(", hdr))
    assert {"ec_route", "ec_moe_forward", "ec_moe_backward", "ec_capacity"} <= names
    L = ctypes.CDLL(os.path.join(ROOT, "paper_2202_09368_b200", "libecmoe.so"))
    for nme in names:
        assert hasattr(L, nme), nme
    assert names == set(B.EXPORTS)


def test_capacity_matches_eq1_and_the_oracle():
    for n, E, c in [(256, 4, 2), (8192, 32, 2), (8192, 64, 0.5), (16384, 64, 2), (10, 3, 1), (8, 8, 8),
                    (262144, 8, 2)]:
        cfg = B.make_config(n, 64, 64, E, c)
        assert B.ec_capacity(cfg) == O.capacity(n, c, E)
    assert B.ec_capacity(B.make_config(4, 64, 64, 8, 0.1)) == -1     # k < 1
    assert B.ec_capacity(B.make_config(4, 64, 64, 2, 3)) == -1       # k > n


def test_sizes_and_rejections():
    cfg = B.make_config(256, 64, 256, 4, 2.0)
    k = 128
    assert B.ec_saved_bytes(cfg) >= 4 * (256 * 4 + 3 * 4 * k + 257) + 4 * 4 * k * (2 * 64 + 2 * 256)
    assert B.ec_workspace_bytes(cfg) > 0
    assert B.ec_workspace_bytes(B.make_config(256, 64, 256, 4, 2.0, groups=0)) == 0
    two = B.make_config(256, 64, 256, 4, 2.0, groups=2)                            # two routing groups: twice the rows and slots
    assert B.ec_capacity(two) == k and B.ec_saved_bytes(two) >= 2 * 4 * (256 * 4 + 3 * 4 * k) + 2 * 4 * 4 * k * (2 * 64 + 2 * 256)
    assert B.ec_workspace_bytes(B.make_config(256, 63, 256, 4, 2.0)) == 0          # rows not 16-byte multiples
    assert B.ec_workspace_bytes(B.make_config(256, 64, 256, 300, 2.0)) == 0        # E > 256
    big = B.make_config(16384, 4096, 16384, 64, 2.0, torch.bfloat16)
    assert B.ec_saved_bytes(big) > 2 * 32768 * (4096 + 16384) * 2
    assert B.status_string(B.EC_ERR_TIMEOUT).startswith("a bounded")


def test_fuse_gather_config():
    """fuse_gather leaves X_in out of the blob and of the forward-only scratch, and is refused where slots can be empty."""
    for dt, es in ((torch.float32, 4), (torch.bfloat16, 2)):
        plain, fused = (B.make_config(256, 64, 256, 4, 2.0, dt, groups=2, fuse_gather=f) for f in (False, True))
        x_in = 4 * 2 * 128 * 64 * es
        assert x_in <= B.ec_saved_bytes(plain) - B.ec_saved_bytes(fused) < x_in + 256
        fwd = lambda cfg: int(B.lib().ec_forward_only_workspace_bytes(ctypes.byref(cfg)))
        assert x_in <= fwd(plain) - fwd(fused) < x_in + 256
        assert B.ec_workspace_bytes(fused) == B.ec_workspace_bytes(plain)
    assert B.ec_saved_bytes(B.make_config(256, 64, 256, 4, 2.0, router="token", fuse_gather=True)) == 0
    bad = B.make_config(256, 64, 256, 4, 2.0)
    bad.fuse_gather = 2
    assert B.ec_saved_bytes(bad) == 0 and B.ec_workspace_bytes(bad) == 0


def test_null_pointers_are_rejected_without_a_gpu():
    cfg = B.make_config(256, 64, 256, 4, 2.0)
    L = B.lib()
    code = L.ec_route(ctypes.byref(cfg), None, None, None, None, None, None, None, None, 0, None)
    assert code == B.EC_ERR_INVALID_ARG
    code = L.ec_moe_forward(ctypes.byref(cfg), None, None, None, None, None, None, None, None, 0, None, 0, None)
    assert code == B.EC_ERR_INVALID_ARG


def test_capped_config_checks():
    """Section 3.3 options: the scratch grows by A, log A and the box factors; infeasible or malformed settings are refused
    by the size functions (host arithmetic only)."""
    ok = B.make_config(256, 64, 128, 8, 2.0, torch.bfloat16, cap_b=2)
    fwd_bytes = lambda cfg: int(B.lib().ec_forward_only_workspace_bytes(ctypes.byref(cfg)))
    assert fwd_bytes(ok) >= fwd_bytes(B.make_config(256, 64, 128, 8, 2.0, torch.bfloat16)) + 3 * 256 * 8 * 4     # A, log A, box factors
    for bad in (B.make_config(256, 64, 128, 8, 2.0, torch.bfloat16, cap_b=1),                 # E*k = 2n slots cannot fit under b = 1
                B.make_config(256, 64, 128, 8, 2.0, torch.bfloat16, cap_b=2, cap_iters=0),
                B.make_config(256, 64, 128, 8, 2.0, torch.bfloat16, cap_b=2, cap_lambda=0.0),
                B.make_config(256, 64, 128, 8, 2.0, torch.bfloat16, cap_b=-1)):
        assert B.ec_workspace_bytes(bad) == 0
