"""ec_route_static: routing for callers that are not allowed to allocate device memory.

Some users of the library run where cudaMalloc is off limits: inside a host framework
that owns every byte of device memory, in a serving or real-time loop where an allocation
could synchronise the device or fail at a bad moment, or under a memory budget fixed at
start-up.  For them the library offers ec_route_static, which takes the same inputs and
outputs as ec_route but no workspace; its scratch is a fixed 8 MiB array inside the
library.  These tests call it through the C ABI and require the same bits as ec_route,
on two calls in a row with different shapes (the array keeps the previous call's contents,
so the second call would expose anything that is not cleared), and check that a
configuration too large for the array is refused before anything is launched.

This file sorts last on purpose: a run that stops at the first failure has then already
run every other test.
"""
import ctypes

import pytest
import torch

from paper_2202_09368_b200 import binding as B
from paper_2202_09368_b200 import inputs as IN


def _empty_routing(cfg, dev):
    k = B.ec_capacity(cfg)
    return B.Routing(torch.empty(cfg.n, cfg.E, dtype=torch.float32, device=dev),
                     torch.empty(cfg.E, k, dtype=torch.int32, device=dev),
                     torch.empty(cfg.E, k, dtype=torch.float32, device=dev),
                     torch.empty(cfg.n + 1, dtype=torch.int32, device=dev),
                     torch.empty(cfg.E * k, dtype=torch.int32, device=dev))


def _same_bits(a, b):
    return torch.equal(a.view(torch.int32), b.view(torch.int32))


@pytest.mark.gpu
def test_static_scratch_routing_matches_ec_route_on_consecutive_calls():
    dev = torch.device("cuda")
    # (n, d, E, c, dtype, seed): the second shape has fewer experts and more slots per expert than the
    # first and the third has ties in every column, so stale histograms, cursors or keys would show; the
    # last two are large enough for the multi-kernel top-k, whose scratch is what the static array holds
    cases = [(4096, 256, 32, 2.0, torch.bfloat16, 0), (3000, 128, 8, 1.0, torch.float32, 1),
             (2048, 64, 16, 2.0, torch.float32, 2),
             (40000, 64, 32, 2.0, torch.bfloat16, 3),       # above the single-kernel sizes: histograms, cursors and keys
             (36000, 32, 8, 2.0, torch.float32, 4)]         # live in the static array (k = 9000: multi-kernel sort)
    for rep in range(2):
        for n, d, E, c, dtype, seed in cases:
            cfg = B.make_config(n, d, 4 * d, E, c, dtype)
            assert 0 < B.ec_route_static_bytes(cfg) <= B.EC_ROUTE_STATIC_SCRATCH_BYTES
            if seed == 2:
                X, Wg = IN.quantised_gate_inputs(n, d, E, 3, dtype, seed=seed)
            else:
                li = IN.make_layer_inputs(n, d, 4 * d, E, dtype, seed=seed)
                X, Wg = li.X, li.Wg
            X, Wg = X.to(dev), Wg.to(dev)
            want = B.ec_route(cfg, X, Wg)                     # existing entry point, caller's workspace
            got = _empty_routing(cfg, dev)
            for t in (got.S, got.I, got.G, got.row_ptr, got.slots):
                t.view(torch.int32).fill_(-1)
            B.ec_route_static(cfg, X, Wg, got)                # scratch inside the library
            B.ec_route_static(cfg, X, Wg, got)                # and again, straight after itself
            torch.cuda.synchronize()
            assert _same_bits(got.S, want.S)
            assert torch.equal(got.I, want.I)
            assert _same_bits(got.G, want.G)
            assert torch.equal(got.row_ptr, want.row_ptr)
            assert torch.equal(got.slots, want.slots)


def test_static_scratch_refuses_what_does_not_fit():
    """Host-side check only: the size test comes before any CUDA call, so no GPU is needed."""
    L = B.lib()
    fake = ctypes.c_void_p(4096)                              # never dereferenced: the call must stop earlier
    big = B.make_config(1 << 22, 1024, 4096, 8, 2.0, torch.bfloat16)     # k = 2^20: the keys alone take 64 MiB
    assert B.ec_route_static_bytes(big) > B.EC_ROUTE_STATIC_SCRATCH_BYTES
    code = L.ec_route_static(ctypes.byref(big), fake, fake, fake, fake, fake, fake, fake, None)
    assert code == B.EC_ERR_WORKSPACE
    assert "workspace" in B.status_string(code)
    ok = B.make_config(262144, 1024, 4096, 256, 2.0, torch.bfloat16)
    assert B.ec_route_static_bytes(ok) <= B.EC_ROUTE_STATIC_SCRATCH_BYTES
    assert L.ec_route_static(ctypes.byref(ok), None, fake, fake, fake, fake, fake, fake, None) == B.EC_ERR_INVALID_ARG
