"""Parity at the benchmark's sizes, in the launch configuration bench.py times.

The 100M/32E-shaped layer is checked in full against the oracle.  The 8B/64E-shaped layer is
26 TFLOP per pass in fp64, so there the routing is checked in full and everything else on
samples the oracle can compute one by one, each stage given inputs that were checked before:
whole experts (Z, H, X_e, dW1, dW2), token rows of X_out (combine given X_e), token rows of dX
for tokens whose experts were all sampled, and dWg from the oracle's softmax backward.
"""
import math

import numpy as np
import pytest
import torch

from oracle import ec_oracle as O
from paper_2202_09368_b200 import binding as B
from paper_2202_09368_b200 import inputs as IN

from _parity import TOL, Bf16Recorder, bf16_assess, bf16_store, check_routing, rel_err, round_bf16, run_and_check, to_np

pytestmark = pytest.mark.gpu
BF16 = torch.bfloat16


def test_100m_32e_layer_full_parity():
    n, d, dff, E, c = 8192, 768, 3072, 32, 2.0
    li = IN.make_layer_inputs(n, d, dff, E, BF16, seed=0, device="cuda")
    errs = run_and_check(n, d, dff, E, c, BF16, li)
    print({k: (f"{v:.3e}" if not isinstance(v, dict) else v) for k, v in errs.items()})


def _check(name, gpu, ref, pre, stored=True):
    """The bf16 acceptance rule of tests/_parity.py for one tensor."""
    a = bf16_assess(gpu, ref, pre, stored, name)
    print(name, {k_: (f"{v_:.3e}" if isinstance(v_, float) else v_) for k_, v_ in a.items()})
    assert a["ok"], (name, a)


def test_8b_64e_layer_sampled_parity():
    n, d, dff, E, c = 16384, 4096, 16384, 64, 2.0
    dev = torch.device("cuda")
    cfg = B.make_config(n, d, dff, E, c, BF16)
    k = B.ec_capacity(cfg)
    chunk = 1 << 26
    X = IN.normal_tensor((n, d), 1.0, 0, IN.TID_X, BF16, dev, chunk)
    Wg = IN.normal_tensor((d, E), 1.0 / math.sqrt(d), 0, IN.TID_WG, BF16, dev, chunk)
    W1 = IN.normal_tensor((E, d, dff), 1.0 / math.sqrt(d), 0, IN.TID_W1, BF16, dev, chunk)
    W2 = IN.normal_tensor((E, d, dff), 1.0 / math.sqrt(dff), 0, IN.TID_W2, BF16, dev, chunk)
    dY = IN.normal_tensor((n, d), 1.0, 0, IN.TID_DXOUT, BF16, dev, chunk)
    ws = B.alloc_workspace(cfg); saved = B.alloc_saved(cfg)
    X_out, _ = B.ec_moe_forward(cfg, X, Wg, W1, W2, saved=saved, ws=ws)
    dX, dWg, dW1, dW2 = B.ec_moe_backward(cfg, X, Wg, W1, W2, dY, saved, ws=ws)
    assert B.ec_read_status(ws) == B.EC_OK
    v = B.saved_view(cfg, saved)

    Xn, Wgn, dYn = to_np(X), to_np(Wg), to_np(dY)
    # (i) gate, (ii) routing in full
    assert rel_err(to_np(v["S"]), O.gate(Xn, Wgn)) <= TOL[BF16]
    I = check_routing(cfg, v["S"], v["I"], v["G"], v["row_ptr"], v["slots"])
    S = to_np(v["S"]); G = to_np(v["G"])
    row_ptr, slots = O.inverse_index(I, n)
    assert torch.equal(v["X_in"][5], X[v["I"][5].long()])                    # the shuffle of Eq. 3 is a copy

    # (iii) whole experts
    sampled = [0, 37, 63]
    ora = {}
    for i in sampled:
        W1i, W2i = to_np(W1[i]), to_np(W2[i])
        X_in = Xn[I[i]]
        Z, H, X_e = O.expert_ffn(X_in, W1i, W2i)
        rec = Bf16Recorder()                                   # the same expert with Z, H, ... rounded where they are stored
        Zf, Hf, X_ef = O.expert_ffn(X_in, W1i, W2i, store=rec)
        _check(f"Z[{i}]", to_np(v["Z"][i]), Z, rec.before("Z", Z))
        _check(f"H[{i}]", to_np(v["H"][i]), H, rec.before("H", H))
        _check(f"X_e[{i}]", to_np(v["X_e"][i]), X_e, X_ef, stored=False)
        dX_e = G[i][:, None] * dYn[I[i]]
        gw1, gw2, dX_in, _, _ = O.expert_ffn_backward(dX_e, X_in, Z, H, W1i, W2i)
        fw1, fw2, dX_in_f, _, _ = O.expert_ffn_backward(rec("dX_e", dX_e), X_in, Zf, Hf, W1i, W2i, store=rec)
        _check(f"dW1[{i}]", to_np(dW1[i]), gw1, rec.before("dW1", gw1))
        _check(f"dW2[{i}]", to_np(dW2[i]), gw2, rec.before("dW2", gw2))
        ora[i] = dict(X_e=X_e, dX_in=dX_in, dX_in_f=dX_in_f)
        del W1i, W2i

    # combine (Eq. 4) on sampled token rows, given the GPU's X_e (checked above on whole experts)
    rng = np.random.default_rng(0)
    rows = rng.choice(n, 1024, replace=False)
    X_e_gpu = v["X_e"].view(E * k, d)
    ref_rows = np.zeros((len(rows), d))
    for a, t in enumerate(rows):
        for s in slots[row_ptr[t]:row_ptr[t + 1]]:
            ref_rows[a] += G.reshape(-1)[s] * to_np(X_e_gpu[int(s)])
    got_rows = to_np(X_out[torch.from_numpy(rows).to(dev)])
    scale = np.sqrt(np.mean(ref_rows ** 2))
    # the only difference left is fp32 summation and the final bf16 rounding of each element
    assert np.all(np.abs(got_rows - ref_rows) <= 2.0 ** -8 * np.abs(ref_rows) + 1e-6 * scale)
    cnt = row_ptr[1:] - row_ptr[:-1]
    assert torch.all(X_out[torch.from_numpy(cnt == 0).to(dev)] == 0)

    # dG for every slot from the GPU's X_e, then the oracle's softmax backward and dWg
    dG = np.empty(E * k)
    X_e_all = v["X_e"].view(E * k, d)
    dY_rows = dY[v["I"].view(-1).long()]
    dG[:] = (dY_rows.float() * X_e_all).double().sum(dim=1).cpu().numpy()    # plain dot products (torch, not the library)
    dS = np.zeros((n, E))
    for i in range(E):
        dS[I[i], i] = dG[i * k:(i + 1) * k]
    dL = S * (dS - (dS * S).sum(axis=1, keepdims=True))
    ref_dWg = Xn.T @ dL
    _check("dWg", to_np(dWg), ref_dWg, Xn.T @ bf16_store("dL", dL))

    # dX rows of tokens all of whose experts were sampled: fully from the oracle
    tok = [t for t in range(n) if cnt[t] > 0 and all((s // k) in ora for s in slots[row_ptr[t]:row_ptr[t + 1]])]
    assert len(tok) >= 32
    ref_dx = dL[tok] @ Wgn.T
    flo_dx = bf16_store("dL", dL[tok]) @ Wgn.T       # the same rows with dL, dX_in and dX rounded where they are stored
    for a, t in enumerate(tok):
        for s in slots[row_ptr[t]:row_ptr[t + 1]]:
            ref_dx[a] += ora[s // k]["dX_in"][s % k]
            flo_dx[a] += ora[s // k]["dX_in_f"][s % k]
    _check("dX rows", to_np(dX[torch.tensor(tok, device=dev)]), ref_dx, flo_dx)
