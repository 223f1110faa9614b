"""Helpers shared by the GPU parity tests: run the CUDA path through the C ABI and
compare it with the CPU oracle following the protocol

  (i)   S_gpu against the oracle's own S, by tolerance;
  (ii)  routing: the oracle's top-k and inverse index evaluated ON S_gpu must equal
        I, G, row_ptr, slots from the GPU bit for bit;
  (iii) every later tensor against the oracle evaluated with S and I fixed to the
        GPU's (a one-ulp difference in S may legitimately flip a boundary token).

Error measure: max|gpu - ref| / RMS(ref), per tensor, ref = the plain fp64 oracle.  Bound: 1e-4 on the fp32 path.
On the bf16 path the stated bound is 2e-2, but the layer keeps Z, H, dX_e, dZ, dX_in, dL and its outputs in bf16
(tensor-core operands and bf16 activations by definition of the path) and its outputs are heavy-tailed (a token's
row scales with its gate weights), so the exact fp64 result rounded once to bf16 can sit above 2e-2 by itself.
For those tensors the tests evaluate, on the CPU, the oracle with the stored tensors rounded to bf16 where they
are stored (tests/test_oracle_store_hook.py pins what that does) and split what storage costs an output element
into the error its operands carried in, eta = pre - ref (pre: the value before the final rounding), and the final
rounding itself, at most h = half a bf16 step at pre.  Three numbers per tensor:
  floor = max|round(pre) - ref| / RMS(ref)   what this particular sequence of roundings costs;
  reach = max(|eta| + h) / RMS(ref)          what exact arithmetic on the stored operands followed by ONE rounding can
                                             cost when a value lands on the other side of a rounding boundary than the
                                             oracle's did (fp32 accumulation moves values by parts in 10^7, enough to
                                             flip a few of them); floor <= reach <= 2 x floor;
  model_rms = RMS(gpu - round(pre)) / RMS(ref)   how far the kernels are from the rounded oracle on average: flipped
                                             roundings are rare, so anything a kernel adds shows here first.
A bf16 tensor passes when  err <= max(2e-2, REACH_SLACK x reach)  AND  model_rms <= MODEL_RMS_TOL (1e-3; 4e-3 for dX, dWg).
"""
import numpy as np
import torch

from oracle import ec_oracle as O
from paper_2202_09368_b200 import binding as B

from _storage import BF16_STORED, Bf16Recorder, bf16_store, half_ulp_bf16, round_bf16  # noqa: F401  (re-exported)

TOL = {torch.float32: 1e-4, torch.bfloat16: 2e-2}
REACH_SLACK = 1.02          # fp32 accumulation and the flipped roundings of upstream tensors, on top of `reach`
# RMS distance from the rounded oracle, relative to RMS(ref).  A twentieth of the 2e-2 bar, except for the two outputs
# that are products with dL, and dL itself: dL = S * (dS - <dS, S>) subtracts nearly equal numbers fed by fp32 dot products over d
# terms, so its bf16 rounding lands on the other side for a few percent of its entries (one bf16 step each).
MODEL_RMS_TOL = {"dX": 4e-3, "dWg": 4e-3, "dL": 4e-3}
MODEL_RMS_DEFAULT = 1e-3


def bf16_assess(gpu, ref, pre, stored=True, name=""):
    """The numbers of the module text for one tensor: err, floor, reach, model_rms, bound, ok
    (and `flipped`: the share of elements that differ from the rounded oracle at all)."""
    gpu = np.asarray(gpu, np.float64); ref = np.asarray(ref, np.float64); pre = np.asarray(pre, np.float64)
    rms = float(np.sqrt(np.mean(ref * ref))) or 1.0
    model = round_bf16(pre) if stored else pre
    h = half_ulp_bf16(pre) if stored else 0.0
    out = dict(err=float(np.max(np.abs(gpu - ref)) / rms), floor=float(np.max(np.abs(model - ref)) / rms),
               reach=float(np.max(np.abs(pre - ref) + h) / rms),
               model_rms=float(np.sqrt(np.mean((gpu - model) ** 2)) / rms), flipped=float(np.mean(gpu != model)))
    out["bound"] = max(TOL[torch.bfloat16], REACH_SLACK * out["reach"])
    out["ok"] = out["err"] <= out["bound"] and out["model_rms"] <= MODEL_RMS_TOL.get(name.split("[")[0].split(" ")[0], MODEL_RMS_DEFAULT)
    return out


def rel_err(got, ref):
    got = np.asarray(got, np.float64); ref = np.asarray(ref, np.float64)
    rms = np.sqrt(np.mean(ref * ref))
    if rms == 0:
        return float(np.max(np.abs(got)))
    return float(np.max(np.abs(got - ref)) / rms)


def to_np(t):
    if not t.is_floating_point():
        return t.cpu().numpy()
    with np.errstate(invalid="ignore"):            # empty slots of the token-choice layer hold unspecified bits (masked by the callers)
        return t.detach().float().cpu().numpy().astype(np.float64)


CAP_ATOL = 2e-3      # on entries of A in [0, 1]: fp32 rounding of log A (|log A| up to 1/lambda) carried through the rounds


def check_token_choice(cfg, S_gpu, I_gpu, G_gpu, row_ptr, slots, load, requested):
    """Step (ii) for the token-choice contrast: the oracle's walk over the GPU's own S must give the same slots,
    gate weights, loads and request counts, and the same token -> slot index over the filled slots."""
    k, n, g = B.ec_capacity(cfg), cfg.n, cfg.groups
    S32 = S_gpu.cpu().numpy()
    parts = [O.token_choice(S32[r * n:(r + 1) * n], k) for r in range(g)]
    I_ref = np.concatenate([np.where(p[1] >= 0, p[1] + r * n, -1) for r, p in enumerate(parts)], axis=1)
    G_ref = np.concatenate([p[0] for p in parts], axis=1)
    assert np.array_equal(I_gpu.cpu().numpy(), I_ref), f"I differs in {(I_gpu.cpu().numpy() != I_ref).sum()} slots"
    assert np.array_equal(G_gpu.cpu().numpy().view(np.uint32), G_ref.astype(np.float32).view(np.uint32))
    assert np.array_equal(load.cpu().numpy(), np.stack([p[2] for p in parts]))
    assert np.array_equal(requested.cpu().numpy(), np.stack([p[3] for p in parts]))
    rp_ref, sl_ref = O.inverse_index(I_ref, n * g)
    assert np.array_equal(row_ptr.cpu().numpy(), rp_ref)
    assert np.array_equal(slots.cpu().numpy()[:len(sl_ref)], sl_ref)
    return I_ref


def check_routing(cfg, S_gpu, I_gpu, G_gpu, row_ptr, slots):
    """Step (ii): bit-exact routing given the GPU's own S.  With a cap (Section 3.3) the GPU's A is compared with
    the oracle's by tolerance and the indices must be the oracle's TopK of the GPU's own A, the gate weights S at them."""
    k, n, g = B.ec_capacity(cfg), cfg.n, cfg.groups
    S32 = S_gpu.cpu().numpy()                      # float32 bits, compared as such
    keys = S32
    if cfg.cap_b:
        A_gpu = B.ec_capped_assignment(cfg, S_gpu.contiguous()).cpu().numpy()
        A_ref = np.concatenate([O.capped_assignment(S32[r * n:(r + 1) * n], k, cfg.cap_b, cfg.cap_lambda, cfg.cap_iters).T
                                for r in range(g)])
        err = np.abs(A_gpu - A_ref).max()
        print(f"capped assignment: max |A - oracle| = {err:.2e}")
        assert A_gpu.min() >= 0 and A_gpu.max() <= 1 and err <= CAP_ATOL, f"A differs by {err}"
        keys = A_gpu
    parts = [O.topk(keys[r * n:(r + 1) * n], k) for r in range(g)]         # every routing group on its own
    I_ref = np.concatenate([p[1] + r * n for r, p in enumerate(parts)], axis=1)
    G_ref = np.stack([S32[I_ref[i], i] for i in range(cfg.E)])             # Eq. 2: G[i, j] = S[I[i, j], i]
    I_np = I_gpu.cpu().numpy()
    assert np.array_equal(I_np, I_ref), f"I differs in {(I_np != I_ref).sum()} of {I_ref.size} slots"
    assert np.array_equal(G_gpu.cpu().numpy().view(np.uint32), G_ref.view(np.uint32))
    rp_ref, sl_ref = O.inverse_index(I_ref, n * g)
    assert np.array_equal(row_ptr.cpu().numpy(), rp_ref)
    assert np.array_equal(slots.cpu().numpy(), sl_ref)
    return I_ref


def run_and_check(n, d, dff, E, c, dtype, li, gelu="erf", backward=True, check_S=True, groups=1, router="expert",
                  biases=None, **cap):
    """Runs forward (+ backward) on the GPU and checks every tensor against the oracle.
    n is the number of tokens per routing group; li holds groups * n rows.  biases = (b1 [E, d'], b2 [E, d]) turns on
    the bias terms Eq. 3 leaves out, and their gradients are then checked too."""
    tol = TOL[dtype]
    cfg = B.make_config(n, d, dff, E, c, dtype, gelu, groups=groups, router=router, **cap)
    dev = "cuda"
    X, Wg, W1, W2 = (t.to(dev) for t in (li.X, li.Wg, li.W1, li.W2))
    ws = B.alloc_workspace(cfg)
    b1, b2 = (t.to(dev) for t in biases) if biases is not None else (None, None)
    b1n, b2n = (to_np(t) for t in biases) if biases is not None else (None, None)
    X_out, saved = B.ec_moe_forward(cfg, X, Wg, W1, W2, ws=ws, b1=b1, b2=b2)
    assert B.ec_read_status(ws) == B.EC_OK
    v = B.saved_view(cfg, saved)
    Xn, Wgn, W1n, W2n = (to_np(t) for t in (li.X, li.Wg, li.W1, li.W2))
    errs = {}
    if check_S:
        errs["S"] = rel_err(to_np(v["S"]), O.gate(Xn, Wgn))
        assert errs["S"] <= tol, errs
    if router == "token":
        check_token_choice(cfg, v["S"], v["I"], v["G"], v["row_ptr"], v["slots"], v["load"], v["requested"])
    else:
        check_routing(cfg, v["S"], v["I"], v["G"], v["row_ptr"], v["slots"])
    f = O.forward(Xn, Wgn, W1n, W2n, c, gelu, S_override=to_np(v["S"]), I_override=v["I"].cpu().numpy(), groups=groups,
                  router=router, b1=b1n, b2=b2n)
    if v["X_in"] is not None:                      # with fuse_gather the shuffle of Eq. 3 is never written
        assert np.array_equal(v["X_in"].float().cpu().numpy(), f["X_in"].astype(np.float32))    # it is a copy
    filled = v["I"].cpu().numpy() >= 0             # all slots with expert choice; token choice leaves some empty, and
    got = {}                                       # what the library keeps for an empty slot is unspecified
    for name in ("Z", "H", "X_e"):
        got[name] = to_np(v[name])
        got[name][~filled] = 0.0
        if biases is not None:
            f[name] = np.where(filled[:, :, None], f[name], 0.0)       # with biases the oracle's empty slots are not zero either
        errs[name] = rel_err(got[name], f[name])
    got["X_out"] = to_np(X_out)
    errs["X_out"] = rel_err(got["X_out"], f["X_out"])
    cnt = O.experts_per_token(f["row_ptr"])
    assert torch.all(X_out[torch.from_numpy(cnt == 0).to(dev)] == 0)
    if backward:
        dY = li.dX_out.to(dev)
        bg = None
        if biases is not None:
            bg = (torch.empty(E, dff, dtype=dtype, device=dev), torch.empty(E, d, dtype=dtype, device=dev))
        dX, dWg, dW1, dW2 = B.ec_moe_backward(cfg, X, Wg, W1, W2, dY, saved, ws=ws, bias_grads=bg)
        assert B.ec_read_status(ws) == B.EC_OK
        b = O.backward(Xn, Wgn, W1n, W2n, to_np(li.dX_out), f, gelu)
        outs = [("dX", dX), ("dWg", dWg), ("dW1", dW1), ("dW2", dW2)] + ([("db1", bg[0]), ("db2", bg[1])] if bg else [])
        for name, t in outs:
            got[name] = to_np(t)
            errs[name] = rel_err(got[name], b[name])
        # the intermediates of the chain rule, as the backward pass left them in the workspace
        wv = B.backward_view(cfg, ws)
        for name in ("dX_e", "dG", "dZ", "dX_in", "dL"):
            got[name] = to_np(wv[name])
            if name != "dL":
                got[name][~filled] = 0.0                               # unspecified for empty slots
                b[name] = np.where(filled.reshape(filled.shape + (1,) * (b[name].ndim - 2)), b[name], 0.0)
            errs[name] = rel_err(got[name], b[name])
    bound = {k_: tol for k_ in errs}
    bad = {k_: (e, bound[k_]) for k_, e in errs.items() if not e <= bound[k_]}
    if dtype == torch.bfloat16:
        rec = Bf16Recorder()
        ff = O.forward(Xn, Wgn, W1n, W2n, c, gelu, S_override=to_np(v["S"]), I_override=v["I"].cpu().numpy(),
                       store=rec, groups=groups, router=router, b1=b1n, b2=b2n)
        refs = dict(f)
        if backward:
            fb = O.backward(Xn, Wgn, W1n, W2n, to_np(li.dX_out), ff, gelu, store=rec)
            refs.update(b)
            ff = {**ff, **fb}
        detail, bad = {}, {k_: v_ for k_, v_ in bad.items() if k_ == "S"}
        for k_, t in got.items():
            stored = k_ in BF16_STORED
            pre = rec.before(k_, refs[k_]) if stored else ff[k_]
            if k_ in ("Z", "H", "X_e", "dX_e", "dG", "dZ", "dX_in"):
                pre = np.where(filled.reshape(filled.shape + (1,) * (pre.ndim - 2)), pre, 0.0)   # empty slots are outside the comparison
            a = bf16_assess(t, refs[k_], pre, stored, k_)
            detail[k_] = a
            if not a["ok"]:
                bad[k_] = a
        errs["_floor"] = {k_: a["floor"] for k_, a in detail.items()}
        errs["_detail"] = detail
    assert not bad, f"over tolerance: {bad} (all: {errs})"
    return errs
