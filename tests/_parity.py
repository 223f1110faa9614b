"""Helpers shared by the GPU parity tests: run the CUDA path through the C ABI and
compare it with the CPU oracle following the protocol

  (i)   S_gpu against the oracle's own S, by tolerance;
  (ii)  routing: the oracle's top-k and inverse index evaluated ON S_gpu must equal
        I, G, row_ptr, slots from the GPU bit for bit;
  (iii) every later tensor against the oracle evaluated with S and I fixed to the
        GPU's (a one-ulp difference in S may legitimately flip a boundary token).

Error measure: max|gpu - ref| / RMS(ref), per tensor.  Bound: 1e-4 on the fp32 path.
On the bf16 path the bound is 2e-2, except where the storage format alone already
costs more: the layer keeps Z, H, dX_e, dZ, dX_in, dL and its outputs in bf16 (they
are tensor-core operands or bf16 activations by definition of the path), and its
outputs are heavy-tailed (a token's row scales with its gate weights), so the
exact fp64 result rounded once to bf16 can sit above 2e-2 by itself.  The test
therefore also evaluates the oracle with those tensors rounded to bf16 where they
are stored (the arithmetic floor, CPU only; tests/test_oracle_store_hook.py pins what
that floor may be) and accepts max(2e-2, FLOOR_SLACK x floor): the kernels may add a
tenth of the format's own rounding on top of it, no more.
"""
import numpy as np
import torch

from oracle import ec_oracle as O
from paper_2202_09368_b200 import binding as B

from _storage import BF16_STORED, bf16_store  # noqa: F401  (re-exported to the test modules)

TOL = {torch.float32: 1e-4, torch.bfloat16: 2e-2}
FLOOR_SLACK = 1.1


def bf16_bound(floor):
    """Bound on a bf16-path tensor whose storage floor (see the module text) is `floor`."""
    return max(TOL[torch.bfloat16], FLOOR_SLACK * floor)


def rel_err(got, ref):
    got = np.asarray(got, np.float64); ref = np.asarray(ref, np.float64)
    rms = np.sqrt(np.mean(ref * ref))
    if rms == 0:
        return float(np.max(np.abs(got)))
    return float(np.max(np.abs(got - ref)) / rms)


def to_np(t):
    return t.detach().float().cpu().numpy().astype(np.float64) if t.is_floating_point() else t.cpu().numpy()


CAP_ATOL = 2e-3      # on entries of A in [0, 1]: fp32 rounding of log A (|log A| up to 1/lambda) carried through the rounds


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


def run_and_check(n, d, dff, E, c, dtype, li, gelu="erf", backward=True, check_S=True, groups=1, **cap):
    """Runs forward (+ backward) on the GPU and checks every tensor against the oracle.
    n is the number of tokens per routing group; li holds groups * n rows."""
    tol = TOL[dtype]
    cfg = B.make_config(n, d, dff, E, c, dtype, gelu, groups=groups, **cap)
    dev = "cuda"
    X, Wg, W1, W2 = (t.to(dev) for t in (li.X, li.Wg, li.W1, li.W2))
    ws = B.alloc_workspace(cfg)
    X_out, saved = B.ec_moe_forward(cfg, X, Wg, W1, W2, ws=ws)
    assert B.ec_read_status(ws) == B.EC_OK
    v = B.saved_view(cfg, saved)
    Xn, Wgn, W1n, W2n = (to_np(t) for t in (li.X, li.Wg, li.W1, li.W2))
    errs = {}
    if check_S:
        errs["S"] = rel_err(to_np(v["S"]), O.gate(Xn, Wgn))
        assert errs["S"] <= tol, errs
    check_routing(cfg, v["S"], v["I"], v["G"], v["row_ptr"], v["slots"])
    f = O.forward(Xn, Wgn, W1n, W2n, c, gelu, S_override=to_np(v["S"]), I_override=v["I"].cpu().numpy(), groups=groups)
    assert np.array_equal(v["X_in"].float().cpu().numpy(), Xn[f["I"]].astype(np.float32))   # gather is a copy
    for name in ("Z", "H", "X_e"):
        errs[name] = rel_err(to_np(v[name]), f[name])
    errs["X_out"] = rel_err(to_np(X_out), f["X_out"])
    cnt = O.experts_per_token(f["row_ptr"])
    assert torch.all(X_out[torch.from_numpy(cnt == 0).to(dev)] == 0)
    if backward:
        dY = li.dX_out.to(dev)
        dX, dWg, dW1, dW2 = B.ec_moe_backward(cfg, X, Wg, W1, W2, dY, saved, ws=ws)
        assert B.ec_read_status(ws) == B.EC_OK
        b = O.backward(Xn, Wgn, W1n, W2n, to_np(li.dX_out), f, gelu)
        for name, t in (("dX", dX), ("dWg", dWg), ("dW1", dW1), ("dW2", dW2)):
            errs[name] = rel_err(to_np(t), b[name])
    bound = {k_: tol for k_ in errs}
    if dtype == torch.bfloat16:
        ff = O.forward(Xn, Wgn, W1n, W2n, c, gelu, S_override=to_np(v["S"]), I_override=v["I"].cpu().numpy(),
                       store=bf16_store, groups=groups)
        floor = {k_: rel_err(ff[k_], f[k_]) for k_ in ("Z", "H", "X_e", "X_out")}
        if backward:
            fb = O.backward(Xn, Wgn, W1n, W2n, to_np(li.dX_out), ff, gelu, store=bf16_store)
            floor.update({k_: rel_err(fb[k_], b[k_]) for k_ in ("dX", "dWg", "dW1", "dW2")})
        bound = {k_: bf16_bound(floor.get(k_, 0.0)) for k_ in errs}
        errs["_floor"] = floor
    bad = {k_: (e, bound[k_]) for k_, e in errs.items() if k_ in bound and not e <= bound[k_]}
    assert not bad, f"over tolerance (err, bound): {bad} (all: {errs})"
    return errs
