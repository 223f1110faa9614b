"""Thin ctypes binding of libecmoe.so (see include/ecmoe.h).

Argument marshalling only: every step of the layer runs in the library's CUDA
kernels.  torch is used to own device memory and to name the current stream.
There is no fallback: if the library is missing, loading raises.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

# ECMOE_DEBUG=1 in the environment selects the build with index checks (python -m paper_2202_09368_b200.build --debug)
_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)),
                         "libecmoe_debug.so" if os.environ.get("ECMOE_DEBUG") == "1" else "libecmoe.so")
_lib = None

EC_OK, EC_ERR_INVALID_ARG, EC_ERR_UNSUPPORTED, EC_ERR_WORKSPACE, EC_ERR_CUDA, EC_ERR_TIMEOUT, EC_ERR_INDEX = range(7)
EC_F32, EC_BF16 = 0, 1
EC_GELU_ERF, EC_GELU_TANH = 0, 1
EC_ROUTER_EXPERT_CHOICE, EC_ROUTER_TOKEN_TOP2 = 0, 1

EXPORTS = ["ec_capacity", "ec_workspace_bytes", "ec_saved_bytes", "ec_saved_view", "ec_route",
           "ec_moe_forward", "ec_moe_backward", "ec_read_status", "ec_status_string",
           "ec_uses_tensor_cores", "ec_launch_count", "ec_profile_enable", "ec_profile_read",
           "ec_route_static", "ec_route_static_bytes", "ec_shuffle", "ec_unshuffle",
           "ec_forward_only_workspace_bytes", "ec_capped_assignment", "ec_route_token_choice", "ec_expert_gemm", "ec_validate_routing", "ec_debug_build", "ec_backward_view"]
EC_GEMM_XW1, EC_GEMM_HW2T, EC_GEMM_ATB = 0, 1, 2
EC_ROUTE_STATIC_SCRATCH_BYTES = 8 << 20


class ec_config(C.Structure):
    _fields_ = [("n", C.c_int64), ("d_model", C.c_int32), ("d_ff", C.c_int32), ("E", C.c_int32),
                ("groups", C.c_int32), ("c", C.c_double), ("dtype", C.c_int32), ("gelu", C.c_int32),
                ("cap_b", C.c_int32), ("cap_iters", C.c_int32), ("cap_lambda", C.c_double),
                ("router", C.c_int32), ("fuse_gather", C.c_int32)]


class ec_saved_ptrs(C.Structure):
    _fields_ = [(name, C.c_void_p) for name in
                ("S", "I", "G", "row_ptr", "slots", "X_in", "Z", "H", "X_e", "load", "requested")]


class ec_backward_ptrs(C.Structure):
    _fields_ = [(name, C.c_void_p) for name in ("dX_e", "dG", "dZ", "dX_in", "dL")] + [("dL_is_bf16", C.c_int32)]


class EcError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        super().__init__(f"{what}: {status_string(code)} ({code})")


def lib():
    """Loads the library once.  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(f"{_LIB_PATH} is missing: run `python -m paper_2202_09368_b200.build`; "
                               "there is no fallback path")
        L = C.CDLL(_LIB_PATH)
        P, V = C.POINTER(ec_config), C.c_void_p
        L.ec_capacity.restype = C.c_int64; L.ec_capacity.argtypes = [P]
        L.ec_workspace_bytes.restype = C.c_size_t; L.ec_workspace_bytes.argtypes = [P]
        L.ec_saved_bytes.restype = C.c_size_t; L.ec_saved_bytes.argtypes = [P]
        L.ec_forward_only_workspace_bytes.restype = C.c_size_t; L.ec_forward_only_workspace_bytes.argtypes = [P]
        L.ec_saved_view.restype = C.c_int; L.ec_saved_view.argtypes = [P, V, C.POINTER(ec_saved_ptrs)]
        L.ec_route.restype = C.c_int
        L.ec_route.argtypes = [P, V, V, V, V, V, V, V, V, C.c_size_t, V]
        L.ec_route_token_choice.restype = C.c_int
        L.ec_route_token_choice.argtypes = [P, V, V, V, V, V, V, V, V, V, V, C.c_size_t, V]
        L.ec_expert_gemm.restype = C.c_int
        L.ec_expert_gemm.argtypes = [P, C.c_int, V, V, V, V, C.c_size_t, V]
        L.ec_validate_routing.restype = C.c_int
        L.ec_validate_routing.argtypes = [P, V, V, V, C.POINTER(C.c_int64), V, C.c_size_t, V]
        L.ec_debug_build.restype = C.c_int; L.ec_debug_build.argtypes = []
        L.ec_backward_view.restype = C.c_int; L.ec_backward_view.argtypes = [P, V, C.POINTER(ec_backward_ptrs)]
        L.ec_route_static.restype = C.c_int
        L.ec_route_static.argtypes = [P, V, V, V, V, V, V, V, V]
        L.ec_route_static_bytes.restype = C.c_size_t; L.ec_route_static_bytes.argtypes = [P]
        L.ec_capped_assignment.restype = C.c_int; L.ec_capped_assignment.argtypes = [P, V, V, V, C.c_size_t, V]
        L.ec_shuffle.restype = C.c_int; L.ec_shuffle.argtypes = [P, V, V, V, V]
        L.ec_unshuffle.restype = C.c_int; L.ec_unshuffle.argtypes = [P, V, V, V, V, V, V]
        L.ec_moe_forward.restype = C.c_int
        L.ec_moe_forward.argtypes = [P, V, V, V, V, V, V, V, V, C.c_size_t, V, C.c_size_t, V]
        L.ec_moe_backward.restype = C.c_int
        L.ec_moe_backward.argtypes = [P, V, V, V, V, V, V, C.c_size_t, V, V, V, V, V, V, V, C.c_size_t, V]
        L.ec_read_status.restype = C.c_int; L.ec_read_status.argtypes = [V, V]
        L.ec_status_string.restype = C.c_char_p; L.ec_status_string.argtypes = [C.c_int]
        L.ec_uses_tensor_cores.restype = C.c_int; L.ec_uses_tensor_cores.argtypes = [P]
        L.ec_launch_count.restype = C.c_longlong; L.ec_launch_count.argtypes = []
        L.ec_profile_enable.restype = None; L.ec_profile_enable.argtypes = [C.c_int]
        L.ec_profile_read.restype = C.c_int
        L.ec_profile_read.argtypes = [C.POINTER(C.c_float), C.POINTER(C.c_char_p), C.c_int]
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().ec_status_string(code).decode()


def make_config(n, d_model, d_ff, E, c, dtype=torch.float32, gelu="erf", groups=1, cap_b=0, cap_iters=100,
                cap_lambda=1e-3, router="expert", fuse_gather=False) -> ec_config:
    """cap_b > 0: at most cap_b experts per token (Section 3.3) with the paper's solver settings as defaults.
    router = "token": the token-choice top-2 contrast of Section 3.1 with expert buffers of n*c/E slots.
    fuse_gather: Eq. 3's X_in = P.X is read in place by the expert GEMMs instead of being written (smaller saved blob)."""
    dt = {torch.float32: EC_F32, torch.bfloat16: EC_BF16}[dtype]
    return ec_config(int(n), int(d_model), int(d_ff), int(E), int(groups), float(c), dt,
                     {"erf": EC_GELU_ERF, "tanh": EC_GELU_TANH}[gelu], int(cap_b), int(cap_iters), float(cap_lambda),
                     {"expert": EC_ROUTER_EXPERT_CHOICE, "token": EC_ROUTER_TOKEN_TOP2}[router], int(bool(fuse_gather)))


def ec_capacity(cfg: ec_config) -> int:
    """Eq. 1 per routing group."""
    return int(lib().ec_capacity(C.byref(cfg)))


def total_tokens(cfg: ec_config) -> int:
    return cfg.n * cfg.groups


def slots_per_expert(cfg: ec_config) -> int:
    return ec_capacity(cfg) * cfg.groups


def ec_workspace_bytes(cfg: ec_config) -> int:
    return int(lib().ec_workspace_bytes(C.byref(cfg)))


def ec_saved_bytes(cfg: ec_config) -> int:
    return int(lib().ec_saved_bytes(C.byref(cfg)))


def ec_uses_tensor_cores(cfg: ec_config) -> bool:
    return bool(lib().ec_uses_tensor_cores(C.byref(cfg)))


def _ptr(t):
    return C.c_void_p(0 if t is None else t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _torch_dtype(cfg):
    return torch.float32 if cfg.dtype == EC_F32 else torch.bfloat16


def _check(code, what):
    if code != EC_OK:
        raise EcError(code, what)


def alloc_workspace(cfg, device="cuda") -> torch.Tensor:
    nb = ec_workspace_bytes(cfg)
    if nb == 0:
        raise EcError(EC_ERR_INVALID_ARG, "ec_workspace_bytes")
    return torch.empty(nb, dtype=torch.uint8, device=device)


def alloc_saved(cfg, device="cuda") -> torch.Tensor:
    nb = ec_saved_bytes(cfg)
    if nb == 0:
        raise EcError(EC_ERR_INVALID_ARG, "ec_saved_bytes")
    return torch.empty(nb, dtype=torch.uint8, device=device)


@dataclass
class Routing:
    S: torch.Tensor
    I: torch.Tensor
    G: torch.Tensor
    row_ptr: torch.Tensor
    slots: torch.Tensor
    load: torch.Tensor | None = None          # token-choice contrast only: slots filled per expert, [groups, E]
    requested: torch.Tensor | None = None     # and tokens that asked for each expert


def ec_route(cfg, X, Wg, ws=None, out: Routing | None = None) -> Routing:
    """Eq. 1-2 on device tensors; returns S, I, G and the token->slot index."""
    if ec_capacity(cfg) < 1:
        raise EcError(EC_ERR_INVALID_ARG, "ec_capacity")
    n, k = total_tokens(cfg), slots_per_expert(cfg)
    dev = X.device
    if out is None:
        out = Routing(torch.empty(n, cfg.E, dtype=torch.float32, device=dev),
                      torch.empty(cfg.E, k, dtype=torch.int32, device=dev),
                      torch.empty(cfg.E, k, dtype=torch.float32, device=dev),
                      torch.empty(n + 1, dtype=torch.int32, device=dev),
                      torch.empty(cfg.E * k, dtype=torch.int32, device=dev))
    ws = alloc_workspace(cfg, dev) if ws is None else ws
    _check(lib().ec_route(C.byref(cfg), _ptr(X), _ptr(Wg), _ptr(out.S), _ptr(out.I), _ptr(out.G),
                          _ptr(out.row_ptr), _ptr(out.slots), _ptr(ws), ws.numel(), _stream()), "ec_route")
    return out


def ec_route_token_choice(cfg, X, Wg, ws=None) -> Routing:
    """The token-choice contrast routing (cfg.router = token): I holds -1 and G holds 0 in empty slots; only the
    first row_ptr[-1] entries of `slots` are meaningful."""
    n, k, dev = total_tokens(cfg), slots_per_expert(cfg), X.device
    out = Routing(torch.empty(n, cfg.E, dtype=torch.float32, device=dev),
                  torch.empty(cfg.E, k, dtype=torch.int32, device=dev),
                  torch.empty(cfg.E, k, dtype=torch.float32, device=dev),
                  torch.empty(n + 1, dtype=torch.int32, device=dev),
                  torch.empty(cfg.E * k, dtype=torch.int32, device=dev),
                  torch.empty(cfg.groups, cfg.E, dtype=torch.int32, device=dev),
                  torch.empty(cfg.groups, cfg.E, dtype=torch.int32, device=dev))
    ws = alloc_workspace(cfg, dev) if ws is None else ws
    _check(lib().ec_route_token_choice(C.byref(cfg), _ptr(X), _ptr(Wg), _ptr(out.S), _ptr(out.I), _ptr(out.G),
                                       _ptr(out.row_ptr), _ptr(out.slots), _ptr(out.load), _ptr(out.requested),
                                       _ptr(ws), ws.numel(), _stream()), "ec_route_token_choice")
    return out


def ec_capped_assignment(cfg, S, ws=None, A=None):
    """Section 3.3: A [n, E] after cfg.cap_iters rounds of the solver, from the gate scores S [n, E]."""
    if A is None:
        A = torch.empty_like(S)
    ws = alloc_workspace(cfg, S.device) if ws is None else ws
    _check(lib().ec_capped_assignment(C.byref(cfg), _ptr(S), _ptr(A), _ptr(ws), ws.numel(), _stream()),
           "ec_capped_assignment")
    return A


def ec_shuffle(cfg, X, I, X_in=None):
    """Eq. 3 shuffle: X_in[i, j, :] = X[I[i, j], :]."""
    k = slots_per_expert(cfg)
    if X_in is None:
        X_in = torch.empty(cfg.E, k, cfg.d_model, dtype=X.dtype, device=X.device)
    _check(lib().ec_shuffle(C.byref(cfg), _ptr(X), _ptr(I), _ptr(X_in), _stream()), "ec_shuffle")
    return X_in


def ec_unshuffle(cfg, X_e, G, row_ptr, slots, X_out=None):
    """Eq. 4 unshuffle: X_out[t, :] = sum over the slots of t of G[s] * X_e[s, :] (X_e, G fp32)."""
    if X_out is None:
        X_out = torch.empty(total_tokens(cfg), cfg.d_model, dtype=_torch_dtype(cfg), device=X_e.device)
    _check(lib().ec_unshuffle(C.byref(cfg), _ptr(X_e), _ptr(G), _ptr(row_ptr), _ptr(slots), _ptr(X_out), _stream()),
           "ec_unshuffle")
    return X_out


def ec_expert_gemm(cfg, kind, A, Bm, out=None, ws=None):
    """One expert-batched product of Eq. 3 / its backward on its own (see ecmoe.h for the three kinds and shapes)."""
    k, E, d, f = slots_per_expert(cfg), cfg.E, cfg.d_model, cfg.d_ff
    shape = {EC_GEMM_XW1: (E, k, f), EC_GEMM_HW2T: (E, k, d), EC_GEMM_ATB: (E, d, f)}[kind]
    out = torch.empty(shape, dtype=A.dtype, device=A.device) if out is None else out
    ws = alloc_workspace(cfg, A.device) if ws is None else ws
    _check(lib().ec_expert_gemm(C.byref(cfg), kind, _ptr(A), _ptr(Bm), _ptr(out), _ptr(ws), ws.numel(), _stream()),
           "ec_expert_gemm")
    return out


def ec_validate_routing(cfg, I, row_ptr, slots, ws=None) -> int:
    """Number of violations found in an index structure (0 = consistent); synchronises the current stream."""
    ws = alloc_workspace(cfg, I.device) if ws is None else ws
    bad = C.c_int64(-1)
    _check(lib().ec_validate_routing(C.byref(cfg), _ptr(I), _ptr(row_ptr), _ptr(slots), C.byref(bad), _ptr(ws), ws.numel(),
                                     _stream()), "ec_validate_routing")
    return int(bad.value)


def ec_debug_build() -> bool:
    return bool(lib().ec_debug_build())


def ec_route_static_bytes(cfg: ec_config) -> int:
    return int(lib().ec_route_static_bytes(C.byref(cfg)))


def ec_route_static(cfg, X, Wg, out: Routing) -> Routing:
    """ec_route without a workspace: the scratch is a fixed array inside the library, for callers
    that cannot allocate device memory.  `out` must be given (this call allocates nothing); calls
    on one device must not overlap on the GPU.  Configurations that need more than
    EC_ROUTE_STATIC_SCRATCH_BYTES of scratch raise EC_ERR_WORKSPACE."""
    _check(lib().ec_route_static(C.byref(cfg), _ptr(X), _ptr(Wg), _ptr(out.S), _ptr(out.I), _ptr(out.G),
                                 _ptr(out.row_ptr), _ptr(out.slots), _stream()), "ec_route_static")
    return out


def ec_moe_forward(cfg, X, Wg, W1, W2, X_out=None, saved=None, ws=None, forward_only=False, b1=None, b2=None):
    """Eq. 2-4.  Returns (X_out, saved); with forward_only nothing is kept for a backward pass (saved is None).
    b1 [E, d'], b2 [E, d]: the bias terms Eq. 3 leaves out (None = none)."""
    dev = X.device
    X_out = torch.empty(total_tokens(cfg), cfg.d_model, dtype=_torch_dtype(cfg), device=dev) if X_out is None else X_out
    if forward_only:
        nb = int(lib().ec_forward_only_workspace_bytes(C.byref(cfg)))
        if ws is None or ws.numel() < nb:
            ws = torch.empty(nb, dtype=torch.uint8, device=dev)
        _check(lib().ec_moe_forward(C.byref(cfg), _ptr(X), _ptr(Wg), _ptr(W1), _ptr(W2), _ptr(b1), _ptr(b2), _ptr(X_out),
                                    None, 0, _ptr(ws), ws.numel(), _stream()), "ec_moe_forward")
        return X_out, None
    saved = alloc_saved(cfg, dev) if saved is None else saved
    ws = alloc_workspace(cfg, dev) if ws is None else ws
    _check(lib().ec_moe_forward(C.byref(cfg), _ptr(X), _ptr(Wg), _ptr(W1), _ptr(W2), _ptr(b1), _ptr(b2), _ptr(X_out),
                                _ptr(saved), saved.numel(), _ptr(ws), ws.numel(), _stream()), "ec_moe_forward")
    return X_out, saved


def ec_moe_backward(cfg, X, Wg, W1, W2, dX_out, saved, grads=None, ws=None, bias_grads=None):
    """Backward of Eq. 2-4.  Returns (dX, dWg, dW1, dW2).  bias_grads = (db1 [E, d'], db2 [E, d]) are filled when given."""
    dev = X.device
    if grads is None:
        grads = (torch.empty_like(X), torch.empty_like(Wg), torch.empty_like(W1), torch.empty_like(W2))
    dX, dWg, dW1, dW2 = grads
    ws = alloc_workspace(cfg, dev) if ws is None else ws
    db1, db2 = bias_grads if bias_grads is not None else (None, None)
    _check(lib().ec_moe_backward(C.byref(cfg), _ptr(X), _ptr(Wg), _ptr(W1), _ptr(W2), _ptr(dX_out),
                                 _ptr(saved), saved.numel(), _ptr(dX), _ptr(dWg), _ptr(dW1), _ptr(dW2), _ptr(db1), _ptr(db2),
                                 _ptr(ws), ws.numel(), _stream()), "ec_moe_backward")
    return dX, dWg, dW1, dW2


def ec_read_status(ws) -> int:
    return int(lib().ec_read_status(_ptr(ws), _stream()))


def ec_launch_count() -> int:
    return int(lib().ec_launch_count())


def ec_profile_enable(on: bool) -> None:
    lib().ec_profile_enable(1 if on else 0)


def ec_profile_read(max_stages: int = 40):
    """[(stage name, milliseconds), ...] of the last profiled forward and backward calls."""
    ms = (C.c_float * max_stages)()
    names = (C.c_char_p * max_stages)()
    cnt = lib().ec_profile_read(ms, names, max_stages)
    if cnt < 0:
        raise EcError(EC_ERR_CUDA, "ec_profile_read")
    return [(names[i].decode(), float(ms[i])) for i in range(cnt)]


def backward_view(cfg, ws) -> dict:
    """Torch views of the backward pass's intermediates in the workspace (no copies; valid until the workspace is used again)."""
    v = ec_backward_ptrs()
    _check(lib().ec_backward_view(C.byref(cfg), _ptr(ws), C.byref(v)), "ec_backward_view")
    k, n, E, d, f = slots_per_expert(cfg), total_tokens(cfg), cfg.E, cfg.d_model, cfg.d_ff
    dt, es, base = _torch_dtype(cfg), (4 if cfg.dtype == EC_F32 else 2), ws.data_ptr()

    def view(addr, shape, dtype, esz):
        cnt = 1
        for s_ in shape:
            cnt *= s_
        return ws[addr - base:addr - base + cnt * esz].view(dtype).view(*shape)

    dl = (torch.bfloat16, 2) if v.dL_is_bf16 else (torch.float32, 4)
    return dict(dX_e=view(v.dX_e, (E, k, d), dt, es), dG=view(v.dG, (E, k), torch.float32, 4), dZ=view(v.dZ, (E, k, f), dt, es),
                dX_in=view(v.dX_in, (E, k, d), dt, es), dL=view(v.dL, (n, E), *dl))


def saved_view(cfg, saved) -> dict:
    """Torch views of the parts of the forward->backward blob (no copies)."""
    v = ec_saved_ptrs()
    _check(lib().ec_saved_view(C.byref(cfg), _ptr(saved), C.byref(v)), "ec_saved_view")
    k = slots_per_expert(cfg)
    base = saved.data_ptr()
    dt = _torch_dtype(cfg)
    es = 4 if cfg.dtype == EC_F32 else 2

    def view(addr, shape, dtype, esz):
        cnt = 1
        for s in shape:
            cnt *= s
        off = addr - base
        return saved[off:off + cnt * esz].view(dtype).view(*shape)

    n, E, d, f = total_tokens(cfg), cfg.E, cfg.d_model, cfg.d_ff
    extra = {}
    if cfg.router == EC_ROUTER_TOKEN_TOP2:
        extra = dict(load=view(v.load, (cfg.groups, E), torch.int32, 4),
                     requested=view(v.requested, (cfg.groups, E), torch.int32, 4))
    return dict(**extra, S=view(v.S, (n, E), torch.float32, 4), I=view(v.I, (E, k), torch.int32, 4),
                G=view(v.G, (E, k), torch.float32, 4), row_ptr=view(v.row_ptr, (n + 1,), torch.int32, 4),
                slots=view(v.slots, (E * k,), torch.int32, 4), X_in=view(v.X_in, (E, k, d), dt, es) if v.X_in else None,
                Z=view(v.Z, (E, k, f), dt, es), H=view(v.H, (E, k, f), dt, es),
                X_e=view(v.X_e, (E, k, d), torch.float32, 4))
