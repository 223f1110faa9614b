"""Seeded synthetic inputs for the expert-choice MoE layer.

This module serves both the CUDA path and the CPU oracle and therefore holds
none of the layer's arithmetic: it only draws tensors.  Values come from a
counter-based generator (a 64-bit mixing hash of seed, tensor id and element
index, then Box-Muller), so any slice of any tensor can be regenerated without
state, on the host or on a GPU, chunk by chunk.

Shapes follow the paper's notation (Section 3.2): X [n, d], Wg [d, E],
W1, W2 [E, d, d'] and the upstream gradient dX_out [n, d].  Distributions:
X ~ N(0, 1), Wg ~ N(0, 1/d), W1 ~ N(0, 1/d), W2 ~ N(0, 1/d') (W2 is applied
transposed, so its fan-in is d'), dX_out ~ N(0, 1).  Every tensor is rounded
once to the path's storage type (fp32 or bf16) here; both sides then see the
same bits.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import torch

# tensor ids mixed into the counter
TID_X, TID_WG, TID_W1, TID_W2, TID_DXOUT, TID_AUX = 1, 2, 3, 4, 5, 6

_M1 = -0x61C8864680B583EB          # 0x9E3779B97F4A7C15 as a signed 64-bit value
_M2 = -0x40A7B892E31B1A47          # 0xBF58476D1CE4E5B9
_M3 = -0x6B2FB644ECCEEE15          # 0x94D049BB133111EB


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical shift right of int64 bit patterns."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix64(z: torch.Tensor) -> torch.Tensor:
    """splitmix64 finaliser on int64 tensors (wrapping arithmetic)."""
    z = z + _M1
    z = (z ^ _lsr(z, 30)) * _M2
    z = (z ^ _lsr(z, 27)) * _M3
    return z ^ _lsr(z, 31)


def normal_chunk(seed: int, tid: int, start: int, count: int, device="cpu") -> torch.Tensor:
    """`count` standard normal fp32 values for elements [start, start+count) of tensor `tid`."""
    idx = torch.arange(start, start + count, dtype=torch.int64, device=device)
    key = ((seed & 0xFFFFFF) << 40) ^ (tid << 56)
    h = _mix64(idx ^ key)
    h2 = _mix64(h ^ 0x5851F42D4C957F2D)
    u1 = (_lsr(h, 40).to(torch.float32) + 1.0) * (1.0 / 16777216.0)   # (0, 1]
    u2 = _lsr(h2, 40).to(torch.float32) * (1.0 / 16777216.0)           # [0, 1)
    r = torch.sqrt(-2.0 * torch.log(u1))
    return r * torch.cos((2.0 * math.pi) * u2)


def normal_tensor(shape, std: float, seed: int, tid: int, dtype=torch.float32,
                  device="cpu", chunk: int = 1 << 24) -> torch.Tensor:
    """A tensor of N(0, std^2) values rounded once to `dtype`, generated chunk by chunk."""
    total = 1
    for s in shape:
        total *= int(s)
    out = torch.empty(total, dtype=dtype, device=device)
    for start in range(0, total, chunk):
        cnt = min(chunk, total - start)
        out[start:start + cnt] = (normal_chunk(seed, tid, start, cnt, device) * std).to(dtype)
    return out.view(*shape)


@dataclass
class LayerInputs:
    X: torch.Tensor
    Wg: torch.Tensor
    W1: torch.Tensor
    W2: torch.Tensor
    dX_out: torch.Tensor


def make_layer_inputs(n: int, d: int, dff: int, E: int, dtype=torch.float32, seed: int = 0,
                      logit_scale: float = 1.0, device="cpu", with_grad: bool = True,
                      expert_skew: float = 0.0) -> LayerInputs:
    """Inputs of one layer call.  `logit_scale` multiplies Wg (varies the token-score skew).

    `expert_skew` > 0 makes some experts popular with every token, the way a trained gate without a balancing
    loss does: feature 0 of every token is set to 1 and row 0 of Wg to expert_skew * z_i with z ~ N(0, 1), which
    adds the same logit offset z_i * expert_skew to expert i for all tokens (the layer has no bias term to carry it).
    """
    X = normal_tensor((n, d), 1.0, seed, TID_X, dtype, device)
    Wg = normal_tensor((d, E), logit_scale / math.sqrt(d), seed, TID_WG, dtype, device)
    if expert_skew:
        X[:, 0] = 1.0
        Wg[0, :] = (normal_chunk(seed, TID_AUX, 1 << 20, E, device) * expert_skew).to(dtype)
    W1 = normal_tensor((E, d, dff), 1.0 / math.sqrt(d), seed, TID_W1, dtype, device)
    W2 = normal_tensor((E, d, dff), 1.0 / math.sqrt(dff), seed, TID_W2, dtype, device)
    dX_out = normal_tensor((n, d), 1.0, seed, TID_DXOUT, dtype, device) if with_grad else None
    return LayerInputs(X, Wg, W1, W2, dX_out)


def quantised_gate_inputs(n: int, d: int, E: int, levels: int, dtype=torch.float32, seed: int = 0):
    """X and Wg whose logits take only a few distinct values, so columns of S hold many exact ties.

    X has one non-zero entry per row (value 1 in column t mod d) and Wg holds small
    integers divided by 4, so X.Wg is exact in any floating type.
    """
    X = torch.zeros(n, d, dtype=torch.float32)
    X[torch.arange(n), torch.arange(n) % d] = 1.0
    raw = normal_chunk(seed, TID_AUX, 0, d * E)
    Wg = torch.round(raw * levels).clamp(-levels, levels).view(d, E) / 4.0
    return X.to(dtype), Wg.to(dtype)
