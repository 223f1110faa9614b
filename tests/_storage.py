"""Which tensors the bf16 path of the layer keeps in bf16, and the rounding itself (numpy only).

Used by the GPU parity tests (to evaluate, on the CPU, how far bf16 storage alone moves each output: the
arithmetic floor of that path) and by tests/golden/make_store_floor.py.  X_in is a copy of bf16 inputs, so
rounding it changes nothing; S, G, X_e, dG, dS, dH are fp32 or never stored on that path and are left alone.
"""
import numpy as np

BF16_STORED = frozenset({"Z", "H", "X_out", "dX_e", "dZ", "dX_in", "dL", "dX", "dWg", "dW1", "dW2", "db1", "db2"})


def round_bf16(x):
    """Round-to-nearest-even to bfloat16 (through float32, as a device that accumulates in fp32 does), returned as float64."""
    u = np.ascontiguousarray(x, np.float32).view(np.uint32)
    u = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return u.view(np.float32).astype(np.float64)


def bf16_store(name, x):
    """`store=` hook for oracle.forward / oracle.backward: the tensors of BF16_STORED are rounded where they are kept."""
    return round_bf16(x) if name in BF16_STORED else x


def half_ulp_bf16(x):
    """Half the spacing of bfloat16 numbers around x (8 significand bits): the most one rounding can move x."""
    _, e = np.frexp(np.asarray(x, np.float64))
    return np.ldexp(1.0, e - 9)


class Bf16Recorder:
    """`store=` hook like bf16_store that also keeps what every rounded tensor was BEFORE it was rounded
    (per-expert tensors in call order), so a test can tell apart the two things bf16 storage does to an output:
    the error its operands carried in (pre - reference) and its own final rounding (at most half_ulp_bf16(pre))."""

    def __init__(self):
        self.pre = {}

    def __call__(self, name, x):
        if name not in BF16_STORED:
            return x
        self.pre.setdefault(name, []).append(np.array(x, np.float64))
        return round_bf16(x)

    def before(self, name, like):
        """The unrounded version of tensor `name`, shaped like `like` (the stack over experts where it is per expert)."""
        got = self.pre[name]
        return got[0] if len(got) == 1 and got[0].shape == like.shape else np.stack(got)
