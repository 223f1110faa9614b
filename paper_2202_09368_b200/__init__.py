"""Expert-choice MoE feed-forward layer for NVIDIA B200 (sm_100a).

The layer lives in a C-ABI shared library built from csrc/ (see include/ecmoe.h);
`paper_2202_09368_b200.binding` marshals torch device tensors into it.  The
library is loaded on first use and its absence is an error: there is no CPU or
eager fallback.  `paper_2202_09368_b200.inputs` draws the seeded synthetic inputs.
"""
__all__ = ["binding", "inputs"]
