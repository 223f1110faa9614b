"""The seeded input generator: stateless, chunk-invariant, right distributions."""
import math

import torch

from paper_2202_09368_b200 import inputs as IN


def test_chunks_agree_with_whole_tensor():
    whole = IN.normal_tensor((1000,), 1.0, 0, IN.TID_X)
    part = IN.normal_chunk(0, IN.TID_X, 137, 50)
    assert torch.equal(whole[137:187], part)
    again = IN.normal_tensor((1000,), 1.0, 0, IN.TID_X, chunk=64)
    assert torch.equal(whole, again)


def test_seed_and_tensor_id_change_the_stream():
    a = IN.normal_tensor((256,), 1.0, 0, IN.TID_X)
    assert not torch.equal(a, IN.normal_tensor((256,), 1.0, 1, IN.TID_X))
    assert not torch.equal(a, IN.normal_tensor((256,), 1.0, 0, IN.TID_WG))


def test_moments_and_fan_in_scaling():
    li = IN.make_layer_inputs(512, 64, 128, 4)
    assert abs(li.X.mean()) < 0.02 and abs(li.X.std() - 1) < 0.02
    assert abs(li.Wg.std() * math.sqrt(64) - 1) < 0.1
    assert abs(li.W1.std() * math.sqrt(64) - 1) < 0.02
    assert abs(li.W2.std() * math.sqrt(128) - 1) < 0.02
    assert li.W1.shape == (4, 64, 128) and li.W2.shape == (4, 64, 128)
    assert torch.isfinite(li.X).all()


def test_bf16_inputs_are_rounded_once():
    a = IN.normal_tensor((300,), 1.0, 0, IN.TID_X, torch.bfloat16)
    b = IN.normal_tensor((300,), 1.0, 0, IN.TID_X, torch.float32)
    assert torch.equal(a, b.to(torch.bfloat16))


def test_quantised_gate_inputs_make_ties():
    X, Wg = IN.quantised_gate_inputs(64, 8, 4, 2)
    L = X @ Wg
    assert L.unique().numel() <= 5
