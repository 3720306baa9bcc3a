"""The seeded input generator: determinism, formats, and bf16 rounding against torch's."""
import numpy as np
import torch

from paper_2601_05732_b200 import synth


def test_streams_are_deterministic_and_distinct():
    a = synth.normal(3, 0, (4, 5)); b = synth.normal(3, 0, (4, 5)); c = synth.normal(3, 1, (4, 5))
    assert (a == b).all() and not (a == c).any()
    big = synth.normal(0, 0, (200000,))
    assert abs(big.mean()) < 0.01 and abs(big.std() - 1) < 0.01


def test_bf16_rounding_matches_torch():
    v = synth.normal(1, 2, (100000,)).astype(np.float32)
    v = np.concatenate([v, np.float32([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.0e38, 1e-40])])
    ours = synth.to_bf16_bits(v)
    ref = torch.from_numpy(v).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert (ours == ref).all()
    back = synth.bf16_bits_to_f32(ours)
    assert (back == torch.from_numpy(v).to(torch.bfloat16).float().numpy()).all()
    # direct rounding of fp64 (no double rounding through fp32)
    x = np.float64(1.0) + 2.0 ** -8 + 2.0 ** -40
    assert synth.bf16_bits_to_f64(synth.to_bf16_bits(np.array([x])))[0] == 1.0 + 2.0 ** -7


def test_layer_inputs_shapes_and_sharding():
    L = synth.make_layer_inputs(4, 16, 8, seed=1, bias_std=0.1)
    assert L["x"].shape == (8, 4, 16) and L["x"].dtype == np.uint16
    assert L["W"].shape == (64, 32) and L["W"].dtype == np.float32 and L["b"].shape == (32,)
    assert L["alpha"].tolist() == [np.float32(0.01)] * 3 and (L["gain"] == 1).all()
    L1 = synth.make_layer_inputs(4, 16, 8, seed=1, bias_std=0.1, shard=1)
    assert (L1["W"] == L["W"]).all() and not (L1["x"] == L["x"]).all()
    S = synth.make_layer_inputs(4, 16, 8, seed=1, kind="sk")
    assert S["W"].shape == (64, 24)
    b = synth.paper_init_bias(4)
    assert b[0] == 0 and (b[1:24] == -8).all() and b[24] == 1 and b[25] == -1
    for w in synth.WORKLOADS.values():
        assert w.C % 8 == 0 and 2 <= w.n <= 5
