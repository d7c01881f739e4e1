"""The seeded input generator: bf16 rounding, determinism, the gap guard and the skewed-routing recipe."""
import numpy as np
import torch

from paper_2608_00916_b200 import synth


def test_bf16_rounding_matches_torch():
    rng = np.random.default_rng(0)
    a = np.concatenate([rng.standard_normal(100000).astype(np.float32) * 3,
                        np.array([0.0, -0.0, 1.0, 1.00390625, 1.0039062, 1.01171875, 3.3895314e38, 1e-40], np.float32)])
    want = torch.from_numpy(a).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = synth.f32_to_bf16_bits(a)
    assert np.array_equal(got, want)
    back = synth.bf16_bits_to_f32(got)
    assert np.array_equal(back, torch.from_numpy(a).to(torch.bfloat16).float().numpy())


def test_deterministic_and_thread_independent():
    a = synth.normal_bf16(7, "W_gate", (16, 512, 1024), 0.02, threads=1)
    b = synth.normal_bf16(7, "W_gate", (16, 512, 1024), 0.02, threads=8)
    assert np.array_equal(a, b)
    c = synth.normal_bf16(8, "W_gate", (16, 512, 1024), 0.02, threads=8)
    assert not np.array_equal(a, c)
    v = synth.bf16_bits_to_f32(a)
    assert abs(v.std() - 0.02) < 2e-4 and abs(v.mean()) < 1e-4


def test_tiny_config_shapes_and_guard():
    inp = synth.make_config("tiny")
    assert inp["x"].shape == (256, 256) and inp["W_r"].shape == (256, 8)
    assert inp["W_gate"].shape == (8, 256, 512) and inp["W_down"].shape == (8, 512, 256)
    l = synth._guard_logits(inp["x"], inp["W_r"], inp["b_r"])
    assert not synth._gap_violations(l, 2).any()
    h = np.array(inp["meta"]["histogram"])
    assert h.sum() == 256 * 2


def test_skew_recipe_on_reduced_shape():
    shape = synth.MoEShape(4096, 256, 128, 8, 64)
    inp = synth.make_inputs(shape, 1002, x_std=1.0, skew=True)
    h = np.array(inp["meta"]["histogram"])
    assert h.sum() == 4096 * 8
    assert (h == 0).sum() >= 3 and h.max() >= 10 * h.mean()
    l = synth._guard_logits(inp["x"], inp["W_r"], inp["b_r"])
    assert not synth._gap_violations(l, 8).any()
