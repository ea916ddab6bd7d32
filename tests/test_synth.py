"""The seeded generator: deterministic, chunk-independent, correct bf16 rounding."""
import numpy as np
import torch

from paper_2310_12109_b200 import synth


def test_counter_based_and_deterministic():
    a = synth.uniform01(7, 1000)
    b = synth.uniform01(7, 400, offset=600)
    assert np.array_equal(a[600:], b)
    assert np.array_equal(a, synth.uniform01(7, 1000))
    assert not np.array_equal(a, synth.uniform01(8, 1000))
    assert a.min() > 0.0 and a.max() < 1.0


def test_normal_moments():
    z = synth.normal(3, (200000,))
    assert abs(z.mean()) < 0.01 and abs(z.std() - 1.0) < 0.01
    assert abs(np.mean(z ** 3)) < 0.03 and abs(np.mean(z ** 4) - 3.0) < 0.1


def test_bf16_rounding_matches_torch():
    z = synth.normal(5, (4096,)) * 3.0
    mine = synth.round_bf16(z)
    ref = torch.from_numpy(z.astype(np.float32)).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(mine, ref)
    bits = synth.bf16_bits(mine)
    assert np.array_equal(synth.from_bf16_bits(bits), mine)


def test_config_shapes():
    c1 = synth.config1()
    assert c1["x"].shape == (1, 4, 256) and c1["k"].shape == (4, 256)
    c2 = synth.config2(B=2, H=3)
    assert c2["x"].shape == (2, 3, 512) and np.array_equal(synth.round_bf16(c2["x"]), c2["x"])
    c3 = synth.config3(T=4, b=8)
    assert c3["X"].shape == (4, 64) and c3["L"].shape == (8, 8, 8)
    # kernel decays: late taps are small
    k = synth.decay_kernel(4, 2, 16384, 0.0005, 128.0)
    assert np.abs(k[:, -100:]).max() < np.abs(k[:, :100]).max()
