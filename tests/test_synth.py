"""Input generators: determinism, shapes, scalings and bf16 rounding."""
import numpy as np
import torch

from paper_2602_12128_b200 import synth


def test_bf16_round_matches_torch():
    x = np.random.default_rng(0).standard_normal(10000).astype(np.float32) * 3
    want = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    np.testing.assert_array_equal(synth.bf16_round(x), want)
    bits = synth.to_bf16_bits(synth.bf16_round(x))
    np.testing.assert_array_equal(synth.from_bf16_bits(bits), want)


def test_configs_shapes_and_scaling():
    c = synth.CONFIGS
    assert (c["dit_bf16"].B, c["dit_bf16"].H, c["dit_bf16"].N, c["dit_bf16"].d) == (1, 24, 21 * 39 * 40, 128)
    assert (c["long_bf16"].H, c["long_bf16"].N) == (40, 21 * 60 * 60)
    assert c["train_bf16"].backward and c["train_bf16"].B == 2
    small = synth.HlaShape("t", 1, 2, 64, 128, "bf16", "rms_qk")
    Q, K, V = synth.make_qkv(small)
    Q2, _, _ = synth.make_qkv(small)
    np.testing.assert_array_equal(Q, Q2)
    assert abs(np.sqrt(np.mean(Q.astype(np.float64) ** 2, axis=-1)).mean() - 1.0) < 5e-3
    assert abs(V.std() - 1.0) < 0.05
    np.testing.assert_array_equal(synth.bf16_round(Q), Q)
    t = synth.HlaShape("t", 1, 1, 4096, 16, "f32", "inv_sqrt_d")
    Q, K, V = synth.make_qkv(t)
    assert abs(Q.std() * 4 - 1.0) < 0.05


def test_weights_and_features():
    pq, pk = synth.make_phi_weights(16, 6, 3, "f32")
    assert len(pk) == 3 and pq[0].shape == (16, 16) and pq[2].shape == (16, 6) and pq[3].shape == (6,)
    qf, kf = synth.make_features(synth.HlaShape("t", 1, 2, 10, 16, "f32", "inv_sqrt_d"))
    assert qf.shape == (1, 2, 10, 6) and kf.shape == (1, 2, 3, 10, 6) and qf.min() >= 0 and kf.min() >= 0
