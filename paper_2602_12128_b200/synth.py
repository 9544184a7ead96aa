"""Seeded synthetic inputs shaped like the paper's video-DiT workloads.

This module holds no attention arithmetic: it only draws random tensors with the
shapes, scalings and seeds of the five benchmark configurations, so that the
CUDA library and the CPU oracle can be fed identical bytes.  The paper's own
workload is the self-attention of Wan2.1-1.3B on flattened video latents
(Section 5: 12 heads x 128 channels, 32760 or 12600 tokens); its datasets and
trained weights are not available, so every tensor here is a stand-in.

Seeds: 0 -> Q, K, V (drawn in that order), 1 -> phi weights, 2 -> upstream
gradient dO, 3 -> non-negative features for the feature-level entry point.
Values meant for a bf16 run are rounded to bf16 (round-to-nearest-even) and
returned as float32 arrays holding exactly those values.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


@dataclass(frozen=True)
class HlaShape:
    name: str
    B: int
    H: int
    N: int
    d: int
    dtype: str            # "f32" | "bf16"
    scale: str            # "inv_sqrt_d" | "rms_qk"
    backward: bool = False
    F: int = 3
    d_phi: int = 6
    causal: bool = False


# The five configurations of the benchmark definition.
CONFIGS = {
    "tiny_f32": HlaShape("tiny_f32", 1, 2, 256, 16, "f32", "inv_sqrt_d"),
    "small_bf16": HlaShape("small_bf16", 2, 12, 4096, 64, "bf16", "inv_sqrt_d"),
    "dit_bf16": HlaShape("dit_bf16", 1, 24, 32760, 128, "bf16", "rms_qk"),          # 21x39x40 latent grid
    "long_bf16": HlaShape("long_bf16", 1, 40, 75600, 128, "bf16", "inv_sqrt_d"),    # 21x60x60 latent grid
    "train_bf16": HlaShape("train_bf16", 2, 24, 32760, 128, "bf16", "inv_sqrt_d", backward=True),
}

# The paper's own two resolutions (Section 5: Wan2.1-1.3B has 12 heads of 128 channels; 81x480x832 video -> 32760
# tokens, 81x320x480 -> 12600 tokens), as extra workloads next to the five benchmark configurations.
CONFIGS["paper_r1_bf16"] = HlaShape("paper_r1_bf16", 1, 12, 32760, 128, "bf16", "rms_qk", backward=True)
CONFIGS["paper_r2_bf16"] = HlaShape("paper_r2_bf16", 1, 12, 12600, 128, "bf16", "rms_qk", backward=True)


# The paper's 2-factor variant (appendix "Defining phi": 12 feature channels for 2 factors; Table 2 row HLA-2F-R1-21) at the training-step shape.
CONFIGS["train_bf16_2f"] = HlaShape("train_bf16_2f", 2, 24, 32760, 128, "bf16", "inv_sqrt_d", backward=True, F=2, d_phi=12)

# Causal HLA (Section 4.4: token i sees the tokens j <= i) at the training-step shape.
CONFIGS["train_bf16_causal"] = HlaShape("train_bf16_causal", 2, 24, 32760, 128, "bf16", "inv_sqrt_d", backward=True, causal=True)


def bf16_round(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bfloat16 (ties to even); result stays float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    r = (u + bias) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Upper 16 bits of float32 values that are already exactly representable in bf16."""
    return (np.ascontiguousarray(x, dtype=np.float32).view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def from_bf16_bits(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def _finish(x: np.ndarray, dtype: str) -> np.ndarray:
    return bf16_round(x) if dtype == "bf16" else x.astype(np.float32)


def make_qkv(shape: HlaShape, seed: int = 0):
    """Q, K, V [B,H,N,d] float32 (bf16-exact when shape.dtype == 'bf16')."""
    rng = np.random.default_rng(seed)
    dims = (shape.B, shape.H, shape.N, shape.d)
    Q = rng.standard_normal(dims, dtype=np.float32)
    K = rng.standard_normal(dims, dtype=np.float32)
    V = rng.standard_normal(dims, dtype=np.float32)
    if shape.scale == "inv_sqrt_d":
        s = np.float32(1.0 / np.sqrt(shape.d))
        Q *= s
        K *= s
        V *= s
    elif shape.scale == "rms_qk":
        # each token's d-vector divided by its root-mean-square, per head; V stays N(0,1)
        Q /= np.sqrt(np.mean(Q * Q, axis=-1, keepdims=True))
        K /= np.sqrt(np.mean(K * K, axis=-1, keepdims=True))
    else:
        raise ValueError(shape.scale)
    return _finish(Q, shape.dtype), _finish(K, shape.dtype), _finish(V, shape.dtype)


def make_dO(shape: HlaShape, seed: int = 2) -> np.ndarray:
    rng = np.random.default_rng(seed)
    dO = rng.standard_normal((shape.B, shape.H, shape.N, shape.d), dtype=np.float32)
    return _finish(dO, shape.dtype)


def make_phi_weights(d: int, d_phi: int, F: int, dtype: str, seed: int = 1):
    """One weight set per map (phi_q, phi_k1..phi_kF): W1 [d,d], b1 [d], W2 [d,d_phi], b2 [d_phi].
    W1, W2 ~ N(0, 1/d); biases small but non-zero so that a dropped bias is visible.
    Returns (phi_q, [phi_k1, ...]) as tuples of float32 arrays (bf16-exact for dtype 'bf16')."""
    rng = np.random.default_rng(seed)
    maps = []
    for _ in range(1 + F):
        W1 = rng.standard_normal((d, d), dtype=np.float32) / np.float32(np.sqrt(d))
        b1 = rng.standard_normal((d,), dtype=np.float32) * np.float32(0.1)
        W2 = rng.standard_normal((d, d_phi), dtype=np.float32) / np.float32(np.sqrt(d))
        b2 = rng.standard_normal((d_phi,), dtype=np.float32) * np.float32(0.1)
        maps.append(tuple(_finish(a, dtype) for a in (W1, b1, W2, b2)))
    return maps[0], maps[1:]


def make_features(shape: HlaShape, seed: int = 3):
    """Non-negative features for the feature-level entry point:
    qf [B,H,N,d_phi], kf [B,H,F,N,d_phi] = |N(0,1)| / sqrt(d_phi), float32."""
    rng = np.random.default_rng(seed)
    s = np.float32(1.0 / np.sqrt(shape.d_phi))
    qf = np.abs(rng.standard_normal((shape.B, shape.H, shape.N, shape.d_phi), dtype=np.float32)) * s
    kf = np.abs(rng.standard_normal((shape.B, shape.H, shape.F, shape.N, shape.d_phi), dtype=np.float32)) * s
    return qf, kf
