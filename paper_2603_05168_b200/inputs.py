"""Seeded synthetic inputs for the Sparse-BitLinear path.

This module holds input generators only -- none of the method's arithmetic.  Everything is drawn
on the host with numpy's PCG64 generator and handed, as the same arrays, to whichever
implementation is being exercised, so no random-number generator has to match across
implementations.

Shapes and distributions follow the workloads the layer is measured on:
  * latent weights  W ~ N(0, sigma^2), fp32, [N][K]  (optionally with heavy-tail outliers)
  * activations     x ~ N(0, 1) rounded to bf16 (round-to-nearest-even), [T][K], optionally with a
                    per-token LogNormal scale
"""
from __future__ import annotations

import numpy as np

# (name, K = d_in, N = d_out) of the BitNet-2B-shaped BitLinears (hidden 2560, FFN 6912,
# 20 query heads / 5 kv heads of dim 128; the QKV projection is one fused matrix).
SHAPES_2B = [
    ("qkv", 2560, 3840),
    ("o", 2560, 2560),
    ("gate_up", 2560, 6912),
    ("down", 6912, 2560),
]

# 7B-class shapes (hidden 4096, FFN 11008).
SHAPES_7B = [
    ("gate_up_7b", 4096, 11008),
    ("down_7b", 11008, 4096),
]

# The seven BitLinears of one 2B-shaped transformer layer when every projection is its own tensor.
LAYER_2B = [
    ("q", 2560, 2560),
    ("k", 2560, 640),
    ("v", 2560, 640),
    ("o", 2560, 2560),
    ("gate", 2560, 6912),
    ("up", 2560, 6912),
    ("down", 6912, 2560),
]


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest-even) and return the 16-bit patterns (finite inputs)."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = u + np.uint32(0x7FFF) + lsb
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def latent_weights(N: int, K: int, seed: int, sigma: float = 0.02,
                   outlier_prob: float = 0.0, outlier_mult: float = 10.0) -> np.ndarray:
    """fp32 [N][K] ~ N(0, sigma^2); each entry independently multiplied by outlier_mult with
    probability outlier_prob."""
    rng = np.random.default_rng(seed)
    W = rng.standard_normal((N, K), dtype=np.float32) * np.float32(sigma)
    if outlier_prob > 0.0:
        hit = rng.random((N, K), dtype=np.float32) < np.float32(outlier_prob)
        W = np.where(hit, W * np.float32(outlier_mult), W).astype(np.float32)
    return np.ascontiguousarray(W)


def activations_bf16(T: int, K: int, seed: int, token_lognormal_sigma: float = 0.0) -> np.ndarray:
    """bf16 bit patterns [T][K] of x ~ N(0,1), optionally times exp(sigma * N(0,1)) per token."""
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((T, K), dtype=np.float32)
    if token_lognormal_sigma > 0.0:
        s = np.exp(np.float32(token_lognormal_sigma) * rng.standard_normal((T, 1), dtype=np.float32))
        x = (x * s).astype(np.float32)
    return f32_to_bf16_bits(x)


def perturb_weights(W: np.ndarray, seed: int, sigma: float = 1e-4) -> np.ndarray:
    """W + N(0, sigma^2): one synthetic optimiser step for the dynamic-mask workload."""
    rng = np.random.default_rng(seed)
    return (W + rng.standard_normal(W.shape, dtype=np.float32) * np.float32(sigma)).astype(np.float32)


def sample_positions(T: int, N: int, count: int, seed: int):
    """Random (t, n) output positions for sampled parity checks on full-size shapes."""
    rng = np.random.default_rng(seed)
    return (rng.integers(0, T, size=count, dtype=np.int64),
            rng.integers(0, N, size=count, dtype=np.int64))
