"""Seeded synthetic inputs shared by the tests, the bench and the CPU oracle's callers.

This module holds no arithmetic of the method (no scales, no rounding to FP4, no random draws the method
makes): it only produces BF16-representable tensors with the shapes and value distributions of the paper's
LLaMA/OLMo-style linear layers (activations ~N(0,1) with a few outlier channels scaled up, weights ~N(0,0.02),
output gradients heavy-tailed Student-t), which stand in for the paper's real training tensors.

Everything is numpy on the host: ``default_rng(seed)``, float32 -> bfloat16 by round-to-nearest-even.
A tensor is returned as float32 (holding exactly BF16-representable values); ``to_bf16_bits`` gives the
uint16 bit patterns to upload.
"""
from __future__ import annotations

import numpy as np


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """float32 -> nearest bfloat16 (ties to even), returned as float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    bias = ((u >> 16) & 1) + np.uint32(0x7FFF)
    r = ((u + bias) >> 16).astype(np.uint32) << 16
    return r.view(np.float32).reshape(x.shape)


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """BF16-representable float32 -> uint16 bit patterns (exact)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    return (x.view(np.uint32) >> 16).astype(np.uint16).reshape(x.shape)


def from_bf16_bits(b: np.ndarray) -> np.ndarray:
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << 16).view(np.float32).reshape(b.shape)


def seed_of(config: int, tensor_id: int) -> int:
    """Seeds are 1000 * config + tensor id (X=1, W=2, dY=3, gate=4, up=5, more weights 10+)."""
    return 1000 * config + tensor_id


def outlier_channels(K: int, n: int, seed: int) -> np.ndarray:
    rng = np.random.default_rng(seed + 500)
    return np.sort(rng.choice(K, size=n, replace=False)).astype(np.int64)


def activations(rows: int, cols: int, seed: int, n_outlier: int = 0, factor: float = 1.0, channel_seed: int | None = None):
    """~N(0,1) with ``n_outlier`` channels multiplied by ``factor``. Returns (tensor, sorted channel list).
    ``channel_seed`` fixes the channel choice independently of the values (the same channels over several steps)."""
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((rows, cols), dtype=np.float32)
    ch = outlier_channels(cols, n_outlier, seed if channel_seed is None else channel_seed) if n_outlier else np.zeros(0, dtype=np.int64)
    if n_outlier:
        x[:, ch] *= np.float32(factor)
    return round_to_bf16(x), ch


def swiglu_activations(rows: int, cols: int, seed_gate: int, seed_up: int, n_outlier: int = 0, factor: float = 1.0):
    """silu(g) * u with g, u ~N(0,1): the input of a SwiGLU down projection."""
    g = np.random.default_rng(seed_gate).standard_normal((rows, cols), dtype=np.float32)
    u = np.random.default_rng(seed_up).standard_normal((rows, cols), dtype=np.float32)
    x = (g / (1.0 + np.exp(-g))) * u
    ch = outlier_channels(cols, n_outlier, seed_gate) if n_outlier else np.zeros(0, dtype=np.int64)
    if n_outlier:
        x[:, ch] *= np.float32(factor)
    return round_to_bf16(x.astype(np.float32)), ch


def weights(rows: int, cols: int, seed: int, std: float = 0.02) -> np.ndarray:
    rng = np.random.default_rng(seed)
    return round_to_bf16(rng.standard_normal((rows, cols), dtype=np.float32) * np.float32(std))


def gradients(rows: int, cols: int, seed: int, scale: float = 1e-3, df: float = 3.0) -> np.ndarray:
    """Heavy-tailed output gradients: Student-t(df) * scale."""
    rng = np.random.default_rng(seed)
    return round_to_bf16((rng.standard_t(df, size=(rows, cols)) * scale).astype(np.float32))


# ---------------------------------------------------------------------------------------------------------
# The benchmark configurations (shapes only; tensors are drawn by the functions above).
# A linear is (name, D_in, C_out).
# ---------------------------------------------------------------------------------------------------------
CONFIGS = {
    1: dict(tokens=256, linears=[("single", 512, 512)], n_outlier=4, factor=50.0, grad_scale=1e-3),
    2: dict(tokens=8192, linears=[("qkv", 1024, 3072), ("o", 1024, 1024)], n_outlier=10, factor=30.0, grad_scale=1e-4),
    3: dict(tokens=8192, linears=[("gate", 1024, 2816), ("up", 1024, 2816), ("down", 2816, 1024)], n_outlier=10,
            factor=30.0, grad_scale=1e-4),
    4: dict(tokens=16384, layers=24,
            linears=[("qkv", 1024, 3072), ("o", 1024, 1024), ("gate", 1024, 2816), ("up", 1024, 2816),
                     ("down", 2816, 1024)], n_outlier=10, factor=30.0, grad_scale=1e-4),
    5: dict(shapes=[(M, N, K) for M in (4096, 16384) for (N, K) in ((4096, 4096), (8192, 8192), (14336, 4096))],
            outlier_frac=0.005, factor=100.0),
}


def layer_inputs(config: int, tokens: int, D: int, C: int, *, n_outlier: int, factor: float, grad_scale: float,
                 weight_id: int = 2, swiglu: bool = False):
    """X [tokens, D], W [C, D], dY [tokens, C] and the planted outlier channel list of one linear layer."""
    if swiglu:
        X, ch = swiglu_activations(tokens, D, seed_of(config, 4), seed_of(config, 5), n_outlier, factor)
    else:
        X, ch = activations(tokens, D, seed_of(config, 1), n_outlier, factor)
    W = weights(C, D, seed_of(config, weight_id))
    dY = gradients(tokens, C, seed_of(config, 3) + 7 * C, grad_scale)
    return X, W, dY, ch


def weight_trajectory(C: int, D: int, steps: int, seed: int, std: float = 0.02, step_scale: float = 2e-3, osc_fraction: float = 0.02):
    """FP32 master weights over ``steps + 1`` optimizer steps, as a list of [C, D] float32 arrays.

    Start ~N(0, std). Every step adds small Gaussian noise (step_scale * std). A planted ``osc_fraction`` of the
    elements additionally alternates by +-1.5 % of its own magnitude from step to step (late-training oscillation:
    the master weight moves little, its quantized value may flip between two bins). Returns (list, planted mask)."""
    rng = np.random.default_rng(seed)
    w = (rng.standard_normal((C, D), dtype=np.float32) * np.float32(std)).astype(np.float32)
    planted = rng.random((C, D)) < osc_fraction
    amp = (np.float32(0.015) * np.abs(w)).astype(np.float32)
    out = [w.copy()]
    for t in range(1, steps + 1):
        w = w + rng.standard_normal((C, D), dtype=np.float32) * np.float32(step_scale * std)
        sign = np.float32(1.0 if t % 2 else -1.0)
        w = np.where(planted, w + sign * amp, w).astype(np.float32)
        out.append(w.copy())
    return out, planted
