"""Seeded synthetic inputs shaped like the paper's workloads.

This module holds none of the method's arithmetic: it only draws Gaussian
tensors with numpy's seeded generator and rounds them to bf16 bit patterns.
Both the CPU oracle's tests and the CUDA path's tests feed from it, so that the
two sides see identical bits.  Depends on numpy only.

Tensors are returned as numpy uint16 arrays holding bf16 bit patterns.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns, round to nearest even (finite inputs)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    return ((u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def gaussian_bf16(seed: int, shape, sigma: float) -> np.ndarray:
    rng = np.random.default_rng(seed)
    x = rng.standard_normal(size=shape, dtype=np.float32) * np.float32(sigma)
    return to_bf16_bits(x)


@dataclass(frozen=True)
class Layer:
    """One S-STE linear: W[O, I], activations X[T, I], output gradient dY[T, O]."""
    name: str
    O: int
    I: int
    T: int
    sigma_w: float = 0.02
    sigma_x: float = 1.0
    sigma_g: float = 1.0


# Shapes of the five benchmark configurations (Gaussian init, std as given).
CONFIGS = {
    # single small layer: the parity configuration
    1: dict(seed=0, fp8=False, layers=[Layer("linear", 256, 256, 512, 0.02, 1.0, 1.0)]),
    # GPT-2-small-shaped MLP, 8 x 1024 tokens
    2: dict(seed=2, fp8=False, layers=[Layer("fc1", 3072, 768, 8192, 0.02, 1.0, 1e-2),
                                       Layer("fc2", 768, 3072, 8192, 0.02, 1.0, 1e-2)]),
    # GPT-2-large-shaped block linears, 16 x 1024 tokens
    3: dict(seed=3, fp8=False, layers=[Layer("qkv", 3840, 1280, 16384, 0.02, 1.0, 1e-2),
                                       Layer("proj", 1280, 1280, 16384, 0.02, 1.0, 1e-2),
                                       Layer("fc1", 5120, 1280, 16384, 0.02, 1.0, 1e-2),
                                       Layer("fc2", 1280, 5120, 16384, 0.02, 1.0, 1e-2)]),
    # the four linear shapes of one GPT-2-124M block (12 identical blocks), 8 x 1024 tokens
    4: dict(seed=4, fp8=False, layers=[Layer("qkv", 2304, 768, 8192, 0.02, 1.0, 1e-2),
                                       Layer("proj", 768, 768, 8192, 0.02, 1.0, 1e-2),
                                       Layer("fc1", 3072, 768, 8192, 0.02, 1.0, 1e-2),
                                       Layer("fc2", 768, 3072, 8192, 0.02, 1.0, 1e-2)]),
    # FP8 whole-process variant, 7B-shaped FFN
    5: dict(seed=5, fp8=True, layers=[Layer("up", 11008, 4096, 16384, 0.02, 1.0, 1e-2),
                                      Layer("gate", 11008, 4096, 16384, 0.02, 1.0, 1e-2),
                                      Layer("down", 4096, 11008, 16384, 0.02, 1.0, 1e-2)]),
}


def layer_tensors(cfg: int, layer_index: int, T: int | None = None):
    """(W, X, dY) bf16 bit patterns for one layer of a configuration; T overrides the token count."""
    c = CONFIGS[cfg]
    L = c["layers"][layer_index]
    T = L.T if T is None else T
    base = c["seed"] * 1000 + 10 * layer_index
    W = gaussian_bf16(base + 0, (L.O, L.I), L.sigma_w)
    X = gaussian_bf16(base + 1, (T, L.I), L.sigma_x)
    dY = gaussian_bf16(base + 2, (T, L.O), L.sigma_g)
    return W, X, dY
