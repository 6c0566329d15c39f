"""Seeded synthetic inputs with the shapes and statistics of LLaMA linear layers.

This module only draws numbers and formats them (fp32 weights, bf16 bit
patterns for activations).  It holds none of the PEQA arithmetic, so both the
CUDA path and the CPU oracle can be fed the very same buffers from here.

Recipe (one ``numpy.random.Generator(PCG64(seed))`` per workload; for every
linear layer of the workload, in layer order, the draws are):
  1. W   = standard_normal(float32) * sigma_w                 [N, K]
  2. if outliers: mask = random() < 1e-3 ; W[mask] *= 20       (heavy-tail entries)
  3. X   = bf16(standard_normal(float32))                      [T, K]
  4. dY  = bf16(standard_normal(float32) * sigma_dy)           [T, N]   (training only)
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Iterator

import numpy as np


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (nearest, ties to even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bfloat16 bit patterns (uint16) to float32 exactly."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


@dataclass(frozen=True)
class LinearSpec:
    name: str
    N: int            # out_features
    K: int            # in_features
    T: int            # tokens (M for decode)
    bits: int
    group_size: int   # 0 = per-channel
    sigma_w: float
    outliers: bool
    sigma_dy: float   # 0.0 = forward-only workload (no dY drawn)


@dataclass(frozen=True)
class Workload:
    name: str
    seed: int
    layers: tuple


def _lin(name, N, K, T, bits, g, sw, out, sdy):
    return LinearSpec(name, N, K, T, bits, g, sw, out, sdy)


WORKLOADS = {
    # 4-bit per-channel toy layer
    "c1": Workload("c1", 0, (_lin("proj", 256, 256, 64, 4, 0, 0.02, False, 1.0),)),
    # LLaMA-7B attention projection, 3-bit, groups of 128 input columns
    "c2": Workload("c2", 0, (_lin("attn_proj", 4096, 4096, 2048, 3, 128, 0.02, True, 1e-2),)),
    # LLaMA-7B SwiGLU MLP, 4-bit per-channel
    "c3": Workload("c3", 1, (
        _lin("gate", 11008, 4096, 4096, 4, 0, 0.02, False, 1e-2),
        _lin("up", 11008, 4096, 4096, 4, 0, 0.02, False, 1e-2),
        _lin("down", 4096, 11008, 4096, 4, 0, 0.02, False, 1e-2),
    )),
    # LLaMA-65B decode shapes, 3-bit per-channel (M is chosen by the caller)
    "c4": Workload("c4", 0, (
        _lin("attn", 8192, 8192, 16, 3, 0, 0.015, False, 0.0),
        _lin("gate_up", 22016, 8192, 16, 3, 0, 0.015, False, 0.0),
        _lin("down", 8192, 22016, 16, 3, 0, 0.015, False, 0.0),
    )),
    # one LLaMA-65B decoder layer, 3-bit, groups of 64
    "c5": Workload("c5", 0, tuple(
        _lin(n, N, K, 4096, 3, 64, 0.015, True, 1e-2)
        for n, N, K in (("q", 8192, 8192), ("k", 8192, 8192), ("v", 8192, 8192), ("o", 8192, 8192),
                        ("gate", 22016, 8192), ("up", 22016, 8192), ("down", 8192, 22016))
    )),
}


def draw_weight(rng: np.random.Generator, N: int, K: int, sigma: float, outliers: bool) -> np.ndarray:
    W = rng.standard_normal((N, K), dtype=np.float32)
    W *= np.float32(sigma)
    if outliers:
        mask = rng.random((N, K), dtype=np.float32) < np.float32(1e-3)
        W[mask] *= np.float32(20.0)
    return W


def draw_act(rng: np.random.Generator, rows: int, cols: int, sigma: float) -> np.ndarray:
    a = rng.standard_normal((rows, cols), dtype=np.float32)
    if sigma != 1.0:
        a *= np.float32(sigma)
    return f32_to_bf16_bits(a)


def draw_layer(rng: np.random.Generator, spec: LinearSpec, T: int | None = None) -> dict:
    """One layer's buffers: W fp32 [N,K], X bf16 bits [T,K], dY bf16 bits [T,N] or None."""
    T = spec.T if T is None else T
    W = draw_weight(rng, spec.N, spec.K, spec.sigma_w, spec.outliers)
    X = draw_act(rng, T, spec.K, 1.0)
    dY = draw_act(rng, T, spec.N, spec.sigma_dy) if spec.sigma_dy > 0.0 else None
    return {"spec": spec, "W": W, "X": X, "dY": dY}


def generate(name: str, T: int | None = None) -> Iterator[dict]:
    """Yield the layers of a named workload in order, all from one seeded stream."""
    wl = WORKLOADS[name]
    rng = np.random.Generator(np.random.PCG64(wl.seed))
    for spec in wl.layers:
        yield draw_layer(rng, spec, T)


def custom(seed: int, N: int, K: int, T: int, bits: int, group_size: int = 0,
           sigma_w: float = 0.02, outliers: bool = False, sigma_dy: float = 1.0) -> dict:
    """A one-layer workload of arbitrary shape (tests use it for ragged and edge sizes)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    return draw_layer(rng, _lin("custom", N, K, T, bits, group_size, sigma_w, outliers, sigma_dy))
