"""Seeded synthetic inputs shared by the CPU oracle's tests and the CUDA path's tests/bench.

This module holds no arithmetic of the method: it only draws random numbers, scales
them, and rounds them to the storage dtype, so that both sides see identical values.
Recipes follow the benchmark configurations: Q, K, V i.i.d. N(0,1)/sqrt(64); mixer input
X ~ N(0,1); short taps N(0, 1/width) (variance); long kernel N(0,1) * exp(-0.001 t);
dense projection weights N(0, 1/D) (variance).
"""
from __future__ import annotations

import numpy as np


def round_bf16(a: np.ndarray) -> np.ndarray:
    """Round float values to the nearest bfloat16 (ties to even); returns float32 holding bf16 values."""
    f = np.ascontiguousarray(a, dtype=np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(f.shape)


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of values that are already bf16-representable."""
    f = np.ascontiguousarray(a, dtype=np.float32)
    return (f.view(np.uint32) >> 16).astype(np.uint16).reshape(f.shape)


def round_storage(a: np.ndarray, dtype: str) -> np.ndarray:
    """Round to the storage dtype ('bf16' or 'f32'); result is float32."""
    if dtype == "bf16":
        return round_bf16(a)
    if dtype == "f32":
        return np.ascontiguousarray(a, dtype=np.float32)
    raise ValueError(dtype)


def qkv(seed: int, B: int, L: int, H: int, d_k: int, d_v: int, dtype: str, std: float = 0.125):
    """Q, K [B,L,H,d_k] and V [B,L,H,d_v], i.i.d. N(0,1)*std, rounded to ``dtype``."""
    rng = np.random.default_rng(seed)
    q = rng.standard_normal((B, L, H, d_k), dtype=np.float32) * np.float32(std)
    k = rng.standard_normal((B, L, H, d_k), dtype=np.float32) * np.float32(std)
    v = rng.standard_normal((B, L, H, d_v), dtype=np.float32) * np.float32(std)
    return round_storage(q, dtype), round_storage(k, dtype), round_storage(v, dtype)


def mixer(seed: int, B: int, L: int, D: int, width: int = 3, dtype: str = "bf16", decay: float = 0.001):
    """Mixer inputs in generation order X, w_short, k_long, W_q, W_k, W_v.

    X and the dense weights are rounded to ``dtype``; the convolution kernels stay float32.
    """
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((B, L, D), dtype=np.float32)
    w_short = rng.standard_normal((D, width), dtype=np.float32) * np.float32(1.0 / np.sqrt(width))
    t = np.arange(L, dtype=np.float64)
    k_long = (rng.standard_normal((D, L), dtype=np.float32).astype(np.float64)
              * np.exp(-decay * t)[None, :]).astype(np.float32)
    s = np.float32(1.0 / np.sqrt(D))
    w_q = rng.standard_normal((D, D), dtype=np.float32) * s
    w_k = rng.standard_normal((D, D), dtype=np.float32) * s
    w_v = rng.standard_normal((D, D), dtype=np.float32) * s
    return dict(x=round_storage(x, dtype), w_short=w_short, k_long=k_long,
                w_q=round_storage(w_q, dtype), w_k=round_storage(w_k, dtype),
                w_v=round_storage(w_v, dtype))


def sweep_shapes(total_tokens: int = 262144, lengths=(1024, 2048, 4096, 8192, 16384, 32768, 65536)):
    """(B, L) pairs of the sequence-length sweep with B*L fixed."""
    return [(total_tokens // L, L) for L in lengths]
