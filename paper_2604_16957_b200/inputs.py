"""Seeded synthetic inputs with the shapes and value distributions of the benchmark configs.

This module holds none of the method's arithmetic: it only draws fp16 tensors.  It is the one
piece of code that both the CUDA path's callers and the CPU oracle's callers use, so that both
see bit-identical inputs.

Config names:
  tiny          B=1, H_q=4,  H_kv=1,  d=64,  alpha=1/8        (context 256, then one appended token)
  llama         B=1, H_q=64, H_kv=8,  d=128, alpha=128**-0.5  (K has 4 seeded outlier channels x10 per KV head)
  gemma         B=1, H_q=32, H_kv=16, d=256, alpha=1.0        (q, k ~ N(0, sigma^2 = d**-0.5) so that q.k ~ N(0,1))
  ragged        B=16, llama heads, per-sequence lengths uniform in [4096, 65536]
"""
from dataclasses import dataclass

import numpy as np


@dataclass(frozen=True)
class Shape:
    name: str
    B: int
    H_q: int
    H_kv: int
    d: int
    alpha: float
    sigma_qk: float = 1.0
    k_outlier_channels: int = 0
    k_outlier_scale: float = 10.0


TINY = Shape("tiny", 1, 4, 1, 64, 64 ** -0.5)
LLAMA = Shape("llama", 1, 64, 8, 128, 128 ** -0.5, k_outlier_channels=4)
GEMMA = Shape("gemma", 1, 32, 16, 256, 1.0, sigma_qk=256 ** -0.25)
RAGGED = Shape("ragged", 16, 64, 8, 128, 128 ** -0.5, k_outlier_channels=4)


def _normal_f16(rng, shape, sigma=1.0):
    x = rng.standard_normal(size=shape, dtype=np.float32)
    if sigma != 1.0:
        x *= np.float32(sigma)
    return x.astype(np.float16)


def outlier_channels(shape: Shape, seed: int) -> np.ndarray:
    """[H_kv][n] channel indices of K that are scaled up, fixed across tokens and sequences."""
    rng = np.random.default_rng([seed, 0x0C])
    n = shape.k_outlier_channels
    return np.stack([rng.choice(shape.d, size=n, replace=False) for _ in range(shape.H_kv)]) if n else \
        np.zeros((shape.H_kv, 0), np.int64)


def make_kv(shape: Shape, T: int, seed: int, stream: int = 0):
    """fp16 K and V of T tokens: each [B][H_kv][T][d].  `stream` separates independent draws
    (prefill, decode step 0, 1, ...) under one seed."""
    rng = np.random.default_rng([seed, 0xA0, stream])
    k = rng.standard_normal(size=(shape.B, shape.H_kv, T, shape.d), dtype=np.float32)
    if shape.sigma_qk != 1.0:
        k *= np.float32(shape.sigma_qk)
    ch = outlier_channels(shape, seed)
    for h in range(shape.H_kv):
        if ch.shape[1]:
            k[:, h, :, ch[h]] *= np.float32(shape.k_outlier_scale)
    k = k.astype(np.float16)
    v = _normal_f16(rng, (shape.B, shape.H_kv, T, shape.d))
    return k, v


def make_q(shape: Shape, seed: int, stream: int = 0) -> np.ndarray:
    """fp16 query of one decode step: [B][H_q][d]."""
    rng = np.random.default_rng([seed, 0xB0, stream])
    return _normal_f16(rng, (shape.B, shape.H_q, shape.d), shape.sigma_qk)


def ragged_lengths(B: int, lo: int, hi: int, seed: int) -> np.ndarray:
    """Per-sequence context lengths, uniform integers in [lo, hi]."""
    rng = np.random.default_rng([seed, 0xC0])
    return rng.integers(lo, hi + 1, size=B).astype(np.int32)
