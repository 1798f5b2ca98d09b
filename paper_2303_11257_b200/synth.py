"""Seeded synthetic inputs for the unit-scaled FFN / linear workloads.

Only random draws and shapes live here -- none of the method's arithmetic -- so the
same tensors can be handed both to the device library and to an independent checker.
Tensor k of a workload with seed s is drawn from numpy's counter-based Philox
generator keyed by (s, k): standard normal float32, optionally multiplied by a
power-of-two sigma (exact in float32).
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


def normal(seed: int, k: int, shape, sigma: float = 1.0) -> np.ndarray:
    """Tensor `k` of workload `seed`: N(0, sigma^2) float32 of the given shape."""
    rng = np.random.Generator(np.random.Philox(key=[int(seed), int(k)]))
    x = rng.standard_normal(size=shape, dtype=np.float32)
    if sigma != 1.0:
        x = x * np.float32(sigma)
    return x


@dataclass(frozen=True)
class FFNShape:
    name: str
    tokens: int      # T = batch x sequence, the paper's b
    d_model: int     # d
    d_ff: int        # f


# Shapes: the character-LM sweep (hidden 128, FFN 512, sequence 256) and
# BERT-large (16 sequences x 512 tokens, hidden 1024, FFN 4096).
FFN_SMALL = FFNShape("ffn_small", 256, 128, 512)
FFN_BERT_LARGE = FFNShape("ffn_bert_large", 8192, 1024, 4096)
# A ragged shape: token and feature counts that are not tile multiples.
FFN_RAGGED = FFNShape("ffn_ragged", 200, 144, 336)


def ffn_tensors(shape: FFNShape, seed: int = 0, sigma_x: float = 1.0):
    """X [T x d], W1 [d x f], W2 [f x d], G [T x d]: unit-normal float32 (X optionally N(0, sigma_x^2))."""
    T, d, f = shape.tokens, shape.d_model, shape.d_ff
    return (
        normal(seed, 0, (T, d), sigma_x),
        normal(seed, 1, (d, f)),
        normal(seed, 2, (f, d)),
        normal(seed, 3, (T, d)),
    )


def linear_tensors(b: int, m: int, n: int, seed: int = 0):
    """X [b x m], W [m x n], G [b x n]: unit-normal float32."""
    return normal(seed, 0, (b, m)), normal(seed, 1, (m, n)), normal(seed, 2, (b, n))
