"""Seeded logits: independent normal draws with standard deviation 2.

bf16 rows are the fp32 draws rounded to nearest-even and are carried as raw
uint16 bit patterns (numpy has no bfloat16).  ``steer`` optionally adds a
constant to every token that contains a structural character; it depends on
the vocabulary only, never on a grammar state, and exists so that greedy
trajectories leave free-text slots often enough to visit every part of a
template.
"""
from __future__ import annotations

from typing import Optional

import numpy as np

SIGMA = 2.0


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even conversion of finite fp32 values to bf16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    rounded = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return rounded.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def make_logits(rows: int, V: int, dtype: str, seed, step: int = 0,
                bonus: Optional[np.ndarray] = None, steer: float = 0.0) -> np.ndarray:
    """[rows, V] logits for one decode step: float32, or uint16 bf16 bit patterns.

    ``seed`` may be an int or a sequence of ints (config id, row base, ...); ``step`` selects
    an independent stream so that every step sees fresh values.
    """
    key = [int(s) for s in (seed if isinstance(seed, (list, tuple)) else [seed])]
    mix = 0x6C6F67
    for k in key:
        mix = (mix * 0x9E3779B1 + k + 1) % (1 << 63)
    rng = np.random.Generator(np.random.Philox(key=[mix, int(step)]))
    x = rng.standard_normal((rows, V), dtype=np.float32) * np.float32(SIGMA)
    if steer != 0.0 and bonus is not None:
        x += np.float32(steer) * bonus.astype(np.float32)[None, :]
    if dtype == "fp32":
        return x
    if dtype == "bf16":
        return f32_to_bf16_bits(x)
    raise ValueError(dtype)
