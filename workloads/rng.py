"""Seeded host-side input generation (numpy Philox bit generator, counter based)."""
from __future__ import annotations

import numpy as np


def generator(seed: int, stream: int = 0) -> np.random.Generator:
    """Independent reproducible stream `stream` of seed `seed`."""
    return np.random.Generator(np.random.Philox(key=[int(seed) & (2**64 - 1), int(stream)]))


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Quantise float32 inputs to bfloat16 storage (uint16 bit patterns, ties to even)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    r = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def normal_f32(g: np.random.Generator, shape, std: float = 1.0, mean: float = 0.0) -> np.ndarray:
    return (g.standard_normal(shape, dtype=np.float32) * np.float32(std) + np.float32(mean)).astype(np.float32)


def normal_bf16(g: np.random.Generator, shape, std: float = 1.0) -> np.ndarray:
    return to_bf16_bits(normal_f32(g, shape, std))


def uniform_f32(g: np.random.Generator, shape, lo: float = -1.0, hi: float = 1.0) -> np.ndarray:
    return (g.random(shape, dtype=np.float32) * np.float32(hi - lo) + np.float32(lo)).astype(np.float32)
