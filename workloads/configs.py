"""Seeded inputs of the five configurations, at full or reduced size.

Distributions (second argument of N(.,.) is the standard deviation):
  C1  a,b,c,d  f32 uniform[-1,1]
  C2  x,h bf16 N(0,1); bias bf16 N(0,0.02)
  C3  x,h bf16 N(0,1); gamma f32 1+N(0,0.02); beta f32 N(0,0.02)
  C4  scores bf16 N(0,4)
  C5  params f32 N(0,0.05); grads f32 N(0,1e-3); m = v = 0, ResNet-50 shapes
"""
from __future__ import annotations

import math

import numpy as np

from . import rng
from .resnet50 import parameter_shapes

FULL = {
    "c1": (1024, 1024),
    "c2": (8192, 4096),
    "c3": (16384, 1024),
    "c4": (16, 2048, 2048),
}


def c1_inputs(seed: int, shape=FULL["c1"]):
    g = rng.generator(seed, 1)
    return [rng.uniform_f32(g, shape) for _ in range(4)]


def c2_inputs(seed: int, shape=FULL["c2"]):
    g = rng.generator(seed, 2)
    x = rng.normal_bf16(g, shape, 1.0)
    h = rng.normal_bf16(g, shape, 1.0)
    bias = rng.normal_bf16(g, (shape[-1],), 0.02)
    return x, h, bias


def c3_inputs(seed: int, shape=FULL["c3"]):
    g = rng.generator(seed, 3)
    x = rng.normal_bf16(g, shape, 1.0)
    h = rng.normal_bf16(g, shape, 1.0)
    gamma = rng.normal_f32(g, (shape[-1],), 0.02, 1.0)
    beta = rng.normal_f32(g, (shape[-1],), 0.02, 0.0)
    return x, h, gamma, beta


def c4_inputs(seed: int, shape=FULL["c4"]):
    g = rng.generator(seed, 4)
    return rng.normal_bf16(g, shape, 4.0)


def c5_inputs(seed: int, shapes=None):
    """Returns (params, grads, ms, vs): lists of f32 arrays, one per parameter tensor."""
    if shapes is None:
        shapes = parameter_shapes()
    g = rng.generator(seed, 5)
    params = [rng.normal_f32(g, s, 0.05) for s in shapes]
    grads = [rng.normal_f32(g, s, 1e-3) for s in shapes]
    ms = [np.zeros(s, dtype=np.float32) for s in shapes]
    vs = [np.zeros(s, dtype=np.float32) for s in shapes]
    return params, grads, ms, vs


def algorithmic_bytes(cfg: str, shape=None) -> int:
    """Fewest bytes a fused flush must move: every input read once, every output written once."""
    if cfg == "c5":
        shapes = shape if shape is not None else parameter_shapes()
        return 28 * sum(math.prod(s) for s in shapes)
    shape = shape if shape is not None else FULL[cfg]
    n = math.prod(shape)
    cols = shape[-1]
    if cfg == "c1":
        return 20 * n
    if cfg == "c2":
        return 6 * n + 2 * cols
    if cfg == "c3":
        return 7 * n + 8 * cols
    if cfg == "c4":
        return 4 * n
    raise KeyError(cfg)
