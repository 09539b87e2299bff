"""The traced programs of the five benchmark configurations.

Each function takes a backend `B` (anything with `scalar`, `op` and `assign`)
plus input handles, issues the configuration's ops one by one, and returns the
handles that stay live.  Intermediate handles go out of scope as the function
runs, so a lazy backend sees only the returned tensors as roots at the next
barrier.  Nothing here computes a value.
"""
from __future__ import annotations

import math

SQRT_2_OVER_PI = math.sqrt(2.0 / math.pi)
GELU_CUBIC = 0.044715


def elementwise_chain(B, a, b, c, d):
    """y = relu(a*b + c) * 0.5 - d."""
    t = B.op("mul", a, b)
    t = B.op("add", t, c)
    t = B.op("relu", t)
    t = B.op("mul", t, B.scalar(0.5))
    return B.op("sub", t, d)


def mlp_epilogue(B, x, h, bias, *, primitive_gelu: bool = True):
    """out = x + GELU_tanh(h + bias); bf16 in, fp32 arithmetic, bf16 out."""
    xf = B.op("convert", x, dtype="f32")
    hf = B.op("convert", h, dtype="f32")
    bf = B.op("convert", bias, dtype="f32")
    t = B.op("add", hf, bf)
    if primitive_gelu:
        u = B.op("mul", t, t)
        u = B.op("mul", u, t)
        u = B.op("mul", u, B.scalar(GELU_CUBIC))
        u = B.op("add", t, u)
        u = B.op("mul", u, B.scalar(SQRT_2_OVER_PI))
        u = B.op("tanh", u)
        u = B.op("add", u, B.scalar(1.0))
        g = B.op("mul", t, B.scalar(0.5))
        g = B.op("mul", g, u)
    else:
        g = B.op("gelu_tanh", t)
    out = B.op("add", xf, g)
    return B.op("convert", out, dtype="bf16")


def dropout_threshold(p: float) -> int:
    """An element is kept when its 32 random bits, as an unsigned integer, are >= floor(p * 2^32)."""
    return int(math.floor(p * 4294967296.0))


def residual_dropout_layernorm(B, x, h, gamma, beta, *, shape, p: float, eps: float, seed: int,
                               offset: int, out_dtype: str = "bf16"):
    """z = LayerNorm(x + dropout(h, p)) * gamma + beta over the last dim; also returns the keep mask."""
    cols = shape[-1]
    xf = B.op("convert", x, dtype="f32")
    hf = B.op("convert", h, dtype="f32")
    bits = B.op("philox_bits", shape=tuple(shape), seed=seed, offset=offset)
    keep = B.op("ge", bits, B.scalar(dropout_threshold(p), "u32"))
    hs = B.op("mul", hf, B.scalar(1.0 / (1.0 - p)))
    hd = B.op("where", keep, hs, B.scalar(0.0))
    t = B.op("add", xf, hd)
    inv_c = B.scalar(1.0 / cols)
    mu = B.op("mul", B.op("row_sum", t), inv_c)
    d = B.op("sub", t, mu)
    var = B.op("mul", B.op("row_sum", B.op("mul", d, d)), inv_c)
    rstd = B.op("rsqrt", B.op("add", var, B.scalar(eps)))
    z = B.op("mul", d, rstd)
    z = B.op("mul", z, gamma)
    z = B.op("add", z, beta)
    if out_dtype != "f32":
        z = B.op("convert", z, dtype=out_dtype)
    return z, keep


def residual_layernorm(B, x, h, gamma, beta, *, shape, eps: float, out_dtype: str = "bf16"):
    """z = LayerNorm(x + h) * gamma + beta over the last dim: the normalisation above without dropout."""
    cols = shape[-1]
    t = B.op("add", B.op("convert", x, dtype="f32"), B.op("convert", h, dtype="f32"))
    inv_c = B.scalar(1.0 / cols)
    d = B.op("sub", t, B.op("mul", B.op("row_sum", t), inv_c))
    var = B.op("mul", B.op("row_sum", B.op("mul", d, d)), inv_c)
    z = B.op("mul", d, B.op("rsqrt", B.op("add", var, B.scalar(eps))))
    z = B.op("add", B.op("mul", z, gamma), beta)
    if out_dtype != "f32":
        z = B.op("convert", z, dtype=out_dtype)
    return z


def causal_softmax(B, scores, *, shape, scale: float, out_dtype: str = "bf16"):
    """softmax over the last dim of scores*scale with columns > row masked to -inf ([heads, q, k] input)."""
    s = B.op("convert", scores, dtype="f32")
    s = B.op("mul", s, B.scalar(scale))
    col = B.op("iota", shape=tuple(shape), dim=len(shape) - 1)
    row = B.op("iota", shape=tuple(shape), dim=len(shape) - 2)
    masked = B.op("gt", col, row)
    s = B.op("where", masked, B.scalar(-math.inf), s)
    mx = B.op("row_max", s)
    e = B.op("exp", B.op("sub", s, mx))
    y = B.op("div", e, B.op("row_sum", e))
    if out_dtype != "f32":
        y = B.op("convert", y, dtype=out_dtype)
    return y


class AdamScalars:
    """Host-side hyper-parameter arithmetic of one Adam step (in double), as dynamic scalars."""

    def __init__(self, B, *, step: int, lr: float = 1e-3, beta1: float = 0.9, beta2: float = 0.999,
                 eps: float = 1e-8):
        bc1 = 1.0 - beta1 ** step
        bc2 = 1.0 - beta2 ** step
        self.beta1 = B.scalar(beta1)
        self.one_minus_beta1 = B.scalar(1.0 - beta1)
        self.beta2 = B.scalar(beta2)
        self.one_minus_beta2 = B.scalar(1.0 - beta2)
        self.sqrt_bc2 = B.scalar(math.sqrt(bc2))
        self.eps = B.scalar(eps)
        self.step_size = B.scalar(lr / bc1)


def adam_update(B, p, g, m, v, s: AdamScalars):
    """One in-place Adam update of (p, m, v) from gradient g; no weight decay, no amsgrad."""
    m_new = B.op("add", B.op("mul", m, s.beta1), B.op("mul", g, s.one_minus_beta1))
    v_new = B.op("add", B.op("mul", v, s.beta2), B.op("mul", B.op("mul", g, g), s.one_minus_beta2))
    denom = B.op("add", B.op("div", B.op("sqrt", v_new), s.sqrt_bc2), s.eps)
    upd = B.op("mul", B.op("div", m_new, denom), s.step_size)
    p_new = B.op("sub", p, upd)
    B.assign(m, m_new)
    B.assign(v, v_new)
    B.assign(p, p_new)


def adam_step(B, params, grads, ms, vs, *, step: int, **hyper):
    s = AdamScalars(B, step=step, **hyper)
    for p, g, m, v in zip(params, grads, ms, vs):
        adam_update(B, p, g, m, v, s)
