"""Traced programs of common fusion groups beyond the five benchmark configurations.

Same conventions as traces.py: a backend `B` with `scalar`, `op`, `assign`; nothing here computes a value.
Each entry of ALL is (name, kinds of its inputs, trace function); input kinds are
"mat:<dtype>" for a [rows, cols] operand and "vec:<dtype>" for a [cols] operand.  The library ships an
ahead-of-time compiled kernel for every one of them; the parity tests run each against the oracle.
"""
from __future__ import annotations


def _f32(B, t, dtype):
    return t if dtype == "f32" else B.op("convert", t, dtype="f32")


def _out(B, t, dtype):
    return t if dtype == "f32" else B.op("convert", t, dtype=dtype)


def bias_relu(B, x, bias, *, cols, dtype="bf16"):
    """out = relu(x + bias)."""
    return _out(B, B.op("relu", B.op("add", _f32(B, x, dtype), _f32(B, bias, dtype))), dtype)


def bias_gelu(B, x, bias, *, cols, dtype="bf16"):
    """out = GELU_tanh(x + bias)."""
    return _out(B, B.op("gelu_tanh", B.op("add", _f32(B, x, dtype), _f32(B, bias, dtype))), dtype)


def residual_add(B, x, y, *, cols, dtype="bf16"):
    """out = x + y."""
    return _out(B, B.op("add", _f32(B, x, dtype), _f32(B, y, dtype)), dtype)


def swiglu(B, gate, up, *, cols, dtype="bf16"):
    """out = gate * sigmoid(gate) * up."""
    g = _f32(B, gate, dtype)
    return _out(B, B.op("mul", B.op("mul", g, B.op("sigmoid", g)), _f32(B, up, dtype)), dtype)


def softmax(B, x, *, cols, dtype="bf16"):
    """Row softmax with the row maximum subtracted."""
    s = _f32(B, x, dtype)
    e = B.op("exp", B.op("sub", s, B.op("row_max", s)))
    return _out(B, B.op("div", e, B.op("row_sum", e)), dtype)


def layernorm(B, x, gamma, beta, *, cols, dtype="bf16", eps=1e-5):
    """LayerNorm over the last dim, biased two-pass variance, f32 gamma / beta."""
    t = _f32(B, x, dtype)
    inv_c = B.scalar(1.0 / cols)
    d = B.op("sub", t, B.op("mul", B.op("row_sum", t), inv_c))
    var = B.op("mul", B.op("row_sum", B.op("mul", d, d)), inv_c)
    z = B.op("mul", d, B.op("rsqrt", B.op("add", var, B.scalar(eps))))
    return _out(B, B.op("add", B.op("mul", z, gamma), beta), dtype)


def rmsnorm(B, x, gamma, *, cols, dtype="bf16", eps=1e-6):
    """x * rsqrt(mean(x^2) + eps) * gamma."""
    t = _f32(B, x, dtype)
    ms = B.op("mul", B.op("row_sum", B.op("mul", t, t)), B.scalar(1.0 / cols))
    return _out(B, B.op("mul", B.op("mul", t, B.op("rsqrt", B.op("add", ms, B.scalar(eps)))), gamma), dtype)


def silu(B, x, *, cols, dtype="bf16"):
    """out = x * sigmoid(x)."""
    t = _f32(B, x, dtype)
    return _out(B, B.op("mul", t, B.op("sigmoid", t)), dtype)


def gelu(B, x, *, cols, dtype="bf16"):
    """out = GELU_tanh(x)."""
    return _out(B, B.op("gelu_tanh", _f32(B, x, dtype)), dtype)


def add_relu(B, x, y, *, cols, dtype="bf16"):
    """out = relu(x + y)."""
    return _out(B, B.op("relu", B.op("add", _f32(B, x, dtype), _f32(B, y, dtype))), dtype)


def scale_to_f32(B, x, *, cols, scale=0.125):
    """out (f32) = x (bf16) * scale."""
    return B.op("mul", B.op("convert", x, dtype="f32"), B.scalar(scale))


def scaled_softmax(B, x, *, cols, dtype="bf16", scale=0.0884):
    """Row softmax of x * scale."""
    s = B.op("mul", _f32(B, x, dtype), B.scalar(scale))
    e = B.op("exp", B.op("sub", s, B.op("row_max", s)))
    return _out(B, B.op("div", e, B.op("row_sum", e)), dtype)


def sgd_momentum(B, params, grads, bufs, *, lr=0.1, momentum=0.9):
    """For every tensor: buf := momentum * buf + g; p := p - lr * buf (in place).  The two scalars are
    shared by all tensors, so the updates are one program over many tensors."""
    lr_s, mom_s = B.scalar(lr), B.scalar(momentum)
    for p, g, buf in zip(params, grads, bufs):
        nb = B.op("add", B.op("mul", buf, mom_s), g)
        B.assign(buf, nb)
        B.assign(p, B.op("sub", p, B.op("mul", nb, lr_s)))


ALL = [
    ("bias_relu_bf16", ("mat:bf16", "vec:bf16"), lambda B, ins, cols: bias_relu(B, *ins, cols=cols)),
    ("bias_gelu_bf16", ("mat:bf16", "vec:bf16"), lambda B, ins, cols: bias_gelu(B, *ins, cols=cols)),
    ("residual_add_bf16", ("mat:bf16", "mat:bf16"), lambda B, ins, cols: residual_add(B, *ins, cols=cols)),
    ("residual_add_f32", ("mat:f32", "mat:f32"), lambda B, ins, cols: residual_add(B, *ins, cols=cols, dtype="f32")),
    ("swiglu_bf16", ("mat:bf16", "mat:bf16"), lambda B, ins, cols: swiglu(B, *ins, cols=cols)),
    ("softmax_bf16", ("mat:bf16",), lambda B, ins, cols: softmax(B, *ins, cols=cols)),
    ("softmax_f32", ("mat:f32",), lambda B, ins, cols: softmax(B, *ins, cols=cols, dtype="f32")),
    ("layernorm_bf16", ("mat:bf16", "vec:f32", "vec:f32"), lambda B, ins, cols: layernorm(B, *ins, cols=cols)),
    ("rmsnorm_bf16", ("mat:bf16", "vec:f32"), lambda B, ins, cols: rmsnorm(B, *ins, cols=cols)),
    ("layernorm_f32", ("mat:f32", "vec:f32", "vec:f32"), lambda B, ins, cols: layernorm(B, *ins, cols=cols, dtype="f32")),
    ("silu_bf16", ("mat:bf16",), lambda B, ins, cols: silu(B, *ins, cols=cols)),
    ("gelu_bf16", ("mat:bf16",), lambda B, ins, cols: gelu(B, *ins, cols=cols)),
    ("add_relu_bf16", ("mat:bf16", "mat:bf16"), lambda B, ins, cols: add_relu(B, *ins, cols=cols)),
    ("scale_to_f32", ("mat:bf16",), lambda B, ins, cols: scale_to_f32(B, *ins, cols=cols)),
    ("scaled_softmax_bf16", ("mat:bf16",), lambda B, ins, cols: scaled_softmax(B, *ins, cols=cols)),
]


# ---- reductions of a computed value (over the rows of every column, or over everything): the value's kernel does the
# first stage of the reduction instead of storing it.  Same signature as ALL.
def _f32(B, t, dtype):
    return t if dtype == "f32" else B.op("convert", t, dtype="f32")


def sum_squares(B, x, *, cols, dtype="f32"):
    """||x||^2, the gradient-norm building block."""
    xf = _f32(B, x, dtype)
    return B.op("all_sum", B.op("mul", xf, xf))


def squared_error_sum(B, a, b, *, cols, dtype="f32"):
    d = B.op("sub", _f32(B, a, dtype), _f32(B, b, dtype))
    return B.op("all_sum", B.op("mul", d, d))


def column_squared_error(B, a, b, *, cols, dtype="f32"):
    d = B.op("sub", _f32(B, a, dtype), _f32(B, b, dtype))
    return B.op("col_sum", B.op("mul", d, d))


def bias_grad(B, dy, *, cols, dtype="bf16"):
    """Gradient of a broadcast bias: column sums of dy, accumulated from its f32 values."""
    return B.op("col_sum", _f32(B, dy, dtype))


def relu_bias_grad(B, dy, x, *, cols, dtype="bf16"):
    """Column sums of dy where the forward input was positive."""
    g = B.op("where", B.op("gt", _f32(B, x, dtype), B.scalar(0.0)), _f32(B, dy, dtype), B.scalar(0.0))
    return B.op("col_sum", g)


def abs_max(B, x, *, cols, dtype="f32"):
    """max |x|: the scale of a tensor."""
    return B.op("all_max", B.op("abs", _f32(B, x, dtype)))


REDUCED = [
    ("sum_squares_f32", ("mat:f32",), lambda B, ins, cols: sum_squares(B, *ins, cols=cols)),
    ("sum_squares_bf16", ("mat:bf16",), lambda B, ins, cols: sum_squares(B, *ins, cols=cols, dtype="bf16")),
    ("squared_error_sum_f32", ("mat:f32", "mat:f32"), lambda B, ins, cols: squared_error_sum(B, *ins, cols=cols)),
    ("column_squared_error_f32", ("mat:f32", "mat:f32"), lambda B, ins, cols: column_squared_error(B, *ins, cols=cols)),
    ("bias_grad_bf16", ("mat:bf16",), lambda B, ins, cols: bias_grad(B, *ins, cols=cols)),
    ("relu_bias_grad_bf16", ("mat:bf16", "mat:bf16"), lambda B, ins, cols: relu_bias_grad(B, *ins, cols=cols)),
    ("abs_max_f32", ("mat:f32",), lambda B, ins, cols: abs_max(B, *ins, cols=cols)),
    ("abs_max_bf16", ("mat:bf16",), lambda B, ins, cols: abs_max(B, *ins, cols=cols, dtype="bf16")),
]
