"""TEST INFRASTRUCTURE -- Python front of the CPU eager oracle.

`EagerOracle` plays the role of an ordinary eager tensor runtime: every `op`
call is evaluated at once by one C routine of `eager_ops.c` into a freshly
allocated array, in the order the ops are traced (LazyTensor paper, Section 3:
a flushed IR graph must be equivalent to running its ops one by one).

Arrays are numpy arrays in storage representation: float32, uint16 holding
bfloat16 bit patterns, uint8 masks, int32, uint32.  Only tests, the smoke
check and the benchmark's CPU-baseline leg may import this module; it shares
no code with the CUDA library.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "eager_ops.c"
_LIB = _HERE / "liblt_oracle.so"

DTYPES = {"f32": 0, "bf16": 1, "u8": 2, "i32": 3, "u32": 4}
_NP = {"f32": np.float32, "bf16": np.uint16, "u8": np.uint8, "i32": np.int32, "u32": np.uint32}
_MAX_RANK = 6


def build(force: bool = False) -> Path:
    """Compile eager_ops.c with gcc (no fast-math, no FMA contraction, OpenMP)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".{os.getpid()}.tmp")
        subprocess.check_call(
            ["gcc", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-fPIC", "-shared",
             "-o", str(tmp), str(_SRC), "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _Arr(ctypes.Structure):
    _fields_ = [("data", ctypes.c_void_p), ("dtype", ctypes.c_int32), ("rank", ctypes.c_int32),
                ("shape", ctypes.c_int64 * _MAX_RANK)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(str(build()))
        P = ctypes.POINTER(_Arr)
        _lib.orc_binary.argtypes = [ctypes.c_char_p, P, P, P]
        _lib.orc_compare.argtypes = [ctypes.c_char_p, P, P, P]
        _lib.orc_where.argtypes = [P, P, P, P]
        _lib.orc_unary.argtypes = [ctypes.c_char_p, P, P]
        _lib.orc_convert.argtypes = [P, P]
        _lib.orc_iota.argtypes = [ctypes.c_int, P]
        _lib.orc_philox_bits.argtypes = [ctypes.c_uint64, ctypes.c_uint64, P]
        _lib.orc_row_reduce.argtypes = [ctypes.c_char_p, P, P]
        _lib.orc_col_reduce.argtypes = [ctypes.c_char_p, P, P]
        _lib.orc_all_reduce.argtypes = [ctypes.c_char_p, P, P]
        _lib.orc_reshape.argtypes = [P, P]
        _lib.orc_narrow.argtypes = [P, ctypes.c_int, ctypes.c_int64, P]
        _lib.orc_permute.argtypes = [P, ctypes.POINTER(ctypes.c_int), P]
        _lib.orc_update_slice.argtypes = [P, P, ctypes.c_int, ctypes.c_int64, P]
        _lib.orc_set_threads.argtypes = [ctypes.c_int]
        _lib.orc_philox4x32_10.argtypes = [ctypes.POINTER(ctypes.c_uint32)] * 3
        _lib.orc_philox4x32_10.restype = None
        _lib.orc_f32_to_bf16.argtypes = [ctypes.c_float]
        _lib.orc_f32_to_bf16.restype = ctypes.c_uint16
        _lib.orc_bf16_to_f32.argtypes = [ctypes.c_uint16]
        _lib.orc_bf16_to_f32.restype = ctypes.c_float
    return _lib


def set_threads(n: int) -> None:
    lib().orc_set_threads(int(n))


def max_threads() -> int:
    return int(lib().orc_max_threads())


class OTensor:
    """A value of the eager oracle: a numpy array plus its dtype tag.

    A tensor made by one of the `view_*` calls holds a numpy view of its base's storage (`shares` is set on
    both): in-place updates of either then write into that storage, which is numpy's own aliasing and not
    something this module computes."""

    __slots__ = ("array", "dtype", "shares")

    def __init__(self, array: np.ndarray, dtype: str, view: bool = False):
        assert array.dtype == _NP[dtype], (array.dtype, dtype)
        self.array = array if view else np.ascontiguousarray(array)
        self.dtype = dtype
        self.shares = view

    @property
    def shape(self):
        return tuple(self.array.shape)

    def _c(self) -> _Arr:
        if not self.array.flags["C_CONTIGUOUS"]:
            # an op reads a strided view: hand the C routine a dense copy (kept alive on the instance below)
            dense = OTensor(np.ascontiguousarray(self.array), self.dtype)
            a = dense._c()
            a._keep = dense
            return a
        a = _Arr()
        a.data = self.array.ctypes.data
        a.dtype = DTYPES[self.dtype]
        a.rank = self.array.ndim
        for i, d in enumerate(self.array.shape):
            a.shape[i] = d
        return a

    def as_f32(self) -> np.ndarray:
        """Numeric view: bf16 widened to float32; other dtypes unchanged."""
        if self.dtype == "bf16":
            return (self.array.astype(np.uint32) << 16).view(np.float32)
        return self.array


def _bshape(*shapes):
    return tuple(np.broadcast_shapes(*shapes))


_BINARY = {"add", "sub", "mul", "div", "max", "min", "and", "or", "xor"}
_COMPARE = {"gt", "ge", "lt", "le", "eq", "ne"}
_UNARY = {"neg", "abs", "relu", "exp", "log", "tanh", "sqrt", "rsqrt", "recip", "square",
          "sigmoid", "gelu_tanh", "not"}
_REDUCE = {"row_sum", "row_max", "row_min"}
_COL_REDUCE = {"col_sum", "col_max", "col_min"}
_ALL_REDUCE = {"all_sum", "all_max", "all_min"}


class _Scalar:
    """A rank-0 operand whose dtype is taken from the tensor it meets."""

    __slots__ = ("value", "dtype")

    def __init__(self, value: float, dtype: str):
        self.value = float(value)
        self.dtype = dtype


class EagerOracle:
    """Evaluates each traced op immediately; `barrier` has nothing left to do."""

    def __init__(self):
        self.ops_run = 0

    # -- factory methods (paper Section 3: from existing data, constant, range, random)
    def leaf(self, array: np.ndarray, dtype: str) -> OTensor:
        return OTensor(np.array(array, dtype=_NP[dtype], copy=True), dtype)

    def scalar(self, value: float, dtype: str = "f32") -> _Scalar:
        return _Scalar(value, dtype)

    def _materialise(self, x, dtype: str) -> OTensor:
        if isinstance(x, OTensor):
            return x
        v = x.value
        if dtype == "f32":
            arr = np.array(v, dtype=np.float64).astype(np.float32)
        elif dtype == "bf16":
            f = np.array(v, dtype=np.float64).astype(np.float32)
            arr = np.array(lib().orc_f32_to_bf16(float(f)), dtype=np.uint16)
        else:
            if v != int(v):
                raise ValueError("integer scalar required")
            arr = np.array(int(v) & 0xFFFFFFFF if dtype != "u8" else int(v), dtype=np.uint64).astype(
                np.uint32 if dtype != "u8" else np.uint8)
            if dtype == "i32":
                arr = arr.view(np.int32)
        return OTensor(arr.reshape(()), dtype)

    def _pair(self, a, b):
        dt = a.dtype if isinstance(a, OTensor) else b.dtype
        return self._materialise(a, dt), self._materialise(b, dt)

    def _new(self, shape, dtype: str) -> OTensor:
        return OTensor(np.empty(shape, dtype=_NP[dtype]), dtype)

    @staticmethod
    def _check(rc: int, name: str):
        if rc != 0:
            raise ValueError(f"oracle op {name!r} failed with code {rc}")

    def op(self, name: str, *inputs, **attrs):
        self.ops_run += 1
        L = lib()
        if name in _BINARY:
            a, b = self._pair(*inputs)
            out = self._new(_bshape(a.shape, b.shape), a.dtype)
            self._check(L.orc_binary(name.encode(), a._c(), b._c(), out._c()), name)
        elif name in _COMPARE:
            a, b = self._pair(*inputs)
            out = self._new(_bshape(a.shape, b.shape), "u8")
            self._check(L.orc_compare(name.encode(), a._c(), b._c(), out._c()), name)
        elif name == "where":
            m = inputs[0]
            a, b = self._pair(inputs[1], inputs[2])
            out = self._new(_bshape(m.shape, a.shape, b.shape), a.dtype)
            self._check(L.orc_where(m._c(), a._c(), b._c(), out._c()), name)
        elif name in _UNARY:
            (a,) = inputs
            out = self._new(a.shape, a.dtype)
            self._check(L.orc_unary(name.encode(), a._c(), out._c()), name)
        elif name == "convert":
            (a,) = inputs
            out = self._new(a.shape, attrs["dtype"])
            self._check(L.orc_convert(a._c(), out._c()), name)
        elif name == "iota":
            out = self._new(tuple(attrs["shape"]), "i32")
            self._check(L.orc_iota(int(attrs["dim"]), out._c()), name)
        elif name == "philox_bits":
            out = self._new(tuple(attrs["shape"]), "u32")
            self._check(L.orc_philox_bits(int(attrs["seed"]), int(attrs["offset"]), out._c()), name)
        elif name == "reshape":
            (a,) = inputs
            out = self._new(tuple(attrs["shape"]), a.dtype)
            self._check(L.orc_reshape(a._c(), out._c()), name)
            out.array = out.array.reshape(tuple(attrs["shape"]))
        elif name == "narrow":
            (a,) = inputs
            d = int(attrs["dim"])
            out = self._new(a.shape[:d] + (int(attrs["length"]),) + a.shape[d + 1:], a.dtype)
            self._check(L.orc_narrow(a._c(), d, int(attrs["start"]), out._c()), name)
        elif name == "permute":
            (a,) = inputs
            perm = [int(p) for p in attrs["perm"]]
            out = self._new(tuple(a.shape[p] for p in perm), a.dtype)
            self._check(L.orc_permute(a._c(), (ctypes.c_int * len(perm))(*perm), out._c()), name)
        elif name == "update_slice":
            base, upd = inputs
            out = self._new(base.shape, base.dtype)
            self._check(L.orc_update_slice(base._c(), upd._c(), int(attrs["dim"]), int(attrs["start"]), out._c()), name)
        elif name in _REDUCE:
            (a,) = inputs
            out = self._new(a.shape[:-1] + (1,), a.dtype)
            self._check(L.orc_row_reduce(name.encode(), a._c(), out._c()), name)
        elif name in _COL_REDUCE:
            (a,) = inputs
            out = self._new((1,) * (len(a.shape) - 1) + a.shape[-1:], a.dtype)
            self._check(L.orc_col_reduce(name.encode(), a._c(), out._c()), name)
        elif name in _ALL_REDUCE:
            (a,) = inputs
            out = self._new((), a.dtype)
            self._check(L.orc_all_reduce(name.encode(), a._c(), out._c()), name)
            out.array = out.array.reshape(())  # rank 0, like the traced op's result
        else:
            raise ValueError(f"unknown op {name!r}")
        return out

    # -- views (paper Section 4.4): numpy views of the base's storage
    def _own_storage(self, t: OTensor) -> None:
        if not t.shares:
            t.array = np.array(t.array, copy=True)  # storage no other value refers to
            t.shares = True

    def view_reshape(self, t: OTensor, shape) -> OTensor:
        self._own_storage(t)
        v = t.array.view()
        v.shape = tuple(shape)  # raises instead of copying when the storage cannot be seen under that shape
        return OTensor(v, t.dtype, view=True)

    def view_narrow(self, t: OTensor, dim: int, start: int, length: int) -> OTensor:
        self._own_storage(t)
        index = [slice(None)] * t.array.ndim
        index[dim] = slice(start, start + length)
        return OTensor(t.array[tuple(index)], t.dtype, view=True)

    def view_permute(self, t: OTensor, perm) -> OTensor:
        self._own_storage(t)
        return OTensor(np.transpose(t.array, tuple(perm)), t.dtype, view=True)

    # -- in-place update: the destination takes over the source's value (paper Section 4.3)
    def assign(self, dst: OTensor, src: OTensor) -> None:
        if dst.shape != src.shape or dst.dtype != src.dtype:
            raise ValueError("assign needs equal shape and dtype")
        if dst.shares:
            dst.array[...] = src.array  # written into the storage its views (or its base) see
        else:
            dst.array = src.array

    def release(self, t) -> None:
        pass

    def barrier(self, blocking: bool = True) -> None:
        pass

    def fetch(self, t: OTensor) -> np.ndarray:
        return t.array.copy()
