"""Python binding of liblazytensor.so (argument marshalling only).

`LazyContext` and `LazyTensor` mirror the C ABI in include/lazytensor.h one to one:
every method forwards to the entry point of the same name.  All recording, hashing,
planning and execution happens in the shared library; there is no Python or CPU
fallback -- if the library is missing, importing this module raises.

PyTorch is used for device memory (its caching allocator backs the allocator
callbacks) and for the CUDA stream the kernels are enqueued on.
"""
from __future__ import annotations

import ctypes
import os
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
LIB_PATH = _HERE / "liblazytensor.so"

if not LIB_PATH.exists():
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -c 'import __graft_entry__ as g; g.build()'` "
        "(there is no fallback implementation)")

_lib = ctypes.CDLL(str(LIB_PATH))

LT_MAX_RANK = 6
LT_DEVICE_NONE = -1
DTYPES = {"f32": 0, "bf16": 1, "u8": 2, "i32": 3, "u32": 4}
DTYPE_NAMES = {v: k for k, v in DTYPES.items()}
NP_DTYPES = {"f32": np.float32, "bf16": np.uint16, "u8": np.uint8, "i32": np.int32, "u32": np.uint32}
OPCODES = {
    "add": 1, "sub": 2, "mul": 3, "div": 4, "max": 5, "min": 6, "and": 7, "or": 8, "xor": 9,
    "gt": 10, "ge": 11, "lt": 12, "le": 13, "eq": 14, "ne": 15, "where": 16,
    "neg": 20, "abs": 21, "relu": 22, "exp": 23, "log": 24, "tanh": 25, "sqrt": 26, "rsqrt": 27,
    "recip": 28, "square": 29, "sigmoid": 30, "gelu_tanh": 31, "not": 32,
    "convert": 40, "iota": 41, "philox_bits": 42, "row_sum": 50, "row_max": 51, "row_min": 52,
    "col_sum": 53, "col_max": 54, "col_min": 55, "all_sum": 56, "all_max": 57, "all_min": 58,
    "reshape": 60, "narrow": 61, "permute": 62, "update_slice": 63,
}
STATUS_NAMES = ["LT_OK", "LT_ERR_INVALID_ARG", "LT_ERR_SHAPE", "LT_ERR_DTYPE", "LT_ERR_DEVICE",
                "LT_ERR_UNSUPPORTED", "LT_ERR_OOM", "LT_ERR_CUDA", "LT_ERR_DEVICE_TIMEOUT"]

ALLOC_FN = ctypes.CFUNCTYPE(ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p, ctypes.c_void_p)
FREE_FN = ctypes.CFUNCTYPE(None, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p)


class lt_allocator(ctypes.Structure):
    _fields_ = [("alloc", ALLOC_FN), ("free", FREE_FN), ("user", ctypes.c_void_p)]


class lt_batch_op(ctypes.Structure):
    _fields_ = [("opcode", ctypes.c_int32), ("n_in", ctypes.c_int32), ("in_", ctypes.c_int32 * 3), ("n_attrs", ctypes.c_int32),
                ("attr_offset", ctypes.c_int32), ("keep", ctypes.c_int32)]


LT_BATCH_ASSIGN = -1


class lt_stats(ctypes.Structure):
    _fields_ = [(n, ctypes.c_uint64) for n in (
        "nodes_recorded", "barriers", "compiles", "cache_hits", "kernels_launched",
        "launches_elementwise", "launches_row", "launches_multi", "bytes_planned",
        "outputs_donated", "outputs_allocated", "temporaries_allocated",
        "ns_record", "ns_canonicalise", "ns_hash_lookup", "ns_plan", "ns_bind_launch", "ns_rebind",
        "launches_compiled", "replays", "launches_reduce", "launches_view", "programs_specialised", "launches_specialised", "allocator_calls", "traces_matched", "traces_diverged")]


class lt_kernel_timing(ctypes.Structure):
    _fields_ = [("launches", ctypes.c_uint64 * 3), ("ms", ctypes.c_double * 3), ("bytes", ctypes.c_uint64 * 3)]


_P = ctypes.POINTER
_vp, _i64, _u64, _int = ctypes.c_void_p, ctypes.c_int64, ctypes.c_uint64, ctypes.c_int

_SIGNATURES = {
    "lt_ctx_create": [_int, _vp, _P(lt_allocator), _P(_vp)],
    "lt_ctx_destroy": [_vp],
    "lt_ctx_set_option": [_vp, ctypes.c_char_p, _i64],
    "lt_tensor_from_device": [_vp, _vp, _int, _int, _P(_i64), _P(_u64)],
    "lt_tensor_from_host": [_vp, _vp, _int, _int, _P(_i64), _P(_u64)],
    "lt_scalar": [_vp, ctypes.c_double, _int, _P(_u64)],
    "lt_scalar_dynamic": [_vp, ctypes.c_double, _int, _P(_u64)],
    "lt_op": [_vp, _int, _P(_u64), _int, _P(_i64), _int, _P(_u64)],
    "lt_assign": [_vp, _u64, _u64],
    "lt_view_reshape": [_vp, _u64, _int, _P(_i64), _P(_u64)],
    "lt_view_narrow": [_vp, _u64, _int, _i64, _i64, _P(_u64)],
    "lt_view_permute": [_vp, _u64, _P(_int), _P(_u64)],
    "lt_release": [_vp, _u64],
    "lt_release_many": [_vp, _P(_u64), ctypes.c_size_t],
    "lt_op_many": [_vp, _P(lt_batch_op), ctypes.c_size_t, _P(_u64), ctypes.c_size_t, _P(_i64), _P(_u64)],
    "lt_barrier": [_vp, _int],
    "lt_barrier_static_scratch": [_vp, _int, _int],
    "lt_debug_bounds_violations": [_vp, _P(_u64)],
    "lt_debug_wait_probe": [_vp, _u64],
    "lt_replay": [_vp, _int],
    "lt_scalar_set": [_vp, _u64, ctypes.c_double],
    "lt_replay_slots": [_vp, _P(ctypes.c_uint32)],
    "lt_replay_set_slot": [_vp, ctypes.c_uint32, _int, ctypes.c_double, _i64],
    "lt_fetch": [_vp, _u64, _vp, ctypes.c_size_t],
    "lt_device_ptr": [_vp, _u64, _P(_vp)],
    "lt_tensor_info": [_vp, _u64, _P(_int), _P(_int), _P(_i64), _P(_int)],
    "lt_get_stats": [_vp, _P(lt_stats)],
    "lt_reset_stats": [_vp],
    "lt_cache_size": [_vp, _P(_u64)],
    "lt_set_kernel_timing": [_vp, _int],
    "lt_get_kernel_timing": [_vp, _P(lt_kernel_timing)],
    "lt_dump_ir": [_vp, ctypes.c_char_p, ctypes.c_size_t, _P(ctypes.c_size_t)],
    "lt_dump_plan": [_vp, ctypes.c_char_p, ctypes.c_size_t, _P(ctypes.c_size_t)],
}
for _name, _args in _SIGNATURES.items():
    _fn = getattr(_lib, _name)
    _fn.argtypes = _args
    _fn.restype = _int
_lib.lt_last_error.argtypes = [_vp]
_lib.lt_last_error.restype = ctypes.c_char_p
_lib.lt_version.argtypes = []
_lib.lt_version.restype = ctypes.c_char_p

EXPORTED_SYMBOLS = sorted(list(_SIGNATURES) + ["lt_last_error", "lt_version"])


class LazyTensorError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else status}: {message}")
        self.status = status


def version() -> str:
    return _lib.lt_version().decode()


def _torch_allocator():
    import torch

    def _alloc(nbytes, stream, user):
        try:
            return torch.cuda.caching_allocator_alloc(int(nbytes), stream=int(stream or 0))
        except Exception:  # out of memory: report NULL, the library turns it into LT_ERR_OOM
            return None

    def _free(ptr, stream, user):
        torch.cuda.caching_allocator_delete(int(ptr))

    return ALLOC_FN(_alloc), FREE_FN(_free)


class LazyTensor:
    """A handle of the C library; its value may still be a pending IR graph (paper Section 3).

    Dropping the last Python reference unregisters the tensor: the handle is queued on the context
    and released in one batch before the next barrier, fetch or dump.
    """

    __slots__ = ("ctx", "handle", "_keep", "_dtype", "_shape", "__weakref__")

    def __init__(self, ctx: "LazyContext", handle: int, dtype: str | None = None, shape=None, keep=None):
        self.ctx = ctx
        self.handle = handle
        self._dtype = dtype
        self._shape = None if shape is None else tuple(shape)
        self._keep = keep  # device storage this tensor borrows

    def __del__(self):
        ctx = self.ctx
        if ctx is not None:
            ctx._dead.append(self.handle)
            if self._keep is not None:
                # a pending graph may still read the borrowed storage: keep it until the next barrier
                ctx._keeps.append(self._keep)

    @property
    def dtype(self) -> str:
        if self._dtype is None:
            self._dtype, _, self._shape, _ = self.ctx._info(self.handle)
        return self._dtype

    @property
    def shape(self) -> tuple:
        if self._shape is None:
            self._dtype, _, self._shape, _ = self.ctx._info(self.handle)
        return self._shape

    # the eager-looking API: every operator only records
    def _bin(self, name, other, swap=False):
        if not isinstance(other, LazyTensor):
            other = self.ctx.scalar(other, self.dtype)
        return self.ctx.op(name, other, self) if swap else self.ctx.op(name, self, other)

    def __add__(self, o): return self._bin("add", o)
    def __radd__(self, o): return self._bin("add", o, True)
    def __sub__(self, o): return self._bin("sub", o)
    def __rsub__(self, o): return self._bin("sub", o, True)
    def __mul__(self, o): return self._bin("mul", o)
    def __rmul__(self, o): return self._bin("mul", o, True)
    def __truediv__(self, o): return self._bin("div", o)
    def __rtruediv__(self, o): return self._bin("div", o, True)
    def __neg__(self): return self.ctx.op("neg", self)
    def __gt__(self, o): return self._bin("gt", o)
    def __ge__(self, o): return self._bin("ge", o)
    def __lt__(self, o): return self._bin("lt", o)
    def __le__(self, o): return self._bin("le", o)

    def __iadd__(self, o):
        self.ctx.assign(self, self + o)
        return self

    def __isub__(self, o):
        self.ctx.assign(self, self - o)
        return self

    def __imul__(self, o):
        self.ctx.assign(self, self * o)
        return self

    def numpy(self) -> np.ndarray:
        return self.ctx.fetch(self)


class _BatchRef:
    """An operand inside a Batch: one of its inputs (index >= 0) or the result of one of its entries (< 0)."""
    __slots__ = ("batch", "index")

    def __init__(self, batch, index):
        self.batch, self.index = batch, index


class Batch:
    """A sequence of operations written once and recorded with one call per use (lt_op_many): what a front end's
    operator expands to, e.g. the thirteen operations and three in-place updates of one Adam parameter update.  It has
    the recording interface of a context (`op`, `assign`), so the same function that traces on a context builds it:

        b = Batch(); p, g, lr = b.input(), b.input(), b.input()
        b.assign(p, b.op("sub", p, b.op("mul", g, lr)))
        ...
        ctx.record(b, [p_tensor, g_tensor, lr_scalar])        # every step, for every parameter
    """

    def __init__(self):
        self._ops, self._attrs, self._n_inputs, self._kept = [], [], 0, []
        self._c = None

    def input(self) -> _BatchRef:
        self._n_inputs += 1
        return _BatchRef(self, self._n_inputs - 1)

    def op(self, name: str, *inputs, **attrs) -> _BatchRef:
        a = _attr_list(name, attrs)
        self._ops.append((OPCODES[name], [r.index for r in inputs], len(self._attrs), len(a), 0))
        self._attrs.extend(a)
        self._c = None
        return _BatchRef(self, -len(self._ops))

    def assign(self, dst: _BatchRef, src: _BatchRef) -> None:
        self._ops.append((LT_BATCH_ASSIGN, [dst.index, src.index], 0, 0, 0))
        self._c = None

    def keep(self, ref: _BatchRef) -> None:
        """The result `ref` is handed back by LazyContext.record (in the order of the keep calls)."""
        k = -ref.index - 1
        op = self._ops[k]
        self._ops[k] = op[:4] + (1,)
        self._kept.append(k)
        self._c = None

    def _compiled(self):
        if self._c is None:
            ops = (lt_batch_op * max(len(self._ops), 1))()
            for k, (code, ins, off, na, keep) in enumerate(self._ops):
                ops[k].opcode, ops[k].n_in, ops[k].n_attrs, ops[k].attr_offset, ops[k].keep = code, len(ins), na, off, keep
                for i, r in enumerate(ins):
                    ops[k].in_[i] = r
            attrs = (_i64 * max(len(self._attrs), 1))(*self._attrs)
            self._c = (ops, attrs, (_u64 * max(len(self._ops), 1))(), (_u64 * max(self._n_inputs, 1))())
        return self._c


def _attr_list(name: str, attrs: dict) -> list:
    if not attrs:
        return []
    if name == "convert":
        return [DTYPES[attrs["dtype"]]]
    if name == "reshape":
        shp = tuple(attrs["shape"])
        return [len(shp), *shp]
    if name == "narrow":
        return [int(attrs["dim"]), int(attrs["start"]), int(attrs["length"])]
    if name == "permute":
        return [int(p) for p in attrs["perm"]]
    if name == "update_slice":
        return [int(attrs["dim"]), int(attrs["start"])]
    if name == "iota":
        shp = tuple(attrs["shape"])
        return [int(attrs["dim"]), len(shp), *shp]
    shp = tuple(attrs["shape"])  # philox_bits
    seed, off = int(attrs["seed"]), int(attrs["offset"])
    # 64-bit patterns travel as signed int64
    return [seed - (1 << 64) if seed >= (1 << 63) else seed, off - (1 << 64) if off >= (1 << 63) else off, len(shp), *shp]


class LazyContext:
    """One per device: the liveness arena, IR recorder, compile cache and executor."""

    def __init__(self, device: int | None = 0, stream: int | None = None, allocator: str = "torch"):
        self._ctx = None
        self.device = LT_DEVICE_NONE if device is None else int(device)
        self._alloc_struct = None
        alloc_ptr = None
        if self.device != LT_DEVICE_NONE and allocator == "torch":
            import torch

            torch.cuda.set_device(self.device)
            if stream is None:
                stream = torch.cuda.current_stream(self.device).cuda_stream
            a, f = _torch_allocator()
            self._alloc_struct = lt_allocator(a, f, None)
            alloc_ptr = ctypes.byref(self._alloc_struct)
        out = _vp()
        st = _lib.lt_ctx_create(self.device, _vp(stream or 0), alloc_ptr, ctypes.byref(out))
        if st != 0:
            raise LazyTensorError(st, "lt_ctx_create failed (is a CUDA device present?)")
        self._ctx = out
        self.stream = stream or 0
        self._h = _u64()
        self._hp = ctypes.byref(self._h)
        self._ins = (_u64 * 3)()
        self._attrs = (_i64 * (3 + LT_MAX_RANK))()
        self._dead: list[int] = []
        self._keeps: list = []

    def close(self):
        if self._ctx:
            ctx, self._ctx = self._ctx, None
            if _lib is not None:  # module globals may already be gone at interpreter shutdown
                _lib.lt_ctx_destroy(ctx)

    def _flush_dead(self):
        """Unregister the tensors Python has dropped since the last flush."""
        dead = self._dead
        if dead and self._ctx:
            self._dead = []
            n = len(dead)
            self._check(_lib.lt_release_many(self._ctx, (_u64 * n)(*dead), n))

    def __del__(self):
        self.close()

    def _check(self, st: int):
        if st != 0:
            raise LazyTensorError(st, _lib.lt_last_error(self._ctx).decode())

    def set_option(self, key: str, value: int) -> None:
        self._check(_lib.lt_ctx_set_option(self._ctx, key.encode(), int(value)))

    # ---- factories
    def from_device_ptr(self, ptr: int, dtype: str, shape, keep=None) -> LazyTensor:
        shp = (_i64 * max(len(shape), 1))(*shape)
        self._check(_lib.lt_tensor_from_device(self._ctx, _vp(ptr), DTYPES[dtype], len(shape), shp, ctypes.byref(self._h)))
        return LazyTensor(self, self._h.value, dtype, shape, keep)

    def from_torch(self, t, dtype: str | None = None) -> LazyTensor:
        """Wrap a contiguous CUDA torch tensor without copying (the tensor is kept alive)."""
        import torch

        names = {torch.float32: "f32", torch.bfloat16: "bf16", torch.uint8: "u8", torch.int32: "i32",
                 torch.uint16: "bf16", torch.int16: "bf16", torch.uint32: "u32"}
        if dtype is None:
            dtype = names[t.dtype]
        if not t.is_contiguous():
            raise ValueError("tensor must be contiguous")
        return self.from_device_ptr(t.data_ptr(), dtype, tuple(t.shape), keep=t)

    def from_host(self, array: np.ndarray, dtype: str) -> LazyTensor:
        a = np.ascontiguousarray(array, dtype=NP_DTYPES[dtype])
        shp = (_i64 * max(a.ndim, 1))(*a.shape)
        self._check(_lib.lt_tensor_from_host(self._ctx, _vp(a.ctypes.data), DTYPES[dtype], a.ndim, shp, ctypes.byref(self._h)))
        return LazyTensor(self, self._h.value, dtype, a.shape, keep=a)

    def leaf(self, array: np.ndarray, dtype: str) -> LazyTensor:
        """Materialised input from a numpy array in storage representation (bf16 as uint16 bits)."""
        a = np.ascontiguousarray(array, dtype=NP_DTYPES[dtype])
        if self.device == LT_DEVICE_NONE:
            return self.from_device_ptr(a.ctypes.data or 16, dtype, a.shape, keep=a)
        import torch

        host = torch.from_numpy(a.view(np.int16) if dtype == "bf16" else a.view(np.int32) if dtype == "u32" else a)
        dev = host.to(f"cuda:{self.device}")
        return self.from_device_ptr(dev.data_ptr(), dtype, a.shape, keep=dev)

    def scalar(self, value: float, dtype: str = "f32", dynamic: bool = False) -> LazyTensor:
        fn = _lib.lt_scalar_dynamic if dynamic else _lib.lt_scalar
        self._check(fn(self._ctx, float(value), DTYPES[dtype], ctypes.byref(self._h)))
        return LazyTensor(self, self._h.value, dtype, ())

    # ---- recording
    def op(self, name: str, *inputs, **attrs) -> LazyTensor:
        ins = self._ins
        n = 0
        for t in inputs:
            ins[n] = t.handle
            n += 1
        at = self._attrs
        na = 0
        if attrs:
            a = _attr_list(name, attrs)
            na = len(a)
            for i in range(na):
                at[i] = a[i]
        st = _lib.lt_op(self._ctx, OPCODES[name], ins, n, at, na, self._hp)
        if st:
            self._check(st)
        return LazyTensor(self, self._h.value)

    def _info(self, handle: int):
        dt, rk, mat = _int(), _int(), _int()
        shp = (_i64 * LT_MAX_RANK)()
        self._check(_lib.lt_tensor_info(self._ctx, handle, ctypes.byref(dt), ctypes.byref(rk), shp, ctypes.byref(mat)))
        return DTYPE_NAMES[dt.value], rk.value, tuple(shp[: rk.value]), bool(mat.value)

    def is_materialised(self, t: LazyTensor) -> bool:
        return self._info(t.handle)[3]

    # ---- views (paper Section 4.4): results that follow, and are followed by, in-place updates of their base
    def view_reshape(self, t: LazyTensor, shape) -> LazyTensor:
        shp = (_i64 * max(len(shape), 1))(*shape)
        self._check(_lib.lt_view_reshape(self._ctx, t.handle, len(shape), shp, ctypes.byref(self._h)))
        return LazyTensor(self, self._h.value, keep=t._keep)

    def view_narrow(self, t: LazyTensor, dim: int, start: int, length: int) -> LazyTensor:
        self._check(_lib.lt_view_narrow(self._ctx, t.handle, int(dim), int(start), int(length), ctypes.byref(self._h)))
        return LazyTensor(self, self._h.value, keep=t._keep)

    def view_permute(self, t: LazyTensor, perm) -> LazyTensor:
        p = (_int * max(len(perm), 1))(*perm)
        self._check(_lib.lt_view_permute(self._ctx, t.handle, p, ctypes.byref(self._h)))
        return LazyTensor(self, self._h.value, keep=t._keep)

    def assign(self, dst: LazyTensor, src: LazyTensor) -> None:
        self._check(_lib.lt_assign(self._ctx, dst.handle, src.handle))

    def record(self, batch: Batch, inputs) -> list:
        """lt_op_many: records the operations of `batch` on `inputs` in one call; returns the results it keeps."""
        ops, attrs, results, ins = batch._compiled()
        n = 0
        for t in inputs:
            ins[n] = t.handle
            n += 1
        if n != batch._n_inputs:
            raise ValueError(f"the batch takes {batch._n_inputs} inputs, {n} given")
        st = _lib.lt_op_many(self._ctx, ops, len(batch._ops), ins, n, attrs, results)
        if st:
            self._check(st)
        return [LazyTensor(self, results[k]) for k in batch._kept]

    def release(self, t: LazyTensor) -> None:
        t.ctx = None
        self._check(_lib.lt_release(self._ctx, t.handle))

    def barrier(self, blocking: bool = False) -> None:
        if self._dead:
            self._flush_dead()
        keeps, self._keeps = self._keeps, []
        st = _lib.lt_barrier(self._ctx, 1 if blocking else 0)
        if st:
            self._keeps.extend(keeps)
            self._check(st)

    def debug_bounds_violations(self) -> int | None:
        """Out-of-bounds accesses the compiled kernels caught (debug build), or None in a release build."""
        n = _u64()
        st = _lib.lt_debug_bounds_violations(self._ctx, ctypes.byref(n))
        if st == STATUS_NAMES.index("LT_ERR_UNSUPPORTED"):
            return None
        self._check(st)
        return n.value

    def debug_wait_probe(self, limit_ns: int) -> None:
        """lt_debug_wait_probe: enqueue a kernel whose bounded wait runs out (see LT_ERR_DEVICE_TIMEOUT)."""
        self._check(_lib.lt_debug_wait_probe(self._ctx, int(limit_ns)))

    def replay(self, blocking: bool = False) -> None:
        """lt_replay: run the previously flushed graph again on the same tensors, without recording it."""
        self._check(_lib.lt_replay(self._ctx, 1 if blocking else 0))

    def scalar_set(self, scalar: LazyTensor, value: float) -> None:
        self._check(_lib.lt_scalar_set(self._ctx, scalar.handle, float(value)))

    def replay_slots(self) -> int:
        n = ctypes.c_uint32()
        self._check(_lib.lt_replay_slots(self._ctx, ctypes.byref(n)))
        return n.value

    def replay_set_slot(self, slot: int, value, integer: bool = False) -> None:
        iv = int(value) if integer else 0
        if iv >= (1 << 63):
            iv -= 1 << 64
        self._check(_lib.lt_replay_set_slot(self._ctx, slot, 1 if integer else 0, 0.0 if integer else float(value), iv))

    def barrier_static_scratch(self, blocking: bool = False, clear_first: bool = False) -> None:
        """lt_barrier_static_scratch: the flush for callers that may not allocate device memory (results go to
        caller buffers via `assign`, temporaries to the library's fixed scratch array)."""
        if self._dead:
            self._flush_dead()
        keeps, self._keeps = self._keeps, []
        st = _lib.lt_barrier_static_scratch(self._ctx, 1 if blocking else 0, 1 if clear_first else 0)
        if st:
            self._keeps.extend(keeps)
            self._check(st)

    def fetch(self, t: LazyTensor) -> np.ndarray:
        self._flush_dead()
        out = np.empty(t.shape, dtype=NP_DTYPES[t.dtype])
        keeps, self._keeps = self._keeps, []
        st = _lib.lt_fetch(self._ctx, t.handle, _vp(out.ctypes.data), out.nbytes)
        if st:
            self._keeps.extend(keeps)
            self._check(st)
        return out

    def fetch_into(self, t: LazyTensor, host_ptr: int, nbytes: int) -> None:
        self._flush_dead()
        keeps, self._keeps = self._keeps, []
        st = _lib.lt_fetch(self._ctx, t.handle, _vp(host_ptr), nbytes)
        if st:
            self._keeps.extend(keeps)
            self._check(st)

    def device_ptr(self, t: LazyTensor) -> int:
        p = _vp()
        self._check(_lib.lt_device_ptr(self._ctx, t.handle, ctypes.byref(p)))
        return p.value or 0

    # ---- introspection
    def stats(self) -> dict:
        s = lt_stats()
        self._check(_lib.lt_get_stats(self._ctx, ctypes.byref(s)))
        return {n: getattr(s, n) for n, _ in lt_stats._fields_}

    def reset_stats(self) -> None:
        self._check(_lib.lt_reset_stats(self._ctx))

    def cache_size(self) -> int:
        n = _u64()
        self._check(_lib.lt_cache_size(self._ctx, ctypes.byref(n)))
        return n.value

    def set_kernel_timing(self, on: bool) -> None:
        self._check(_lib.lt_set_kernel_timing(self._ctx, 1 if on else 0))

    def kernel_timing(self) -> dict:
        t = lt_kernel_timing()
        self._check(_lib.lt_get_kernel_timing(self._ctx, ctypes.byref(t)))
        names = ("elementwise", "row", "multi")
        return {n: {"launches": t.launches[i], "ms": t.ms[i], "bytes": t.bytes[i]} for i, n in enumerate(names)}

    def _text(self, fn) -> str:
        need = ctypes.c_size_t()
        self._check(fn(self._ctx, None, 0, ctypes.byref(need)))
        buf = ctypes.create_string_buffer(need.value)
        self._check(fn(self._ctx, buf, need.value, ctypes.byref(need)))
        return buf.value.decode()

    def dump_ir(self) -> str:
        self._flush_dead()
        return self._text(_lib.lt_dump_ir)

    def dump_plan(self) -> str:
        return self._text(_lib.lt_dump_plan)
