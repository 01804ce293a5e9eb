"""ctypes front end of the BF16 CPU oracle (oracle/pd_oracle_bf16.c).

TEST INFRASTRUCTURE ONLY.  Imported by the tests, by the smoke check and by the benchmark's
CPU legs; never by the product package.  bfloat16 tensors travel as numpy uint16 arrays (the
upper halves of binary32 values); the scale vectors are numpy float16.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

AXIS_ROW = 0
AXIS_COL = 1

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pd_oracle_bf16.c")
_LIB = os.path.join(_HERE, "libpd_oracle_bf16.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle if the shared object is missing or older than its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-frounding-math", "-fopenmp", "-shared", "-fPIC",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _bind(path):
    lib = ctypes.CDLL(path)
    p, i64, i32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32
    lib.pdb_bf16_to_double.argtypes = [ctypes.c_uint16]
    lib.pdb_bf16_to_double.restype = ctypes.c_double
    lib.pdb_double_to_bf16.argtypes = [ctypes.c_double]
    lib.pdb_double_to_bf16.restype = ctypes.c_uint16
    lib.pdb_pack.argtypes = [p, p, i64, i64, p, p, p]
    lib.pdb_pack.restype = ctypes.c_int
    lib.pdb_reconstruct.argtypes = [p, p, p, ctypes.c_int, i64, i64, p]
    lib.pdb_reconstruct.restype = None
    lib.pdb_merge.argtypes = [p, p, p, ctypes.c_int, i64, i64, p]
    lib.pdb_merge.restype = None
    lib.pdb_linear.argtypes = [p, i64, i64, p, p, p, ctypes.c_int, i64, i64, p]
    lib.pdb_linear.restype = None
    lib.pdb_linear_multivariant.argtypes = [p, i64, i64, p, p, p, p, i64, p, i32, i64, i64, p]
    lib.pdb_linear_multivariant.restype = ctypes.c_int
    return lib


def _load():
    global _lib
    if _lib is None:
        _lib = _bind(build())
    return _lib


class use_library:
    """Context manager: route every call of this module to another build of the C file
    (the mutation tests compile deliberately broken copies and check that the pins notice)."""

    def __init__(self, path):
        self.path = path

    def __enter__(self):
        global _lib
        self.saved = _lib
        _lib = _bind(self.path)
        return self

    def __exit__(self, *exc):
        global _lib
        _lib = self.saved
        return False


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _u16(a, name):
    a = np.ascontiguousarray(a)
    if a.dtype != np.uint16:
        raise TypeError(f"{name} must be uint16 (bfloat16 bit patterns)")
    return a


def _f16(a, name):
    a = np.ascontiguousarray(a)
    if a.dtype != np.float16:
        raise TypeError(f"{name} must be float16")
    return a


def bf16_to_double(bits: int) -> float:
    return _load().pdb_bf16_to_double(int(bits))


def double_to_bf16(value: float) -> int:
    return _load().pdb_double_to_bf16(float(value))


def pack(w_f, w_b, want_row=True, want_col=True):
    """(mask uint32 [d_out, d_in/32], v_row fp16 [d_out] | None, v_col fp16 [d_in] | None)."""
    w_f, w_b = _u16(w_f, "w_f"), _u16(w_b, "w_b")
    d_out, d_in = w_b.shape
    assert w_f.shape == w_b.shape and d_in % 32 == 0
    mask = np.empty((d_out, d_in // 32), dtype=np.uint32)
    v_row = np.empty(d_out, dtype=np.float16) if want_row else None
    v_col = np.empty(d_in, dtype=np.float16) if want_col else None
    bad = _load().pdb_pack(_ptr(w_f), _ptr(w_b), d_out, d_in, _ptr(mask), _ptr(v_row), _ptr(v_col))
    if bad:
        raise OverflowError("sum of |dW| units >= 2^53: fp64 accumulation no longer exact")
    return mask, v_row, v_col


def reconstruct(w_b, mask, v, axis):
    w_b, v = _u16(w_b, "w_b"), _f16(v, "v")
    mask = np.ascontiguousarray(mask, dtype=np.uint32)
    d_out, d_in = w_b.shape
    assert v.shape[0] == (d_out if axis == AXIS_ROW else d_in)
    out = np.empty((d_out, d_in), dtype=np.float64)
    _load().pdb_reconstruct(_ptr(w_b), _ptr(mask), _ptr(v), axis, d_out, d_in, _ptr(out))
    return out


def merge(w_b, mask, v, axis):
    """bfloat16 bit patterns [d_out, d_in] of bf16(fp32(W_b) +- fp32(v))."""
    w_b, v = _u16(w_b, "w_b"), _f16(v, "v")
    mask = np.ascontiguousarray(mask, dtype=np.uint32)
    d_out, d_in = w_b.shape
    assert v.shape[0] == (d_out if axis == AXIS_ROW else d_in)
    out = np.empty((d_out, d_in), dtype=np.uint16)
    _load().pdb_merge(_ptr(w_b), _ptr(mask), _ptr(v), axis, d_out, d_in, _ptr(out))
    return out


def linear(x, w_b, mask, v, axis):
    """y fp64 [M, d_out] = x . (W_b + v (.) B)^T with unrounded W_hat; x and w_b are bfloat16 bit patterns."""
    x, w_b, v = _u16(x, "x"), _u16(w_b, "w_b"), _f16(v, "v")
    mask = np.ascontiguousarray(mask, dtype=np.uint32)
    d_out, d_in = w_b.shape
    m = x.shape[0]
    assert x.shape[1] == d_in and v.shape[0] == (d_out if axis == AXIS_ROW else d_in)
    y = np.empty((m, d_out), dtype=np.float64)
    _load().pdb_linear(_ptr(x), m, d_in, _ptr(w_b), _ptr(mask), _ptr(v), axis, d_out, d_in, _ptr(y))
    return y


def linear_multivariant(x, ids, w_b, masks, vs, axes):
    """Row m uses variant ids[m]; masks [V, d_out, d_in/32], vs fp16 [V, v_stride], axes uint8 [V]."""
    x, w_b, vs = _u16(x, "x"), _u16(w_b, "w_b"), _f16(vs, "vs")
    masks = np.ascontiguousarray(masks, dtype=np.uint32)
    ids = np.ascontiguousarray(ids, dtype=np.int32)
    axes = np.ascontiguousarray(axes, dtype=np.uint8)
    d_out, d_in = w_b.shape
    m, n_var = x.shape[0], masks.shape[0]
    assert masks.shape == (n_var, d_out, d_in // 32) and vs.shape[0] == n_var
    y = np.empty((m, d_out), dtype=np.float64)
    bad = _load().pdb_linear_multivariant(_ptr(x), m, d_in, _ptr(ids), _ptr(w_b), _ptr(masks), _ptr(vs),
                                          vs.shape[1], _ptr(axes), n_var, d_out, d_in, _ptr(y))
    return y, bad
