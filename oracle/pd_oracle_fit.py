"""ctypes front end of the scale-fitting CPU oracle (oracle/pd_oracle_fit.c).  TEST INFRASTRUCTURE ONLY."""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

AXIS_ROW, AXIS_COL, AXIS_SCALAR = 0, 1, 2

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pd_oracle_fit.c")
_LIB = os.path.join(_HERE, "libpd_oracle_fit.so")
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _bind(path):
    lib = ctypes.CDLL(path)
    p, i64, d = ctypes.c_void_p, ctypes.c_int64, ctypes.c_double
    lib.pdf_loss_grad.argtypes = [p, p, i64, p, p, p, ctypes.c_int, i64, i64, p]
    lib.pdf_loss_grad.restype = d
    lib.pdf_adamw_step.argtypes = [p, p, p, p, i64, i64, d, d, d, d, d]
    lib.pdf_adamw_step.restype = None
    return lib


def _load():
    global _lib
    if _lib is None:
        _lib = _bind(build())
    return _lib


class use_library:
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


def vector_length(axis, d_out, d_in):
    return d_out if axis == AXIS_ROW else (d_in if axis == AXIS_COL else 1)


def loss_grad(x, y, w_b, mask, v, axis, want_grad=True):
    """(loss, grad fp64) of the output-matching objective; x, y, w_b float16, v any float array of the axis' length."""
    x, y, w_b = (np.ascontiguousarray(a) for a in (x, y, w_b))
    assert x.dtype == y.dtype == w_b.dtype == np.float16
    mask = np.ascontiguousarray(mask, dtype=np.uint32)
    d_out, d_in = w_b.shape
    m = x.shape[0]
    assert x.shape == (m, d_in) and y.shape == (m, d_out)
    v = np.ascontiguousarray(v, dtype=np.float64)
    assert v.shape == (vector_length(axis, d_out, d_in),)
    grad = np.empty_like(v) if want_grad else None
    loss = _load().pdf_loss_grad(_ptr(x), _ptr(y), m, _ptr(w_b), _ptr(mask), _ptr(v), int(axis), d_out, d_in, _ptr(grad))
    return loss, grad


def adamw_step(v, m1, m2, g, t, lr, b1=0.9, b2=0.999, eps=1e-8, wd=0.01):
    """In place on the fp64 arrays v, m1, m2."""
    for a in (v, m1, m2):
        assert a.dtype == np.float64 and a.flags.c_contiguous
    g = np.ascontiguousarray(g, dtype=np.float64)
    _load().pdf_adamw_step(_ptr(v), _ptr(m1), _ptr(m2), _ptr(g), v.shape[0], int(t), lr, b1, b2, eps, wd)


def train(x_tr, y_tr, x_val, y_val, w_b, mask, v0, axis, epochs, batch, lr, b1=0.9, b2=0.999, eps=1e-8, wd=0.01, cosine=False):
    """Algorithm "Train per-row/column scaling vectors via activation matching": for each epoch, for each minibatch
    (consecutive `batch` tokens of the training cache, the last one possibly shorter): loss, gradient with respect to
    v only, one AdamW step; with `cosine` the step k = 0 .. T-1 (T = all steps) uses lr * (1 + cos(pi k / T)) / 2.
    Then the validation loss without gradient.  Returns (v, validation loss)."""
    v = np.array(v0, dtype=np.float64)
    m1, m2 = np.zeros_like(v), np.zeros_like(v)
    m_tr = x_tr.shape[0]
    total = epochs * ((m_tr + batch - 1) // batch)
    k = 0
    for _ in range(epochs):
        for b0 in range(0, m_tr, batch):
            _, g = loss_grad(x_tr[b0:b0 + batch], y_tr[b0:b0 + batch], w_b, mask, v, axis)
            lr_k = lr * 0.5 * (1.0 + np.cos(np.pi * k / total)) if cosine else lr
            k += 1
            adamw_step(v, m1, m2, g, k, lr_k, b1, b2, eps, wd)
    val, _ = loss_grad(x_val, y_val, w_b, mask, v, axis, want_grad=False)
    return v, val


def fit_layer(x_tr, y_tr, x_val, y_val, w_b, mask, v_row0, v_col0, epochs, batch, lr, **kw):
    """Algorithm "Per-layer compression with Row/Col selection": both variants start from the packed scales and get
    the same budget; the row variant is kept when E_row <= E_col.  The error compared is the validation loss of the
    layer's outputs (the paper's training paragraph: "selected by validation MSE on the held-out shard").
    Returns (axis, v of that axis, (E_row, E_col), (v_row, v_col))."""
    v_col, e_col = train(x_tr, y_tr, x_val, y_val, w_b, mask, np.asarray(v_col0, dtype=np.float64), AXIS_COL, epochs, batch, lr, **kw)
    v_row, e_row = train(x_tr, y_tr, x_val, y_val, w_b, mask, np.asarray(v_row0, dtype=np.float64), AXIS_ROW, epochs, batch, lr, **kw)
    axis = AXIS_ROW if e_row <= e_col else AXIS_COL
    return axis, (v_row if axis == AXIS_ROW else v_col), (e_row, e_col), (v_row, v_col)
