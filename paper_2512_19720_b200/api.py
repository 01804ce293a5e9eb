"""Thin Python binding of the C ABI in include/pd.h (ctypes, argument marshalling only).

Every function takes torch CUDA tensors, passes their device pointers and the current
stream to the library and returns torch tensors.  No arithmetic of the method happens in
Python.  If the CUDA library is missing the import fails loudly: there is no CPU fallback.
"""
from __future__ import annotations

import ctypes
import os

import torch

AXIS_ROW = 0
AXIS_COL = 1
AXIS_SCALAR = 2  # pd_fit_* only
OP_PACK, OP_LINEAR, OP_LINEAR_MULTIVARIANT, OP_MERGE, OP_FIT, OP_FIT_LAYER = 0, 1, 2, 3, 4, 5

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpd.so")

EXPORTS = ["pd_pack_delta", "pd_pack_delta_static", "pd_linear_host", "pd_linear", "pd_linear_ex", "pd_linear_multivariant", "pd_merge",
           "pd_workspace_bytes", "pd_device_status", "pd_status_string", "pd_launch_count", "pd_selftest_bounded_wait",
           "pd_pack_delta_bf16", "pd_merge_bf16", "pd_linear_bf16", "pd_linear_multivariant_bf16",
           "pd_artifact_bytes", "pd_load_merged",
           "pd_transpose_mask", "pd_fit_loss_grad", "pd_fit_adamw_step", "pd_fit_layer"]
LINEAR_WEIGHTS_RESIDENT = 1


class PdModule(ctypes.Structure):
    """pd_module of include/pd.h."""
    _fields_ = [("w_b", ctypes.c_void_p), ("w_hat", ctypes.c_void_p), ("artifact", ctypes.c_void_p),
                ("d_out", ctypes.c_int64), ("d_in", ctypes.c_int64), ("axis", ctypes.c_int32), ("bf16", ctypes.c_int32)]


class PdAdamW(ctypes.Structure):
    """pd_adamw of include/pd.h."""
    _fields_ = [("lr", ctypes.c_float), ("beta1", ctypes.c_float), ("beta2", ctypes.c_float), ("eps", ctypes.c_float),
                ("weight_decay", ctypes.c_float)]


class PdError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} (pd_status {code})")


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2512_19720_b200.build` "
                          "(there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    p, i64, i32, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_size_t
    lib.pd_pack_delta.argtypes = [p, p, i64, i64, p, p, p, p, sz, p]
    lib.pd_pack_delta.restype = ctypes.c_int
    lib.pd_pack_delta_static.argtypes = [p, p, i64, i64, p, p, p, p]
    lib.pd_pack_delta_static.restype = ctypes.c_int
    lib.pd_linear.argtypes = [p, i64, i64, p, p, p, ctypes.c_int, i64, i64, p, i64, p, sz, p]
    lib.pd_linear.restype = ctypes.c_int
    lib.pd_linear_ex.argtypes = [p, i64, i64, p, p, p, ctypes.c_int, i64, i64, p, i64, p, sz, p, ctypes.c_uint32]
    lib.pd_linear_ex.restype = ctypes.c_int
    lib.pd_linear_host.argtypes = [p, p, i64, p, p, p, ctypes.c_int, i64, i64, p, p, p, sz, p, ctypes.c_uint32]
    lib.pd_linear_host.restype = ctypes.c_int
    lib.pd_selftest_bounded_wait.argtypes = [p, i64, p]
    lib.pd_selftest_bounded_wait.restype = ctypes.c_int
    lib.pd_linear_multivariant.argtypes = [p, i64, i64, p, p, p, p, i64, p, i32, i64, i64, p, i64, p, sz, p]
    lib.pd_linear_multivariant.restype = ctypes.c_int
    lib.pd_merge.argtypes = [p, p, p, ctypes.c_int, i64, i64, p, p]
    lib.pd_merge.restype = ctypes.c_int
    lib.pd_workspace_bytes.argtypes = [ctypes.c_int, i64, i32, i64, i64]
    lib.pd_workspace_bytes.restype = sz
    lib.pd_device_status.argtypes = [p, p]
    lib.pd_device_status.restype = ctypes.c_int
    lib.pd_status_string.argtypes = [ctypes.c_int]
    lib.pd_status_string.restype = ctypes.c_char_p
    lib.pd_artifact_bytes.argtypes = [i64, i64, ctypes.c_int]
    lib.pd_artifact_bytes.restype = sz
    lib.pd_load_merged.argtypes = [ctypes.POINTER(PdModule), i32, p, sz, p, p]
    lib.pd_load_merged.restype = ctypes.c_int
    lib.pd_transpose_mask.argtypes = [p, i64, i64, p, p]
    lib.pd_transpose_mask.restype = ctypes.c_int
    lib.pd_fit_loss_grad.argtypes = [p, p, i64, p, p, p, p, ctypes.c_int, i64, i64, p, p, p, sz, p]
    lib.pd_fit_loss_grad.restype = ctypes.c_int
    lib.pd_fit_adamw_step.argtypes = [p, p, p, p, i64, i64, ctypes.POINTER(PdAdamW), p]
    lib.pd_fit_adamw_step.restype = ctypes.c_int
    lib.pd_fit_layer.argtypes = [p, p, i64, p, p, i64, p, p, p, p, i64, i64, i32, i64, ctypes.POINTER(PdAdamW), i32, p, p, p, p, sz, p]
    lib.pd_fit_layer.restype = ctypes.c_int
    lib.pd_launch_count.argtypes = []
    lib.pd_launch_count.restype = i64
    for name, proto in (("pd_pack_delta_bf16", lib.pd_pack_delta), ("pd_merge_bf16", lib.pd_merge),
                        ("pd_linear_bf16", lib.pd_linear_ex), ("pd_linear_multivariant_bf16", lib.pd_linear_multivariant)):
        fn = getattr(lib, name)
        fn.argtypes, fn.restype = proto.argtypes, ctypes.c_int
        assert fn.argtypes is not None
    return lib


lib = _load()


def status_string(code: int) -> str:
    return lib.pd_status_string(int(code)).decode()


def launch_count() -> int:
    return int(lib.pd_launch_count())


def workspace_bytes(op: int, m: int = 0, n_variants: int = 0, d_out: int = 0, d_in: int = 0) -> int:
    return int(lib.pd_workspace_bytes(op, m, n_variants, d_out, d_in))


_ws_cache: dict = {}


def _workspace(nbytes: int, device) -> torch.Tensor:
    """A cached scratch tensor of at least nbytes on `device` (torch allocations are 512-byte aligned)."""
    key = (device.type, device.index)
    ws = _ws_cache.get(key)
    if ws is None or ws.numel() < nbytes:
        ws = torch.zeros(max(nbytes, 1 << 20), dtype=torch.uint8, device=device)
        _ws_cache[key] = ws
    return ws


_pack_ws_cache: dict = {}


def _pack_workspace(nbytes: int, device) -> torch.Tensor:
    """The pack call's own scratch tensor: it must be all zero on entry, and the call leaves it all zero, so it is
    kept apart from the workspace the linear calls write into."""
    key = (device.type, device.index)
    ws = _pack_ws_cache.get(key)
    if ws is None or ws.numel() < nbytes:
        ws = torch.zeros(max(nbytes, 1 << 20), dtype=torch.uint8, device=device)
        _pack_ws_cache[key] = ws
    return ws


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _check(code: int, where: str):
    if code != 0:
        raise PdError(code, where)


def _ptr(t):
    return None if t is None else t.data_ptr()


def _want(t, dtype, name):
    if not t.is_cuda or t.dtype != dtype:
        raise TypeError(f"{name} must be a CUDA tensor of {dtype}")


def _elem(t, name):
    """True for bfloat16 weights / activations, False for float16 (the two storage types the library has)."""
    if not t.is_cuda or t.dtype not in (torch.float16, torch.bfloat16):
        raise TypeError(f"{name} must be a CUDA tensor of float16 or bfloat16")
    return t.dtype == torch.bfloat16


def pd_pack_delta(w_f, w_b, want_row=True, want_col=True, mask=None, v_row=None, v_col=None, workspace=None):
    """mask uint32-as-int32 [d_out, d_in/32], v_row fp16 [d_out] | None, v_col fp16 [d_in] | None.
    A workspace passed in must be all zero (the call leaves it so)."""
    bf16 = _elem(w_b, "w_b")
    _want(w_f, w_b.dtype, "w_f")
    assert w_f.shape == w_b.shape and w_f.is_contiguous() and w_b.is_contiguous()
    d_out, d_in = w_b.shape
    dev = w_b.device
    if mask is None:
        mask = torch.empty((d_out, d_in // 32), dtype=torch.int32, device=dev)
    if want_row and v_row is None:
        v_row = torch.empty(d_out, dtype=torch.float16, device=dev)
    if want_col and v_col is None:
        v_col = torch.empty(d_in, dtype=torch.float16, device=dev)
    need = workspace_bytes(OP_PACK, 0, 0, d_out, d_in)
    ws = workspace if workspace is not None else _pack_workspace(need, dev)
    fn = lib.pd_pack_delta_bf16 if bf16 else lib.pd_pack_delta
    _check(fn(_ptr(w_f), _ptr(w_b), d_out, d_in, _ptr(mask), _ptr(v_row if want_row else None),
              _ptr(v_col if want_col else None), _ptr(ws), ws.numel() * ws.element_size(), _stream()), "pd_pack_delta")
    return mask, (v_row if want_row else None), (v_col if want_col else None)


def pd_pack_delta_static(w_f, w_b, mask, v_row=None, v_col=None):
    """pd_pack_delta for callers that cannot allocate: every output is a tensor the caller already
    owns, the scratch sums live in a fixed array inside the library (d_out + d_in <= 65536), and
    neither this wrapper nor the library call allocates anything.  Calls that overlap on one GPU
    race on that array; calls queued on one stream do not."""
    _want(w_f, torch.float16, "w_f"), _want(w_b, torch.float16, "w_b")
    assert w_f.shape == w_b.shape and w_f.is_contiguous() and w_b.is_contiguous()
    d_out, d_in = w_b.shape
    _check(lib.pd_pack_delta_static(_ptr(w_f), _ptr(w_b), d_out, d_in, _ptr(mask), _ptr(v_row), _ptr(v_col),
                                    _stream()), "pd_pack_delta_static")
    return mask, v_row, v_col


def pd_linear(x, w_b, mask, v, axis, y=None, workspace=None, weights_resident=False):
    """y fp16 [M, d_out] = x . (W_b + v (.) B)^T; mask None = base weights only.  weights_resident=True passes
    PD_LINEAR_WEIGHTS_RESIDENT: no earlier work on the stream writes w_b, mask or v."""
    bf16 = _elem(w_b, "w_b")
    _want(x, w_b.dtype, "x")
    assert x.dim() == 2 and x.stride(1) == 1 and w_b.is_contiguous()
    m, d_in = x.shape
    d_out = w_b.shape[0]
    assert w_b.shape[1] == d_in
    if y is None:
        y = torch.empty((m, d_out), dtype=w_b.dtype, device=x.device)
    assert y.dtype == w_b.dtype
    need = workspace_bytes(OP_LINEAR, m, 0, d_out, d_in)
    ws = workspace if workspace is not None else _workspace(need, x.device)
    fn = lib.pd_linear_bf16 if bf16 else lib.pd_linear_ex
    _check(fn(_ptr(x), m, x.stride(0), _ptr(w_b), _ptr(mask), _ptr(v), int(axis), d_out, d_in, _ptr(y),
              y.stride(0), _ptr(ws), ws.numel() * ws.element_size(), _stream(),
              LINEAR_WEIGHTS_RESIDENT if weights_resident else 0), "pd_linear")
    return y


def pd_linear_host(x_host, x_dev, w_b, mask, v, axis, y_dev, y_host, workspace=None, weights_resident=False):
    """pd_linear with the activations in host memory: x_host (CPU fp16 [M, d_in], ideally pinned) is copied to the
    staging tensor x_dev, the linear runs, y_dev is copied to y_host; all on the current stream, nothing synchronised."""
    assert x_host.dtype == torch.float16 and y_host.dtype == torch.float16 and not x_host.is_cuda and not y_host.is_cuda
    assert x_host.is_contiguous() and y_host.is_contiguous() and x_dev.is_contiguous() and y_dev.is_contiguous()
    m, d_in = x_host.shape
    d_out = w_b.shape[0]
    assert x_dev.numel() >= m * d_in and y_dev.numel() >= m * d_out and tuple(y_host.shape) == (m, d_out)
    need = workspace_bytes(OP_LINEAR, m, 0, d_out, d_in)
    ws = workspace if workspace is not None else _workspace(need, w_b.device)
    _check(lib.pd_linear_host(x_host.data_ptr(), _ptr(x_dev), m, _ptr(w_b), _ptr(mask), _ptr(v), int(axis), d_out, d_in,
                              _ptr(y_dev), y_host.data_ptr(), _ptr(ws), ws.numel() * ws.element_size(), _stream(),
                              LINEAR_WEIGHTS_RESIDENT if weights_resident else 0), "pd_linear_host")
    return y_host


def pd_linear_multivariant(x, variant_ids, w_b, masks, vs, axes, y=None, workspace=None):
    """Row m of x uses variant variant_ids[m] (-1 = base only).  masks [V, d_out, d_in/32], vs fp16
    [V, v_stride], axes: sequence of V axis codes (host)."""
    bf16 = _elem(w_b, "w_b")
    _want(x, w_b.dtype, "x"), _want(variant_ids, torch.int32, "variant_ids"), _want(vs, torch.float16, "vs")
    assert x.dim() == 2 and x.stride(1) == 1 and w_b.is_contiguous() and masks.is_contiguous() and vs.is_contiguous()
    m, d_in = x.shape
    d_out = w_b.shape[0]
    n_var = masks.shape[0]
    if y is None:
        y = torch.empty((m, d_out), dtype=w_b.dtype, device=x.device)
    assert y.dtype == w_b.dtype
    axes_arr = (ctypes.c_uint8 * n_var)(*[int(a) for a in axes])
    need = workspace_bytes(OP_LINEAR_MULTIVARIANT, m, n_var, d_out, d_in)
    ws = workspace if workspace is not None else _workspace(need, x.device)
    fn = lib.pd_linear_multivariant_bf16 if bf16 else lib.pd_linear_multivariant
    _check(fn(_ptr(x), m, x.stride(0), _ptr(variant_ids), _ptr(w_b), _ptr(masks), _ptr(vs),
              vs.stride(0), axes_arr, n_var, d_out, d_in, _ptr(y), y.stride(0), _ptr(ws),
              ws.numel() * ws.element_size(), _stream()), "pd_linear_multivariant")
    return y


def pd_merge(w_b, mask, v, axis, w_hat=None):
    """Dense fp16 W_hat = fp16(fp32(W_b) +- fp32(v)); w_hat may be w_b itself."""
    bf16 = _elem(w_b, "w_b")
    assert w_b.is_contiguous()
    d_out, d_in = w_b.shape
    if w_hat is None:
        w_hat = torch.empty_like(w_b)
    assert w_hat.dtype == w_b.dtype
    _check((lib.pd_merge_bf16 if bf16 else lib.pd_merge)(_ptr(w_b), _ptr(mask), _ptr(v), int(axis), d_out, d_in, _ptr(w_hat), _stream()), "pd_merge")
    return w_hat


def artifact_bytes(d_out: int, d_in: int, axis: int) -> int:
    return int(lib.pd_artifact_bytes(d_out, d_in, int(axis)))


def make_artifact(mask, v, pin=True):
    """One contiguous host buffer (uint8): the mask words, then the scales (the layout pd_load_merged copies)."""
    d_out, words = mask.shape
    mask_bytes = (d_out * words * 4 + 15) // 16 * 16
    buf = torch.zeros(mask_bytes + (v.numel() * 2 + 15) // 16 * 16, dtype=torch.uint8)
    buf[:d_out * words * 4] = mask.detach().cpu().contiguous().view(torch.uint8).reshape(-1)
    buf[mask_bytes:mask_bytes + v.numel() * 2] = v.detach().cpu().contiguous().view(torch.uint8).reshape(-1)
    return buf.pin_memory() if pin else buf


def pd_load_merged(modules, staging, copy_stream):
    """modules: sequence of (w_b, w_hat, artifact (host uint8 tensor from make_artifact), axis).  The copies go to
    copy_stream (a torch.cuda.Stream), the merges to the current stream; nothing is synchronised."""
    arr = (PdModule * len(modules))()
    for i, (w_b, w_hat, art, axis) in enumerate(modules):
        bf16 = _elem(w_b, "w_b")
        assert w_hat.dtype == w_b.dtype and w_b.is_contiguous() and w_hat.is_contiguous() and not art.is_cuda
        d_out, d_in = w_b.shape
        assert art.numel() >= artifact_bytes(d_out, d_in, axis)
        arr[i] = PdModule(w_b.data_ptr(), w_hat.data_ptr(), art.data_ptr(), d_out, d_in, int(axis), int(bf16))
    _check(lib.pd_load_merged(arr, len(modules), _ptr(staging), staging.numel() * staging.element_size(),
                              copy_stream.cuda_stream, _stream()), "pd_load_merged")


def pd_transpose_mask(mask, d_out, d_in, mask_t=None):
    """mask_t [d_in, ceil(d_out/32)]: the sign mask with the roles of rows and columns exchanged."""
    _want(mask, torch.int32, "mask")
    if mask_t is None:
        mask_t = torch.empty(d_in, (d_out + 31) // 32, dtype=torch.int32, device=mask.device)
    _check(lib.pd_transpose_mask(_ptr(mask), d_out, d_in, _ptr(mask_t), _stream()), "pd_transpose_mask")
    return mask_t


def adamw(lr=1e-4, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01) -> PdAdamW:
    return PdAdamW(lr, beta1, beta2, eps, weight_decay)


def pd_fit_loss_grad(x, y, w_b, mask, v, axis, mask_t=None, want_grad=True, loss=None, grad=None, workspace=None):
    """Loss of the batch (x, y) and its gradient with respect to the fp32 scales v; returns (loss, grad) device tensors."""
    _want(x, torch.float16, "x"), _want(y, torch.float16, "y"), _want(w_b, torch.float16, "w_b")
    _want(mask, torch.int32, "mask"), _want(v, torch.float32, "v")
    m, d_in = x.shape
    d_out = w_b.shape[0]
    if loss is None:
        loss = torch.empty(1, dtype=torch.float32, device=x.device)
    if grad is None and want_grad:
        grad = torch.empty_like(v)
    need = workspace_bytes(OP_FIT, m, 0, d_out, d_in)
    ws = workspace if workspace is not None else _workspace(need, x.device)
    _check(lib.pd_fit_loss_grad(_ptr(x), _ptr(y), m, _ptr(w_b), _ptr(mask), _ptr(mask_t), _ptr(v), int(axis), d_out, d_in,
                                _ptr(loss), _ptr(grad) if want_grad else None, _ptr(ws), ws.numel(), _stream()), "pd_fit_loss_grad")
    return loss, grad


def pd_fit_adamw_step(v, m1, m2, grad, t, opt: PdAdamW):
    for name, a in (("v", v), ("m1", m1), ("m2", m2), ("grad", grad)):
        _want(a, torch.float32, name)
    _check(lib.pd_fit_adamw_step(_ptr(v), _ptr(m1), _ptr(m2), _ptr(grad), v.numel(), int(t), ctypes.byref(opt), _stream()),
           "pd_fit_adamw_step")


def pd_fit_layer(x_tr, y_tr, x_val, y_val, w_b, mask, v_row0, v_col0, epochs, batch, opt: PdAdamW, cosine=False, workspace=None):
    """Trains both axis variants and keeps the one with the lower validation loss.
    Returns (v_out fp16 [max(d_out, d_in)], axis_out int32 [1], val_loss fp32 [2]) as device tensors."""
    for name, a in (("x_tr", x_tr), ("y_tr", y_tr), ("x_val", x_val), ("y_val", y_val), ("w_b", w_b), ("v_row0", v_row0), ("v_col0", v_col0)):
        _want(a, torch.float16, name)
    _want(mask, torch.int32, "mask")
    d_out, d_in = w_b.shape
    dev = w_b.device
    v_out = torch.zeros(max(d_out, d_in), dtype=torch.float16, device=dev)
    axis_out = torch.zeros(1, dtype=torch.int32, device=dev)
    val_loss = torch.zeros(2, dtype=torch.float32, device=dev)
    m_max = max(min(batch, x_tr.shape[0]), x_val.shape[0])
    need = workspace_bytes(OP_FIT_LAYER, m_max, 0, d_out, d_in)
    ws = workspace if workspace is not None else _workspace(need, dev)
    _check(lib.pd_fit_layer(_ptr(x_tr), _ptr(y_tr), x_tr.shape[0], _ptr(x_val), _ptr(y_val), x_val.shape[0], _ptr(w_b), _ptr(mask),
                            _ptr(v_row0), _ptr(v_col0), d_out, d_in, int(epochs), int(batch), ctypes.byref(opt), int(bool(cosine)),
                            _ptr(v_out), _ptr(axis_out), _ptr(val_loss), _ptr(ws), ws.numel(), _stream()), "pd_fit_layer")
    return v_out, axis_out, val_loss


def pd_selftest_bounded_wait(limit_cycles=100000, workspace=None, device=None):
    """Launches the probe whose bounded wait runs out after limit_cycles; pd_device_status() then reports 7 once."""
    ws = workspace if workspace is not None else _workspace(256, device or torch.device("cuda", torch.cuda.current_device()))
    _check(lib.pd_selftest_bounded_wait(_ptr(ws), int(limit_cycles), _stream()), "pd_selftest_bounded_wait")


def pd_device_status(workspace=None, device=None) -> int:
    """Synchronise the current stream and return the status a linear call latched (0 = ok)."""
    ws = workspace if workspace is not None else _workspace(256, device or torch.device("cuda", torch.cuda.current_device()))
    return int(lib.pd_device_status(_ptr(ws), _stream()))
