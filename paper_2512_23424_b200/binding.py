"""Thin ctypes binding of ``libakg.so`` - argument marshalling only.

Every operator runs in the CUDA library; this module turns torch tensors into
(device pointer, rows, cols, strides, dtype, stream) and checks the returned
status.  There is no CPU path: a missing library raises, it is never replaced.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

from . import build as _build

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_CUDA, ERR_DEVICE_TIMEOUT = range(5)
F32, BF16, F16 = 0, 1, 2
VARIANT_AUTO, VARIANT_STREAM, VARIANT_REG, VARIANT_TMA, VARIANT_CLUSTER = range(5)
VARIANTS = {"auto": 0, "stream": 1, "reg": 2, "tma": 3, "cluster": 4}


class AkgError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str):
        super().__init__(f"{where}: {status_string(status)} - {detail}")
        self.status = status


class Mask(ctypes.Structure):
    """Mirror of ``akg_mask`` (see include/akg.h)."""
    _fields_ = [("additive", ctypes.c_void_p), ("add_rows", ctypes.c_int64),
                ("add_row_stride", ctypes.c_int64), ("causal", ctypes.c_int32),
                ("causal_period", ctypes.c_int64), ("causal_offset", ctypes.c_int64)]


_lib: Optional[ctypes.CDLL] = None


def lib() -> ctypes.CDLL:
    """Load ``libakg.so`` (the in-tree build); raises if it is not there."""
    global _lib
    if _lib is None:
        path = _build.LIB_PATH
        if not os.path.exists(path):
            raise FileNotFoundError(
                f"{path} is missing: build it with `python -m paper_2512_23424_b200.build` "
                "(nvcc, sm_100a); there is no fallback path")
        L = ctypes.CDLL(path)
        vp, i64, ci, cf = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_float
        mp = ctypes.POINTER(Mask)
        for name in ("akg_softmax", "akg_log_softmax"):
            getattr(L, name).argtypes = [vp, vp, i64, i64, i64, i64, ci, mp, vp]
            getattr(L, name).restype = ci
        L.akg_layernorm.argtypes = [vp, vp, i64, i64, i64, i64, ci, vp, vp, cf, vp]
        L.akg_layernorm.restype = ci
        L.akg_rmsnorm.argtypes = [vp, vp, i64, i64, i64, i64, ci, vp, cf, vp]
        L.akg_rmsnorm.restype = ci
        L.akg_status_string.argtypes = [ci]
        L.akg_status_string.restype = ctypes.c_char_p
        L.akg_last_error_string.argtypes = []
        L.akg_last_error_string.restype = ctypes.c_char_p
        L.akg_last_kernel_name.argtypes = []
        L.akg_last_kernel_name.restype = ctypes.c_char_p
        L.akg_version.argtypes = []
        L.akg_version.restype = ci
        L.akg_set_variant.argtypes = [ci]
        L.akg_set_variant.restype = ci
        L.akg_set_tuning.argtypes = [ctypes.c_char_p, ci]
        L.akg_set_tuning.restype = ci
        L.akg_device_status.argtypes = [ctypes.POINTER(ci)]
        L.akg_device_status.restype = ci
        L.akg_rowop_host.argtypes = [ci, vp, vp, i64, i64, i64, i64, ci, vp, vp, cf, mp, vp,
                                     ctypes.c_size_t, vp]
        L.akg_rowop_host.restype = ci
        L.akg_host_workspace_bytes.argtypes = [i64, i64, ci, ci, ci]
        L.akg_host_workspace_bytes.restype = ctypes.c_size_t
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().akg_status_string(int(status)).decode()


def last_error() -> str:
    return lib().akg_last_error_string().decode()


def last_kernel() -> str:
    return lib().akg_last_kernel_name().decode()


def last_host_copy_bytes():
    """(host -> device, device -> host) bytes copied by the last rowop_host call of this thread."""
    up, down = ctypes.c_size_t(0), ctypes.c_size_t(0)
    fn = lib().akg_last_host_copy_bytes
    fn.restype = ctypes.c_int
    fn.argtypes = [ctypes.POINTER(ctypes.c_size_t), ctypes.POINTER(ctypes.c_size_t)]
    fn(ctypes.byref(up), ctypes.byref(down))
    return up.value, down.value


def set_variant(variant) -> None:
    code = VARIANTS[variant] if isinstance(variant, str) else int(variant)
    _check(lib().akg_set_variant(code), "akg_set_variant")


def set_tuning(key: str, value: int) -> None:
    _check(lib().akg_set_tuning(key.encode(), int(value)), "akg_set_tuning")


def device_status() -> int:
    word = ctypes.c_int(0)
    st = lib().akg_device_status(ctypes.byref(word))
    if st not in (OK, ERR_DEVICE_TIMEOUT):
        _check(st, "akg_device_status")
    return word.value


def _check(status: int, where: str) -> None:
    if status != OK:
        raise AkgError(status, where, last_error())


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    if t.dtype == torch.float16:
        return F16
    raise TypeError(f"unsupported dtype {t.dtype}: the library handles float32, bfloat16 and float16")


def _matrix(t: torch.Tensor, what: str):
    if t.dim() != 2:
        raise ValueError(f"{what} must be 2-D [rows, cols]")
    if not t.is_cuda:
        raise ValueError(f"{what} must live on a CUDA device")
    rows, cols = t.shape
    if cols > 1 and t.stride(1) != 1:
        raise ValueError(f"{what}: the last axis must be contiguous")
    return rows, cols, (t.stride(0) if rows > 1 else cols)


def _vector(v: Optional[torch.Tensor], like: torch.Tensor, cols: int, what: str):
    if v is None:
        return None
    if v.dtype != like.dtype or v.dim() != 1 or v.numel() != cols or not v.is_contiguous() \
            or v.device != like.device:
        raise ValueError(f"{what} must be a contiguous {like.dtype} vector of cols elements on x's device")
    return v.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def make_mask(x: torch.Tensor, additive: Optional[torch.Tensor] = None, causal: bool = False,
              causal_period: int = 1, causal_offset: int = 0) -> Optional[Mask]:
    if additive is None and not causal:
        return None
    m = Mask()
    if additive is not None:
        if additive.dim() != 2 or additive.dtype != x.dtype or additive.device != x.device:
            raise ValueError("additive mask must be a 2-D tensor of x's dtype on x's device")
        if additive.shape[1] > 1 and additive.stride(1) != 1:
            raise ValueError("additive mask: the last axis must be contiguous")
        m.additive = additive.data_ptr()
        m.add_rows = additive.shape[0]
        m.add_row_stride = additive.stride(0) if additive.shape[0] > 1 else max(additive.shape[1], 1)
        m._keep = additive
    m.causal = 1 if causal else 0
    m.causal_period = int(causal_period)
    m.causal_offset = int(causal_offset)
    return m


class PreparedCall:
    """One operator call with its arguments marshalled once; ``launch()`` only makes
    the C call (about a microsecond of host time), for loops that re-issue the same
    call.  The tensors are kept alive by the object; the stream is fixed at creation."""

    def __init__(self, fn_name: str, args: tuple, keep: tuple, out: torch.Tensor):
        self._fn = getattr(lib(), fn_name)
        self._name, self._args, self._keep, self.out = fn_name, args, keep, out

    def launch(self) -> torch.Tensor:
        st = self._fn(*self._args)
        if st != OK:
            raise AkgError(st, self._name, last_error())
        return self.out


def prepare(op: str, x: torch.Tensor, out: Optional[torch.Tensor] = None, *,
            gamma: Optional[torch.Tensor] = None, beta: Optional[torch.Tensor] = None,
            eps: float = 1e-5, mask: Optional[Mask] = None, stream=None) -> PreparedCall:
    """Marshal a call of ``op`` (softmax | log_softmax | layernorm | rmsnorm) once."""
    rows, cols, xs = _matrix(x, "x")
    if out is None:
        out = torch.empty_like(x)
    orow, ocol, ys = _matrix(out, "out")
    if (orow, ocol) != (rows, cols) or out.dtype != x.dtype or out.device != x.device:
        raise ValueError("out must match x in shape, dtype and device")
    with torch.cuda.device(x.device):
        s = ctypes.c_void_p(_stream(stream))
    vp, i64 = ctypes.c_void_p, ctypes.c_int64
    head = (vp(x.data_ptr()), vp(out.data_ptr()), i64(rows), i64(cols), i64(xs), i64(ys),
            ctypes.c_int(_dtype_code(x)))
    if op in ("softmax", "log_softmax"):
        args = head + (ctypes.byref(mask) if mask is not None else None, s)
        return PreparedCall("akg_" + op, args, (x, mask), out)
    if op == "layernorm":
        args = head + (vp(_vector(gamma, x, cols, "gamma")), vp(_vector(beta, x, cols, "beta")),
                       ctypes.c_float(eps), s)
        return PreparedCall("akg_layernorm", args, (x, gamma, beta), out)
    if op == "rmsnorm":
        args = head + (vp(_vector(gamma, x, cols, "weight")), ctypes.c_float(eps), s)
        return PreparedCall("akg_rmsnorm", args, (x, gamma), out)
    raise ValueError(f"unknown operator {op}")


OPS = {"softmax": 0, "log_softmax": 1, "layernorm": 2, "rmsnorm": 3}


def host_workspace_bytes(rows: int, cols: int, dtype: torch.dtype, has_gamma: bool = False,
                         has_beta: bool = False) -> int:
    code = F32 if dtype == torch.float32 else BF16
    return int(lib().akg_host_workspace_bytes(rows, cols, code, int(has_gamma), int(has_beta)))


def rowop_host(op: str, x: torch.Tensor, out: torch.Tensor, workspace: torch.Tensor, *,
               gamma: Optional[torch.Tensor] = None, beta: Optional[torch.Tensor] = None,
               eps: float = 1e-5, causal_period: int = 0, causal_offset: int = 0, stream=None) -> torch.Tensor:
    """akg_rowop_host: x, out, gamma, beta are HOST tensors (pinned for overlap), workspace
    is a device byte tensor the caller owns.  Enqueues on the current stream and returns."""
    if x.is_cuda or out.is_cuda or not workspace.is_cuda:
        raise ValueError("x / out must be host tensors and workspace a device tensor")
    if x.dim() != 2 or out.shape != x.shape or out.dtype != x.dtype:
        raise ValueError("x and out must be 2-D host tensors of the same shape and dtype")
    if x.shape[1] > 1 and (x.stride(1) != 1 or out.stride(1) != 1):
        raise ValueError("the last axis must be contiguous")
    rows, cols = x.shape
    xs = x.stride(0) if rows > 1 else cols
    ys = out.stride(0) if rows > 1 else cols
    mask = None
    if causal_period > 0:
        mask = Mask()
        mask.causal, mask.causal_period, mask.causal_offset = 1, int(causal_period), int(causal_offset)
    for v, what in ((gamma, "gamma"), (beta, "beta")):
        if v is not None and (v.is_cuda or v.dtype != x.dtype or v.numel() != cols or not v.is_contiguous()):
            raise ValueError(f"{what} must be a contiguous host vector of cols elements of x's dtype")
    with torch.cuda.device(workspace.device):
        st = lib().akg_rowop_host(OPS[op], x.data_ptr(), out.data_ptr(), rows, cols, xs, ys, _dtype_code(x),
                                  None if gamma is None else gamma.data_ptr(),
                                  None if beta is None else beta.data_ptr(), float(eps),
                                  ctypes.byref(mask) if mask is not None else None,
                                  workspace.data_ptr(), workspace.numel() * workspace.element_size(),
                                  _stream(stream))
    _check(st, "akg_rowop_host")
    return out


def rowop_axis(op: str, x: torch.Tensor, out: Optional[torch.Tensor] = None, *,
               gamma: Optional[torch.Tensor] = None, beta: Optional[torch.Tensor] = None,
               eps: float = 1e-5, stream=None) -> torch.Tensor:
    """akg_rowop_axis: `op` over axis 1 of a 3-D CUDA tensor [outer, reduce, inner] whose
    last axis is contiguous (the layout of the paper's RMSNorm sketch).  gamma / beta are
    device vectors of `reduce` elements."""
    if x.dim() != 3 or not x.is_cuda:
        raise ValueError("x must be a 3-D CUDA tensor [outer, reduce, inner]")
    if out is None:
        out = torch.empty_like(x)
    if out.shape != x.shape or out.dtype != x.dtype or out.device != x.device:
        raise ValueError("out must match x in shape, dtype and device")
    outer, red, inner = x.shape
    for t in (x, out):
        if inner > 1 and t.stride(2) != 1:
            raise ValueError("the last axis must be contiguous")

    def strides(t):
        sf = t.stride(1) if red > 1 else inner
        so = t.stride(0) if outer > 1 else (red - 1) * sf + inner
        return so, sf

    (xso, xsf), (yso, ysf) = strides(x), strides(out)
    fn = lib().akg_rowop_axis
    if not fn.argtypes:
        vp, i64, ci = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int
        fn.argtypes = [ci, vp, vp, i64, i64, i64, i64, i64, i64, i64, ci, vp, vp, ctypes.c_float, vp]
        fn.restype = ci
    with torch.cuda.device(x.device):
        st = fn(OPS[op], x.data_ptr(), out.data_ptr(), outer, red, inner, xso, xsf, yso, ysf, _dtype_code(x),
                _vector(gamma, x, red, "gamma"), _vector(beta, x, red, "beta"), float(eps), _stream(stream))
    _check(st, "akg_rowop_axis")
    return out


_NO_SUM = object()


def add_norm(op: str, x: torch.Tensor, residual: torch.Tensor, *, gamma: Optional[torch.Tensor] = None,
             beta: Optional[torch.Tensor] = None, eps: float = 1e-5, out: Optional[torch.Tensor] = None,
             sum_out=_NO_SUM, stream=None):
    """akg_add_norm: s = x + residual, returns (LayerNorm or RMSNorm of s, s) for 2-D CUDA tensors.
    `out` / `sum_out` default to new tensors; pass sum_out=None to skip storing the sum (the second
    result is then None); either may be `x` or `residual` themselves (in place)."""
    if op not in ("layernorm", "rmsnorm"):
        raise ValueError("op must be 'layernorm' or 'rmsnorm'")
    rows, cols, xs = _matrix(x, "x")
    rrows, rcols, rs = _matrix(residual, "residual")
    if out is None:
        out = torch.empty_like(x)
    if sum_out is _NO_SUM:
        sum_out = torch.empty_like(x)
    orow, ocol, ys = _matrix(out, "out")
    others = [(residual, rrows, rcols, "residual"), (out, orow, ocol, "out")]
    ss = cols
    if sum_out is not None:
        srow, scol, ss = _matrix(sum_out, "sum_out")
        others.append((sum_out, srow, scol, "sum_out"))
    for t, r, c, what in others:
        if (r, c) != (rows, cols) or t.dtype != x.dtype or t.device != x.device:
            raise ValueError(f"{what} must match x in shape, dtype and device")
    fn = lib().akg_add_norm
    if not fn.argtypes:
        vp, i64, ci = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int
        fn.argtypes = [ci, vp, vp, vp, vp, i64, i64, i64, i64, i64, i64, ci, vp, vp, ctypes.c_float, vp]
        fn.restype = ci
    with torch.cuda.device(x.device):
        st = fn(OPS[op], x.data_ptr(), residual.data_ptr(), out.data_ptr(),
                None if sum_out is None else sum_out.data_ptr(), rows, cols, xs, rs, ys, ss, _dtype_code(x),
                _vector(gamma, x, cols, "gamma"), _vector(beta, x, cols, "beta") if op == "layernorm" else None,
                float(eps), _stream(stream))
    _check(st, "akg_add_norm")
    return out, sum_out


ACTS = {"silu": 0, "gelu": 1, "gelu_tanh": 2}


def act_mul(act: str, x: torch.Tensor, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """akg_act_mul: act(x[:, :d]) * x[:, d:] for a 2-D CUDA tensor [rows, 2 d]; act is "silu",
    "gelu" or "gelu_tanh".  `out` ([rows, d]) defaults to a new tensor."""
    rows, cols, xs = _matrix(x, "x")
    if cols % 2:
        raise ValueError("x must have an even number of columns (gate | factor)")
    d = cols // 2
    if out is None:
        out = torch.empty((rows, d), dtype=x.dtype, device=x.device)
    orow, ocol, ys = _matrix(out, "out")
    if (orow, ocol) != (rows, d) or out.dtype != x.dtype or out.device != x.device:
        raise ValueError("out must be [rows, d] of x's dtype on x's device")
    fn = lib().akg_act_mul
    if not fn.argtypes:
        vp, i64, ci = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int
        fn.argtypes = [ci, vp, vp, i64, i64, i64, i64, ci, vp]
        fn.restype = ci
    with torch.cuda.device(x.device):
        st = fn(ACTS[act], x.data_ptr(), out.data_ptr(), rows, d, xs if rows > 1 else max(xs, 2 * d), ys,
                _dtype_code(x), _stream(stream))
    _check(st, "akg_act_mul")
    return out


def _argreduce(want_min: int, x: torch.Tensor, out, stream):
    rows, cols, xs = _matrix(x, "x")
    if out is None:
        out = torch.empty((rows,), dtype=torch.int64, device=x.device)
    if out.shape != (rows,) or out.dtype != torch.int64 or out.device != x.device or not out.is_contiguous():
        raise ValueError("out must be a contiguous int64 vector of `rows` entries on x's device")
    fn = lib().akg_argreduce
    if not fn.argtypes:
        vp, i64, ci = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int
        fn.argtypes = [ci, vp, vp, i64, i64, i64, ci, vp]
        fn.restype = ci
    with torch.cuda.device(x.device):
        st = fn(want_min, x.data_ptr(), out.data_ptr(), rows, cols, xs, _dtype_code(x), _stream(stream))
    _check(st, "akg_argreduce")
    return out


def argmax(x: torch.Tensor, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """akg_argreduce(0): first index of the row maximum (NaN counts as the maximum), int64 [rows]."""
    return _argreduce(0, x, out, stream)


def argmin(x: torch.Tensor, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """akg_argreduce(1): first index of the row minimum (NaN counts as the minimum), int64 [rows]."""
    return _argreduce(1, x, out, stream)


def _cumulative(want_prod: int, x: torch.Tensor, out, stream):
    rows, cols, xs = _matrix(x, "x")
    if out is None:
        out = torch.empty_like(x)
    orow, ocol, ys = _matrix(out, "out")
    if (orow, ocol) != (rows, cols) or out.dtype != x.dtype or out.device != x.device:
        raise ValueError("out must match x in shape, dtype and device")
    fn = lib().akg_cumulative
    if not fn.argtypes:
        vp, i64, ci = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int
        fn.argtypes = [ci, vp, vp, i64, i64, i64, i64, ci, vp]
        fn.restype = ci
    with torch.cuda.device(x.device):
        st = fn(want_prod, x.data_ptr(), out.data_ptr(), rows, cols, xs, ys, _dtype_code(x), _stream(stream))
    _check(st, "akg_cumulative")
    return out


def cumsum(x: torch.Tensor, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """akg_cumulative(0): inclusive running sum along the last axis of a 2-D CUDA tensor."""
    return _cumulative(0, x, out, stream)


def cumprod(x: torch.Tensor, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """akg_cumulative(1): inclusive running product along the last axis of a 2-D CUDA tensor."""
    return _cumulative(1, x, out, stream)


def colnorm_workspace_bytes(rows: int, cols: int) -> int:
    """akg_colnorm_workspace_bytes: the workspace with which akg_colnorm fills the GPU."""
    fn = lib().akg_colnorm_workspace_bytes
    fn.argtypes = [ctypes.c_int64, ctypes.c_int64]
    fn.restype = ctypes.c_size_t
    return int(fn(rows, cols))


def colnorm(x: torch.Tensor, gamma: Optional[torch.Tensor] = None, beta: Optional[torch.Tensor] = None,
            eps: float = 1e-5, out: Optional[torch.Tensor] = None, want_stats: bool = False,
            workspace: Optional[torch.Tensor] = None, stream=None):
    """akg_colnorm: every column of a 2-D CUDA tensor normalised with its own mean and biased variance
    over the rows (BatchNorm-style), per-column gamma / beta.  Returns y, or (y, mean, var) with
    float32 statistics when want_stats.  `workspace` (a CUDA byte tensor) defaults to a new one."""
    rows, cols, xs = _matrix(x, "x")
    if out is None:
        out = torch.empty_like(x)
    orow, ocol, ys = _matrix(out, "out")
    if (orow, ocol) != (rows, cols) or out.dtype != x.dtype or out.device != x.device:
        raise ValueError("out must match x in shape, dtype and device")
    L = lib()
    fn = L.akg_colnorm
    if not fn.argtypes:
        vp, i64, ci = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int
        fn.argtypes = [vp, vp, i64, i64, i64, i64, ci, vp, vp, ctypes.c_float, vp, vp, vp, ctypes.c_size_t, vp]
        fn.restype = ci
    if workspace is None:
        workspace = torch.empty(max(colnorm_workspace_bytes(rows, cols), 8), dtype=torch.uint8, device=x.device)
    mean = torch.empty(cols, dtype=torch.float32, device=x.device) if want_stats else None
    var = torch.empty(cols, dtype=torch.float32, device=x.device) if want_stats else None
    with torch.cuda.device(x.device):
        st = fn(x.data_ptr(), out.data_ptr(), rows, cols, xs, ys, _dtype_code(x), _vector(gamma, x, cols, "gamma"),
                _vector(beta, x, cols, "beta"), float(eps), mean.data_ptr() if want_stats else None,
                var.data_ptr() if want_stats else None, workspace.data_ptr(), workspace.numel(), _stream(stream))
    _check(st, "akg_colnorm")
    return (out, mean, var) if want_stats else out


STATIC_STAGING_BYTES = 16 << 20


def rowop_host_static(op: str, x: torch.Tensor, out: torch.Tensor, *, gamma: Optional[torch.Tensor] = None,
                      beta: Optional[torch.Tensor] = None, eps: float = 1e-5, causal_period: int = 0,
                      causal_offset: int = 0, stream=None) -> torch.Tensor:
    """akg_rowop_host_static: like rowop_host, for callers that cannot hand over a device
    workspace (no allocator at hand, or allocation not allowed where they run).  The chunks
    are staged in the 16 MiB area built into the library; nothing is allocated, on the
    device or by this wrapper.  x, out, gamma, beta are HOST tensors.  All work is enqueued
    on one stream (the current one unless given); calls that overlap on the GPU from
    different streams race on the shared staging area."""
    if x.is_cuda or out.is_cuda:
        raise ValueError("x / out must be host tensors")
    if x.dim() != 2 or out.shape != x.shape or out.dtype != x.dtype:
        raise ValueError("x and out must be 2-D host tensors of the same shape and dtype")
    if x.shape[1] > 1 and (x.stride(1) != 1 or out.stride(1) != 1):
        raise ValueError("the last axis must be contiguous")
    rows, cols = x.shape
    xs = x.stride(0) if rows > 1 else cols
    ys = out.stride(0) if rows > 1 else cols
    mask = None
    if causal_period > 0:
        mask = Mask()
        mask.causal, mask.causal_period, mask.causal_offset = 1, int(causal_period), int(causal_offset)
    for v, what in ((gamma, "gamma"), (beta, "beta")):
        if v is not None and (v.is_cuda or v.dtype != x.dtype or v.numel() != cols or not v.is_contiguous()):
            raise ValueError(f"{what} must be a contiguous host vector of cols elements of x's dtype")
    fn = lib().akg_rowop_host_static
    if not fn.argtypes:
        vp, i64, ci = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int
        fn.argtypes = [ci, vp, vp, i64, i64, i64, i64, ci, vp, vp, ctypes.c_float, ctypes.POINTER(Mask), vp]
        fn.restype = ci
    st = fn(OPS[op], x.data_ptr(), out.data_ptr(), rows, cols, xs, ys, _dtype_code(x),
            None if gamma is None else gamma.data_ptr(), None if beta is None else beta.data_ptr(),
            float(eps), ctypes.byref(mask) if mask is not None else None, _stream(stream))
    _check(st, "akg_rowop_host_static")
    return out


def _softmax_like(fn_name, x, out, mask, stream):
    rows, cols, xs = _matrix(x, "x")
    if out is None:
        out = torch.empty_like(x)
    orow, ocol, ys = _matrix(out, "out")
    if (orow, ocol) != (rows, cols) or out.dtype != x.dtype or out.device != x.device:
        raise ValueError("out must match x in shape, dtype and device")
    with torch.cuda.device(x.device):
        st = getattr(lib(), fn_name)(x.data_ptr(), out.data_ptr(), rows, cols, xs, ys,
                                     _dtype_code(x), ctypes.byref(mask) if mask is not None else None,
                                     _stream(stream))
    _check(st, fn_name)
    return out


def softmax(x: torch.Tensor, out: Optional[torch.Tensor] = None, mask: Optional[Mask] = None,
            stream=None) -> torch.Tensor:
    """akg_softmax over the last axis of a 2-D CUDA tensor."""
    return _softmax_like("akg_softmax", x, out, mask, stream)


def log_softmax(x: torch.Tensor, out: Optional[torch.Tensor] = None, mask: Optional[Mask] = None,
                stream=None) -> torch.Tensor:
    """akg_log_softmax over the last axis of a 2-D CUDA tensor."""
    return _softmax_like("akg_log_softmax", x, out, mask, stream)


def softmax_scaled(x: torch.Tensor, scale: float, out: Optional[torch.Tensor] = None, mask: Optional[Mask] = None,
                   log: bool = False, stream=None) -> torch.Tensor:
    """akg_softmax_scaled: softmax (log=False) or log-softmax (log=True) of scale * x + additive
    mask under the causal rule, over the last axis of a 2-D CUDA tensor; scale > 0."""
    rows, cols, xs = _matrix(x, "x")
    if out is None:
        out = torch.empty_like(x)
    orow, ocol, ys = _matrix(out, "out")
    if (orow, ocol) != (rows, cols) or out.dtype != x.dtype or out.device != x.device:
        raise ValueError("out must match x in shape, dtype and device")
    fn = lib().akg_softmax_scaled
    if not fn.argtypes:
        vp, i64, ci = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int
        fn.argtypes = [vp, vp, i64, i64, i64, i64, ci, ctypes.c_float, vp, ci, vp]
        fn.restype = ci
    with torch.cuda.device(x.device):
        st = fn(x.data_ptr(), out.data_ptr(), rows, cols, xs, ys, _dtype_code(x), float(scale),
                ctypes.cast(ctypes.byref(mask), ctypes.c_void_p) if mask is not None else None, 1 if log else 0,
                _stream(stream))
    _check(st, "akg_softmax_scaled")
    return out


def layernorm(x: torch.Tensor, gamma: Optional[torch.Tensor] = None, beta: Optional[torch.Tensor] = None,
              eps: float = 1e-5, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """akg_layernorm over the last axis of a 2-D CUDA tensor."""
    rows, cols, xs = _matrix(x, "x")
    if out is None:
        out = torch.empty_like(x)
    orow, ocol, ys = _matrix(out, "out")
    if (orow, ocol) != (rows, cols) or out.dtype != x.dtype or out.device != x.device:
        raise ValueError("out must match x in shape, dtype and device")
    with torch.cuda.device(x.device):
        st = lib().akg_layernorm(x.data_ptr(), out.data_ptr(), rows, cols, xs, ys, _dtype_code(x),
                                 _vector(gamma, x, cols, "gamma"), _vector(beta, x, cols, "beta"),
                                 float(eps), _stream(stream))
    _check(st, "akg_layernorm")
    return out


def rmsnorm(x: torch.Tensor, weight: Optional[torch.Tensor] = None, eps: float = 1e-6,
            out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """akg_rmsnorm over the last axis of a 2-D CUDA tensor."""
    rows, cols, xs = _matrix(x, "x")
    if out is None:
        out = torch.empty_like(x)
    orow, ocol, ys = _matrix(out, "out")
    if (orow, ocol) != (rows, cols) or out.dtype != x.dtype or out.device != x.device:
        raise ValueError("out must match x in shape, dtype and device")
    with torch.cuda.device(x.device):
        st = lib().akg_rmsnorm(x.data_ptr(), out.data_ptr(), rows, cols, xs, ys, _dtype_code(x),
                               _vector(weight, x, cols, "weight"), float(eps), _stream(stream))
    _check(st, "akg_rmsnorm")
    return out
