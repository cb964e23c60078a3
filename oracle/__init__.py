"""ctypes front end of the fp64 CPU oracle (``oracle.c``).

TEST INFRASTRUCTURE ONLY.  The oracle is the plain definition of softmax,
log-softmax, LayerNorm and RMSNorm (with additive / causal masking) written out
in double precision; the test-suite, the smoke check and the benchmark's
CPU-baseline leg are its only callers.  It shares nothing with the CUDA
library and never imports it.

Arrays are numpy: float32 / float64 as themselves, bf16 as ``uint16`` holding
the raw bits.  Every driver returns a ``float64`` array of shape (rows, cols).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "oracle.c")
_HDR = os.path.join(_HERE, "oracle.h")
_LIB = os.path.join(_HERE, "liboracle.so")

F32, BF16, F64, F16 = 0, 1, 2, 3


def build(force: bool = False) -> str:
    """Compile ``oracle.c`` with gcc (no fast-math) when the library is stale."""
    stale = force or not os.path.exists(_LIB) or any(
        os.path.getmtime(s) > os.path.getmtime(_LIB) for s in (_SRC, _HDR))
    if stale:
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.run(
            ["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-Wall",
             "-Wextra", _SRC, "-o", tmp, "-lm"], check=True)
        os.replace(tmp, _LIB)
    return _LIB


class _Mask(ctypes.Structure):
    _fields_ = [("additive", ctypes.c_void_p), ("add_rows", ctypes.c_int64),
                ("add_row_stride", ctypes.c_int64), ("causal", ctypes.c_int32),
                ("causal_period", ctypes.c_int64), ("causal_offset", ctypes.c_int64)]


@dataclass
class Mask:
    """additive: 2-D array [add_rows, >= cols] of x's storage type (or None);
    causal: entry (r, c) is masked iff c > (r % causal_period) + causal_offset."""
    additive: Optional[np.ndarray] = None
    causal: bool = False
    causal_period: int = 1
    causal_offset: int = 0


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        dp = ctypes.POINTER(ctypes.c_double)
        i64, vp, ci, cd = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int, ctypes.c_double
        for name in ("oracle_softmax_row", "oracle_log_softmax_row"):
            getattr(L, name).argtypes = [dp, i64, dp]
            getattr(L, name).restype = None
        L.oracle_logsumexp_row.argtypes = [dp, i64]
        L.oracle_logsumexp_row.restype = cd
        L.oracle_layernorm_row.argtypes = [dp, i64, dp, dp, cd, dp]
        L.oracle_layernorm_row.restype = None
        L.oracle_rmsnorm_row.argtypes = [dp, i64, dp, cd, dp]
        L.oracle_rmsnorm_row.restype = None
        for name in ("oracle_softmax", "oracle_log_softmax"):
            getattr(L, name).argtypes = [vp, ci, i64, i64, i64, vp,
                                         ctypes.POINTER(_Mask), dp, ci]
            getattr(L, name).restype = ci
        L.oracle_layernorm.argtypes = [vp, ci, i64, i64, i64, vp, vp, cd, dp, ci]
        L.oracle_layernorm.restype = ci
        L.oracle_rmsnorm.argtypes = [vp, ci, i64, i64, i64, vp, cd, dp, ci]
        L.oracle_rmsnorm.restype = ci
        L.oracle_verifier_fraction.argtypes = [dp, dp, i64, cd, cd]
        L.oracle_verifier_fraction.restype = cd
        L.oracle_last_threads.argtypes = []
        L.oracle_last_threads.restype = ci
        _lib = L
    return _lib


def _dtype_code(a: np.ndarray) -> int:
    if a.dtype == np.float32:
        return F32
    if a.dtype == np.uint16:
        return BF16
    if a.dtype == np.float64:
        return F64
    if a.dtype == np.float16:
        return F16
    raise TypeError(f"oracle: unsupported storage dtype {a.dtype}")


def _dptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _as2d(x: np.ndarray):
    """Return (array kept alive, rows, cols, row stride in elements)."""
    if x.ndim != 2:
        raise ValueError("oracle: x must be 2-D")
    if x.shape[1] > 1 and x.strides[1] != x.itemsize:
        x = np.ascontiguousarray(x)
    if x.shape[0] > 1 and (x.strides[0] % x.itemsize or x.strides[0] < x.shape[1] * x.itemsize):
        x = np.ascontiguousarray(x)
    stride = x.strides[0] // x.itemsize if x.shape[0] > 1 else max(x.shape[1], 1)
    return x, x.shape[0], x.shape[1], stride


def _vec(v: Optional[np.ndarray], like: np.ndarray, cols: int):
    if v is None:
        return None, None
    v = np.ascontiguousarray(v)
    if v.dtype != like.dtype or v.shape != (cols,):
        raise ValueError("oracle: gamma/beta/weight must match x's dtype and have cols elements")
    return v, v.ctypes.data


def _softmax_like(fn_name, x, mask, row_ids, nthreads, scale=None, want_log=0):
    x, rows, cols, stride = _as2d(x)
    out = np.empty((rows, cols), dtype=np.float64)
    cm, keep = None, None
    if mask is not None:
        cm = _Mask()
        if mask.additive is not None:
            keep, ar, ac, astr = _as2d(mask.additive)
            if keep.dtype != x.dtype or ac < cols:
                raise ValueError("oracle: additive mask must share x's dtype and cover cols")
            cm.additive, cm.add_rows, cm.add_row_stride = keep.ctypes.data, ar, astr
        cm.causal = 1 if mask.causal else 0
        cm.causal_period, cm.causal_offset = mask.causal_period, mask.causal_offset
    ids = None
    if row_ids is not None:
        ids = np.ascontiguousarray(row_ids, dtype=np.int64)
        if ids.shape != (rows,):
            raise ValueError("oracle: row_ids must have one entry per row")
    if scale is not None:
        fn = lib().oracle_softmax_scaled
        if not fn.argtypes:
            i64, vp, ci = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int
            fn.argtypes = [vp, ci, i64, i64, i64, ctypes.c_double, vp, vp, ci, ctypes.POINTER(ctypes.c_double), ci]
            fn.restype = ci
        rc = fn(x.ctypes.data, _dtype_code(x), rows, cols, stride, float(scale),
                ids.ctypes.data if ids is not None else None,
                ctypes.cast(ctypes.byref(cm), ctypes.c_void_p) if cm is not None else None, int(want_log),
                _dptr(out), int(nthreads))
    else:
        rc = getattr(lib(), fn_name)(
            x.ctypes.data, _dtype_code(x), rows, cols, stride,
            ids.ctypes.data if ids is not None else None,
            ctypes.byref(cm) if cm is not None else None, _dptr(out), int(nthreads))
    if rc != 0:
        raise ValueError(f"{fn_name}: malformed argument")
    return out


def softmax(x, mask: Optional[Mask] = None, row_ids=None, nthreads: int = 1):
    return _softmax_like("oracle_softmax", x, mask, row_ids, nthreads)


def log_softmax(x, mask: Optional[Mask] = None, row_ids=None, nthreads: int = 1):
    return _softmax_like("oracle_log_softmax", x, mask, row_ids, nthreads)


def softmax_scaled(x, scale: float, mask: Optional[Mask] = None, log: bool = False, row_ids=None,
                   nthreads: int = 1):
    """softmax (or log-softmax) of scale * x + additive mask under the causal rule: the fused
    pre-scale variant.  The additive mask is not scaled."""
    return _softmax_like("oracle_softmax_scaled", x, mask, row_ids, nthreads, scale=scale, want_log=1 if log else 0)


def logsumexp_row(z: np.ndarray) -> float:
    z = np.ascontiguousarray(z, dtype=np.float64)
    return float(lib().oracle_logsumexp_row(_dptr(z), z.size))


def layernorm(x, gamma=None, beta=None, eps: float = 1e-5, nthreads: int = 1):
    x, rows, cols, stride = _as2d(x)
    out = np.empty((rows, cols), dtype=np.float64)
    g, gp = _vec(gamma, x, cols)
    b, bp = _vec(beta, x, cols)
    rc = lib().oracle_layernorm(x.ctypes.data, _dtype_code(x), rows, cols, stride,
                                gp, bp, float(eps), _dptr(out), int(nthreads))
    if rc != 0:
        raise ValueError("oracle_layernorm: malformed argument")
    return out


def rmsnorm(x, weight=None, eps: float = 1e-6, nthreads: int = 1):
    x, rows, cols, stride = _as2d(x)
    out = np.empty((rows, cols), dtype=np.float64)
    w, wp = _vec(weight, x, cols)
    rc = lib().oracle_rmsnorm(x.ctypes.data, _dtype_code(x), rows, cols, stride,
                              wp, float(eps), _dptr(out), int(nthreads))
    if rc != 0:
        raise ValueError("oracle_rmsnorm: malformed argument")
    return out


def add_norm(op: str, x, res, gamma=None, beta=None, eps: float = 1e-5, nthreads: int = 1):
    """Fused residual add + LayerNorm / RMSNorm (a fused variant of Section 3.6):
    returns (norm(x + res), x + res), both float64 [rows, cols]."""
    x, rows, cols, xs = _as2d(x)
    res, rrows, rcols, rs = _as2d(res)
    if (rrows, rcols) != (rows, cols) or res.dtype != x.dtype:
        raise ValueError("oracle: res must match x's shape and dtype")
    out_y = np.empty((rows, cols), dtype=np.float64)
    out_s = np.empty((rows, cols), dtype=np.float64)
    g, gp = _vec(gamma, x, cols)
    b, bp = _vec(beta, x, cols)
    L = lib()
    if not L.oracle_add_norm.argtypes:
        i64, vp, ci, cd = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int, ctypes.c_double
        dp = ctypes.POINTER(ctypes.c_double)
        L.oracle_add_norm.argtypes = [ci, vp, vp, ci, i64, i64, i64, i64, vp, vp, cd, dp, dp, ci]
        L.oracle_add_norm.restype = ci
    rc = L.oracle_add_norm({"layernorm": 2, "rmsnorm": 3}[op], x.ctypes.data, res.ctypes.data, _dtype_code(x),
                           rows, cols, xs, rs, gp, bp, float(eps), _dptr(out_y), _dptr(out_s), int(nthreads))
    if rc != 0:
        raise ValueError("oracle_add_norm: malformed argument")
    return out_y, out_s


ACTS = {"silu": 0, "gelu": 1, "gelu_tanh": 2}


def act_mul(act: str, x, nthreads: int = 1):
    """SiLU-and-Mul / GELU-and-Mul (named in Section 3.6): x is [rows, 2 d]; returns
    act(x[:, :d]) * x[:, d:] as float64 [rows, d]."""
    x, rows, cols, stride = _as2d(x)
    if cols % 2:
        raise ValueError("oracle: x must have an even number of columns")
    d = cols // 2
    out = np.empty((rows, d), dtype=np.float64)
    L = lib()
    if not L.oracle_act_mul.argtypes:
        i64, vp, ci = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int
        L.oracle_act_mul.argtypes = [ci, vp, ci, i64, i64, i64, ctypes.POINTER(ctypes.c_double), ci]
        L.oracle_act_mul.restype = ci
        L.oracle_activation.argtypes = [ci, ctypes.c_double]
        L.oracle_activation.restype = ctypes.c_double
    rc = L.oracle_act_mul(ACTS[act], x.ctypes.data, _dtype_code(x), rows, d, stride, _dptr(out), int(nthreads))
    if rc != 0:
        raise ValueError("oracle_act_mul: malformed argument")
    return out


def argreduce(op: str, x, nthreads: int = 1) -> np.ndarray:
    """"argmax" / "argmin" over the last axis (Section 3.6): int64 [rows]; first index on ties,
    NaN counts as the extreme."""
    x, rows, cols, stride = _as2d(x)
    out = np.empty((rows,), dtype=np.int64)
    L = lib()
    if not L.oracle_argreduce.argtypes:
        i64, vp, ci = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int
        L.oracle_argreduce.argtypes = [ci, vp, ci, i64, i64, i64, vp, ci]
        L.oracle_argreduce.restype = ci
    rc = L.oracle_argreduce({"argmax": 0, "argmin": 1}[op], x.ctypes.data, _dtype_code(x), rows, cols, stride,
                            out.ctypes.data, int(nthreads))
    if rc != 0:
        raise ValueError("oracle_argreduce: malformed argument")
    return out


def cumulative(op: str, x, nthreads: int = 1) -> np.ndarray:
    """"cumsum" / "cumprod" along the last axis (Section 3.6), inclusive: float64 [rows, cols]."""
    x, rows, cols, stride = _as2d(x)
    out = np.empty((rows, cols), dtype=np.float64)
    L = lib()
    if not L.oracle_cumulative.argtypes:
        i64, vp, ci = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int
        L.oracle_cumulative.argtypes = [ci, vp, ci, i64, i64, i64, ctypes.POINTER(ctypes.c_double), ci]
        L.oracle_cumulative.restype = ci
    rc = L.oracle_cumulative({"cumsum": 0, "cumprod": 1}[op], x.ctypes.data, _dtype_code(x), rows, cols, stride,
                             _dptr(out), int(nthreads))
    if rc != 0:
        raise ValueError("oracle_cumulative: malformed argument")
    return out


def colnorm(x, gamma=None, beta=None, eps: float = 1e-5, nthreads: int = 1):
    """BatchNorm-style normalisation of every column of x[rows, cols] with its own mean and
    biased variance over the rows; returns (y, mean, var) as float64."""
    x, rows, cols, stride = _as2d(x)
    y = np.empty((rows, cols), dtype=np.float64)
    mean, var = np.empty(cols, dtype=np.float64), np.empty(cols, dtype=np.float64)
    g, gp = _vec(gamma, x, cols)
    b, bp = _vec(beta, x, cols)
    L = lib()
    if not L.oracle_colnorm.argtypes:
        i64, vp, ci, dp = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int, ctypes.POINTER(ctypes.c_double)
        L.oracle_colnorm.argtypes = [vp, ci, i64, i64, i64, vp, vp, ctypes.c_double, dp, dp, dp, ci]
        L.oracle_colnorm.restype = ci
    rc = L.oracle_colnorm(x.ctypes.data, _dtype_code(x), rows, cols, stride, gp, bp, float(eps), _dptr(y),
                          _dptr(mean), _dptr(var), int(nthreads))
    if rc != 0:
        raise ValueError("oracle_colnorm: malformed argument")
    return y, mean, var


AXIS_OPS = {"softmax": 0, "log_softmax": 1, "layernorm": 2, "rmsnorm": 3}


def rowop_axis(op: str, x: np.ndarray, gamma=None, beta=None, eps: float = 1e-5, nthreads: int = 1):
    """Operator `op` over axis 1 of a 3-D array [outer, reduce, inner] (inner contiguous):
    the layout of the paper's RMSNorm sketch.  gamma / beta have `reduce` elements."""
    if x.ndim != 3:
        raise ValueError("oracle: x must be 3-D [outer, reduce, inner]")
    if x.shape[2] > 1 and x.strides[2] != x.itemsize:
        x = np.ascontiguousarray(x)
    if any(s % x.itemsize for s in x.strides[:2]):
        x = np.ascontiguousarray(x)
    outer, reduce_n, inner = x.shape
    so = x.strides[0] // x.itemsize if outer > 1 else reduce_n * max(x.strides[1] // x.itemsize, inner)
    sf = x.strides[1] // x.itemsize if reduce_n > 1 else inner
    if sf < inner or so < (reduce_n - 1) * sf + inner:
        x = np.ascontiguousarray(x)
        so, sf = reduce_n * inner, inner
    out = np.empty((outer, reduce_n, inner), dtype=np.float64)
    g, gp = _vec(gamma, x, reduce_n)
    b, bp = _vec(beta, x, reduce_n)
    L = lib()
    if not L.oracle_rowop_axis.argtypes:
        i64, vp, ci, cd = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int, ctypes.c_double
        L.oracle_rowop_axis.argtypes = [ci, vp, ci, i64, i64, i64, i64, i64, vp, vp, cd,
                                        ctypes.POINTER(ctypes.c_double), ci]
        L.oracle_rowop_axis.restype = ci
    rc = L.oracle_rowop_axis(AXIS_OPS[op], x.ctypes.data, _dtype_code(x), outer, reduce_n, inner, so, sf,
                             gp, bp, float(eps), _dptr(out), int(nthreads))
    if rc != 0:
        raise ValueError("oracle_rowop_axis: malformed argument")
    return out


def verifier_fraction(gen, ref, eps_switch: float = 1e-8, tau: float = 1e-3) -> float:
    """Fraction of elements whose error (Section 3.2.3, Eq. 2) exceeds tau."""
    g = np.ascontiguousarray(gen, dtype=np.float64).ravel()
    r = np.ascontiguousarray(ref, dtype=np.float64).ravel()
    if g.size != r.size:
        raise ValueError("verifier_fraction: size mismatch")
    return float(lib().oracle_verifier_fraction(_dptr(g), _dptr(r), g.size,
                                                float(eps_switch), float(tau)))


def widen(a: np.ndarray) -> np.ndarray:
    """The exact values of a stored array (float32, float16, float64, or uint16 bf16 bits)."""
    a = np.ascontiguousarray(a)
    out = np.empty(a.shape, dtype=np.float64)
    L = lib()
    L.oracle_widen.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.POINTER(ctypes.c_double)]
    L.oracle_widen.restype = ctypes.c_int
    if L.oracle_widen(a.ctypes.data, _dtype_code(a), a.size, _dptr(out)) != 0:
        raise ValueError("oracle_widen: malformed argument")
    return out


def last_threads() -> int:
    return int(lib().oracle_last_threads())
