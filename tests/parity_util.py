"""Helpers for the GPU parity tests: run a workload through the C-ABI library and
through the fp64 oracle, and compare under the stated tolerances.

Tolerances (the build contract's):
  fp32 I/O : max |y_gpu - y_ref| <= 1e-5 over finite reference values; infinities
             and NaNs must sit at the same positions (infinities with equal sign)
  bf16 I/O : per element |y_gpu - y_ref| <= 2 ulp_bf16(y_ref), where
             ulp_bf16(v) = 2^(max(floor(log2 |v|), -126) - 7); a flushed zero is
             accepted when |y_ref| < 2^-126.  LayerNorm (+ beta) and log-softmax
             (- logsumexp) end in an addition that can cancel, so "output magnitude"
             is read there as the magnitude of the two addends: the bound gains
             2^-22 * (|addend 1| + |addend 2|), i.e. 4 fp32 ulps of the terms that
             the fp32 arithmetic actually rounds (nothing for softmax / RMSNorm).
             compare() counts the elements that need it (stats["rescued"])
  masked softmax entries and rows with no live entry: +0, bit for bit
"""
from __future__ import annotations

import os
from typing import Optional, Sequence

import numpy as np
import torch

import oracle
import paper_2512_23424_b200 as akg
from paper_2512_23424_b200 import workloads as wl

FP32_ATOL = 1e-5
BF16_ULPS = 2.0
#: 16-bit LayerNorm / log-softmax: slack per unit of |addend 1| + |addend 2| (four fp32 ulps)
CANCEL_16BIT = 2.0 ** -22


def to_torch(a: Optional[np.ndarray], dtype: int, device="cuda") -> Optional[torch.Tensor]:
    """Host array (float32, or uint16 bf16 bits) -> device tensor of the same bits."""
    if a is None:
        return None
    if dtype == wl.F32:
        return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(device)
    if dtype == wl.F16:
        return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float16)).to(device)
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.uint16).view(np.int16)).to(device)
    return t.view(torch.bfloat16)


def to_numpy(t: torch.Tensor) -> np.ndarray:
    """Device tensor -> host array holding the same bits (float32 or uint16)."""
    t = t.detach().contiguous().cpu()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16).copy()
    return t.numpy().copy()


def widen(a: np.ndarray) -> np.ndarray:
    """Stored output (float32 or bf16 bits) -> float64, exactly."""
    if a.dtype == np.uint16:
        return wl.bf16_bits_to_f32(a).astype(np.float64)
    return a.astype(np.float64)


def strided_device_matrix(host: np.ndarray, dtype: int, stride: int, offset_elems: int = 0,
                          sentinel: float = float("nan")):
    """Place `host` [rows, cols] in a device buffer with the given row stride and a
    leading element offset; padding holds the sentinel.  Returns (buffer, view)."""
    rows, cols = host.shape
    tdt = {wl.F32: torch.float32, wl.BF16: torch.bfloat16, wl.F16: torch.float16}[dtype]
    buf = torch.full((offset_elems + rows * stride + 8,), sentinel, dtype=tdt, device="cuda")
    view = torch.as_strided(buf, (rows, cols), (stride, 1), storage_offset=offset_elems)
    view.copy_(to_torch(host, dtype))
    return buf, view


def run_gpu(w: wl.Workload, *, x_dev: Optional[torch.Tensor] = None, out: Optional[torch.Tensor] = None,
            additive: Optional[torch.Tensor] = None, causal_offset: int = 0) -> torch.Tensor:
    """One call of the operator through the binding (and so through the C ABI)."""
    x = to_torch(w.x, w.dtype) if x_dev is None else x_dev
    if out is None:
        out = torch.full_like(x, float("nan")) if x.is_contiguous() else None
    if w.op in ("softmax", "log_softmax"):
        mask = akg.make_mask(x, additive=additive, causal=w.causal_period > 0,
                             causal_period=max(w.causal_period, 1), causal_offset=causal_offset)
        fn = akg.softmax if w.op == "softmax" else akg.log_softmax
        return fn(x, out=out, mask=mask)
    g = to_torch(w.gamma, w.dtype)
    if w.op == "layernorm":
        return akg.layernorm(x, g, to_torch(w.beta, w.dtype), eps=w.eps, out=out)
    return akg.rmsnorm(x, g, eps=w.eps, out=out)


def run_oracle(w: wl.Workload, rows: Optional[Sequence[int]] = None,
               additive: Optional[np.ndarray] = None, causal_offset: int = 0,
               nthreads: int = 0) -> np.ndarray:
    """fp64 reference for all rows, or for the listed global row indices."""
    x = w.x if rows is None else np.ascontiguousarray(w.x[np.asarray(rows)])
    ids = None if rows is None else np.asarray(rows, dtype=np.int64)
    eps = float(np.float32(w.eps))          # the library takes eps as a float
    nthreads = nthreads or min(32, os.cpu_count() or 1)
    if w.op in ("softmax", "log_softmax"):
        mask = None
        if additive is not None or w.causal_period > 0:
            mask = oracle.Mask(additive=additive, causal=w.causal_period > 0,
                               causal_period=max(w.causal_period, 1), causal_offset=causal_offset)
        fn = oracle.softmax if w.op == "softmax" else oracle.log_softmax
        return fn(x, mask=mask, row_ids=ids, nthreads=nthreads)
    if w.op == "layernorm":
        return oracle.layernorm(x, w.gamma, w.beta, eps=eps, nthreads=nthreads)
    return oracle.rmsnorm(x, w.gamma, eps=eps, nthreads=nthreads)


def f16_ulp(ref: np.ndarray) -> np.ndarray:
    """Spacing of IEEE half at |ref|: 2^(max(floor(log2 |ref|), -14) - 10) (2^-24 in the subnormal range)."""
    a = np.abs(ref)
    e = np.floor(np.log2(np.where(a > 0, a, 1.0)))
    e = np.where(a > 0, e, -14.0)
    return np.exp2(np.maximum(e, -14.0) - 10.0)


def bf16_ulp(ref: np.ndarray) -> np.ndarray:
    a = np.abs(ref)
    e = np.floor(np.log2(np.where(a > 0, a, 1.0)))
    e = np.where(a > 0, e, -126.0)
    return np.exp2(np.maximum(e, -126.0) - 7.0)


def cancel_magnitude(w: wl.Workload, ref: np.ndarray, additive: Optional[np.ndarray] = None):
    """Absolute slack added to the tolerance, per element (None = none).

    bf16 LayerNorm / log-softmax: CANCEL_16BIT * (|addend 1| + |addend 2|) of the final
    addition (see the module docstring).
    LayerNorm, both dtypes: 2^-23 * max|x_row| * rstd_row * |gamma_c|.  The row mean is
    a real number that fp32 holds to half an ulp of |mean| <= max|x_row| at best; that
    error passes through (x - mean) * rstd * gamma whatever the implementation, so the
    term is the conditioning of the operator in fp32, not a kernel allowance.  It is
    below 1e-6 for ordinary rows (benchmark configuration 2: about 8e-7) and only
    matters for rows whose spread is tiny against their mean."""
    if w.op == "layernorm":
        x = widen(w.x)
        eps = float(np.float32(w.eps))
        rstd = 1.0 / np.sqrt(x.var(axis=1, keepdims=True) + eps)
        gamma = 1.0 if w.gamma is None else np.abs(widen(w.gamma))[None, :]
        slack = 2.0 ** -23 * np.abs(x).max(axis=1, keepdims=True) * rstd * gamma * np.ones_like(ref)
        if w.dtype != wl.F32:
            beta = 0.0 if w.beta is None else widen(w.beta)[None, :]
            slack = slack + CANCEL_16BIT * (np.abs(ref - beta) + np.abs(beta))
        return slack
    if w.op == "log_softmax" and w.dtype != wl.F32:
        z = widen(w.x)
        if additive is not None:
            a = widen(additive)
            z = z + a[np.arange(w.rows) % a.shape[0], :w.cols]
        with np.errstate(invalid="ignore"):
            mag = np.abs(z) + np.abs(z - ref)
        return CANCEL_16BIT * np.where(np.isfinite(mag), mag, 0.0)
    return None


#: one entry per comparison that was given a slack: (what, elements, rescued) where `rescued`
#: counts the elements beyond the strict bound that only the slack lets pass.  Written to the
#: file named by AKG_PARITY_LOG at the end of the session (see conftest.py).
RESCUE_LOG = []


def compare(got_stored: np.ndarray, ref: np.ndarray, dtype: int, what: str = "",
            cancel_mag: Optional[np.ndarray] = None, tiny: float = 2.0 ** -126,
            max_rescued: Optional[int] = None) -> dict:
    """Assert parity under the tolerances above; returns error statistics.  `tiny`: bf16 results
    whose reference is below it in magnitude may be returned as a flushed zero.  `cancel_mag`
    widens the bound per element; stats["rescued"] counts the elements that needed it and
    `max_rescued` (where given) limits that count."""
    got = widen(got_stored)
    assert got.shape == ref.shape, (what, got.shape, ref.shape)
    ref_nan, got_nan = np.isnan(ref), np.isnan(got)
    assert np.array_equal(ref_nan, got_nan), f"{what}: NaN positions differ ({got_nan.sum()} vs {ref_nan.sum()})"
    ref_inf = np.isinf(ref)
    assert np.array_equal(ref_inf, np.isinf(got)), f"{what}: infinity positions differ"
    if ref_inf.any():
        assert np.array_equal(np.sign(ref[ref_inf]), np.sign(got[ref_inf])), f"{what}: infinity signs differ"
    fin = ~(ref_nan | ref_inf)
    err = np.abs(got[fin] - ref[fin])
    stats = {"max_abs": float(err.max()) if err.size else 0.0, "n": int(fin.sum()), "rescued": 0}
    if dtype == wl.F32:
        bound = np.full(err.shape, FP32_ATOL)
        excused = np.zeros(err.shape, dtype=bool)
    else:
        # fp16 I/O: the same rule with the spacing of IEEE half (2 ulps; no flush below its range)
        ulp = f16_ulp(ref[fin]) if dtype == wl.F16 else bf16_ulp(ref[fin])
        bound = BF16_ULPS * ulp
        excused = (np.abs(ref[fin]) < (0.0 if dtype == wl.F16 else tiny)) & (got[fin] == 0)
        stats["max_ulp"] = float((err / ulp).max()) if err.size else 0.0
    strict_bad = (err > bound) & ~excused
    bad = strict_bad
    if cancel_mag is not None:
        bad = (err > bound + cancel_mag[fin]) & ~excused
        stats["rescued"] = int(strict_bad.sum() - bad.sum())
        stats["max_abs_after_slack"] = float(np.maximum(err - cancel_mag[fin], 0.0).max()) if err.size else 0.0
        RESCUE_LOG.append((what, stats["n"], stats["rescued"]))
    if dtype == wl.F32:
        assert not bad.any(), f"{what}: max abs error {stats['max_abs']:.3e} > {FP32_ATOL}"
    else:
        assert not bad.any(), (f"{what}: {bad.sum()} elements beyond {BF16_ULPS} ulps of the storage type "
                               f"(max {stats['max_ulp']:.3f})")
    if max_rescued is not None:
        assert stats["rescued"] <= max_rescued, (f"{what}: {stats['rescued']} elements pass only with the "
                                                 f"cancellation slack (allowed: {max_rescued})")
    return stats


def assert_positive_zero(stored: np.ndarray, where: np.ndarray, what: str = ""):
    """Entries selected by `where` must be +0 bit for bit."""
    bits = stored.view(np.uint32) if stored.dtype == np.float32 else stored
    assert (bits[where] == 0).all(), f"{what}: masked entries are not +0 bit-exactly"


def verifier_passes(got_stored: np.ndarray, ref: np.ndarray, dtype: int) -> bool:
    """The paper's own criterion (Section 3.2.3, Eq. 2-3): tau = 1e-3 for fp32; the
    paper's float16 threshold 4e-3 is borrowed for bf16 (it gives none)."""
    tau = 1e-3 if dtype == wl.F32 else 4e-3          # 4e-3 is the paper's own float16 threshold (Section 4.1)
    # Eq. 3 tolerates a fraction tau of mismatching elements.  An array of fewer than 1 / tau elements would
    # be allowed less than one: there a single element whose reference nearly cancels (a LayerNorm output
    # close to zero in a three-column row) decides the test by the luck of its rounding, so one is allowed.
    allowed = max(tau, 1.0 / max(ref.size, 1))
    return oracle.verifier_fraction(widen(got_stored), ref, eps_switch=1e-8, tau=tau) <= allowed
