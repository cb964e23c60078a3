"""Seeded synthetic inputs for the five benchmark configurations.

This module holds input generation only - none of the operators' arithmetic -
so that the CPU oracle and the CUDA library can consume the very same bytes.
Everything is numpy on the host; bf16 arrays are ``uint16`` holding raw bits.

The operator workloads (row-wise softmax / LayerNorm / RMSNorm over LLM-like
hidden sizes, a vocabulary-like axis, and an attention-score block) stand in for
the paper's operator benchmark (Section 3.6) and the third-party suite of
Section 4.1, neither of which is reproduced here.

Seeding: configuration k (1-based) uses base seed k-1; independent sub-streams
come from ``numpy.random.SeedSequence(seed).spawn(4)`` in the fixed order
x, gamma/weight, beta, positions, each driving a ``Generator(PCG64)``.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, Optional

import numpy as np

F32, BF16, F16 = 0, 1, 2      # F16 arrays are numpy float16


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (nearest, ties to even); returns uint16 bits.
    NaN inputs map to a quiet NaN."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    bits = a.view(np.uint32)
    rounded = ((bits + (np.uint32(0x7FFF) + ((bits >> np.uint32(16)) & np.uint32(1))))
               >> np.uint32(16)).astype(np.uint16)
    nan = np.isnan(a)
    if nan.any():
        rounded = np.where(nan, np.uint16(0x7FC0), rounded)
    return rounded


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact widening of raw bf16 bits to float32."""
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


@dataclass
class Workload:
    """One operator call: what to run and the host arrays it runs on."""
    name: str
    op: str                      # softmax | log_softmax | layernorm | rmsnorm
    dtype: int                   # F32 | BF16
    rows: int
    cols: int
    x: np.ndarray                # [rows, cols] float32, or uint16 bf16 bits
    eps: float = 0.0
    gamma: Optional[np.ndarray] = None   # LayerNorm gamma or RMSNorm weight
    beta: Optional[np.ndarray] = None
    causal_period: int = 0       # > 0: entry (r, c) masked iff c > r % period
    extra: Dict[str, object] = field(default_factory=dict)

    @property
    def itemsize(self) -> int:
        return 4 if self.dtype == F32 else 2

    def algorithmic_bytes(self) -> int:
        """Bytes the method must move: every live input element read once,
        every output element written once, gamma / beta / weight once."""
        e = self.itemsize
        if self.causal_period > 0:
            p = self.causal_period
            full, rem = divmod(self.rows, p)
            # row r has min(cols, r % p + 1) live entries
            per_period = sum(min(self.cols, i + 1) for i in range(p)) if p <= 1 << 16 else None
            if per_period is None:
                raise ValueError("causal period too large for the byte count")
            live = full * per_period + sum(min(self.cols, i + 1) for i in range(rem))
        else:
            live = self.rows * self.cols
        vec = sum(self.cols for v in (self.gamma, self.beta) if v is not None)
        return (live + vec + self.rows * self.cols) * e


_SHAPES = {
    1: ("softmax", F32, 64, 1024),
    2: ("layernorm", F32, 4096, 4096),
    3: ("rmsnorm", BF16, 16384, 8192),
    4: ("log_softmax", F32, 256, 262144),
    5: ("softmax", BF16, 32 * 4096, 4096),
}

CONFIG_NAMES = {
    1: "softmax_f32_64x1024",
    2: "layernorm_f32_4096x4096",
    3: "rmsnorm_bf16_16384x8192",
    4: "log_softmax_f32_256x262144",
    5: "causal_softmax_bf16_32x4096x4096",
}


def config_shape(k: int):
    """(rows, cols) of configuration k at full size."""
    return _SHAPES[k][2], _SHAPES[k][3]


def _normal_f32(rng: np.random.Generator, rows: int, cols: int) -> np.ndarray:
    out = np.empty((rows, cols), dtype=np.float32)
    block = max(1, (1 << 24) // max(cols, 1))
    for r0 in range(0, rows, block):
        r1 = min(rows, r0 + block)
        out[r0:r1] = rng.standard_normal((r1 - r0, cols), dtype=np.float32)
    return out


def make_config(k: int, rows: Optional[int] = None, seed_offset: int = 0) -> Workload:
    """Build configuration k (1..5).  ``rows`` truncates the row count (the
    column count, value distribution and seeds are unchanged, so the first rows
    of a truncated workload equal the first rows of the full one for k != 5's
    blockwise generator as well).  ``seed_offset`` shifts the base seed (used to
    give each rank of a multi-GPU run its own rows)."""
    op, dtype, full_rows, cols = _SHAPES[k]
    rows = full_rows if rows is None else int(rows)
    seed = (k - 1) + 1000 * int(seed_offset)
    s_x, s_g, s_b, s_p = np.random.SeedSequence(seed).spawn(4)
    rx, rg, rb, rp = (np.random.Generator(np.random.PCG64(s)) for s in (s_x, s_g, s_b, s_p))
    name = CONFIG_NAMES[k]
    if k == 1:
        return Workload(name, op, dtype, rows, cols, _normal_f32(rx, rows, cols))
    if k == 2:
        x = _normal_f32(rx, rows, cols)
        x *= np.float32(2.0)
        x += np.float32(3.0)
        gamma = rg.uniform(0.5, 1.5, cols).astype(np.float32)
        beta = (rb.standard_normal(cols) * 0.1).astype(np.float32)
        return Workload(name, op, dtype, rows, cols, x, eps=1e-5, gamma=gamma, beta=beta)
    if k == 3:
        x = f32_to_bf16_bits(_normal_f32(rx, rows, cols))
        w = f32_to_bf16_bits(rg.uniform(0.5, 1.5, cols).astype(np.float32))
        return Workload(name, op, dtype, rows, cols, x, eps=1e-6, gamma=w)
    if k == 4:
        x = _normal_f32(rx, rows, cols)
        x *= np.float32(4.0)
        n_out = (cols * 1) // 10000          # 0.01 % of the row, rounded down
        pos = np.empty((rows, n_out), dtype=np.int64)
        for r in range(rows):
            pos[r] = rp.choice(cols, size=n_out, replace=False)
            x[r, pos[r]] = np.float32(30.0)
        return Workload(name, op, dtype, rows, cols, x, extra={"outlier_cols": pos})
    if k == 5:
        scale = np.float32(1.0 / np.sqrt(128.0))
        x = _normal_f32(rx, rows, cols)
        x *= scale
        return Workload(name, op, dtype, rows, cols, f32_to_bf16_bits(x), causal_period=4096)
    raise ValueError(f"unknown configuration {k}")


def make_random(op: str, dtype: int, rows: int, cols: int, seed: int,
                loc: float = 0.0, scale: float = 1.0, affine: bool = True,
                eps: float = 1e-5) -> Workload:
    """Free-form seeded workload for shape sweeps."""
    s_x, s_g, s_b = np.random.SeedSequence(seed).spawn(3)
    rx, rg, rb = (np.random.Generator(np.random.PCG64(s)) for s in (s_x, s_g, s_b))
    x = _normal_f32(rx, rows, cols) * np.float32(scale) + np.float32(loc)
    gamma = beta = None
    if op in ("layernorm", "rmsnorm") and affine:
        gamma = rg.uniform(0.5, 1.5, cols).astype(np.float32)
        if op == "layernorm":
            beta = (rb.standard_normal(cols) * 0.1).astype(np.float32)
    if dtype == BF16:
        x = f32_to_bf16_bits(x)
        gamma = None if gamma is None else f32_to_bf16_bits(gamma)
        beta = None if beta is None else f32_to_bf16_bits(beta)
    if dtype == F16:
        x = x.astype(np.float16)
        gamma = None if gamma is None else gamma.astype(np.float16)
        beta = None if beta is None else beta.astype(np.float16)
    return Workload(f"{op}_{ {F32: 'f32', BF16: 'bf16', F16: 'f16'}[dtype]}_{rows}x{cols}", op, dtype,
                    rows, cols, x, eps=eps if op in ("layernorm", "rmsnorm") else 0.0,
                    gamma=gamma, beta=beta)


# ---------------------------------------------------------------------------------------------
# Operators over a non-last axis: x[outer, reduce, inner], inner contiguous.  The first shape is
# the one of the paper's RMSNorm sketch (Unified Sketch figure: X[B, F, D1, D2] normalised over
# the feature axis F) with B = 16, F = 64, D1 = D2 = 256; the long-axis shapes exercise the
# two-pass kernel.
# ---------------------------------------------------------------------------------------------
AXIS_CONFIGS: Dict[str, tuple] = {
    "axis_sketch_rmsnorm_f32_16x64x65536": ("rmsnorm", F32, 16, 64, 65536),
    "axis_softmax_f32_16x64x65536": ("softmax", F32, 16, 64, 65536),
    "axis_layernorm_f32_16x64x65536": ("layernorm", F32, 16, 64, 65536),
    "axis_sketch_rmsnorm_bf16_16x64x65536": ("rmsnorm", BF16, 16, 64, 65536),
    "axis_softmax_bf16_16x64x65536": ("softmax", BF16, 16, 64, 65536),
    "axis_layernorm_bf16_16x64x65536": ("layernorm", BF16, 16, 64, 65536),
    "axis_rmsnorm_f32_8x512x16384": ("rmsnorm", F32, 8, 512, 16384),
    "axis_softmax_f32_2x1024x32768": ("softmax", F32, 2, 1024, 32768),
}


@dataclass
class AxisWorkload:
    name: str
    op: str
    dtype: int                         # F32 / BF16
    x: np.ndarray                      # [outer, reduce, inner]; float32, or uint16 bf16 bits
    eps: float = 0.0
    gamma: Optional[np.ndarray] = None  # [reduce]
    beta: Optional[np.ndarray] = None

    @property
    def itemsize(self) -> int:
        return 4 if self.dtype == F32 else 2

    def algorithmic_bytes(self) -> int:
        """One read and one write of every element (gamma / beta are negligible)."""
        return 2 * self.x.size * self.itemsize


def make_axis(name: str, outer: Optional[int] = None, seed_offset: int = 0) -> AxisWorkload:
    """Seeded input of a non-last-axis configuration; `outer` truncates the outer axis."""
    op, dtype, o, f, d = AXIS_CONFIGS[name]
    o = o if outer is None else min(o, outer)
    seed = 100 + sorted(AXIS_CONFIGS).index(name) + 1000 * seed_offset
    s_x, s_g, s_b = np.random.SeedSequence(seed).spawn(3)
    rx, rg, rb = (np.random.Generator(np.random.PCG64(s)) for s in (s_x, s_g, s_b))
    x = (_normal_f32(rx, o * f, d) * np.float32(1.5) + np.float32(0.25)).reshape(o, f, d)
    gamma = beta = None
    if op in ("layernorm", "rmsnorm"):
        gamma = rg.uniform(0.5, 1.5, f).astype(np.float32)
        if op == "layernorm":
            beta = (rb.standard_normal(f) * 0.1).astype(np.float32)
    if dtype == BF16:
        x = f32_to_bf16_bits(x)
        gamma = None if gamma is None else f32_to_bf16_bits(gamma)
        beta = None if beta is None else f32_to_bf16_bits(beta)
    return AxisWorkload(name, op, dtype, x, eps=1e-5 if gamma is not None else 0.0, gamma=gamma, beta=beta)


# ---------------------------------------------------------------------------------------------
# Fused residual add + normalisation (a "fused variant" of the paper's operator benchmark,
# Section 3.6): the pre-norm residual step of a transformer block at the hidden sizes of
# configurations 2 and 3; x is the branch output, res the residual stream.
# ---------------------------------------------------------------------------------------------
FUSED_CONFIGS: Dict[str, tuple] = {
    "add_rmsnorm_bf16_16384x8192": ("rmsnorm", BF16, 16384, 8192, 1e-6),
    "add_layernorm_f32_4096x4096": ("layernorm", F32, 4096, 4096, 1e-5),
    "add_rmsnorm_f32_8192x4096": ("rmsnorm", F32, 8192, 4096, 1e-6),
    "add_layernorm_bf16_16384x4096": ("layernorm", BF16, 16384, 4096, 1e-5),
}


@dataclass
class FusedWorkload:
    name: str
    op: str
    dtype: int
    x: np.ndarray                      # [rows, cols]; float32, or uint16 bf16 bits
    res: np.ndarray                    # same shape and storage
    eps: float
    gamma: Optional[np.ndarray] = None
    beta: Optional[np.ndarray] = None

    @property
    def itemsize(self) -> int:
        return 4 if self.dtype == F32 else 2

    def algorithmic_bytes(self) -> int:
        """x and res read once, y and the sum written once, gamma / beta once."""
        vec = sum(v.size for v in (self.gamma, self.beta) if v is not None)
        return (4 * self.x.size + vec) * self.itemsize


def make_fused(name: str, rows: Optional[int] = None, seed_offset: int = 0) -> FusedWorkload:
    op, dtype, r, c, eps = FUSED_CONFIGS[name]
    r = r if rows is None else min(r, rows)
    seed = 200 + sorted(FUSED_CONFIGS).index(name) + 1000 * seed_offset
    s_x, s_r, s_g, s_b = np.random.SeedSequence(seed).spawn(4)
    rx, rr, rg, rb = (np.random.Generator(np.random.PCG64(s)) for s in (s_x, s_r, s_g, s_b))
    x = _normal_f32(rx, r, c)                                        # branch output ~ N(0, 1)
    res = _normal_f32(rr, r, c) * np.float32(2.0) + np.float32(0.5)  # residual stream: wider, offset
    gamma = rg.uniform(0.5, 1.5, c).astype(np.float32)
    beta = (rb.standard_normal(c) * 0.1).astype(np.float32) if op == "layernorm" else None
    if dtype == BF16:
        x, res, gamma = f32_to_bf16_bits(x), f32_to_bf16_bits(res), f32_to_bf16_bits(gamma)
        beta = None if beta is None else f32_to_bf16_bits(beta)
    return FusedWorkload(name, op, dtype, x, res, eps, gamma=gamma, beta=beta)


# ---------------------------------------------------------------------------------------------
# Gated activations (SiLU-and-Mul, GELU-and-Mul; named in Section 3.6): x = [gate | factor] of
# a feed-forward block, [tokens, 2 d] with d the intermediate size.
# ---------------------------------------------------------------------------------------------
ACT_CONFIGS: Dict[str, tuple] = {
    "silu_and_mul_bf16_8192x14336": ("silu", BF16, 8192, 14336),
    "gelu_and_mul_bf16_8192x14336": ("gelu", BF16, 8192, 14336),
    "gelu_tanh_and_mul_bf16_8192x14336": ("gelu_tanh", BF16, 8192, 14336),
    "silu_and_mul_f32_4096x11008": ("silu", F32, 4096, 11008),
    "gelu_and_mul_f32_4096x11008": ("gelu", F32, 4096, 11008),
}


@dataclass
class ActWorkload:
    name: str
    act: str
    dtype: int
    x: np.ndarray                      # [rows, 2 d]; float32, or uint16 bf16 bits

    @property
    def itemsize(self) -> int:
        return 4 if self.dtype == F32 else 2

    def algorithmic_bytes(self) -> int:
        """Gate and factor read once, the product written once."""
        return (self.x.size + self.x.size // 2) * self.itemsize


def make_act(name: str, rows: Optional[int] = None, seed_offset: int = 0) -> ActWorkload:
    act, dtype, r, d = ACT_CONFIGS[name]
    r = r if rows is None else min(r, rows)
    seed = 300 + sorted(ACT_CONFIGS).index(name) + 1000 * seed_offset
    rx = np.random.Generator(np.random.PCG64(np.random.SeedSequence(seed)))
    x = _normal_f32(rx, r, 2 * d) * np.float32(1.5)                  # pre-activations ~ N(0, 1.5^2)
    if dtype == BF16:
        x = f32_to_bf16_bits(x)
    return ActWorkload(name, act, dtype, x)


def make_scaled_causal(rows: Optional[int] = None, seed_offset: int = 0) -> Workload:
    """Configuration 5 with its 1/sqrt(128) moved out of the input and into the call: x holds
    the unscaled bf16 scores N(0, 1); `extra["scale"]` is the pre-scale to pass to the fused
    softmax (same seed, shape and causal period as configuration 5)."""
    k = 5
    op, dtype, r, c = _SHAPES[k]
    name = "scaled_causal_softmax_bf16_32x4096x4096"
    r = r if rows is None else min(r, rows)
    s_x = np.random.SeedSequence(k - 1 + 1000 * seed_offset).spawn(4)[0]
    x = _normal_f32(np.random.Generator(np.random.PCG64(s_x)), r, c)
    return Workload(name, op, dtype, r, c, f32_to_bf16_bits(x), causal_period=4096,
                    extra={"scale": float(np.float32(1.0 / np.sqrt(128.0)))})


# ---------------------------------------------------------------------------------------------
# Other reduction-category operators of Section 3.6 (arg-max / arg-min, cumulative sum /
# product) on the shapes of configurations 2 and 3 and on a vocabulary-like axis.
# ---------------------------------------------------------------------------------------------
REDUCTION_CONFIGS: Dict[str, tuple] = {
    "argmax_f32_16384x8192": ("argmax", F32, 16384, 8192),
    "argmax_bf16_16384x8192": ("argmax", BF16, 16384, 8192),
    "argmin_f32_1024x131072": ("argmin", F32, 1024, 131072),
    "cumsum_f32_16384x8192": ("cumsum", F32, 16384, 8192),
    "cumsum_bf16_16384x8192": ("cumsum", BF16, 16384, 8192),
    "cumprod_f32_16384x8192": ("cumprod", F32, 16384, 8192),
    "cumsum_f32_256x262144": ("cumsum", F32, 256, 262144),
    "cumsum_bf16_256x262144": ("cumsum", BF16, 256, 262144),
    "cumsum_bf16_1048576x256": ("cumsum", BF16, 1048576, 256),
}


@dataclass
class ReductionWorkload:
    name: str
    op: str                            # argmax | argmin | cumsum | cumprod
    dtype: int
    x: np.ndarray                      # [rows, cols]; float32, or uint16 bf16 bits

    @property
    def itemsize(self) -> int:
        return 4 if self.dtype == F32 else 2

    def algorithmic_bytes(self) -> int:
        """Every element read once; an int64 index per row, or every element written once."""
        if self.op in ("argmax", "argmin"):
            return self.x.size * self.itemsize + self.x.shape[0] * 8
        return 2 * self.x.size * self.itemsize


def make_reduction(name: str, rows: Optional[int] = None, seed_offset: int = 0) -> ReductionWorkload:
    op, dtype, r, c = REDUCTION_CONFIGS[name]
    r = r if rows is None else min(r, rows)
    seed = 400 + sorted(REDUCTION_CONFIGS).index(name) + 1000 * seed_offset
    rx = np.random.Generator(np.random.PCG64(np.random.SeedSequence(seed)))
    x = _normal_f32(rx, r, c)
    if op == "cumprod":                                 # factors near one keep the product in range
        x = np.float32(1.0) + np.float32(0.002) * x
    if dtype == BF16:
        x = f32_to_bf16_bits(x)
    return ReductionWorkload(name, op, dtype, x)


def as_f16(w: Workload) -> Workload:
    """The same workload stored as IEEE half (the paper's float16 regime, Section 4.1): every
    array is converted from its stored values with numpy's round-to-nearest-even."""
    def conv(a):
        if a is None:
            return None
        f = bf16_bits_to_f32(a) if a.dtype == np.uint16 else a
        return f.astype(np.float16)
    name = w.name.replace("bf16", "f16").replace("f32", "f16")
    return Workload(name, w.op, F16, w.rows, w.cols, conv(w.x), eps=w.eps, gamma=conv(w.gamma), beta=conv(w.beta),
                    causal_period=w.causal_period, extra=dict(w.extra))


# ---------------------------------------------------------------------------------------------
# BatchNorm-style column normalisation (BatchNorm is listed in Section 3.6): activations
# [N * H * W, C] in channels-last layout, statistics per channel over all rows.
# ---------------------------------------------------------------------------------------------
COLNORM_CONFIGS: Dict[str, tuple] = {
    "colnorm_f32_16384x8192": (F32, 16384, 8192),
    "colnorm_bf16_65536x1024": (BF16, 65536, 1024),
    "colnorm_f32_1048576x64": (F32, 1048576, 64),
}


def make_colnorm(name: str, rows: Optional[int] = None, seed_offset: int = 0) -> Workload:
    """x ~ N(1, 2^2), gamma ~ U(0.5, 1.5), beta ~ N(0, 0.1^2), eps 1e-5; `op` is "colnorm"."""
    dtype, r, c = COLNORM_CONFIGS[name]
    r = r if rows is None else min(r, rows)
    seed = 500 + sorted(COLNORM_CONFIGS).index(name) + 1000 * seed_offset
    s_x, s_g, s_b = np.random.SeedSequence(seed).spawn(3)
    rx, rg, rb = (np.random.Generator(np.random.PCG64(s)) for s in (s_x, s_g, s_b))
    x = _normal_f32(rx, r, c) * np.float32(2.0) + np.float32(1.0)
    gamma = rg.uniform(0.5, 1.5, c).astype(np.float32)
    beta = (rb.standard_normal(c) * 0.1).astype(np.float32)
    if dtype == BF16:
        x, gamma, beta = f32_to_bf16_bits(x), f32_to_bf16_bits(gamma), f32_to_bf16_bits(beta)
    return Workload(name, "colnorm", dtype, r, c, x, eps=1e-5, gamma=gamma, beta=beta)
