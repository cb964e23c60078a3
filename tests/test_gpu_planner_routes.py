"""GPU parity on the shapes that steer the planner into its specialised routes: every case asserts
the kernel family that ran (so the route is really exercised) and compares with the oracle through
the C ABI under the tolerances of parity_util."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
import paper_2512_23424_b200 as akg
from paper_2512_23424_b200 import binding
from paper_2512_23424_b200 import workloads as wl
from parity_util import (assert_positive_zero, cancel_magnitude, compare, run_gpu, run_oracle, to_numpy, to_torch,
                         widen)

pytestmark = pytest.mark.gpu
DTYPES = [wl.F32, wl.BF16, wl.F16]


def check(w, expect, rows=None, what=""):
    """Run w on the GPU, require `expect` (substrings) in the kernel name, compare all rows (or the
    sampled `rows`) with the oracle."""
    got = to_numpy(run_gpu(w))
    name = akg.last_kernel()
    for part in expect:
        assert part in name, f"{w.name}: expected {expect}, ran {name}"
    if rows is None:
        ref = run_oracle(w)
        compare(got, ref, w.dtype, f"{what}{w.name} [{name}]", cancel_magnitude(w, ref))
    else:
        ref = run_oracle(w, rows=rows)
        sub = dataclasses.replace(w, x=np.ascontiguousarray(w.x[rows]), rows=len(rows))
        compare(got[rows], ref, w.dtype, f"{what}{w.name} [{name}] sampled", cancel_magnitude(sub, ref))
    return got, name


# ---- a warp per row with 3, 5, 6 or 7 vectors per lane (768, 1280, 1536, 1792 columns) ------------

@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("op", ["layernorm", "rmsnorm"])
def test_norm_rows_of_odd_vectors_per_lane(op, dtype):
    epv = 4 if dtype == wl.F32 else 8
    for per_lane in (3, 5, 6, 7):
        cols = 32 * per_lane * epv
        w = wl.make_random(op, dtype, 4100, cols, seed=300 + per_lane, loc=0.5)
        warp_fit = per_lane * epv <= 40 or per_lane == 7
        check(w, ("g32", f"v{per_lane}", "full") if warp_fit else (("flex",) if dtype == wl.F32 else ("packed",)))


# ---- exact fits that are not a warp's: fat threads first ------------------------------------------

@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16])
def test_flex_rows_prefer_fat_threads(dtype):
    # few rows, so the warp-per-row route is not taken
    for cols, expect in ((1280, "g64,t64,v5") if dtype == wl.F32 else (1536, "g64,t64,v3"),
                         (1792, "g64,t64,v7") if dtype == wl.F32 else (3072, "g64,t64,v6")):
        for op in ("layernorm", "rmsnorm"):
            if dtype != wl.F32 and op == "rmsnorm" and cols == 3072:
                check(wl.make_random(op, dtype, 333, cols, seed=310), ("g96,t96,v4", "packed"))   # four per thread
            else:
                check(wl.make_random(op, dtype, 333, cols, seed=310), (expect, "flex" if dtype == wl.F32 else "packed"))


@pytest.mark.parametrize("dtype", [wl.BF16, wl.F16])
def test_sixteen_bit_norm_rows_grid_stride(dtype):
    # more rows than the persistent grid holds CTAs: every CTA walks several rows
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    rows = sms * 64 + 777
    for op, cols in (("layernorm", 2048), ("layernorm", 2560), ("rmsnorm", 5120)):
        w = wl.make_random(op, dtype, rows, cols, seed=320, loc=-0.25)
        sample = np.unique(np.concatenate([np.arange(0, 40), np.arange(rows - 40, rows),
                                           np.random.default_rng(5).integers(0, rows, 200)]))
        check(w, ("reg<",), rows=sample)


# ---- long rows: cluster size follows the row length, slices are whole unrolled steps ---------------

@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16])
def test_long_rows_cluster_size_follows_length(dtype):
    epv = 4 if dtype == wl.F32 else 8
    cases = [  # rows, cols, expected cluster size (many rows: by length; few rows: by fill)
        (320, 4096 * epv * 4, 4),
        (300, 32064 * epv // 2, 4),            # 16032 vectors: slices of 4096, a ragged last slice
        (40, 4096 * epv * 2, 8),               # few rows: 8 CTAs per row fill the GPU
        (3, 50304, 16),
    ]
    for rows, cols, cs in cases:
        for op in ("softmax", "log_softmax", "layernorm", "rmsnorm"):
            if dtype == wl.F32 and cols // epv <= 8192 and op in ("layernorm", "rmsnorm"):
                continue                       # exact fits of fp32 normalisations stay in registers
            # the fp32 softmax pair and RMSNorm take slices of about 2048 vectors: twice the CTAs by length;
            # so do the 16-bit RMSNorm and log-softmax
            by_length = rows >= 300 and ((dtype == wl.F32 and op != "layernorm") or
                                         (dtype != wl.F32 and op in ("rmsnorm", "log_softmax")))
            w = wl.make_random(op, dtype, rows, cols, seed=330 + cs, scale=2.0)
            check(w, ("split", f"cs{2 * cs if by_length else cs},"))


@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16])
def test_long_causal_rows_mix_merged_and_plain_steps(dtype):
    # a causal mask makes consecutive rows of a cluster differ in their live slices, so the
    # interleaved loop, the separate passes and wholly masked slices all occur in one launch
    rows, cols = 96, 40960
    w = wl.make_random("softmax", dtype, rows, cols, seed=340)
    w = dataclasses.replace(w, causal_period=48)
    x = w.x.copy()
    poison = np.float32(np.nan) if dtype == wl.F32 else np.uint16(0x7FC0)
    for r in range(rows):
        x[r, (r % 48) + 1:] = poison            # masked inputs must never be used
    w = dataclasses.replace(w, x=x)
    got, _ = check(w, ("split",))
    live = (np.arange(rows) % 48) + 1
    masked = np.arange(cols)[None, :] >= live[:, None]
    assert_positive_zero(got, masked, "masked tail")
    for op in ("log_softmax",):
        w2 = dataclasses.replace(w, op=op, name="causal_log_softmax")
        got2, _ = check(w2, ("split",))
        assert np.all(np.isneginf(widen(got2)[masked]))


@pytest.mark.parametrize("dtype", [wl.BF16, wl.F16])
def test_sixteen_bit_rows_beyond_2048_vectors_leave_the_register_form(dtype):
    # unmasked rows stay in registers (packed form) while eight vectors per thread fit a CTA
    # (given rows for about a full wave of threads) ...
    for op in ("layernorm", "rmsnorm", "softmax", "log_softmax"):
        check(wl.make_random(op, dtype, 600, 20480, seed=350), ("reg<", "t320,v8,packed"))
        check(wl.make_random(op, dtype, 200, 65536, seed=352), ("reg<", "t1024,v8,packed"))
        check(wl.make_random(op, dtype, 200, 20480, seed=355), ("split", "cs2,"))    # ... and leave them with few rows,
        check(wl.make_random(op, dtype, 200, 65536 + 256, seed=353), ("split",))    # beyond 8192 vectors,
        check(wl.make_random(op, dtype, 600, 20480 + 8, seed=354), ("split",))      # or where the fit is not exact
    # a mask keeps the softmax pair out of the packed form
    w = wl.make_random("softmax", dtype, 600, 20480, seed=356, scale=2.0)
    check(dataclasses.replace(w, causal_period=64), ("split",))
    check(wl.make_random("log_softmax", dtype, 100, 16384, seed=358, scale=2.0), ("reg<", "packed"))
    # the fp32 normalisations stay in registers while the row is an exact fit, ragged rows do not
    check(wl.make_random("rmsnorm", wl.F32, 300, 32768, seed=352), ("reg", "flex"))
    check(wl.make_random("layernorm", wl.F32, 300, 32000, seed=353), ("split",))
    # ... and, with a thousand rows or more, leave one CTA of 576 - 1024 threads for a cluster of two
    check(wl.make_random("layernorm", wl.F32, 1100, 20480, seed=359, loc=0.5), ("split", "cs2,"), rows=list(range(0, 1100, 37)))
    check(wl.make_random("layernorm", wl.F32, 300, 20480, seed=359, loc=0.5), ("reg", "flex"))
    # fp32 softmax pair and RMSNorm rows of 4097 .. 6143 vectors: no thin CTA
    check(wl.make_random("rmsnorm", wl.F32, 300, 20480, seed=360), ("split", "cs2,"))
    check(wl.make_random("rmsnorm", wl.F32, 300, 24576, seed=360), ("reg", "flex"))
    # the fp32 softmax pair leaves the registers beyond 4096 vectors, masked or not (slices of about 2048 vectors)
    check(wl.make_random("softmax", wl.F32, 300, 32768, seed=354), ("split", "cs4,"))
    check(wl.make_random("log_softmax", wl.F32, 300, 16384, seed=357), ("reg<", "t512,v8,flex"))
    check(dataclasses.replace(wl.make_random("softmax", wl.F32, 300, 32768, seed=354), causal_period=77), ("split", "cs4,"))


@pytest.mark.parametrize("dtype", DTYPES)
def test_softmax_rows_in_the_registers_of_a_cluster(dtype):
    """cluster_mode 3: an unmasked softmax row held in the registers of a cluster of CTAs (no automatic choice)."""
    epv = 4 if dtype == wl.F32 else 8
    try:
        akg.set_tuning("cluster_mode", 3)
        for rows, nvec, cs in ((9, 16 * 512 * 8, 16), (70, 4 * 1024 * 8, 4), (5, 2 * 1024 * 8, 2), (300, 8 * 160 * 8, 8)):
            akg.set_tuning("cluster_size", cs)
            for op in ("softmax", "log_softmax"):
                w = wl.make_random(op, dtype, rows, nvec * epv, seed=370 + cs, scale=2.5)
                x = w.x.copy()
                if rows > 4:                       # a row without a live entry, and infinities in another
                    x[1, :] = np.float32(-np.inf) if dtype == wl.F32 else np.uint16(0xFF80)
                    x[2, 5] = np.float32(-np.inf) if dtype == wl.F32 else np.uint16(0xFF80)
                check(dataclasses.replace(w, x=x), ("reg<", f"cs{cs},"))
    finally:
        akg.set_tuning("cluster_mode", 0)
        akg.set_tuning("cluster_size", 0)
    assert akg.device_status() == 0


# ---- softmax, a CTA per row: the next row is loaded ahead -------------------------------------------

@pytest.mark.parametrize("dtype", DTYPES)
def test_softmax_prefetch_over_persistent_grid(dtype):
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    rows, cols = sms * 12 + 301, 4096            # more rows than CTAs: each CTA prefetches its next row
    for op in ("softmax", "log_softmax"):
        w = wl.make_random(op, dtype, rows, cols, seed=360, scale=3.0)
        w = dataclasses.replace(w, causal_period=4096)     # (unmasked rows take the packed / flex kernels)
        if w.causal_period:
            x = w.x.copy()
            bad = np.float32(np.nan) if dtype == wl.F32 else (np.uint16(0x7FC0) if dtype == wl.BF16 else np.float16(np.nan))
            for r in range(rows):
                x[r, (r % 4096) + 1:] = bad
            w = dataclasses.replace(w, x=x)
        sample = np.unique(np.concatenate([np.arange(0, 64), np.arange(rows - 64, rows),
                                           np.random.default_rng(6).integers(0, rows, 150)]))
        check(w, ("reg<", "v4>"), rows=sample)
    try:
        akg.set_tuning("grid_cap", 3)             # a handful of CTAs walk every row
        w = wl.make_random("softmax", dtype, 41, 3000 if dtype == wl.F32 else 3000 // 8 * 8, seed=361)
        check(w, ("reg<",))
    finally:
        akg.set_tuning("grid_cap", 0)


# ---- reductions: a warp per row, and the CTA per row that loads ahead -------------------------------

def store(x32, dtype):
    if dtype == wl.F32:
        return x32
    return wl.f32_to_bf16_bits(x32) if dtype == wl.BF16 else x32.astype(np.float16)


@pytest.mark.parametrize("dtype", DTYPES)
def test_argreduce_routes(dtype):
    rng = np.random.default_rng(370)
    es = 4 if dtype == wl.F32 else 2
    warp_cols = (8192 if dtype == wl.F32 else 16384) // es
    for rows, cols, expect in ((530, warp_cols, "g32"), (530, warp_cols + 64, "g256"), (3100, 8192, None),
                               (64, 1024, "g32")):
        x = np.round(rng.normal(0, 2, (rows, cols)) * 8).astype(np.float32) / 8      # many ties
        x[rng.integers(0, rows, 9), rng.integers(0, cols, 9)] = np.nan
        xs = store(x, dtype)
        for op, fn in (("argmax", binding.argmax), ("argmin", binding.argmin)):
            got = fn(to_torch(xs, dtype)).cpu().numpy()
            name = akg.last_kernel()
            if expect is not None:
                assert expect in name, (rows, cols, name)
            assert np.array_equal(got, oracle.argreduce(op, xs, nthreads=8)), (op, rows, cols, name)
    # the CTA-per-row kernel on a grid far smaller than the rows (every CTA loads ahead many times)
    try:
        akg.set_tuning("grid_cap", 7)
        x = store(rng.normal(0, 1, (300, 8192 + 4096)).astype(np.float32), dtype)
        got = binding.argmax(to_torch(x, dtype)).cpu().numpy()
        assert "g256" in akg.last_kernel() and "grid7" in akg.last_kernel()
        assert np.array_equal(got, oracle.argreduce("argmax", x, nthreads=8))
    finally:
        akg.set_tuning("grid_cap", 0)


@pytest.mark.parametrize("dtype", DTYPES)
def test_cumulative_routes(dtype):
    from test_gpu_reduction import tree_slack
    rng = np.random.default_rng(380)
    es = 4 if dtype == wl.F32 else 2
    warp_cols = (2048 if dtype == wl.F32 else 32768) // es
    for rows, cols, expect in ((270, warp_cols, "g32"), (270, warp_cols + 64, "vec,t"), (1000, 256, "scan_short"),
                               (1000, 128 * 16 // es, "g32"), (9, 40000, ",t256")):
        x = store(rng.normal(0.05, 1, (rows, cols)).astype(np.float32), dtype)
        ref = oracle.cumulative("cumsum", x, nthreads=8)
        got = to_numpy(binding.cumsum(to_torch(x, dtype)))
        name = akg.last_kernel()
        assert expect in name, (rows, cols, name)
        mag = np.cumsum(np.abs(widen(x)), axis=1)
        compare(got, ref, dtype, f"cumsum {rows}x{cols} [{name}]", tree_slack(cols, mag))
        f = store((1.0 + 0.002 * rng.normal(0, 1, (rows, cols))).astype(np.float32), dtype)
        ref = oracle.cumulative("cumprod", f, nthreads=8)
        got = to_numpy(binding.cumprod(to_torch(f, dtype)))
        compare(got, ref, dtype, f"cumprod {rows}x{cols} [{akg.last_kernel()}]", tree_slack(cols, np.abs(ref)))
    try:
        akg.set_tuning("grid_cap", 5)             # rows and chunks are both loaded ahead across a small grid
        for cols in (1024, 9000 // 8 * 8):
            x = store(rng.normal(0, 1, (77, cols)).astype(np.float32), dtype)
            ref = oracle.cumulative("cumsum", x, nthreads=8)
            got = to_numpy(binding.cumsum(to_torch(x, dtype)))
            compare(got, ref, dtype, f"cumsum capped {cols}", tree_slack(cols, np.cumsum(np.abs(widen(x)), axis=1)))
    finally:
        akg.set_tuning("grid_cap", 0)


# ---- short rows: several rows per warp ----------------------------------------------------------------

@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("op", ["softmax", "log_softmax", "layernorm", "rmsnorm"])
def test_short_rows_share_a_warp(op, dtype):
    epv = 4 if dtype == wl.F32 else 8
    norm = op in ("layernorm", "rmsnorm")
    # vectors per row -> lanes per row: 1..16 -> 4, ..32 -> 8, ..64 -> 16, ..128 -> 32
    for nv, lanes in ((1, 4), (3, 4), (16, 4), (17, 8), (32, 8), (33, 16), (50, 16), (64, 16), (80, 32), (112, 32)):
        if nv > 64 and not norm and dtype == wl.F32 and nv > 96:
            continue
        for rows in (1, 37, 1031):                       # rows that do not fill the last warp or CTA
            w = wl.make_random(op, dtype, rows, nv * epv, seed=390 + nv, loc=0.3, scale=1.7)
            check(w, ("short<", f"l{lanes},"))
    # non-finite rows keep the semantics of the other kernels: NaN rows, +inf rows, rows of -inf
    w = wl.make_random(op, dtype, 8, 16 * epv, seed=399)
    x = widen(w.x).copy()
    x[1, 3] = np.nan
    x[4, :] = 0.0
    if not norm:                                         # infinities: pinned for the softmax pair only
        x[2, 5] = np.inf
        x[3, :] = -np.inf
        x[5, 7] = -np.inf
    w = dataclasses.replace(w, x=store(x.astype(np.float32), dtype))
    check(w, ("short<",))
    # strided rows and a grid smaller than the work
    try:
        akg.set_tuning("grid_cap", 2)
        w = wl.make_random(op, dtype, 700, 24 * epv, seed=398)
        check(w, ("short<", "grid2>"))
    finally:
        akg.set_tuning("grid_cap", 0)
    # the causal rule: live prefixes of every length, masked inputs poisoned, masked outputs exact
    if not norm:
        for nv, period in ((16, 16 * epv), (50, 37), (64, 1000)):
            cols = nv * epv
            rows = 3 * period + 5
            w = dataclasses.replace(wl.make_random(op, dtype, rows, cols, seed=397 + nv), causal_period=period)
            x = w.x.copy()
            bad = np.float32(np.nan) if dtype == wl.F32 else (np.uint16(0x7FC0) if dtype == wl.BF16 else np.float16(np.nan))
            live = np.minimum(np.arange(rows) % period + 1, cols)
            for r in range(rows):
                x[r, live[r]:] = bad
            w = dataclasses.replace(w, x=x)
            got, name = check(w, ("short<",))
            dead = np.arange(cols)[None, :] >= live[:, None]
            if op == "softmax":
                assert_positive_zero(got, dead, name)
            else:
                assert np.all(np.isneginf(widen(got)[dead]))
