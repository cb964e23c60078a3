"""GPU parity of akg_argreduce (bit-exact indices) and akg_cumulative (within the tolerance the
tree of additions / multiplications implies) against the oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
import paper_2512_23424_b200 as akg
from paper_2512_23424_b200 import binding
from paper_2512_23424_b200 import workloads as wl
from parity_util import compare, to_numpy, to_torch, widen

pytestmark = pytest.mark.gpu
DTYPES = [wl.F32, wl.BF16]
SHAPES = [(1, 1), (3, 7), (64, 1024), (9, 4096), (5, 40000), (300, 130), (17, 2048), (2, 262144), (33, 520), (4, 8)]


def store(x32, dtype):
    return x32 if dtype == wl.F32 else wl.f32_to_bf16_bits(x32)


# ---- arg-max / arg-min: indices must match exactly -----------------------------------------------

def check_arg(x, dtype, what):
    xd = to_torch(x, dtype)
    for op, fn in (("argmax", binding.argmax), ("argmin", binding.argmin)):
        got = fn(xd).cpu().numpy()
        want = oracle.argreduce(op, x, nthreads=8)
        assert got.dtype == np.int64
        assert np.array_equal(got, want), f"{what} {op} [{akg.last_kernel()}]: rows {np.nonzero(got != want)[0][:5]}"


@pytest.mark.parametrize("dtype", DTYPES)
def test_argreduce_shapes_ties_and_special_values(dtype):
    rng = np.random.default_rng(21)
    kernels = set()
    for rows, cols in SHAPES:
        x = rng.normal(0, 1, (rows, cols)).astype(np.float32)
        check_arg(store(x, dtype), dtype, f"{rows}x{cols}")
        kernels.add(akg.last_kernel().split(",grid")[0])
        # heavy ties: a handful of distinct values, so first-index rules decide almost every row
        q = np.round(x * 2).astype(np.float32) / 2
        q[q == 0] = np.where(rng.random(np.count_nonzero(q == 0)) < 0.5, -0.0, 0.0)
        check_arg(store(q, dtype), dtype, f"ties {rows}x{cols}")
        # NaN and infinities at seeded places, a constant row, a row of one sign of infinity
        s = x.copy()
        for r in range(rows):
            k = rng.integers(0, 6)
            pos = rng.integers(0, cols, size=3)
            if k == 0:
                s[r, pos[0]] = np.nan
            elif k == 1:
                s[r, pos] = np.nan
            elif k == 2:
                s[r, pos[0]], s[r, pos[1]] = np.inf, -np.inf
            elif k == 3:
                s[r, :] = 1.25
            elif k == 4:
                s[r, :] = -np.inf if r % 2 else np.inf
        check_arg(store(s, dtype), dtype, f"special {rows}x{cols}")
    assert len(kernels) >= 3 and any(k.startswith("arg_split") for k in kernels), kernels
    # few long rows with and without the split into segments: same indices, ties and NaN across segments
    x = np.round(rng.normal(0, 1, (3, 200000)) * 4).astype(np.float32) / 4
    x[1, 150000] = np.nan
    x[1, 70000] = np.nan
    x[2, :] = 0.5
    try:
        for general in (0, 1):
            akg.set_tuning("reg_general", general)
            check_arg(store(x, dtype), dtype, f"long rows, split {1 - general}")
            assert akg.last_kernel().startswith("arg_split") == (general == 0)
    finally:
        akg.set_tuning("reg_general", 0)


@pytest.mark.parametrize("dtype", DTYPES)
def test_argreduce_strides_misalignment_and_clipped_grid(dtype):
    rng = np.random.default_rng(22)
    rows, cols = 37, 1032
    x = store(np.round(rng.normal(0, 3, (rows, cols))).astype(np.float32), dtype)
    tdt = torch.float32 if dtype == wl.F32 else torch.bfloat16
    big = torch.full((rows, cols + 24), 99.0, dtype=tdt, device="cuda")     # padding would win an arg-max
    big[:, :cols].copy_(to_torch(x, dtype))
    for op, fn in (("argmax", binding.argmax), ("argmin", binding.argmin)):
        assert np.array_equal(fn(big[:, :cols]).cpu().numpy(), oracle.argreduce(op, x))
    flat = torch.zeros(rows * (cols + 1) + 3, dtype=tdt, device="cuda")
    v = flat[1:1 + rows * (cols + 1)].view(rows, cols + 1)[:, :cols]
    v.copy_(to_torch(x, dtype))
    got = binding.argmax(v).cpu().numpy()
    assert "scalar" in akg.last_kernel()
    assert np.array_equal(got, oracle.argreduce("argmax", x))
    try:
        akg.set_tuning("grid_cap", 2)
        for shape in ((50, 256), (50, 9000)):
            y = store(rng.normal(0, 1, shape).astype(np.float32), dtype)
            assert np.array_equal(binding.argmin(to_torch(y, dtype)).cpu().numpy(), oracle.argreduce("argmin", y))
    finally:
        akg.set_tuning("grid_cap", 0)


# ---- cumulative sum / product ------------------------------------------------------------------------

def tree_slack(cols, magnitude):
    """First-order error bound of the kernel's association order.  A prefix is assembled from the
    totals of the groups of 1024 columns (a warp-level tree of at most 16 operations each, plus its
    own merge) that precede it and a tree of at most 32 operations inside its own group, so element
    c has passed through at most 32 + 20 * floor(c / 1024) roundings of half an fp32 ulp of the
    running magnitude (the sum of |x| so far for a sum, |result| for a product)."""
    depth = 32.0 + 20.0 * np.floor(np.arange(cols) / 1024.0)
    return depth[None, :] * 2.0 ** -24 * magnitude


def check_cum(op, x, dtype, what):
    ref = oracle.cumulative(op, x, nthreads=8)
    fn = binding.cumsum if op == "cumsum" else binding.cumprod
    got = to_numpy(fn(to_torch(x, dtype)))
    mag = np.cumsum(np.abs(widen(x)), axis=1) if op == "cumsum" else np.abs(ref)
    compare(got, ref, dtype, f"{what} {op} [{akg.last_kernel()}]", tree_slack(x.shape[1], mag))


@pytest.mark.parametrize("dtype", DTYPES)
def test_cumulative_shapes(dtype):
    rng = np.random.default_rng(23)
    kernels = set()
    for rows, cols in SHAPES:
        x = rng.normal(0.1, 1, (rows, cols)).astype(np.float32)
        check_cum("cumsum", store(x, dtype), dtype, f"{rows}x{cols}")
        kernels.add(akg.last_kernel().split(",grid")[0])
        # factors near one, a few sign flips: the running product stays inside the fp32 range
        f = (1.0 + 0.002 * rng.normal(0, 1, (rows, cols))).astype(np.float32)
        f[rng.random((rows, cols)) < 0.01] *= -1
        check_cum("cumprod", store(f, dtype), dtype, f"{rows}x{cols}")
    assert len(kernels) >= 4, kernels


@pytest.mark.parametrize("dtype", DTYPES)
def test_cumulative_short_rows_several_per_warp(dtype):
    """Rows of at most 64 vectors: 4, 8 or 16 lanes per row (every group size, ragged row counts, rows that
    do not fill their lanes, more rows than the grid holds warps)."""
    rng = np.random.default_rng(26)
    epv = 4 if dtype == wl.F32 else 8
    seen = set()
    try:
        for rows, nvec, cap in [(1, 1, 0), (7, 3, 0), (1000, 8, 0), (37, 16, 0), (999, 17, 0), (5000, 32, 0), (130, 33, 0),
                                (3001, 64, 0), (20000, 32, 5), (8, 64, 0), (65, 12, 1)]:
            akg.set_tuning("grid_cap", cap)
            cols = nvec * epv
            x = rng.normal(0.05, 1, (rows, cols)).astype(np.float32)
            check_cum("cumsum", store(x, dtype), dtype, f"{rows}x{cols}")
            assert akg.last_kernel().startswith("scan_short<"), akg.last_kernel()
            seen.add(akg.last_kernel().split(",")[2])
            f = (1.0 + 0.01 * rng.normal(0, 1, (rows, cols))).astype(np.float32)
            check_cum("cumprod", store(f, dtype), dtype, f"{rows}x{cols}")
        assert seen == {"l4", "l8", "l16"}, seen
        # exact arithmetic and padded rows in place
        akg.set_tuning("grid_cap", 0)
        x = rng.integers(-3, 4, (77, 24 * epv)).astype(np.float32)
        tdt = torch.float32 if dtype == wl.F32 else torch.bfloat16
        big = torch.full((77, 24 * epv + 2 * epv), 9.0, dtype=tdt, device="cuda")
        big[:, :24 * epv].copy_(to_torch(store(x, dtype), dtype))
        binding.cumsum(big[:, :24 * epv], out=big[:, :24 * epv])
        torch.cuda.synchronize()
        assert akg.last_kernel().startswith("scan_short<")
        ref = oracle.cumulative("cumsum", x)
        got = widen(to_numpy(big[:, :24 * epv].contiguous()))
        exact = np.abs(ref) < (2 ** 24 if dtype == wl.F32 else 256)
        assert np.array_equal(got[exact], ref[exact])
        assert torch.all(big[:, 24 * epv:] == 9.0)
    finally:
        akg.set_tuning("grid_cap", 0)


@pytest.mark.parametrize("dtype", DTYPES)
def test_cumulative_long_rows_split_over_a_cluster(dtype):
    """Few, long rows: a cluster per row, a slice per CTA, the carry of a slice from the peers' totals."""
    rng = np.random.default_rng(25)
    epv = 4 if dtype == wl.F32 else 8
    try:
        for rows, cols, cs in [(3, 65536 * epv // 4, 0), (2, 262144 + 8, 0), (5, 100000, 4), (7, 40960, 2),
                               (2, 70000 * epv // 4 + epv, 16), (300, 9000 * epv, 8), (1, 4096 * epv, 8)]:
            akg.set_tuning("cluster_size", cs)
            x = rng.normal(0.05, 1, (rows, cols)).astype(np.float32)
            check_cum("cumsum", store(x, dtype), dtype, f"{rows}x{cols} cs{cs}")
            assert akg.last_kernel().startswith("scan_split<"), akg.last_kernel()
            if cs:
                assert f"cs{cs}," in akg.last_kernel()
            f = (1.0 + 0.002 * rng.normal(0, 1, (rows, cols))).astype(np.float32)
            f[rng.random((rows, cols)) < 0.01] *= -1
            check_cum("cumprod", store(f, dtype), dtype, f"{rows}x{cols} cs{cs}")
            assert akg.last_kernel().startswith("scan_split<")
        # exact arithmetic across slices: small integers, and in place with padded rows
        akg.set_tuning("cluster_size", 4)
        x = rng.integers(-2, 3, (3, 24576)).astype(np.float32)
        ref = oracle.cumulative("cumsum", x)
        tdt = torch.float32 if dtype == wl.F32 else torch.bfloat16
        big = torch.full((3, 24576 + 8 * epv), 7.0, dtype=tdt, device="cuda")
        big[:, :24576].copy_(to_torch(store(x, dtype), dtype))
        binding.cumsum(big[:, :24576], out=big[:, :24576])
        torch.cuda.synchronize()
        assert akg.last_kernel().startswith("scan_split<")
        got = widen(to_numpy(big[:, :24576].contiguous()))
        exact = np.abs(ref) < (2 ** 24 if dtype == wl.F32 else 256)
        assert np.array_equal(got[exact], ref[exact])
        assert torch.all(big[:, 24576:] == 7.0)
    finally:
        akg.set_tuning("cluster_size", 0)
    assert akg.device_status() == 0


@pytest.mark.parametrize("dtype", DTYPES)
def test_cumulative_few_long_rows_load_three_chunks_ahead(dtype):
    """A CTA per row with few CTAs: the loads run three chunks ahead of the scan, across row ends as well."""
    rng = np.random.default_rng(26)
    epv = 4 if dtype == wl.F32 else 8
    try:
        # (ragged last chunks, rows of exactly three and of four chunks, one chunk only, more rows than CTAs)
        for rows, cols, cap in [(37, 5000 * epv, 0), (200, 4096 * epv, 0), (9, 3072 * epv + epv, 0), (50, 7777 * epv, 7),
                                (11, 1024 * epv, 3), (5, 300 * epv, 2)]:
            akg.set_tuning("reg_vpt", 3)
            akg.set_tuning("cluster_size", 1)
            akg.set_tuning("grid_cap", cap)
            x = rng.normal(0.05, 1, (rows, cols)).astype(np.float32)
            check_cum("cumsum", store(x, dtype), dtype, f"{rows}x{cols} ahead3")
            if ",t256," in akg.last_kernel() and "g32" not in akg.last_kernel():     # a CTA of 256 threads per row
                assert "ahead3" in akg.last_kernel(), akg.last_kernel()
            f = (1.0 + 0.002 * rng.normal(0, 1, (rows, cols))).astype(np.float32)
            check_cum("cumprod", store(f, dtype), dtype, f"{rows}x{cols} ahead3")
        akg.set_tuning("reg_vpt", 0)
        akg.set_tuning("grid_cap", 0)
        akg.set_tuning("cluster_size", 0)
        # the automatic choice (16-bit only): fewer CTAs than two per SM, rows of at least four chunks, no cluster
        x = rng.integers(-2, 3, (200, 5120 * epv)).astype(np.float32)
        ref = oracle.cumulative("cumsum", x)
        got = widen(to_numpy(binding.cumsum(to_torch(store(x, dtype), dtype))))
        assert akg.last_kernel().startswith("scan<") and ("ahead3" in akg.last_kernel()) == (dtype != wl.F32), \
            akg.last_kernel()
        exact = np.abs(ref) < (2 ** 24 if dtype == wl.F32 else 256)
        assert np.array_equal(got[exact], ref[exact])
    finally:
        akg.set_tuning("reg_vpt", 0)
        akg.set_tuning("grid_cap", 0)
        akg.set_tuning("cluster_size", 0)


@pytest.mark.parametrize("dtype", DTYPES)
def test_cumulative_exact_cases_in_place_and_strides(dtype):
    tdt = torch.float32 if dtype == wl.F32 else torch.bfloat16
    # small integers: every partial sum is exact in fp32 (and in bf16 while below 256)
    rng = np.random.default_rng(24)
    x = rng.integers(-3, 4, (19, 1000)).astype(np.float32)
    ref = oracle.cumulative("cumsum", x)
    got = widen(to_numpy(binding.cumsum(to_torch(store(x, dtype), dtype))))
    exact = np.abs(ref) < (2 ** 24 if dtype == wl.F32 else 256)
    assert np.array_equal(got[exact], ref[exact])
    # powers of two multiply exactly
    p = np.where(rng.random((7, 90)) < 0.5, 2.0, 0.5).astype(np.float32)
    assert np.array_equal(widen(to_numpy(binding.cumprod(to_torch(store(p, dtype), dtype)))), oracle.cumulative("cumprod", p))
    # zero, infinity and NaN travel as the arithmetic says
    s = np.array([[1.0, 2.0, np.inf, 1.0, -np.inf, 3.0, 0.0, 1.0] * 40], dtype=np.float32)
    got = widen(to_numpy(binding.cumsum(to_torch(store(s, dtype), dtype))))
    ref = oracle.cumulative("cumsum", s)
    assert np.array_equal(np.isnan(got), np.isnan(ref)) and np.array_equal(got[~np.isnan(ref)], ref[~np.isnan(ref)])
    z = np.array([[3.0, 0.5, 0.0, 7.0, 2.0, 1.0, 1.0, 1.0] * 5], dtype=np.float32)
    assert np.array_equal(widen(to_numpy(binding.cumprod(to_torch(store(z, dtype), dtype)))), oracle.cumulative("cumprod", z))
    # in place, padded rows, misaligned base
    y = store(rng.normal(0, 1, (11, 1032)).astype(np.float32), dtype)
    big = torch.full((11, 1032 + 8), 5.0, dtype=tdt, device="cuda")
    big[:, :1032].copy_(to_torch(y, dtype))
    binding.cumsum(big[:, :1032], out=big[:, :1032])
    torch.cuda.synchronize()
    ref = oracle.cumulative("cumsum", y)
    compare(to_numpy(big[:, :1032].contiguous()), ref, dtype, "in place", tree_slack(1032, np.cumsum(np.abs(widen(y)), axis=1)))
    assert torch.all(big[:, 1032:] == 5.0)
    flat = torch.zeros(11 * 1033 + 3, dtype=tdt, device="cuda")
    v = flat[1:1 + 11 * 1033].view(11, 1033)[:, :1032]
    v.copy_(to_torch(y, dtype))
    out = binding.cumsum(v)
    assert "scalar" in akg.last_kernel()
    compare(to_numpy(out), ref, dtype, "misaligned", tree_slack(1032, np.cumsum(np.abs(widen(y)), axis=1)))


def test_reduction_argument_errors():
    L = akg.lib()
    x = torch.zeros((4, 64), device="cuda")
    idx = torch.empty(4, dtype=torch.int64, device="cuda")
    y = torch.empty_like(x)
    binding.argmax(x, out=idx)
    binding.cumsum(x, out=y)
    P = lambda t: t.data_ptr()
    arg = lambda wm=0, xp=P(x), op=P(idx), rows=4, cols=64, xs=64, dt=0: L.akg_argreduce(wm, xp, op, rows, cols, xs, dt, None)
    assert arg() == 0 and arg(wm=1) == 0
    assert arg(wm=2) == 1 and arg(dt=4) == 1 and arg(rows=-1) == 1 and arg(xs=63) == 1
    assert arg(xp=None) == 1 and arg(op=None) == 1
    assert arg(cols=0, xs=0) == 1 and arg(rows=0) == 0
    cum = lambda wp=0, xp=P(x), yp=P(y), rows=4, cols=64, xs=64, ys=64, dt=0: L.akg_cumulative(wp, xp, yp, rows, cols, xs, ys, dt, None)
    assert cum() == 0 and cum(wp=1) == 0 and cum(yp=P(x)) == 0
    assert cum(wp=3) == 1 and cum(dt=9) == 1 and cum(ys=10) == 1 and cum(yp=P(x) + 8) == 1 and cum(xp=None) == 1
    assert cum(rows=0) == 0 and cum(cols=0, xs=0, ys=0) == 0
    torch.cuda.synchronize()
