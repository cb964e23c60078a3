"""GPU parity: the CUDA library (through its C ABI) against the fp64 oracle,
element by element, on the same seeded inputs."""
import os

import numpy as np
import pytest
import torch

import oracle
import paper_2512_23424_b200 as akg
from golden_io import worked_examples
from paper_2512_23424_b200 import workloads as wl
from parity_util import (assert_positive_zero, cancel_magnitude, compare, run_gpu, run_oracle, strided_device_matrix,
                         to_numpy, to_torch, verifier_passes, widen)

pytestmark = pytest.mark.gpu

VARIANTS = ["auto", "stream", "reg", "tma", "tma_smem", "cluster", "split"]
GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


@pytest.fixture(autouse=True)
def _reset_variant():
    yield
    akg.set_variant("auto")
    for key in ("reg_threads", "reg_vpt", "reg_group", "reg_general", "grid_cap", "cluster_size",
                "smem_nbuf", "smem_threads", "smem_ctas"):
        akg.set_tuning(key, 0)


def run_variant(variant, fn):
    """Run fn() under a forced kernel family; None if that family cannot take the call."""
    # "split" is the cluster family's two-pass mode (second pass served by L2)
    # "tma" prefers the ring-fed register kernels; "tma_smem" forces the shared-memory passes
    family = {"split": "cluster", "tma_smem": "tma"}.get(variant, variant)
    akg.set_variant(family)
    akg.set_tuning("cluster_mode", 2 if variant == "split" else (1 if variant == "cluster" else 0))
    akg.set_tuning("tma_mode", 2 if variant == "tma_smem" else 0)
    try:
        return fn()
    except akg.AkgError as e:
        if variant != "auto" and e.status == akg.binding.ERR_UNSUPPORTED:
            return None
        raise
    finally:
        akg.set_variant("auto")
        akg.set_tuning("cluster_mode", 0)
        akg.set_tuning("tma_mode", 0)


def check_workload(w, variants=VARIANTS, **kw):
    ref = run_oracle(w, additive=kw.get("additive_host"), causal_offset=kw.get("causal_offset", 0))
    mag = cancel_magnitude(w, ref, kw.get("additive_host"))
    ran = []
    for v in variants:
        add_dev = to_torch(kw["additive_host"], w.dtype) if kw.get("additive_host") is not None else None
        out = run_variant(v, lambda: run_gpu(w, additive=add_dev, causal_offset=kw.get("causal_offset", 0)))
        if out is None:
            continue
        torch.cuda.synchronize()
        got = to_numpy(out)
        compare(got, ref, w.dtype, f"{w.name}[{v}:{akg.last_kernel()}]", mag)
        assert verifier_passes(got, ref, w.dtype)
        ran.append(v)
    assert "auto" in ran
    return ref


# ---- the five configurations, at sizes the oracle finishes in seconds ---------------------

@pytest.mark.parametrize("k,rows", [(1, None), (2, 300), (3, 301), (4, 5), (5, 4096 + 130)])
def test_configs_reduced(k, rows):
    w = wl.make_config(k, rows=rows)
    ref = check_workload(w)
    if k == 5:
        out = to_numpy(run_gpu(w))
        r = np.arange(w.rows)[:, None] % 4096
        c = np.arange(w.cols)[None, :]
        assert_positive_zero(out, c > r, "config 5")
        np.testing.assert_allclose(ref.sum(axis=1), 1.0, atol=1e-12)


# ---- worked examples through the GPU ------------------------------------------------------------

@pytest.mark.parametrize("dtype", [wl.F32])
def test_worked_examples_on_gpu(dtype):
    for case in worked_examples(GOLDEN):
        x = np.array(case["x"], dtype=np.float32)
        want = np.array(case["expect"], dtype=np.float64)
        w = wl.Workload(case["name"], case["op"], dtype, x.shape[0], x.shape[1], x, eps=case["eps"],
                        causal_period=case["causal_period"])
        add = np.array(case["additive"], dtype=np.float32) if "additive" in case else None
        if case["op"] == "layernorm":
            w.gamma = np.array(case["gamma"], dtype=np.float32) if "gamma" in case else None
            w.beta = np.array(case["beta"], dtype=np.float32) if "beta" in case else None
        if case["op"] == "rmsnorm":
            w.gamma = np.array(case["weight"], dtype=np.float32) if "weight" in case else None
        for v in VARIANTS:
            add_dev = to_torch(add, dtype) if add is not None else None
            out = run_variant(v, lambda: run_gpu(w, additive=add_dev))
            if out is None:
                continue
            got = to_numpy(out)
            keep = [r for r in range(x.shape[0]) if r not in case["skip_rows"]]
            # eps given as float32 to the library: compare with a tolerance that covers it
            np.testing.assert_allclose(widen(got)[keep], want[keep], rtol=0, atol=2e-6,
                                       err_msg=f"{case['name']}[{v}]")
            if case["op"] == "softmax":
                assert_positive_zero(got[keep], want[keep] == 0, case["name"])


# ---- shape sweep: ragged sizes, strides, misaligned bases ---------------------------------------

SWEEP_COLS = [1, 2, 3, 4, 5, 7, 8, 9, 31, 32, 33, 127, 128, 129, 1000, 1023, 1024, 1025, 4095, 4096,
              4097, 8191, 8192, 32768 + 8,
              # hidden sizes that are (a multiple of 32 threads) x (1..8 vectors), not a power of two
              1536, 2560, 5120, 6144, 7168, 12288, 20480]
SWEEP_ROWS = [1, 2, 3, 63, 65, 148, 149]
# long rows around the sizes a tile size would divide (two or three rows each): odd, a multiple of
# one fp32 vector only, of one 16-bit vector only, and a row of a million columns
SWEEP_LONG_COLS = [262144 - 1, 262144 + 4, 262144 + 8, 1048576 + 12]


@pytest.mark.parametrize("op", ["softmax", "log_softmax", "layernorm", "rmsnorm"])
@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16])
def test_shape_sweep(op, dtype):
    seed = 100
    for cols in SWEEP_COLS:
        for rows in (SWEEP_ROWS if cols <= 1025 else [3, 65]):
            seed += 1
            if op in ("softmax", "log_softmax"):
                w = wl.make_random(op, dtype, rows, cols, seed, scale=2.0)
            else:
                w = wl.make_random(op, dtype, rows, cols, seed, loc=1.0, scale=1.5, eps=1e-5)
            check_workload(w)
    for i, cols in enumerate(SWEEP_LONG_COLS):
        rows = 2 + i % 2
        if op in ("softmax", "log_softmax"):
            w = wl.make_random(op, dtype, rows, cols, 900 + i, scale=2.0)
        else:
            w = wl.make_random(op, dtype, rows, cols, 900 + i, loc=1.0, scale=1.5, eps=1e-5)
        check_workload(w)


# LayerNorm rows whose mean is thirty standard deviations from zero: a mean that is off by one part in 2^24
# (a thread's sum times a rounded 1 / 24, 1 / 56, ...; warp means times a rounded 1 / 3, 1 / 7, ...) moves the
# results next to zero by more than two ulps of a 16-bit type.  Shapes with a number of values per thread and a
# number of warps per row that are no powers of two, and short rows (1 / cols).
@pytest.mark.parametrize("dtype,rows,cols,seed,affine", [
    (wl.BF16, 585, 5376, 112391494, True), (wl.F16, 585, 5376, 98737495, True), (wl.F16, 585, 5376, 98737495, False),
    (wl.BF16, 585, 5376, 5, True), (wl.BF16, 585, 10752, 5, True), (wl.BF16, 2000, 768, 6, True),
    (wl.BF16, 4100, 264, 7, True), (wl.F16, 4100, 200, 8, True), (wl.F32, 300, 5120, 9, True),
    (wl.F32, 300, 2560, 10, True)])
def test_layernorm_mean_far_from_zero(dtype, rows, cols, seed, affine):
    base = wl.make_random("layernorm", wl.F32 if dtype == wl.F16 else dtype, rows, cols, seed, loc=-3.0, scale=0.1,
                          affine=affine)
    check_workload(wl.as_f16(base) if dtype == wl.F16 else base, variants=["auto"])


@pytest.mark.parametrize("op", ["softmax", "log_softmax", "layernorm", "rmsnorm"])
@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16])
def test_strides_offsets_and_no_stray_writes(op, dtype):
    """Row stride > cols, base pointer off by one element, output padding untouched."""
    sentinel = 12345.0
    for cols, rows in [(1000, 9), (1024, 33), (33, 70), (4096, 5), (260, 300)]:
        for stride, off in [(cols + 1, 0), (cols + 8, 0), (2 * cols, 0), (cols, 1), (cols + 8, 1)]:
            w = wl.make_random(op, dtype, rows, cols, seed=cols + stride + off, loc=0.5, eps=1e-5)
            ref = run_oracle(w)
            for v in VARIANTS:
                _, xv = strided_device_matrix(w.x, dtype, stride, off)
                ybuf, yv = strided_device_matrix(np.zeros_like(w.x), dtype, stride, off, sentinel=sentinel)
                yv.fill_(float("nan"))
                before = ybuf.clone()
                out = run_variant(v, lambda: run_gpu(w, x_dev=xv, out=yv))
                if out is None:
                    continue
                torch.cuda.synchronize()
                compare(to_numpy(yv), ref, dtype, f"{w.name} stride {stride} off {off} [{v}]",
                        cancel_magnitude(w, ref))
                # everything outside the rows x cols window is unchanged
                ybuf2 = ybuf.clone()
                torch.as_strided(ybuf2, (rows, cols), (stride, 1), off).copy_(
                    torch.as_strided(before, (rows, cols), (stride, 1), off))
                assert torch.equal(ybuf2.view(torch.int16 if dtype == wl.BF16 else torch.int32),
                                   before.view(torch.int16 if dtype == wl.BF16 else torch.int32))


# ---- masks ---------------------------------------------------------------------------------------

@pytest.mark.parametrize("op", ["softmax", "log_softmax"])
@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16])
def test_causal_masks(op, dtype):
    for rows, cols, period, offset in [(70, 64, 64, 0), (130, 1024, 100, 0), (50, 1000, 7, 3),
                                       (40, 4096, 4096, 0), (64, 512, 16, -2), (33, 129, 5, 0),
                                       (20, 256, 1000, 250)]:
        w = wl.make_random(op, dtype, rows, cols, seed=rows + cols + period)
        w.causal_period = period
        ref = check_workload(w, causal_offset=offset)
        # masked inputs are never read: poison them with NaN, the result must not change
        poisoned = widen(w.x).astype(np.float32)
        r = (np.arange(rows)[:, None] % period) + offset
        dead = np.arange(cols)[None, :] > r
        poisoned[dead] = np.nan
        wp = wl.Workload(w.name + "_poison", op, dtype, rows, cols,
                         poisoned if dtype == wl.F32 else wl.f32_to_bf16_bits(poisoned),
                         causal_period=period)
        for v in VARIANTS:
            out = run_variant(v, lambda: run_gpu(wp, causal_offset=offset))
            if out is None:
                continue
            got = to_numpy(out)
            compare(got, ref, dtype, f"{wp.name}[{v}]", cancel_magnitude(w, ref))
            if op == "softmax":
                assert_positive_zero(got, dead, wp.name)


@pytest.mark.parametrize("op", ["softmax", "log_softmax"])
@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16])
def test_additive_masks(op, dtype):
    rng = np.random.default_rng(7)
    for rows, cols, add_rows in [(64, 256, 1), (64, 256, 64), (96, 1024, 32), (10, 1000, 3), (17, 33, 5),
                                 (12, 8192, 4)]:
        w = wl.make_random(op, dtype, rows, cols, seed=rows * cols + add_rows)
        add = rng.normal(0, 1, size=(add_rows, cols)).astype(np.float32)
        add[rng.random(size=add.shape) < 0.3] = -np.inf
        if add_rows > 1:
            add[1, :] = -np.inf                      # a whole row with no live entry
        add_host = add if dtype == wl.F32 else wl.f32_to_bf16_bits(add)
        ref = check_workload(w, additive_host=add_host)
        if op == "softmax":
            out = to_numpy(run_gpu(w, additive=to_torch(add_host, dtype)))
            dead = np.isneginf(np.tile(add, (rows // add_rows + 1, 1))[:rows])
            assert_positive_zero(out, dead, w.name)
        # both masks at once
        w.causal_period = 16
        check_workload(w, additive_host=add_host)


@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16])
def test_rows_without_live_entries_and_non_finite_inputs(dtype):
    cols = 1024
    x = np.random.default_rng(3).normal(size=(6, cols)).astype(np.float32)
    x[0, :] = -np.inf
    x[1, 5] = np.nan
    x[2, 1000] = np.inf
    x[3, ::2] = -np.inf
    x[4, :] = np.nan                       # nothing but NaN
    x[5, :] = -np.inf                      # NaN among masked entries only
    x[5, 77] = np.nan
    xs = x if dtype == wl.F32 else wl.f32_to_bf16_bits(x)
    for op in ("softmax", "log_softmax"):
        w = wl.Workload("special", op, dtype, 6, cols, xs)
        check_workload(w)
        out = to_numpy(run_gpu(w))
        if op == "softmax":
            assert_positive_zero(out, np.isneginf(x) & ~np.isnan(widen(out)), "special")
            bits = out.view(np.uint32) if dtype == wl.F32 else out
            assert (bits[0] == 0).all()
    # causal offset that masks entire rows
    w = wl.make_random("softmax", dtype, 8, 256, seed=5)
    w.causal_period = 4
    check_workload(w, causal_offset=-2)
    out = to_numpy(run_gpu(w, causal_offset=-2))
    bits = out.view(np.uint32) if dtype == wl.F32 else out
    assert (bits[0] == 0).all() and (bits[1] == 0).all() and (bits[4] == 0).all()


# ---- in place, empty shapes, bad arguments ---------------------------------------------------------

@pytest.mark.parametrize("op", ["softmax", "log_softmax", "layernorm", "rmsnorm"])
@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16])
def test_in_place(op, dtype):
    for cols in (1000, 4096, 1023):
        w = wl.make_random(op, dtype, 37, cols, seed=cols, loc=0.3, eps=1e-5)
        ref = run_oracle(w)
        for v in VARIANTS:
            x = to_torch(w.x, dtype)
            out = run_variant(v, lambda: run_gpu(w, x_dev=x, out=x))
            if out is None:
                continue
            compare(to_numpy(x), ref, dtype, f"in-place {w.name}[{v}]", cancel_magnitude(w, ref))


def test_interleaved_column_windows_of_one_buffer():
    """x = buf[:, :cols] and y = buf[:, cols:] share rows of one buffer but no element: accepted."""
    for dtype in (wl.F32, wl.BF16):
        w = wl.make_random("rmsnorm", dtype, 48, 512, seed=77, eps=1e-6)
        tdt = torch.float32 if dtype == wl.F32 else torch.bfloat16
        buf = torch.zeros((w.rows, 2 * w.cols), dtype=tdt, device="cuda")
        buf[:, :w.cols] = to_torch(w.x, dtype)
        before = buf[:, :w.cols].clone()
        run_gpu(w, x_dev=buf[:, :w.cols], out=buf[:, w.cols:])
        torch.cuda.synchronize()
        compare(to_numpy(buf[:, w.cols:]), run_oracle(w), dtype, "interleaved windows")
        assert torch.equal(buf[:, :w.cols], before)
    # windows that do share elements are still refused
    L = akg.lib()
    f = torch.zeros(4 * 24, device="cuda")
    assert L.akg_softmax(f.data_ptr(), f.data_ptr() + 4 * 4, 4, 8, 24, 24, 0, None, None) == 1
    assert L.akg_softmax(f.data_ptr(), f.data_ptr() + 4 * 20, 4, 8, 24, 24, 0, None, None) == 1
    assert L.akg_softmax(f.data_ptr(), f.data_ptr() + 4 * 8, 3, 8, 24, 24, 0, None, None) == 0


def test_empty_and_invalid_arguments():
    x = torch.zeros((4, 8), device="cuda")
    y = torch.empty_like(x)
    L = akg.lib()
    assert L.akg_softmax(None, None, 0, 8, 8, 8, 0, None, None) == 0
    assert L.akg_softmax(None, None, 8, 0, 8, 8, 0, None, None) == 0
    assert L.akg_softmax(x.data_ptr(), y.data_ptr(), 4, 8, 7, 8, 0, None, None) == 1
    assert L.akg_softmax(x.data_ptr(), y.data_ptr(), 4, 8, 8, 8, 9, None, None) == 1
    assert L.akg_layernorm(x.data_ptr(), y.data_ptr(), 4, 8, 8, 8, 0, None, None, -1.0, None) == 1
    assert L.akg_rmsnorm(x.data_ptr(), y.data_ptr(), 4, 8, 8, 8, 0, None, float("nan"), None) == 1
    # partial overlap of x and y
    buf = torch.zeros(64, device="cuda")
    assert L.akg_softmax(buf.data_ptr(), buf.data_ptr() + 16, 4, 8, 8, 8, 0, None, None) == 1
    torch.cuda.synchronize()
    assert akg.device_status() == 0
