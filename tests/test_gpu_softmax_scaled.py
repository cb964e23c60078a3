"""GPU parity of akg_softmax_scaled (softmax / log-softmax with a fused pre-scale) against the fp64
oracle, element by element, through the C ABI, with every kernel family forced in turn."""
import numpy as np
import pytest
import torch

import oracle
import paper_2512_23424_b200 as akg
from paper_2512_23424_b200 import binding
from paper_2512_23424_b200 import workloads as wl
from parity_util import CANCEL_16BIT, assert_positive_zero, compare, to_numpy, to_torch, verifier_passes, widen

pytestmark = pytest.mark.gpu
VARIANTS = ["auto", "stream", "reg", "tma", "tma_smem", "cluster", "split"]
SCALES = [0.125, 0.08838834764831845, 1.0, 3.0]


@pytest.fixture(autouse=True)
def _reset():
    yield
    akg.set_variant("auto")
    for key in ("cluster_mode", "tma_mode", "reg_general"):
        akg.set_tuning(key, 0)


def forced(variant, fn):
    family = {"split": "cluster", "tma_smem": "tma"}.get(variant, variant)
    akg.set_variant(family)
    akg.set_tuning("cluster_mode", 2 if variant == "split" else (1 if variant == "cluster" else 0))
    akg.set_tuning("tma_mode", 2 if variant == "tma_smem" else 0)
    try:
        return fn()
    except akg.AkgError as e:
        if "cannot run this call" in str(e):
            return None
        raise
    finally:
        akg.set_variant("auto")


def check_all(x, dtype, scale, log, additive=None, causal_period=0, variants=VARIANTS, what=""):
    rows, cols = x.shape
    omask = None
    if additive is not None or causal_period:
        omask = oracle.Mask(additive=additive, causal=causal_period > 0, causal_period=max(causal_period, 1))
    ref = oracle.softmax_scaled(x, float(np.float32(scale)), mask=omask, log=log, nthreads=8)
    mag = None
    if log and dtype == wl.BF16:                           # the final subtraction can cancel (see parity_util)
        z = float(np.float32(scale)) * widen(x)
        if additive is not None:
            z = z + widen(additive)[np.arange(rows) % additive.shape[0], :cols]
        with np.errstate(invalid="ignore"):
            m = np.abs(z) + np.abs(z - ref)
        mag = CANCEL_16BIT * np.where(np.isfinite(m), m, 0.0)
    ran = []
    for v in variants:
        xd = to_torch(x, dtype)
        mask = akg.make_mask(xd, additive=to_torch(additive, dtype) if additive is not None else None,
                             causal=causal_period > 0, causal_period=max(causal_period, 1))
        out = forced(v, lambda: binding.softmax_scaled(xd, scale, mask=mask, log=log))
        if out is None:
            continue
        torch.cuda.synchronize()
        got = to_numpy(out)
        compare(got, ref, dtype, f"{what} scale {scale} log {log} [{v}:{akg.last_kernel()}]", mag)
        assert verifier_passes(got, ref, dtype)
        if not log:
            assert_positive_zero(got, ref == 0, what)
        ran.append(v)
    assert "auto" in ran
    return ran


def make_x(dtype, rows, cols, seed, spread=4.0):
    x = (np.random.default_rng(seed).normal(0, 1, (rows, cols)) * spread).astype(np.float32)
    return x if dtype == wl.F32 else wl.f32_to_bf16_bits(x)


@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16])
@pytest.mark.parametrize("log", [False, True])
def test_scaled_softmax_shapes_and_families(dtype, log):
    families = set()
    for i, (rows, cols) in enumerate([(64, 1024), (33, 4096), (7, 1000), (3, 129), (5, 40000), (2, 8192), (9, 2560)]):
        x = make_x(dtype, rows, cols, seed=600 + i)
        for scale in SCALES[:2] if cols > 8192 else SCALES:
            families.update(check_all(x, dtype, scale, log, what=f"{rows}x{cols}"))
    assert {"auto", "stream", "reg", "split"} <= families


@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16])
def test_scaled_softmax_with_masks(dtype):
    rng = np.random.default_rng(17)
    for rows, cols, period in [(40, 1024, 16), (130, 4096, 128), (6, 33000, 4), (11, 200, 8)]:
        x = make_x(dtype, rows, cols, seed=rows + cols)
        a = rng.normal(0, 2, (3, cols)).astype(np.float32)
        a[1, ::7] = -np.inf
        a[2, :] = -np.inf                                   # every third row fully masked
        if dtype == wl.BF16:
            a = wl.f32_to_bf16_bits(a)
        for log in (False, True):
            check_all(x, dtype, 0.08838834764831845, log, causal_period=period, what=f"causal {rows}x{cols}")
            check_all(x, dtype, 2.5, log, additive=a, what=f"additive {rows}x{cols}")
            check_all(x, dtype, 0.5, log, additive=a, causal_period=period, what=f"both {rows}x{cols}")


def test_scale_one_is_bit_identical_and_errors():
    for dtype in (wl.F32, wl.BF16):
        x = make_x(dtype, 50, 4096, seed=3)
        xd = to_torch(x, dtype)
        mask = akg.make_mask(xd, causal=True, causal_period=32)
        for log in (False, True):
            plain = (akg.log_softmax if log else akg.softmax)(xd, mask=mask)
            scaled = binding.softmax_scaled(xd, 1.0, mask=mask, log=log)
            bits = torch.int32 if dtype == wl.F32 else torch.int16
            assert torch.equal(plain.view(bits), scaled.view(bits))
    xd = torch.zeros((2, 8), device="cuda")
    for bad in (0.0, -1.0, float("inf"), float("nan")):
        with pytest.raises(akg.AkgError):
            binding.softmax_scaled(xd, bad)
    torch.cuda.synchronize()
