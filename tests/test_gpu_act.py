"""GPU parity of akg_act_mul (SiLU-and-Mul / GELU-and-Mul) against the fp64 oracle, element by
element, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
import paper_2512_23424_b200 as akg
from paper_2512_23424_b200 import binding
from paper_2512_23424_b200 import workloads as wl
from parity_util import compare, to_numpy, to_torch, verifier_passes

pytestmark = pytest.mark.gpu
ACTS = ["silu", "gelu", "gelu_tanh"]
DTYPES = [wl.F32, wl.BF16]


def make(dtype, rows, d, seed, scale=1.5):
    x = (np.random.default_rng(seed).normal(0.0, 1.0, (rows, 2 * d)) * scale).astype(np.float32)
    return x if dtype == wl.F32 else wl.f32_to_bf16_bits(x)


def check(act, dtype, x, got, what):
    ref = oracle.act_mul(act, x, nthreads=8)
    # the kernels flush a sigmoid / distribution value below 2^-126 to zero before the two
    # multiplications, so a product below 2^-126 * |gate * factor| (< 2^-110 for any input these
    # tests draw) may come back as zero; everything else is held to the usual tolerance
    compare(got, ref, dtype, what, tiny=2.0 ** -110)
    assert verifier_passes(got, ref, dtype)


@pytest.mark.parametrize("act", ACTS)
@pytest.mark.parametrize("dtype", DTYPES)
def test_act_mul_shapes(act, dtype):
    kernels = set()
    for i, (rows, d) in enumerate([(1, 1), (3, 7), (5, 128), (2, 1000), (4, 4096), (3, 11008), (2, 14336), (70000, 8),
                                   (1, 40960), (9, 264), (2, 6)]):
        x = make(dtype, rows, d, seed=400 + i)
        y = binding.act_mul(act, to_torch(x, dtype))
        torch.cuda.synchronize()
        kernels.add("vec" if ",vec," in akg.last_kernel() else "scalar")
        check(act, dtype, x, to_numpy(y), f"{act}_and_mul {rows}x{d} [{akg.last_kernel()}]")
    assert kernels == {"vec", "scalar"}


@pytest.mark.parametrize("act", ACTS)
@pytest.mark.parametrize("dtype", DTYPES)
def test_act_mul_strides_in_place_and_tails(act, dtype):
    rows, d = 6, 520
    x = make(dtype, rows, d, seed=9)
    tdt = torch.float32 if dtype == wl.F32 else torch.bfloat16
    # padded rows on both sides
    bigx = torch.full((rows, 2 * d + 16), 3.0, dtype=tdt, device="cuda")
    bigx[:, :2 * d].copy_(to_torch(x, dtype))
    bigy = torch.full((rows, d + 8), -7.0, dtype=tdt, device="cuda")
    binding.act_mul(act, bigx[:, :2 * d], out=bigy[:, :d])
    torch.cuda.synchronize()
    check(act, dtype, x, to_numpy(bigy[:, :d].contiguous()), f"{act} strided")
    assert torch.all(bigy[:, d:] == -7.0) and torch.all(bigx[:, 2 * d:] == 3.0)
    # in place: the result replaces the gate half, the factor half is untouched
    xt = to_torch(x, dtype).clone()
    keep = xt[:, d:].clone()
    binding.act_mul(act, xt, out=xt[:, :d])
    torch.cuda.synchronize()
    check(act, dtype, x, to_numpy(xt[:, :d].contiguous()), f"{act} in place")
    assert torch.equal(xt[:, d:], keep)
    # odd stride and misaligned base take the scalar kernel
    flat = torch.zeros(rows * (2 * d + 1) + 3, dtype=tdt, device="cuda")
    v = flat[1:1 + rows * (2 * d + 1)].view(rows, 2 * d + 1)[:, :2 * d]
    v.copy_(to_torch(x, dtype))
    y = binding.act_mul(act, v)
    torch.cuda.synchronize()
    assert ",scalar," in akg.last_kernel()
    check(act, dtype, x, to_numpy(y), f"{act} misaligned")
    # a clipped grid walks the rest in its loops
    try:
        akg.set_tuning("grid_cap", 1)
        xl = make(dtype, 3, 9000, seed=10)
        y = binding.act_mul(act, to_torch(xl, dtype))
        torch.cuda.synchronize()
        check(act, dtype, xl, to_numpy(y), f"{act} clipped grid")
    finally:
        akg.set_tuning("grid_cap", 0)


def test_act_mul_special_values_and_errors():
    x = np.array([[0.0, -0.0, 30.0, -30.0, 100.0, -100.0, np.inf, np.nan, 1.0, 2.0, 3.0, 4.0, 5.0, 6.0, 7.0, 8.0]],
                 dtype=np.float32)
    for act in ACTS:
        y = to_numpy(binding.act_mul(act, to_torch(x, wl.F32)))
        ref = oracle.act_mul(act, x)
        assert np.isnan(y[0, 7]) and np.isnan(ref[0, 7])
        fin = np.isfinite(ref[0])
        assert np.allclose(y[0][fin], ref[0][fin], rtol=2e-6, atol=1e-30)
        assert y[0, 6] == np.inf and ref[0, 6] == np.inf
    L = akg.lib()
    xt = torch.zeros((4, 64), device="cuda")
    yt = torch.empty((4, 32), device="cuda")
    binding.act_mul("silu", xt, out=yt)
    P = lambda t: t.data_ptr()
    call = lambda act=0, xp=P(xt), yp=P(yt), rows=4, d=32, xs=64, ys=32, dt=0: L.akg_act_mul(act, xp, yp, rows, d, xs, ys, dt, None)
    assert call() == 0
    assert call(act=3) == 1 and call(dt=5) == 1 and call(rows=-1) == 1 and call(d=-2) == 1
    assert call(xs=63) == 1 and call(ys=31) == 1
    assert call(xp=None) == 1 and call(yp=None) == 1
    assert call(yp=P(xt) + 4) == 1                      # overlaps x without being x
    assert call(yp=P(xt), ys=64) == 0 and call(yp=P(xt), ys=32) == 1
    assert call(rows=0) == 0 and call(d=0, xs=0, ys=0) == 0
    torch.cuda.synchronize()
