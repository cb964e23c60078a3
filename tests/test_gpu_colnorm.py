"""GPU parity of akg_colnorm (BatchNorm-style column normalisation) against the fp64 oracle, element
by element, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
import paper_2512_23424_b200 as akg
from paper_2512_23424_b200 import binding
from paper_2512_23424_b200 import workloads as wl
from parity_util import CANCEL_16BIT, compare, to_numpy, to_torch, widen

pytestmark = pytest.mark.gpu
DTYPES = [wl.F32, wl.BF16, wl.F16]


def store(a, dtype):
    if a is None:
        return None
    a = a.astype(np.float32)
    return a if dtype == wl.F32 else (wl.f32_to_bf16_bits(a) if dtype == wl.BF16 else a.astype(np.float16))


def check(x, g, b, dtype, eps, got_y, got_mean, got_var, what):
    ref_y, ref_mean, ref_var = oracle.colnorm(x, g, b, eps=float(np.float32(eps)), nthreads=8)
    xv = widen(x)
    rstd = 1.0 / np.sqrt(ref_var + float(np.float32(eps)))
    gam = np.ones(x.shape[1]) if g is None else np.abs(widen(g))
    # the conditioning of the operator in fp32 (as for LayerNorm): an ulp of the column's largest
    # value passes through (x - mean) * rstd * gamma; 16-bit outputs add the cancellation of + beta
    slack = 2.0 ** -23 * np.abs(xv).max(axis=0)[None, :] * (rstd * gam)[None, :] * np.ones_like(ref_y)
    if dtype != wl.F32:
        beta = np.zeros(x.shape[1]) if b is None else widen(b)
        slack = slack + CANCEL_16BIT * (np.abs(ref_y - beta[None, :]) + np.abs(beta)[None, :])
    compare(got_y, ref_y, dtype, what, slack)
    if got_mean is not None:
        scale = np.abs(xv).max(axis=0) + 1e-30
        assert np.max(np.abs(got_mean - ref_mean) / scale) < 4e-7, what
        assert np.max(np.abs(got_var - ref_var) / (ref_var + scale * scale * 1e-6 + 1e-30)) < 2e-5, what


@pytest.mark.parametrize("dtype", DTYPES)
def test_colnorm_shapes(dtype):
    rng = np.random.default_rng(31)
    kernels = set()
    for rows, cols in [(1, 1), (7, 5), (300, 64), (4096, 1024), (1000, 132), (33, 4096), (20000, 8), (257, 260), (64, 16384)]:
        x = store(rng.normal(1.0, 2.0, (rows, cols)), dtype)
        g = store(rng.uniform(0.5, 1.5, cols), dtype)
        b = store(rng.normal(0, 0.2, cols), dtype)
        y, mean, var = binding.colnorm(to_torch(x, dtype), to_torch(g, dtype), to_torch(b, dtype), eps=1e-5, want_stats=True)
        torch.cuda.synchronize()
        kernels.add(akg.last_kernel().split(",grid")[0])
        check(x, g, b, dtype, 1e-5, to_numpy(y), mean.cpu().numpy().astype(np.float64), var.cpu().numpy().astype(np.float64),
              f"colnorm {rows}x{cols} [{akg.last_kernel()}]")
    assert len(kernels) >= 3, kernels


@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16])
def test_colnorm_in_place_strides_small_workspace_and_no_affine(dtype):
    rng = np.random.default_rng(32)
    rows, cols = 1500, 264
    x = store(rng.normal(-0.5, 3.0, (rows, cols)), dtype)
    tdt = torch.float32 if dtype == wl.F32 else torch.bfloat16
    big = torch.full((rows, cols + 8), 7.0, dtype=tdt, device="cuda")
    big[:, :cols].copy_(to_torch(x, dtype))
    binding.colnorm(big[:, :cols], eps=1e-3, out=big[:, :cols])                       # in place, padded rows, no affine
    torch.cuda.synchronize()
    check(x, None, None, dtype, 1e-3, to_numpy(big[:, :cols].contiguous()), None, None, "in place")
    assert torch.all(big[:, cols:] == 7.0)
    # the smallest workspace (one row block) and a few sizes in between give the same answer
    for blocks in (1, 2, 5):
        ws = torch.empty(blocks * cols * 8, dtype=torch.uint8, device="cuda")
        y = binding.colnorm(to_torch(x, dtype), eps=1e-3, workspace=ws)
        assert int(akg.last_kernel().rsplit("x", 1)[1].rstrip(">")) <= blocks
        check(x, None, None, dtype, 1e-3, to_numpy(y), None, None, f"workspace of {blocks} blocks")
    # misaligned base: element path
    flat = torch.zeros(rows * (cols + 1) + 3, dtype=tdt, device="cuda")
    v = flat[1:1 + rows * (cols + 1)].view(rows, cols + 1)[:, :cols]
    v.copy_(to_torch(x, dtype))
    y = binding.colnorm(v, eps=1e-3)
    assert "scalar" in akg.last_kernel()
    check(x, None, None, dtype, 1e-3, to_numpy(y), None, None, "misaligned")


def test_colnorm_constant_column_and_errors():
    x = np.random.default_rng(33).normal(0, 1, (100, 8)).astype(np.float32)
    x[:, 3] = 2.5
    b = np.arange(8, dtype=np.float32)
    y = to_numpy(binding.colnorm(to_torch(x, wl.F32), beta=to_torch(b, wl.F32), eps=1e-5))
    assert np.array_equal(y[:, 3], np.full(100, 3.0, dtype=np.float32))            # a constant column returns beta
    L = akg.lib()
    xt = torch.zeros((16, 64), device="cuda")
    yt = torch.empty_like(xt)
    ws = torch.empty(binding.colnorm_workspace_bytes(16, 64), dtype=torch.uint8, device="cuda")
    P = lambda t: t.data_ptr()

    def call(xp=P(xt), yp=P(yt), rows=16, cols=64, xs=64, ys=64, dt=0, eps=1e-5, wp=P(ws), wb=ws.numel()):
        import ctypes
        return L.akg_colnorm(xp, yp, rows, cols, xs, ys, dt, None, None, ctypes.c_float(eps), None, None, wp, wb, None)

    assert call() == 0
    assert call(dt=7) == 1 and call(eps=-1.0) == 1 and call(xs=10) == 1 and call(xp=None) == 1
    assert call(wp=None) == 1 and call(wb=100) == 1 and call(wp=P(ws) + 4) == 1
    assert call(wb=64 * 8) == 0                                                       # one block fits
    assert call(yp=P(xt)) == 0 and call(yp=P(xt) + 16) == 1
    assert call(rows=0) == 0
    assert L.akg_colnorm_workspace_bytes(16, 64) == 256 * 64 * 8 and L.akg_colnorm_workspace_bytes(0, 64) == 0
    assert L.akg_colnorm_workspace_bytes(16, 1 << 20) <= 4 * (1 << 20) * 8
    torch.cuda.synchronize()
