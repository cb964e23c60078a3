"""GPU parity of akg_add_norm (fused residual add + LayerNorm / RMSNorm) against the fp64 oracle,
element by element, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
import paper_2512_23424_b200 as akg
from paper_2512_23424_b200 import binding
from paper_2512_23424_b200 import workloads as wl
from parity_util import cancel_magnitude, compare, to_numpy, to_torch, verifier_passes

pytestmark = pytest.mark.gpu
OPS = ["layernorm", "rmsnorm"]
DTYPES = [wl.F32, wl.BF16]


def make(op, dtype, rows, cols, seed):
    rng = np.random.default_rng(seed)
    x = rng.normal(0.5, 1.5, (rows, cols)).astype(np.float32)
    r = rng.normal(-0.25, 2.0, (rows, cols)).astype(np.float32)
    g = rng.uniform(0.5, 1.5, cols).astype(np.float32)
    b = rng.normal(0, 0.1, cols).astype(np.float32) if op == "layernorm" else None
    if dtype == wl.BF16:
        x, r, g = wl.f32_to_bf16_bits(x), wl.f32_to_bf16_bits(r), wl.f32_to_bf16_bits(g)
        b = None if b is None else wl.f32_to_bf16_bits(b)
    return x, r, g, b


def check(op, dtype, x, r, g, b, eps, got_y, got_s, what):
    ref_y, ref_s = oracle.add_norm(op, x, r, g, b, eps=float(np.float32(eps)), nthreads=8)
    s32 = ref_s.astype(np.float32)
    w = wl.Workload(what, op, dtype, x.shape[0], x.shape[1], s32 if dtype == wl.F32 else wl.f32_to_bf16_bits(s32),
                    eps=eps, gamma=g, beta=b)
    compare(got_y, ref_y, dtype, what + " y", cancel_magnitude(w, ref_y))
    assert verifier_passes(got_y, ref_y, dtype)
    if got_s is not None:
        compare(got_s, ref_s, dtype, what + " sum")


SHAPES = [(1, 1), (4, 128), (7, 1024), (33, 4096), (5, 5120), (3, 8192), (2, 768), (9, 100), (3, 130), (6, 2560),
          (2, 32768), (2, 12288), (3, 1000)]


@pytest.mark.parametrize("op", OPS)
@pytest.mark.parametrize("dtype", DTYPES)
def test_add_norm_shapes(op, dtype):
    eps = 1e-5
    kernels = set()
    for i, (rows, cols) in enumerate(SHAPES):
        x, r, g, b = make(op, dtype, rows, cols, seed=200 + i)
        y, s = binding.add_norm(op, to_torch(x, dtype), to_torch(r, dtype), gamma=to_torch(g, dtype),
                                beta=to_torch(b, dtype), eps=eps)
        torch.cuda.synchronize()
        kernels.add(akg.last_kernel().split("<")[0])
        check(op, dtype, x, r, g, b, eps, to_numpy(y), to_numpy(s), f"add_{op} {rows}x{cols} [{akg.last_kernel()}]")
    assert kernels == {"add_flex", "add_stream"}


@pytest.mark.parametrize("op", OPS)
@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("cols", [1024, 100])
def test_add_norm_in_place_strides_and_no_sum(op, dtype, cols):
    rows, eps = 11, 1e-6
    x, r, g, b = make(op, dtype, rows, cols, seed=31)
    tdt = torch.float32 if dtype == wl.F32 else torch.bfloat16

    def padded(a, pad):
        big = torch.full((rows, cols + pad), 9.0, dtype=tdt, device="cuda")
        big[:, :cols].copy_(to_torch(a, dtype))
        return big, big[:, :cols]

    # the residual stream updated in place, y over x, all four with their own strides
    bigx, vx = padded(x, 8)
    bigr, vr = padded(r, 16)
    y, s = binding.add_norm(op, vx, vr, gamma=to_torch(g, dtype), beta=to_torch(b, dtype), eps=eps, out=vx, sum_out=vr)
    torch.cuda.synchronize()
    assert y.data_ptr() == vx.data_ptr() and s.data_ptr() == vr.data_ptr()
    check(op, dtype, x, r, g, b, eps, to_numpy(vx.contiguous()), to_numpy(vr.contiguous()), f"add_{op} in place {cols}")
    assert torch.all(bigx[:, cols:] == 9.0) and torch.all(bigr[:, cols:] == 9.0)
    # y over the residual, the sum over x
    _, vx = padded(x, 0)
    _, vr = padded(r, 24)
    binding.add_norm(op, vx, vr, gamma=to_torch(g, dtype), beta=to_torch(b, dtype), eps=eps, out=vr, sum_out=vx)
    torch.cuda.synchronize()
    check(op, dtype, x, r, g, b, eps, to_numpy(vr.contiguous()), to_numpy(vx.contiguous()), f"add_{op} crossed {cols}")
    # no sum output; residual untouched
    _, vx = padded(x, 0)
    _, vr = padded(r, 0)
    y, s = binding.add_norm(op, vx, vr, gamma=to_torch(g, dtype), beta=to_torch(b, dtype), eps=eps, sum_out=None)
    torch.cuda.synchronize()
    assert s is None
    check(op, dtype, x, r, g, b, eps, to_numpy(y), None, f"add_{op} no sum {cols}")
    assert torch.equal(vr.view(torch.int16 if dtype == wl.BF16 else torch.int32),
                       to_torch(r, dtype).view(torch.int16 if dtype == wl.BF16 else torch.int32))
    # misaligned base: the scalar kernel
    flat = torch.zeros(rows * cols + 8, dtype=tdt, device="cuda")
    vx = flat[1:1 + rows * cols].view(rows, cols)
    vx.copy_(to_torch(x, dtype))
    y, s = binding.add_norm(op, vx, to_torch(r, dtype), gamma=to_torch(g, dtype), beta=to_torch(b, dtype), eps=eps)
    torch.cuda.synchronize()
    assert akg.last_kernel().startswith("add_stream")
    check(op, dtype, x, r, g, b, eps, to_numpy(y), to_numpy(s), f"add_{op} misaligned {cols}")


def test_add_norm_without_affine_and_vpt_sweep():
    eps = 1e-5
    try:
        for dtype in DTYPES:
            x, r, _, _ = make("rmsnorm", dtype, 5, 6144, seed=77)
            for vpt in (0, 1, 2, 3, 4, 6, 8):
                akg.set_tuning("reg_vpt", vpt)
                for op in OPS:
                    y, s = binding.add_norm(op, to_torch(x, dtype), to_torch(r, dtype), eps=eps)
                    torch.cuda.synchronize()
                    check(op, dtype, x, r, None, None, eps, to_numpy(y), to_numpy(s), f"add_{op} vpt {vpt} [{akg.last_kernel()}]")
    finally:
        akg.set_tuning("reg_vpt", 0)


def test_add_norm_argument_errors():
    L = akg.lib()
    x = torch.zeros((4, 256), device="cuda")
    r, y, s = torch.zeros_like(x), torch.empty_like(x), torch.empty_like(x)
    binding.add_norm("rmsnorm", x, r, out=y, sum_out=s)                       # sets the ctypes signature
    P = lambda t: t.data_ptr()

    def call(op=3, xp=P(x), rp=P(r), yp=P(y), sp=P(s), rows=4, cols=256, xs=256, rs=256, ys=256, ss=256, dt=0, eps=1e-5):
        return L.akg_add_norm(op, xp, rp, yp, sp, rows, cols, xs, rs, ys, ss, dt, None, None, eps, None)

    assert call() == 0
    assert call(op=0) == 1 and call(op=1) == 1 and call(op=7) == 1
    assert call(rp=None) == 1
    assert call(rs=255) == 1 and call(ss=100) == 1 and call(xs=1) == 1
    assert call(dt=3) == 1 and call(eps=-1.0) == 1 and call(rows=-1) == 1
    assert call(sp=None) == 0
    assert call(sp=P(y)) == 1                                   # the two outputs overlap
    assert call(sp=P(y) + 64, rows=1) == 1
    assert call(yp=P(x) + 16) == 1                              # y partially over x
    assert call(sp=P(r) + 16) == 1                              # sum partially over the residual
    assert call(yp=P(r), ys=512, rows=1) == 0                   # one row: the stride plays no part
    assert call(yp=P(r), ys=512) == 1
    assert call(yp=P(x), sp=P(r)) == 0 and call(yp=P(r), sp=P(x)) == 0
    assert call(rows=0) == 0 and call(cols=0, xs=0, rs=0, ys=0, ss=0) == 0
    assert "overlap" in akg.last_error() or akg.last_error() == ""
    torch.cuda.synchronize()
