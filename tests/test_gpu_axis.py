"""GPU parity of akg_rowop_axis (operators over a non-last axis, the layout of the paper's
RMSNorm sketch) against the fp64 oracle, element by element."""
import numpy as np
import pytest
import torch

import oracle
import paper_2512_23424_b200 as akg
from paper_2512_23424_b200 import binding
from paper_2512_23424_b200 import workloads as wl
from parity_util import cancel_magnitude, compare, to_numpy, to_torch, verifier_passes

pytestmark = pytest.mark.gpu
OPS = ["softmax", "log_softmax", "layernorm", "rmsnorm"]


def make(op, dtype, outer, red, inner, seed):
    rng = np.random.default_rng(seed)
    x = rng.normal(0.7, 1.5, size=(outer, red, inner)).astype(np.float32)
    gamma = rng.uniform(0.5, 1.5, red).astype(np.float32) if op in ("layernorm", "rmsnorm") else None
    beta = rng.normal(0, 0.1, red).astype(np.float32) if op == "layernorm" else None
    if dtype == wl.BF16:
        x = wl.f32_to_bf16_bits(x)
        gamma = None if gamma is None else wl.f32_to_bf16_bits(gamma)
        beta = None if beta is None else wl.f32_to_bf16_bits(beta)
    return x, gamma, beta


def as_lines(a):
    """[outer, reduce, inner] -> [outer * inner, reduce]: one row per reduced line."""
    return np.ascontiguousarray(a.transpose(0, 2, 1)).reshape(-1, a.shape[1])


def check(op, dtype, x, gamma, beta, got, eps, what):
    ref = oracle.rowop_axis(op, x, gamma, beta, eps=float(np.float32(eps)), nthreads=8)
    w = wl.Workload(what, op, dtype, x.shape[0] * x.shape[2], x.shape[1], as_lines(x), eps=eps, gamma=gamma, beta=beta)
    ref2, got2 = as_lines(ref), as_lines(got)
    compare(got2, ref2, dtype, what, cancel_magnitude(w, ref2))
    assert verifier_passes(got2, ref2, dtype)


@pytest.mark.parametrize("op", OPS)
@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16])
def test_axis_shapes(op, dtype):
    eps = 1e-5
    shapes = [(1, 2, 2), (2, 7, 5), (3, 33, 128), (2, 64, 1000), (1, 257, 260), (4, 16, 4096), (2, 300, 36),
              (1, 1, 64), (5, 1000, 8), (2, 8, 1028)]
    for i, (outer, red, inner) in enumerate(shapes):
        x, g, b = make(op, dtype, outer, red, inner, seed=50 + i)
        out = binding.rowop_axis(op, to_torch(x.reshape(outer * red, inner), dtype).view(outer, red, inner),
                                 gamma=to_torch(g, dtype), beta=to_torch(b, dtype), eps=eps)
        torch.cuda.synchronize()
        got = to_numpy(out.view(outer * red, inner)).reshape(outer, red, inner)
        check(op, dtype, x, g, b, got, eps, f"axis {op} {outer}x{red}x{inner} [{akg.last_kernel()}]")


# LayerNorm lines whose mean lies thirty standard deviations from zero.  The mean has to come out within an ulp
# or so: partial means merged as "first partial + weighted mean of the differences from it", the thread's own
# mean as "first row + mean of the differences".  (Summing the values, or count x partial mean, rounds at the
# magnitude count x |mean|, and a rounded 1 / count biases the quotient: 2e-5 on fp32 results before.)  Only
# the element-wise bound is asserted: the relative criterion of Eq. 2-3 has no meaning for the results next
# to zero of such lines.
@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16])
def test_axis_layernorm_mean_far_from_zero(dtype):
    eps = 1e-5
    kernels = set()
    for i, (outer, red, inner) in enumerate([(3, 16, 1024), (2, 1000, 1024), (2, 257, 8), (1, 1000, 8), (4, 512, 8),
                                             (2, 64, 4096), (2, 100, 264)]):
        rng = np.random.default_rng(700 + i)
        x = rng.normal(-3.0, 0.1, size=(outer, red, inner)).astype(np.float32)
        g = rng.uniform(0.5, 1.5, red).astype(np.float32)
        b = rng.normal(0, 0.1, red).astype(np.float32)
        if dtype == wl.BF16:
            x, g, b = wl.f32_to_bf16_bits(x), wl.f32_to_bf16_bits(g), wl.f32_to_bf16_bits(b)
        out = binding.rowop_axis("layernorm", to_torch(x.reshape(outer * red, inner), dtype).view(outer, red, inner),
                                 gamma=to_torch(g, dtype), beta=to_torch(b, dtype), eps=eps)
        torch.cuda.synchronize()
        kernels.add(akg.last_kernel().split("<")[0])
        got = to_numpy(out.view(outer * red, inner)).reshape(outer, red, inner)
        ref = oracle.rowop_axis("layernorm", x, g, b, eps=float(np.float32(eps)), nthreads=8)
        what = f"axis layernorm {outer}x{red}x{inner} [{akg.last_kernel()}]"
        w = wl.Workload(what, "layernorm", dtype, outer * inner, red, as_lines(x), eps=eps, gamma=g, beta=b)
        compare(as_lines(got), as_lines(ref), dtype, what, cancel_magnitude(w, as_lines(ref)))
    assert kernels == {"axis", "axis_reg"}


@pytest.mark.parametrize("op", ["softmax", "rmsnorm"])
@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16])
def test_axis_strides_in_place_and_padding(op, dtype):
    outer, red, inner, eps = 3, 40, 264, 1e-6
    x, g, b = make(op, dtype, outer, red, inner, seed=7)
    tdt = torch.float32 if dtype == wl.F32 else torch.bfloat16
    bits = torch.int16 if dtype == wl.BF16 else torch.int32
    xd = to_torch(x.reshape(outer * red, inner), dtype).view(outer, red, inner)
    for pad_inner, pad_red in [(8, 2), (1, 0), (0, 1), (3, 5)]:
        big = torch.full((outer, red + pad_red, inner + pad_inner), 5.0, dtype=tdt, device="cuda")
        view = big[:, :red, :inner]
        view.copy_(xd)
        binding.rowop_axis(op, view, out=view, gamma=to_torch(g, dtype), eps=eps)        # in place, strided
        torch.cuda.synchronize()
        got = to_numpy(view.contiguous().view(outer * red, inner)).reshape(outer, red, inner)
        check(op, dtype, x, g, None, got, eps, f"axis in place, padding {pad_inner},{pad_red}")
        outside = torch.ones(big.shape, dtype=torch.bool, device="cuda")
        outside[:, :red, :inner] = False
        assert torch.equal(big[outside].view(bits), torch.full_like(big[outside], 5.0).view(bits))
    # base pointer off by one element (breaks 16-byte alignment)
    flat = torch.full((outer * red * inner + 8,), 5.0, dtype=tdt, device="cuda")
    view = flat[1:1 + outer * red * inner].view(outer, red, inner)
    view.copy_(xd)
    out = torch.empty_like(flat)[1:1 + outer * red * inner].view(outer, red, inner)
    binding.rowop_axis(op, view, out=out, gamma=to_torch(g, dtype), eps=eps)
    torch.cuda.synchronize()
    assert "scalar" in akg.last_kernel()
    got = to_numpy(out.contiguous().view(outer * red, inner)).reshape(outer, red, inner)
    check(op, dtype, x, g, None, got, eps, "axis misaligned base")


@pytest.mark.parametrize("op", OPS)
@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16])
def test_axis_every_kernel_shape(op, dtype):
    """Each lane layout (16-byte vectors, widened 8-byte bf16 vectors, elements), each rows-per-
    thread count, several column blocks per CTA, and the two-pass kernel, on ragged shapes."""
    eps = 1e-5
    shapes = [(2, 64, 512), (3, 37, 264), (2, 5, 1032), (1, 128, 96), (2, 19, 4100)]
    settings = [dict(axis_mode=m, axis_r=r, axis_nc=nc)
                for m in (1, 2, 3) for r, nc in ((8, 0), (4, 2), (2, 3), (0, 1))] + [dict(axis_r=-1)]
    try:
        for i, (outer, red, inner) in enumerate(shapes):
            x, g, b = make(op, dtype, outer, red, inner, seed=90 + i)
            xd = to_torch(x.reshape(outer * red, inner), dtype).view(outer, red, inner)
            seen = set()
            for st in settings:
                for k in ("axis_mode", "axis_r", "axis_nc"):
                    akg.set_tuning(k, st.get(k, 0))
                out = binding.rowop_axis(op, xd, gamma=to_torch(g, dtype), beta=to_torch(b, dtype), eps=eps)
                torch.cuda.synchronize()
                name = akg.last_kernel()
                if name in seen:
                    continue
                seen.add(name)
                got = to_numpy(out.view(outer * red, inner)).reshape(outer, red, inner)
                check(op, dtype, x, g, b, got, eps, f"axis {op} {outer}x{red}x{inner} [{name}]")
            assert len(seen) >= 2
    finally:
        for k in ("axis_mode", "axis_r", "axis_nc"):
            akg.set_tuning(k, 0)


def test_axis_sketch_workload_and_special_columns():
    # the sketch's shape class: X[B, F, D1, D2] fp32, reduced over F
    B, F, D1, D2 = 4, 96, 16, 64
    x, _, _ = make("rmsnorm", wl.F32, B, F, D1 * D2, seed=3)
    out = binding.rowop_axis("rmsnorm", to_torch(x.reshape(B * F, D1 * D2), wl.F32).view(B, F, D1 * D2), eps=1e-6)
    check("rmsnorm", wl.F32, x, None, None, to_numpy(out.view(B * F, -1)).reshape(B, F, -1), 1e-6, "sketch")
    # columns that are all -inf, hold a NaN, or a +inf maximum
    xs = np.random.default_rng(1).normal(size=(1, 9, 8)).astype(np.float32)
    xs[0, :, 1] = -np.inf
    xs[0, 4, 2] = np.nan
    xs[0, 5, 3] = np.inf
    for op in ("softmax", "log_softmax"):
        out = binding.rowop_axis(op, to_torch(xs.reshape(9, 8), wl.F32).view(1, 9, 8))
        got = to_numpy(out.view(9, 8)).reshape(1, 9, 8)
        check(op, wl.F32, xs, None, None, got, 0.0, f"axis special {op}")
        if op == "softmax":
            assert (got[0, :, 1].view(np.uint32) == 0).all()


@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16])
def test_axis_softmax_large_magnitudes(dtype):
    """Logits of magnitude 1e3..1e4: the rounding of max * log2(e) must not reach the output."""
    rng = np.random.default_rng(11)
    for scale, shape in ((3.0e3, (2, 64, 512)), (2.0e4, (1, 24, 264)), (5.0e2, (2, 7, 40))):
        x = (rng.normal(0.0, 1.0, size=shape) * scale + rng.normal(0.0, 2.0, size=shape)).astype(np.float32)
        x[0, : shape[1] // 2, 3] = x[0, 0, 3]                      # ties at the maximum
        if dtype == wl.BF16:
            x = wl.f32_to_bf16_bits(x)
        # (log-softmax is left out: its outputs are of the inputs' magnitude, where fp32 values
        # are spaced 1e-3 apart and no kernel can meet an absolute 1e-5)
        out = binding.rowop_axis("softmax", to_torch(x.reshape(-1, shape[2]), dtype).view(*shape))
        torch.cuda.synchronize()
        got = to_numpy(out.view(-1, shape[2])).reshape(shape)
        check("softmax", dtype, x, None, None, got, 0.0, f"axis softmax scale {scale} [{akg.last_kernel()}]")


def test_axis_argument_errors():
    L = akg.lib()
    x = torch.zeros((2, 4, 8), device="cuda")
    y = torch.empty_like(x)
    binding.rowop_axis("softmax", x, out=y)                     # sets the ctypes signature
    args = lambda **k: (k.get("op", 0), x.data_ptr(), y.data_ptr(), 2, 4, 8, k.get("xso", 32), k.get("xsf", 8), 32, 8,
                        k.get("dtype", 0), None, None, k.get("eps", 0.0), None)
    assert L.akg_rowop_axis(*args()) == 0
    assert L.akg_rowop_axis(*args(op=5)) == 1
    assert L.akg_rowop_axis(*args(dtype=3)) == 1
    assert L.akg_rowop_axis(*args(xsf=7)) == 1
    assert L.akg_rowop_axis(*args(xso=31)) == 1
    assert L.akg_rowop_axis(*args(op=3, eps=-1.0)) == 1
    assert L.akg_rowop_axis(0, x.data_ptr(), x.data_ptr() + 64, 2, 4, 8, 32, 8, 32, 8, 0, None, None, 0.0, None) == 1
    assert L.akg_rowop_axis(0, None, None, 0, 4, 8, 32, 8, 32, 8, 0, None, None, 0.0, None) == 0
    torch.cuda.synchronize()
