"""Parity at the benchmark's full sizes, in the launch configuration bench.py times
(automatic kernel choice, contiguous inputs): sampled rows are compared with the fp64
oracle element by element, and properties that hold at any size are checked on every
row (torch is used here only to read the results back and to sum them)."""
import numpy as np
import pytest
import torch

import paper_2512_23424_b200 as akg
from paper_2512_23424_b200 import workloads as wl
from parity_util import assert_positive_zero, cancel_magnitude, compare, run_gpu, run_oracle, to_numpy, widen

pytestmark = pytest.mark.gpu


def sample_rows(rows, n, extra=()):
    rng = np.random.default_rng(rows)
    picks = set(int(r) for r in rng.choice(rows, size=min(n, rows), replace=False))
    picks.update(r for r in (0, 1, rows - 1, *extra) if 0 <= r < rows)
    return np.array(sorted(picks))


def compare_sample(w, out, rows):
    ref = run_oracle(w, rows=rows)
    sub = wl.Workload(w.name, w.op, w.dtype, len(rows), w.cols, w.x[rows], eps=w.eps, gamma=w.gamma, beta=w.beta)
    got = to_numpy(out[torch.from_numpy(rows).cuda()])
    return compare(got, ref, w.dtype, f"{w.name} (sampled rows)", cancel_magnitude(sub, ref)), ref, got


def test_config1_full():
    w = wl.make_config(1)
    out = run_gpu(w)
    ref = run_oracle(w)
    compare(to_numpy(out), ref, w.dtype, w.name)


def test_config2_layernorm_full():
    w = wl.make_config(2)
    out = run_gpu(w)
    assert "reg<f32" in akg.last_kernel()
    ref = run_oracle(w)                                           # all 4096 rows
    stats = compare(to_numpy(out), ref, w.dtype, w.name, cancel_magnitude(w, ref))
    assert stats["max_abs"] < 5e-6


def test_config3_rmsnorm_full():
    w = wl.make_config(3)
    out = run_gpu(w)
    assert "ring<bf16" in akg.last_kernel()
    compare_sample(w, out, sample_rows(w.rows, 384))
    # every row: mean((y / w)^2) = ms / (ms + eps), up to the bf16 rounding of y
    wgt = torch.from_numpy(wl.bf16_bits_to_f32(w.gamma)).cuda().double()
    for r0 in range(0, w.rows, 2048):
        y = out[r0:r0 + 2048].double()
        ms = ((y / wgt) ** 2).mean(dim=1)
        assert torch.all((ms - 1).abs() < 2e-3), "row mean square off"


def test_config4_log_softmax_full():
    w = wl.make_config(4)
    out = run_gpu(w)
    assert "split<f32" in akg.last_kernel() or "cluster<f32" in akg.last_kernel()
    stats, ref, _ = compare_sample(w, out, sample_rows(w.rows, 24))
    # every row: the exponentials of a log-softmax row sum to one; the outliers sit at -ln(S)
    s = torch.exp(out.double()).sum(dim=1)
    assert torch.all((s - 1).abs() < 1e-5)
    lse = np.array([np.log(np.exp(widen(w.x[r]) - 30.0).sum()) + 30.0 for r in (0, 100, 255)])
    got_top = to_numpy(out[torch.tensor([0, 100, 255]).cuda()]).max(axis=1)
    np.testing.assert_allclose(got_top, 30.0 - lse, atol=1e-5)


def test_config5_causal_softmax_full():
    w = wl.make_config(5)
    x = torch.from_numpy(w.x.view(np.int16)).cuda().view(torch.bfloat16)
    out = torch.full_like(x, float("nan"))
    mask = akg.make_mask(x, causal=True, causal_period=4096)
    akg.softmax(x, out=out, mask=mask)
    torch.cuda.synchronize()
    assert "reg<bf16" in akg.last_kernel()
    rows = sample_rows(w.rows, 512, extra=(4095, 4096, 4097, 8191, 65536, 131071 - 4096))
    ref = run_oracle(w, rows=rows)
    got = to_numpy(out[torch.from_numpy(rows).cuda()])
    compare(got, ref, w.dtype, "config 5 (sampled rows)")
    dead = np.arange(w.cols)[None, :] > (rows[:, None] % 4096)
    assert_positive_zero(got, dead, "config 5")
    # every row: masked tail is +0 bit for bit, the live prefix sums to one (bf16 rounding aside)
    col = torch.arange(w.cols, device="cuda")[None, :]
    for r0 in range(0, w.rows, 8192):
        blk = out[r0:r0 + 8192]
        live = (torch.arange(r0, r0 + blk.shape[0], device="cuda") % 4096)[:, None]
        bits = blk.view(torch.int16)
        assert torch.all(bits[col > live] == 0)
        sums = blk.float().sum(dim=1)
        assert torch.all((sums - 1).abs() < 2e-2)
    # masked inputs are never read: poisoning them with NaN leaves the result unchanged
    for r0 in range(0, w.rows, 8192):
        live = (torch.arange(r0, r0 + 8192, device="cuda") % 4096)[:, None]
        x[r0:r0 + 8192][col > live] = float("nan")
    out2 = torch.full_like(x, float("nan"))
    akg.softmax(x, out=out2, mask=mask)
    torch.cuda.synchronize()
    assert torch.equal(out.view(torch.int16), out2.view(torch.int16))
    assert akg.device_status() == 0
