"""Parity at the benchmark's full sizes, in the launch configuration bench.py times
(automatic kernel choice, contiguous inputs): EVERY row of every configuration is
compared with the fp64 oracle element by element at the strict tolerance (1e-5 absolute
for fp32, 2 bf16 ulps; no cancellation slack), the oracle streamed over blocks of rows
so that its fp64 output never has to exist at once.  Properties that hold at any size
are checked on top (torch is used here only to read the results back and to sum them)."""
import numpy as np
import pytest
import torch

import paper_2512_23424_b200 as akg
from paper_2512_23424_b200 import workloads as wl
from parity_util import assert_positive_zero, compare, run_gpu, run_oracle, to_numpy, widen

pytestmark = pytest.mark.gpu


def compare_all_rows(w, out, block_elems=1 << 24):
    """Every row against the oracle, in blocks of about `block_elems` elements; returns the
    worst figures over the blocks."""
    block = max(1, block_elems // w.cols)
    worst = {"max_abs": 0.0, "max_ulp": 0.0, "n": 0}
    for r0 in range(0, w.rows, block):
        rows = np.arange(r0, min(w.rows, r0 + block))
        ref = run_oracle(w, rows=rows)                               # global row numbers: the causal rule sees them
        got = to_numpy(out[r0:r0 + len(rows)])
        st = compare(got, ref, w.dtype, f"{w.name} rows {r0}..{r0 + len(rows) - 1}")
        worst["max_abs"] = max(worst["max_abs"], st["max_abs"])
        worst["max_ulp"] = max(worst["max_ulp"], st.get("max_ulp", 0.0))
        worst["n"] += st["n"]
    return worst


def test_config1_full():
    w = wl.make_config(1)
    out = run_gpu(w)
    ref = run_oracle(w)
    compare(to_numpy(out), ref, w.dtype, w.name)


def test_config2_layernorm_full():
    w = wl.make_config(2)
    out = run_gpu(w)
    assert "reg<f32" in akg.last_kernel()
    ref = run_oracle(w)                                           # all 4096 rows, no slack
    stats = compare(to_numpy(out), ref, w.dtype, w.name)
    assert stats["max_abs"] < 5e-6


def test_config3_rmsnorm_full():
    w = wl.make_config(3)
    out = run_gpu(w)
    assert "packed>" in akg.last_kernel()
    stats = compare_all_rows(w, out)
    assert stats["n"] == w.rows * w.cols
    # every row: mean((y / w)^2) = ms / (ms + eps), up to the bf16 rounding of y
    wgt = torch.from_numpy(wl.bf16_bits_to_f32(w.gamma)).cuda().double()
    for r0 in range(0, w.rows, 2048):
        y = out[r0:r0 + 2048].double()
        ms = ((y / wgt) ** 2).mean(dim=1)
        assert torch.all((ms - 1).abs() < 2e-3), "row mean square off"


def test_config4_log_softmax_full():
    w = wl.make_config(4)
    out = run_gpu(w)
    assert "split<f32" in akg.last_kernel()
    stats = compare_all_rows(w, out)
    assert stats["n"] == w.rows * w.cols and stats["max_abs"] < 5e-6
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
    stats = compare_all_rows(w, out)                               # all 131072 rows
    assert stats["n"] == w.rows * w.cols
    rows = np.array([0, 1, 4095, 4096, 4097, 8191, 65536, 131071 - 4096, 131071])
    got = to_numpy(out[torch.from_numpy(rows).cuda()])
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
