"""GPU parity of the host-buffer entry point (akg_rowop_host) against the fp64 oracle."""
import numpy as np
import pytest
import torch

import paper_2512_23424_b200 as akg
from paper_2512_23424_b200 import binding
from paper_2512_23424_b200 import workloads as wl
from parity_util import cancel_magnitude, compare, run_oracle, to_numpy

pytestmark = pytest.mark.gpu


def host_tensor(a, dtype, pinned=True):
    if a is None:
        return None
    t = torch.from_numpy(np.ascontiguousarray(a) if dtype == wl.F32 else np.ascontiguousarray(a).view(np.int16))
    t = t if dtype == wl.F32 else t.view(torch.bfloat16)
    return t.pin_memory() if pinned else t


def run_host(w, workspace_bytes=None, pinned=True, stride_pad=0):
    tdt = torch.float32 if w.dtype == wl.F32 else torch.bfloat16
    x = host_tensor(w.x, w.dtype, pinned)
    if stride_pad:
        wide = torch.full((w.rows, w.cols + stride_pad), 7.0, dtype=tdt)
        wide[:, :w.cols] = x
        x = wide[:, :w.cols]
        out_wide = torch.full((w.rows, w.cols + stride_pad), float("nan"), dtype=tdt)
        out = out_wide[:, :w.cols]
    else:
        out = torch.full((w.rows, w.cols), float("nan"), dtype=tdt)
        out = out.pin_memory() if pinned else out
    gamma, beta = host_tensor(w.gamma, w.dtype, pinned), host_tensor(w.beta, w.dtype, pinned)
    n = workspace_bytes or binding.host_workspace_bytes(w.rows, w.cols, tdt, gamma is not None, beta is not None)
    ws = torch.empty(n, dtype=torch.uint8, device="cuda")
    binding.rowop_host(w.op, x, out, ws, gamma=gamma, beta=beta, eps=w.eps, causal_period=w.causal_period)
    torch.cuda.synchronize()
    if stride_pad:
        assert (out_wide[:, w.cols:].float() != out_wide[:, w.cols:].float()).all()   # padding untouched (NaN)
    return to_numpy(out.contiguous())


@pytest.mark.parametrize("op", ["softmax", "log_softmax", "layernorm", "rmsnorm"])
@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16])
def test_host_entry_matches_oracle(op, dtype):
    for rows, cols in [(5, 1000), (300, 4096), (2049, 1024), (70, 33)]:
        w = wl.make_random(op, dtype, rows, cols, seed=rows + cols, loc=0.4, eps=1e-5)
        ref = run_oracle(w)
        compare(run_host(w), ref, dtype, f"host {w.name}", cancel_magnitude(w, ref))
    # a workspace of three single rows forces one chunk per row; pageable memory; padded strides
    w = wl.make_random(op, dtype, 37, 512, seed=9, eps=1e-5)
    ref = run_oracle(w)
    es = 4 if dtype == wl.F32 else 2
    tiny = 3 * 512 * es + 2 * 512 * es + 1024
    compare(run_host(w, workspace_bytes=tiny), ref, dtype, "host tiny workspace", cancel_magnitude(w, ref))
    compare(run_host(w, pinned=False), ref, dtype, "host pageable", cancel_magnitude(w, ref))
    compare(run_host(w, stride_pad=8), ref, dtype, "host strided", cancel_magnitude(w, ref))


@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16])
def test_host_entry_causal_chunks_keep_global_rows(dtype):
    """The causal rule uses the global row index although rows are processed in chunks."""
    w = wl.make_random("softmax", dtype, 3000, 1024, seed=3)
    w.causal_period = 700
    ref = run_oracle(w)
    es = 4 if dtype == wl.F32 else 2
    got = run_host(w, workspace_bytes=3 * 64 * 1024 * es)         # 64-row chunks
    compare(got, ref, dtype, "host causal")
    r = np.arange(3000)[:, None] % 700
    dead = np.arange(1024)[None, :] > r
    bits = got.view(np.uint32) if dtype == wl.F32 else got
    assert (bits[dead] == 0).all()


@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16])
def test_host_entry_uploads_only_live_columns_and_ramps_its_chunks(dtype):
    """Under a causal mask the masked columns of a chunk are not uploaded (the kernels never read them):
    NaN in the masked part of the host matrix does not show, the byte counter reports the smaller upload,
    and the result is the oracle's.  Without a mask the first and last chunks are smaller than the rest;
    the counter then reports the whole matrix."""
    es = 4 if dtype == wl.F32 else 2
    rows, cols, period = 6144, 2048, 2048
    w = wl.make_random("softmax", dtype, rows, cols, seed=5)
    w.causal_period = period
    ref = run_oracle(w)
    dead = np.arange(cols)[None, :] > (np.arange(rows)[:, None] % period)
    x = w.x.copy()
    x[dead] = np.float32(np.nan) if dtype == wl.F32 else np.uint16(0x7FC0)
    wp = wl.Workload(w.name, w.op, dtype, rows, cols, x, causal_period=period)
    got = run_host(wp)
    compare(got, ref, dtype, "host causal, poisoned masked columns")
    up, down = binding.last_host_copy_bytes()
    assert down == rows * cols * es
    # chunks of a quarter period: 1/4, 2/4, 3/4, 4/4 of the columns -> 62.5 % of the matrix (chunks of at
    # least 4 MiB: 512 rows of 8 KiB for fp32, 1024 rows of 4 KiB otherwise, i.e. a quarter / a half period)
    assert up < 0.80 * rows * cols * es and up >= 0.5 * rows * cols * es, (up, rows * cols * es)
    try:
        akg.set_tuning("host_full_upload", 1)
        got2 = run_host(w)
        assert binding.last_host_copy_bytes()[0] == rows * cols * es
        assert np.array_equal(got2, got)
    finally:
        akg.set_tuning("host_full_upload", 0)
    # no mask: ramped chunks (1/8, 1/8, 1/4, 1/2, 1, ... of a chunk), every row exactly once
    wn = wl.make_random("rmsnorm", dtype, 40000, 1024, seed=6, eps=1e-6)
    gotn = run_host(wn)
    compare(gotn, run_oracle(wn), dtype, "host ramped chunks")
    assert binding.last_host_copy_bytes() == (40000 * 1024 * es + 1024 * es, 40000 * 1024 * es)


def test_host_entry_argument_errors():
    L = akg.lib()
    x = torch.zeros((4, 8)).pin_memory()
    y = torch.zeros((4, 8)).pin_memory()
    ws = torch.empty(1 << 20, dtype=torch.uint8, device="cuda")
    args = (x.data_ptr(), y.data_ptr(), 4, 8, 8, 8, 0, None, None, 0.0, None)
    assert L.akg_rowop_host(0, *args, ws.data_ptr(), 1 << 20, None) == 0
    assert L.akg_rowop_host(7, *args, ws.data_ptr(), 1 << 20, None) == 1
    assert L.akg_rowop_host(0, *args, None, 1 << 20, None) == 1
    assert L.akg_rowop_host(0, *args, ws.data_ptr(), 16, None) == 1
    assert L.akg_rowop_host(0, *args, ws.data_ptr() + 4, 1 << 19, None) == 1
    torch.cuda.synchronize()
    assert L.akg_host_workspace_bytes(0, 8, 0, 0, 0) == 0
    assert L.akg_host_workspace_bytes(4096, 4096, 0, 1, 1) >= 3 * 4096 * 4 + 2 * 4096 * 4
