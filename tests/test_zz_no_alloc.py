"""The allocation-free host entry point (akg_rowop_host_static), checked against the
existing host entry point (akg_rowop_host) through the C ABI.

Who needs it: code that gets host buffers and a stream but cannot obtain device memory of
its own - a plug-in that may not touch its host application's memory pool, a service that
must not allocate once it is running.  Such a caller cannot give akg_rowop_host the staging
workspace it asks for, so the library carries a fixed 16 MiB staging area instead.  The
area is shared by all calls and keeps the previous call's bytes, hence the test runs
different problems back to back and checks that neither sees the other's leftovers.  Every
result is also compared with the fp64 oracle at the parity tests' strict tolerance, so an
error common to both entry points cannot hide.

This file is named so that pytest collects it last.
"""
import numpy as np
import pytest
import torch

import paper_2512_23424_b200 as akg
from paper_2512_23424_b200 import binding
from paper_2512_23424_b200 import workloads as wl
from parity_util import BF16_ULPS, FP32_ATOL, bf16_ulp, compare, run_oracle, to_numpy, widen

pytestmark = pytest.mark.gpu


def host(a, dtype):
    if a is None:
        return None
    t = torch.from_numpy(np.ascontiguousarray(a) if dtype == wl.F32 else np.ascontiguousarray(a).view(np.int16))
    return (t if dtype == wl.F32 else t.view(torch.bfloat16)).pin_memory()


def run_both(w):
    """The same problem through the existing entry point (caller workspace) and the new one."""
    tdt = torch.float32 if w.dtype == wl.F32 else torch.bfloat16
    x, gamma, beta = host(w.x, w.dtype), host(w.gamma, w.dtype), host(w.beta, w.dtype)
    want = torch.full((w.rows, w.cols), float("nan"), dtype=tdt).pin_memory()
    got = torch.full((w.rows, w.cols), float("nan"), dtype=tdt).pin_memory()
    ws = torch.empty(binding.host_workspace_bytes(w.rows, w.cols, tdt, gamma is not None, beta is not None),
                     dtype=torch.uint8, device="cuda")
    binding.rowop_host(w.op, x, want, ws, gamma=gamma, beta=beta, eps=w.eps, causal_period=w.causal_period)
    binding.rowop_host_static(w.op, x, got, gamma=gamma, beta=beta, eps=w.eps, causal_period=w.causal_period)
    torch.cuda.synchronize()
    return to_numpy(want), to_numpy(got)


def assert_same(want, got, dtype, what):
    """Same tolerance as the parity tests, with the existing entry point as the reference
    (the two may cut the rows into different chunks and so pick different kernels)."""
    a, b = widen(want), widen(got)
    assert np.array_equal(np.isnan(a), np.isnan(b)), what
    assert np.array_equal(np.isinf(a), np.isinf(b)), what
    fin = np.isfinite(a)
    err = np.abs(a[fin] - b[fin])
    if dtype == wl.F32:
        assert err.max(initial=0.0) <= FP32_ATOL, f"{what}: {err.max():.3e}"
    else:
        assert (err <= BF16_ULPS * bf16_ulp(a[fin])).all(), what


def test_static_entry_matches_workspace_entry_twice_in_a_row():
    # first call: LayerNorm fp32, 40 MiB of rows -> several chunks through the 16 MiB area
    w1 = wl.make_random("layernorm", wl.F32, 2560, 4096, seed=11, loc=3.0, scale=2.0, eps=1e-5)
    want, got = run_both(w1)
    got_first = got.copy()
    assert not np.isnan(widen(got)).any()
    assert_same(want, got, w1.dtype, "first call (layernorm f32)")
    compare(got, run_oracle(w1), w1.dtype, "first call against the oracle")
    # second call, straight after: a smaller causal bf16 softmax; leftovers of call one in
    # the staging area must not show (masked entries are exactly +0, live ones match)
    w2 = wl.make_random("softmax", wl.BF16, 700, 1024, seed=12)
    w2.causal_period = 256
    want, got = run_both(w2)
    assert_same(want, got, w2.dtype, "second call (causal softmax bf16)")
    dead = np.arange(1024)[None, :] > (np.arange(700)[:, None] % 256)
    assert (got[dead] == 0).all()
    compare(got, run_oracle(w2), w2.dtype, "second call against the oracle")
    # third call: a causal softmax larger than the staging area (3000 x 4096 bf16 = 23 MiB), so the
    # rows go through it in chunks of 2048 and the second chunk starts in the middle of a causal
    # period (1500 rows, not a power of two): the rule has to see global row numbers
    w3 = wl.make_random("softmax", wl.BF16, 3000, 4096, seed=13)
    w3.causal_period = 1500
    want, got = run_both(w3)
    assert_same(want, got, w3.dtype, "third call (causal softmax bf16, chunked)")
    compare(got, run_oracle(w3), w3.dtype, "third call against the oracle")
    dead = np.arange(4096)[None, :] > (np.arange(3000)[:, None] % 1500)
    assert (got[dead] == 0).all()
    # and the first problem again gives the first answer again
    want1, got1 = run_both(w1)
    assert np.array_equal(got1.view(np.uint32), got_first.view(np.uint32))
    assert_same(want1, got1, w1.dtype, "fourth call (layernorm f32 again)")
    assert akg.device_status() == 0


def test_static_entry_rejects_rows_beyond_the_staging_area():
    L = akg.lib()
    cols = (16 << 20) // 4 + 64                        # one fp32 row larger than the area
    x = torch.zeros((1, cols)).pin_memory()
    y = torch.zeros((1, cols)).pin_memory()
    with pytest.raises(akg.AkgError) as info:
        binding.rowop_host_static("rmsnorm", x, y, eps=1e-6)
    assert info.value.status == binding.ERR_UNSUPPORTED
    assert "staging area" in str(info.value) and "akg_rowop_host" in str(info.value)
    # a row that fits alone but not together with gamma and beta is rejected as well
    cols = (16 << 20) // 4 // 2
    x = torch.zeros((1, cols)).pin_memory()
    g = torch.ones(cols).pin_memory()
    with pytest.raises(akg.AkgError):
        binding.rowop_host_static("layernorm", x, x.clone().pin_memory(), gamma=g, beta=g)
    # the same row without vectors is accepted
    out = torch.empty_like(x).pin_memory()
    binding.rowop_host_static("rmsnorm", x + 1.0, out, eps=0.0)
    torch.cuda.synchronize()
    assert torch.allclose(out, torch.ones_like(out))
    assert L.akg_rowop_host_static(9, x.data_ptr(), out.data_ptr(), 1, cols, cols, cols, 0, None, None, 0.0,
                                   None, None) == 1
