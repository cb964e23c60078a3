"""The device-side failure path: a bounded wait that runs out.

Every wait of a kernel on a bulk copy (and on its cluster's partial statistics) is bounded by the
global timer.  This test makes such a wait run out in the one safe way: a test-only setting stops
the ring kernel from issuing any bulk copy at all, so nothing is ever in flight towards a CTA,
and another shortens the limit from two seconds to 200 microseconds.  No fault, no trap, no
out-of-bounds access and no endless loop is involved; the kernel returns by itself.

Expected: the status word is set (akg_device_status reports AKG_ERR_DEVICE_TIMEOUT once, then is
clean again), the output still holds its sentinel (a CTA whose wait ran out stores nothing), and
the next ordinary call on the same context is correct.
"""
import ctypes

import numpy as np
import pytest
import torch

import paper_2512_23424_b200 as akg
from paper_2512_23424_b200 import binding
from paper_2512_23424_b200 import workloads as wl
from parity_util import compare, run_gpu, run_oracle, to_numpy, to_torch

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _reset():
    yield
    akg.set_tuning("test_no_copies", 0)
    akg.set_tuning("test_wait_us", 0)
    akg.set_variant("auto")
    akg.set_tuning("tma_mode", 0)


def status_once():
    word = ctypes.c_int(-1)
    st = akg.lib().akg_device_status(ctypes.byref(word))
    return st, word.value


@pytest.mark.parametrize("case", ["ring_norm", "ring_softmax", "smem_resident"])
def test_wait_runs_out_and_the_context_stays_usable(case):
    if case == "ring_norm":                      # forced: the ring-fed normalisation kernel
        w = wl.make_random("rmsnorm", wl.BF16, 2304, 4096, seed=71)
        prepare, family = (lambda: akg.set_variant("tma")), "ring<bf16"
    elif case == "ring_softmax":                 # forced: the ring-fed softmax kernel
        w = wl.make_random("softmax", wl.BF16, 600, 2048, seed=72)
        prepare, family = (lambda: akg.set_variant("tma")), "ring<bf16"
    else:                                        # forced: row resident in shared memory, two sweeps
        w = wl.make_random("layernorm", wl.F32, 300, 8192, seed=73, eps=1e-5)
        prepare, family = (lambda: (akg.set_variant("tma"), akg.set_tuning("tma_mode", 2))), "tma<f32"
    torch.cuda.synchronize()
    assert status_once() == (binding.OK, 0)
    x = to_torch(w.x, w.dtype)
    sentinel = torch.full_like(x, float("nan"))
    out = sentinel.clone()

    prepare()
    akg.set_tuning("test_no_copies", 1)
    akg.set_tuning("test_wait_us", 200)
    run_gpu(w, x_dev=x, out=out)
    torch.cuda.synchronize()                     # the kernel ends by itself
    assert family in akg.last_kernel(), akg.last_kernel()
    st, word = status_once()
    assert st == binding.ERR_DEVICE_TIMEOUT and word != 0
    assert status_once() == (binding.OK, 0)      # reported once, then clean
    bits = torch.int16 if w.dtype != wl.F32 else torch.int32
    assert torch.equal(out.view(bits), sentinel.view(bits)), "a CTA whose wait ran out stored something"

    # the same call with the copies back on, on the same context, is correct
    akg.set_tuning("test_no_copies", 0)
    akg.set_tuning("test_wait_us", 0)
    run_gpu(w, x_dev=x, out=out)
    torch.cuda.synchronize()
    assert family in akg.last_kernel()
    compare(to_numpy(out), run_oracle(w), w.dtype, f"{w.name} after a timeout")
    assert status_once() == (binding.OK, 0)
