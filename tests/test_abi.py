"""The C-ABI library loads without a GPU and exports every symbol the header declares;
argument validation answers before any CUDA call."""
import ctypes
import os
import re

import numpy as np

import paper_2512_23424_b200 as akg
from paper_2512_23424_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "akg.h")


def declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(akg_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    names = declared_functions()
    assert {"akg_softmax", "akg_log_softmax", "akg_layernorm", "akg_rmsnorm", "akg_rowop_host",
            "akg_status_string", "akg_version"} <= set(names)
    L = akg.lib()
    for name in names:
        assert hasattr(L, name), f"{name} is declared in akg.h but not exported by libakg.so"


def test_header_documents_each_entry_point():
    text = open(HEADER).read()
    for name in declared_functions():
        idx = text.index(name + "(")
        before = text[:idx]
        assert before.rstrip().endswith(("*/", "akg_status", "char*", "int", "size_t")), name
        assert "*/" in before[-2500:], f"{name} has no comment block before it"


def test_status_strings_and_version():
    assert akg.status_string(0) == "AKG_OK"
    assert akg.status_string(1) == "AKG_ERR_INVALID_ARG"
    assert akg.status_string(2) == "AKG_ERR_UNSUPPORTED"
    assert akg.status_string(3) == "AKG_ERR_CUDA"
    assert akg.status_string(4) == "AKG_ERR_DEVICE_TIMEOUT"
    assert akg.lib().akg_version() >= 100


def test_argument_validation_needs_no_gpu():
    L = akg.lib()
    buf = np.zeros(256, dtype=np.float32)
    p = buf.ctypes.data
    q = p + 512
    ok_shape = (4, 8, 8, 8)
    # empty problems are fine and launch nothing
    assert L.akg_softmax(None, None, 0, 8, 8, 8, 0, None, None) == 0
    assert L.akg_rmsnorm(None, None, 4, 0, 0, 0, 1, None, 1e-6, None) == 0
    # NULL data, negative sizes, short strides, unknown dtype
    assert L.akg_softmax(None, q, *ok_shape, 0, None, None) == 1
    assert "NULL" in akg.last_error()
    assert L.akg_softmax(p, q, -1, 8, 8, 8, 0, None, None) == 1
    assert L.akg_softmax(p, q, 4, 8, 7, 8, 0, None, None) == 1
    assert L.akg_softmax(p, q, 4, 8, 8, 7, 0, None, None) == 1
    assert L.akg_log_softmax(p, q, *ok_shape, 5, None, None) == 1
    # eps must be >= 0, finite, not NaN
    assert L.akg_layernorm(p, q, *ok_shape, 0, None, None, -1e-5, None) == 1
    assert L.akg_layernorm(p, q, *ok_shape, 0, None, None, float("nan"), None) == 1
    assert L.akg_rmsnorm(p, q, *ok_shape, 0, None, float("inf"), None) == 1
    # partial overlap of x and y is rejected, identical matrices are not an argument error
    assert L.akg_softmax(p, p + 16, *ok_shape, 0, None, None) == 1
    assert "overlap" in akg.last_error()
    # malformed masks
    m = binding.Mask()
    m.causal, m.causal_period = 1, 0
    assert L.akg_softmax(p, q, *ok_shape, 0, ctypes.byref(m), None) == 1
    m.causal, m.causal_period = 2, 4
    assert L.akg_softmax(p, q, *ok_shape, 0, ctypes.byref(m), None) == 1
    m = binding.Mask()
    m.additive, m.add_rows, m.add_row_stride = p, 0, 8
    assert L.akg_softmax(p, q, *ok_shape, 0, ctypes.byref(m), None) == 1
    m.add_rows, m.add_row_stride = 1, 7
    assert L.akg_softmax(p, q, *ok_shape, 0, ctypes.byref(m), None) == 1
    # knobs
    assert L.akg_set_variant(9) == 1
    assert L.akg_set_variant(0) == 0
    assert L.akg_set_tuning(b"no_such_key", 1) == 1
    assert L.akg_set_tuning(None, 1) == 1
    assert L.akg_set_tuning(b"grid_cap", 0) == 0
    # host entry point
    assert L.akg_rowop_host(9, p, q, *ok_shape, 0, None, None, 0.0, None, p, 4096, None) == 1
    assert L.akg_rowop_host(0, p, q, *ok_shape, 0, None, None, 0.0, None, None, 4096, None) == 1
    assert L.akg_host_workspace_bytes(-1, 8, 0, 0, 0) == 0
    assert L.akg_host_workspace_bytes(16, 8, 0, 1, 1) > 0
