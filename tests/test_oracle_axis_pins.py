"""Pins for the oracle's non-last-axis driver (no GPU): x is [outer, reduce, inner] and the
operator runs over `reduce` for every (outer, inner) pair - the layout of the paper's RMSNorm
sketch (Unified Sketch figure, Section 3.2.1: X[B, F, D1, D2] reduced over F)."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2512_23424_b200 import workloads as wl

RNG = np.random.default_rng(2024)
OPS = ["softmax", "log_softmax", "layernorm", "rmsnorm"]


def last_axis(op, rows, gamma, beta, eps):
    if op == "softmax":
        return oracle.softmax(rows)
    if op == "log_softmax":
        return oracle.log_softmax(rows)
    if op == "layernorm":
        return oracle.layernorm(rows, gamma, beta, eps=eps)
    return oracle.rmsnorm(rows, gamma, eps=eps)


@pytest.mark.parametrize("op", OPS)
def test_axis_equals_last_axis_of_the_transposed_array(op):
    outer, red, inner = 3, 7, 5
    x = RNG.normal(1.0, 2.0, size=(outer, red, inner))
    gamma = RNG.uniform(0.5, 1.5, red) if op in ("layernorm", "rmsnorm") else None
    beta = RNG.normal(0, 0.3, red) if op == "layernorm" else None
    got = oracle.rowop_axis(op, x, gamma, beta, eps=1e-3)
    rows = np.ascontiguousarray(x.transpose(0, 2, 1)).reshape(outer * inner, red)     # numpy does the indexing
    want = last_axis(op, rows, gamma, beta, 1e-3).reshape(outer, inner, red).transpose(0, 2, 1)
    np.testing.assert_array_equal(got, want)


def test_sketch_shaped_worked_example():
    # X[B=1, F=2, D1=1, D2=2]: column 0 holds (3, 4), column 1 holds (1, 1); eps = 0
    x = np.array([[[3.0, 1.0], [4.0, 1.0]]])
    y = oracle.rowop_axis("rmsnorm", x, eps=0.0)
    r = math.sqrt((9 + 16) / 2)
    np.testing.assert_allclose(y[0, :, 0], [3 / r, 4 / r], rtol=2e-16)
    np.testing.assert_allclose(y[0, :, 1], [1.0, 1.0], rtol=2e-16)
    # the weight is indexed by f (the reduced axis), not by the column
    yw = oracle.rowop_axis("rmsnorm", x, gamma=np.array([2.0, 0.5]), eps=0.0)
    np.testing.assert_allclose(yw[0, :, 0], [2 * 3 / r, 0.5 * 4 / r], rtol=2e-16)
    np.testing.assert_allclose(yw[0, :, 1], [2.0, 0.5], rtol=2e-16)
    # softmax over f: columns are independent logistic pairs
    s = oracle.rowop_axis("softmax", x)
    np.testing.assert_allclose(s[0, :, 0], [1 / (1 + math.e), math.e / (1 + math.e)], rtol=3e-16)
    np.testing.assert_allclose(s[0, :, 1], [0.5, 0.5], rtol=2e-16)
    # LayerNorm over f with beta indexed by f
    ln = oracle.rowop_axis("layernorm", x, gamma=np.array([1.0, 1.0]), beta=np.array([10.0, 20.0]), eps=0.0)
    np.testing.assert_allclose(ln[0, :, 0], [9.0, 21.0], rtol=2e-16)


def test_axis_against_torch_float64():
    x = RNG.normal(0.5, 1.5, size=(4, 11, 9))
    xt = torch.from_numpy(x)
    np.testing.assert_allclose(oracle.rowop_axis("softmax", x), torch.softmax(xt, 1).numpy(), rtol=1e-13)
    np.testing.assert_allclose(oracle.rowop_axis("log_softmax", x), torch.log_softmax(xt, 1).numpy(), atol=1e-13)
    g = RNG.uniform(0.5, 1.5, 11)
    b = RNG.normal(0, 0.2, 11)
    perm = xt.permute(0, 2, 1)
    ln = torch.nn.functional.layer_norm(perm, (11,), torch.from_numpy(g), torch.from_numpy(b), 1e-5)
    np.testing.assert_allclose(oracle.rowop_axis("layernorm", x, g, b, eps=1e-5), ln.permute(0, 2, 1).numpy(),
                               atol=1e-13)
    rn = torch.nn.functional.rms_norm(perm, (11,), torch.from_numpy(g), 1e-6)
    np.testing.assert_allclose(oracle.rowop_axis("rmsnorm", x, g, eps=1e-6), rn.permute(0, 2, 1).numpy(), rtol=1e-13)


def test_axis_strides_dtypes_and_threads():
    big = RNG.normal(size=(3, 6, 10)).astype(np.float32)
    view = big[:, :4, :7]                                  # outer stride 60, reduce stride 10, inner 7
    want = oracle.rowop_axis("softmax", np.ascontiguousarray(view))
    np.testing.assert_array_equal(oracle.rowop_axis("softmax", view), want)
    np.testing.assert_array_equal(oracle.rowop_axis("softmax", view, nthreads=3), want)
    bits = wl.f32_to_bf16_bits(big)
    wide = wl.bf16_bits_to_f32(bits).astype(np.float64)
    np.testing.assert_array_equal(oracle.rowop_axis("rmsnorm", bits, eps=1e-6), oracle.rowop_axis("rmsnorm", wide, eps=1e-6))
    # invariants per column: softmax sums to one over f; RMSNorm scales the mean square to ms / (ms + eps)
    s = oracle.rowop_axis("softmax", big.astype(np.float64))
    np.testing.assert_allclose(s.sum(axis=1), 1.0, atol=2e-15)
    y = oracle.rowop_axis("rmsnorm", big.astype(np.float64), eps=1e-2)
    ms = (big.astype(np.float64) ** 2).mean(axis=1)
    np.testing.assert_allclose((y ** 2).mean(axis=1), ms / (ms + 1e-2), rtol=1e-13)
