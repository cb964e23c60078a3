"""Pins of the oracle's gated activations (SiLU-and-Mul, GELU-and-Mul), no GPU: worked examples
re-derived at 40 digits, identities of the activations, a library second opinion, brute force."""
import math
import os

import numpy as np
import pytest
import torch
from mpmath import erf as mperf, exp as mpexp, mp, mpf, pi as mppi, sqrt as mpsqrt, tanh as mptanh

import oracle
from golden_io import _mat, read_records
from paper_2512_23424_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
RECORDS = read_records(os.path.join(GOLDEN, "act_mul_examples.txt"))
ACTS = ["silu", "gelu", "gelu_tanh"]


def mp_act(act, a):
    mp.dps = 100                    # 1 + erf and 1 + tanh cancel up to 60 digits at the gates tested below
    a = mpf(float(a))
    if act == "silu":
        return a / (1 + mpexp(-a))
    if act == "gelu":
        return a * (1 + mperf(a / mpsqrt(2))) / 2
    return a * (1 + mptanh(mpsqrt(2 / mppi) * (a + mpf("0.044715") * a ** 3))) / 2


@pytest.mark.parametrize("rec", RECORDS, ids=[r["name"] for r in RECORDS])
def test_worked_examples_and_their_derivation(rec):
    x = np.array(_mat(rec["x"]))
    want = np.array(_mat(rec["expect"]))
    d = x.shape[1] // 2
    mine = np.array([[float(mp_act(rec["act"], x[0, c]) * mpf(float(x[0, d + c]))) for c in range(d)]])
    assert np.max(np.abs(mine - want)) <= 4e-16
    got = oracle.act_mul(rec["act"], x)
    assert got.shape == want.shape
    assert np.max(np.abs(got - want)) <= 1e-15


def test_identities_of_the_activations():
    rng = np.random.default_rng(3)
    a = rng.normal(0, 3, (5, 64))
    one = np.ones_like(a)
    for act in ACTS:
        f = oracle.act_mul(act, np.concatenate([a, one], axis=1))
        fm = oracle.act_mul(act, np.concatenate([-a, one], axis=1))
        # act(a) - act(-a) = a for all three (sigmoid, Phi and the tanh form are odd about 1/2)
        assert np.max(np.abs((f - fm) - a)) < 1e-14
        # the second half is a plain factor
        b = rng.normal(0, 2, a.shape)
        fb = oracle.act_mul(act, np.concatenate([a, b], axis=1))
        assert np.max(np.abs(fb - f * b)) < 1e-14
        # act(0) = 0; act(a) -> a for large a; act(a) -> 0 for very negative a
        edge = oracle.act_mul(act, np.array([[0.0, 40.0, -40.0, 1.0, 1.0, 1.0]]))
        assert edge[0, 0] == 0.0 and abs(edge[0, 1] - 40.0) < 1e-12 and abs(edge[0, 2]) < 1e-12
    # SiLU at ln 3: sigmoid = 3/4; GELU at 0.6744897501960817 (the upper quartile of N(0,1)): Phi = 3/4
    s = oracle.act_mul("silu", np.array([[math.log(3.0), 2.0]]))
    assert abs(s[0, 0] - 1.5 * math.log(3.0)) < 1e-15
    q = 0.6744897501960817
    g = oracle.act_mul("gelu", np.array([[q, 4.0]]))
    assert abs(g[0, 0] - 3.0 * q) < 1e-14
    # the tanh form approximates the exact GELU to 5e-4 everywhere, and is not equal to it
    t = oracle.act_mul("gelu_tanh", np.concatenate([a, one], axis=1))
    e = oracle.act_mul("gelu", np.concatenate([a, one], axis=1))
    assert 1e-6 < np.max(np.abs(t - e)) < 5e-4


def test_left_tail_keeps_its_relative_accuracy():
    """1 + erf and 1 + tanh cancel for very negative gates; the oracle must not (the GPU kernels
    are checked against it to a relative tolerance there)."""
    a = np.array([[-4.0, -6.0, -8.0, -10.0, -12.5, -7.625, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0]])
    for act in ACTS:
        got = oracle.act_mul(act, a)[0]
        want = np.array([float(mp_act(act, v)) for v in a[0, :6]])
        assert np.all(want < 0) and np.all(got < 0)
        assert np.max(np.abs(got - want) / np.abs(want)) < 1e-12


def test_against_torch_float64():
    rng = np.random.default_rng(4)
    x = rng.normal(0, 2.5, (37, 258))
    tx = torch.from_numpy(x)
    a, b = tx[:, :129], tx[:, 129:]
    F = torch.nn.functional
    for act, want in (("silu", F.silu(a) * b), ("gelu", F.gelu(a) * b), ("gelu_tanh", F.gelu(a, approximate="tanh") * b)):
        assert np.max(np.abs(oracle.act_mul(act, x) - want.numpy())) < 1e-13


def test_storage_types_strides_and_threads():
    rng = np.random.default_rng(5)
    xf = rng.normal(0, 2, (9, 80)).astype(np.float32)
    for act in ACTS:
        y = oracle.act_mul(act, xf)
        assert np.array_equal(y, oracle.act_mul(act, xf.astype(np.float64)))
        xb = wl.f32_to_bf16_bits(xf)
        assert np.array_equal(oracle.act_mul(act, xb), oracle.act_mul(act, wl.bf16_bits_to_f32(xb).astype(np.float64)))
        big = np.full((9, 100), 3.0, np.float32)
        big[:, :80] = xf
        assert np.array_equal(oracle.act_mul(act, big[:, :80], nthreads=4), y)
    with pytest.raises(ValueError):
        oracle.act_mul("silu", xf[:, :79])


@pytest.mark.parametrize("seed", range(3))
def test_brute_force_mpmath(seed):
    rng = np.random.default_rng(300 + seed)
    rows, d = int(rng.integers(1, 4)), int(rng.integers(1, 7))
    x = rng.normal(0, 3, (rows, 2 * d))
    for act in ACTS:
        got = oracle.act_mul(act, x)
        want = np.array([[float(mp_act(act, x[i, c]) * mpf(float(x[i, d + c]))) for c in range(d)] for i in range(rows)])
        assert np.max(np.abs(got - want) / np.maximum(1.0, np.abs(want))) < 1e-14
