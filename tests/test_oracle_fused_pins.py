"""Pins of the oracle's fused residual add + normalisation (no GPU): worked examples re-derived
at 40 digits, special cases with known answers, a library second opinion, brute force."""
import os

import numpy as np
import pytest
import torch
from mpmath import mp, mpf, sqrt as mpsqrt

import oracle
from golden_io import _mat, _vec, read_records
from paper_2512_23424_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
ALL_RECORDS = read_records(os.path.join(GOLDEN, "fused_examples.txt"))
RECORDS = [r for r in ALL_RECORDS if "res" in r]
SCALED = [r for r in ALL_RECORDS if "scale" in r]
OPS = ["layernorm", "rmsnorm"]


def mp_add_norm(op, x, res, gamma, beta, eps):
    """The definition, written independently of the oracle, at 40 digits."""
    mp.dps = 40
    ys, ss = [], []
    for xr, rr in zip(x, res):
        s = [mpf(float(a)) + mpf(float(b)) for a, b in zip(xr, rr)]
        n = len(s)
        g = [mpf(float(v)) for v in gamma] if gamma is not None else [mpf(1)] * n
        b = [mpf(float(v)) for v in beta] if beta is not None else [mpf(0)] * n
        if op == "layernorm":
            mean = sum(s) / n
            var = sum((v - mean) ** 2 for v in s) / n
            y = [(v - mean) / mpsqrt(var + mpf(repr(eps))) * gi + bi for v, gi, bi in zip(s, g, b)]
        else:
            ms = sum(v * v for v in s) / n
            y = [v / mpsqrt(ms + mpf(repr(eps))) * gi for v, gi in zip(s, g)]
        ys.append(y)
        ss.append(s)
    return ys, ss


@pytest.mark.parametrize("rec", RECORDS, ids=[r["name"] for r in RECORDS])
def test_worked_examples_and_their_derivation(rec):
    x, res = np.array(_mat(rec["x"])), np.array(_mat(rec["res"]))
    gamma = np.array(_vec(rec.get("gamma", rec.get("weight", "")))) if ("gamma" in rec or "weight" in rec) else None
    beta = np.array(_vec(rec["beta"])) if "beta" in rec else None
    eps = float(rec.get("eps", "0"))
    want_y, want_s = np.array(_mat(rec["expect"])), np.array(_mat(rec["expect_sum"]))
    # the file against an independent 40-digit evaluation of the definition
    my, ms = mp_add_norm(rec["op"], x, res, gamma, beta, eps)
    assert np.allclose(np.array([[float(v) for v in r] for r in my]), want_y, rtol=0, atol=2e-16 * 8)
    assert np.array_equal(np.array([[float(v) for v in r] for r in ms]), want_s)
    # the oracle against the file
    y, s = oracle.add_norm(rec["op"], x, res, gamma, beta, eps=eps)
    assert np.array_equal(s, want_s)
    assert np.max(np.abs(y - want_y)) <= 1e-15 * max(1.0, np.max(np.abs(want_y)))


@pytest.mark.parametrize("op", OPS)
def test_special_cases_with_known_answers(op):
    rng = np.random.default_rng(5)
    x = rng.normal(1.0, 2.0, (7, 33))
    g, b = rng.uniform(0.5, 1.5, 33), rng.normal(0, 0.3, 33)
    beta = b if op == "layernorm" else None
    plain = oracle.layernorm(x, g, b, eps=1e-5) if op == "layernorm" else oracle.rmsnorm(x, g, eps=1e-5)
    # zero residual: the plain operator, and the sum is x itself
    y, s = oracle.add_norm(op, x, np.zeros_like(x), g, beta, eps=1e-5)
    assert np.array_equal(s, x) and np.array_equal(y, plain)
    # res = -x: the sum vanishes; LayerNorm returns beta, RMSNorm returns 0
    y, s = oracle.add_norm(op, x, -x, g, beta, eps=1e-5)
    assert np.all(s == 0)
    assert np.array_equal(y, np.broadcast_to(b, x.shape)) if op == "layernorm" else np.all(y == 0)
    # the operands commute; splitting x differently does not change anything
    r = rng.normal(0, 1, x.shape)
    y1, s1 = oracle.add_norm(op, x, r, g, beta, eps=1e-5)
    y2, s2 = oracle.add_norm(op, r, x, g, beta, eps=1e-5)
    assert np.array_equal(y1, y2) and np.array_equal(s1, s2)
    assert np.array_equal(s1, x + r)
    # the normalisation sees the sum, not x: moments of y are those of a normalised row
    y, s = oracle.add_norm(op, x, r, None, None, eps=0.0)
    if op == "layernorm":
        assert np.max(np.abs(y.mean(axis=1))) < 1e-14 and np.max(np.abs((y * y).mean(axis=1) - 1)) < 1e-13
        assert np.max(np.abs(y - (s - s.mean(axis=1, keepdims=True)) / s.std(axis=1, keepdims=True))) < 1e-13
    else:
        assert np.max(np.abs((y * y).mean(axis=1) - 1)) < 1e-13
        assert np.max(np.abs(y * np.sqrt((s * s).mean(axis=1, keepdims=True)) - s)) < 1e-13
    # RMSNorm ignores beta
    if op == "rmsnorm":
        assert np.array_equal(oracle.add_norm(op, x, r, g, b, eps=1e-5)[0], oracle.add_norm(op, x, r, g, None, eps=1e-5)[0])


@pytest.mark.parametrize("op", OPS)
def test_against_torch_float64(op):
    rng = np.random.default_rng(6)
    x, r = rng.normal(0.5, 3.0, (37, 129)), rng.normal(-1.0, 2.0, (37, 129))
    g, b = rng.uniform(0.5, 1.5, 129), rng.normal(0, 0.3, 129)
    tx, tr, tg, tb = (torch.from_numpy(a) for a in (x, r, g, b))
    if op == "layernorm":
        want = torch.nn.functional.layer_norm(tx + tr, (129,), tg, tb, eps=1e-5).numpy()
        y, s = oracle.add_norm(op, x, r, g, b, eps=1e-5)
    else:
        want = torch.nn.functional.rms_norm(tx + tr, (129,), tg, eps=1e-6).numpy()
        y, s = oracle.add_norm(op, x, r, g, eps=1e-6)
    assert np.max(np.abs(y - want)) < 1e-12
    assert np.array_equal(s, (tx + tr).numpy())


@pytest.mark.parametrize("op", OPS)
def test_storage_types_strides_and_threads(op):
    rng = np.random.default_rng(7)
    xf = rng.normal(0, 2, (9, 40)).astype(np.float32)
    rf = rng.normal(1, 1, (9, 40)).astype(np.float32)
    gf = rng.uniform(0.5, 1.5, 40).astype(np.float32)
    # fp32 storage: the sum is the exact sum of the widened values
    y, s = oracle.add_norm(op, xf, rf, gf, eps=1e-5)
    assert np.array_equal(s, xf.astype(np.float64) + rf.astype(np.float64))
    y64, _ = oracle.add_norm(op, xf.astype(np.float64), rf.astype(np.float64), gf.astype(np.float64), eps=1e-5)
    assert np.array_equal(y, y64)
    # bf16 storage: bits widen exactly
    xb, rb, gb = wl.f32_to_bf16_bits(xf), wl.f32_to_bf16_bits(rf), wl.f32_to_bf16_bits(gf)
    yb, sb = oracle.add_norm(op, xb, rb, gb, eps=1e-5)
    yw, sw = oracle.add_norm(op, wl.bf16_bits_to_f32(xb).astype(np.float64), wl.bf16_bits_to_f32(rb).astype(np.float64),
                             wl.bf16_bits_to_f32(gb).astype(np.float64), eps=1e-5)
    assert np.array_equal(yb, yw) and np.array_equal(sb, sw)
    # independent row strides of x and res, several threads
    bigx, bigr = np.full((9, 64), 7.0, np.float32), np.full((9, 51), -3.0, np.float32)
    bigx[:, :40], bigr[:, :40] = xf, rf
    y2, s2 = oracle.add_norm(op, bigx[:, :40], bigr[:, :40], gf, eps=1e-5, nthreads=4)
    assert np.array_equal(y2, y) and np.array_equal(s2, s)
    with pytest.raises(ValueError):
        oracle.add_norm(op, xf, rf[:, :39], gf)
    with pytest.raises(ValueError):
        oracle.add_norm(op, xf, rf.astype(np.float64), gf)


@pytest.mark.parametrize("seed", range(4))
def test_brute_force_mpmath(seed):
    rng = np.random.default_rng(100 + seed)
    rows, cols = int(rng.integers(1, 5)), int(rng.integers(1, 9))
    x, r = rng.normal(0, 3, (rows, cols)), rng.normal(2, 1, (rows, cols))
    g, b = rng.uniform(0.5, 1.5, cols), rng.normal(0, 1, cols)
    for op in OPS:
        eps = 1e-5 if op == "layernorm" else 1e-6
        if op == "layernorm" and cols == 1:
            continue                                   # 0 / sqrt(eps): fine, but nothing to compare beyond beta
        y, s = oracle.add_norm(op, x, r, g, b if op == "layernorm" else None, eps=eps)
        my, ms = mp_add_norm(op, x, r, g, b if op == "layernorm" else None, eps)
        want = np.array([[float(v) for v in row] for row in my])
        assert np.max(np.abs(y - want) / np.maximum(1.0, np.abs(want))) < 1e-13
        assert np.array_equal(s, np.array([[float(v) for v in row] for row in ms]))


# ---- softmax with a fused pre-scale ---------------------------------------------------------

def mp_scaled_softmax(x, scale, additive, log):
    """softmax / log-softmax of scale * x + additive, written independently at 40 digits."""
    from mpmath import exp as mpexp, log as mplog
    mp.dps = 40
    out = []
    for i, row in enumerate(x):
        z = [mpf(float(scale)) * mpf(float(v)) + (mpf(float(additive[i % len(additive)][c])) if additive is not None else 0)
             for c, v in enumerate(row)]
        m = max(z)
        s = sum(mpexp(v - m) for v in z)
        out.append([(v - m) - mplog(s) if log else mpexp(v - m) / s for v in z])
    return out


@pytest.mark.parametrize("rec", SCALED, ids=[r["name"] for r in SCALED])
def test_scaled_softmax_worked_examples(rec):
    x = np.array(_mat(rec["x"]))
    add = np.array(_mat(rec["additive"])) if "additive" in rec else None
    scale, log = float(rec["scale"]), rec["op"] == "log_softmax"
    want = np.array(_mat(rec["expect"]))
    mine = np.array([[float(v) for v in r] for r in mp_scaled_softmax(x, scale, add, log)])
    assert np.max(np.abs(mine - want)) <= 4e-16
    mask = oracle.Mask(additive=add) if add is not None else None
    got = oracle.softmax_scaled(x, scale, mask=mask, log=log)
    assert np.max(np.abs(got - want)) <= 1e-15


def test_scaled_softmax_identities_and_torch():
    rng = np.random.default_rng(8)
    x = rng.normal(0, 2, (9, 37))
    for s in (0.125, 1.0, 0.08838834764831845, 3.0):
        p = oracle.softmax_scaled(x, s)
        lp = oracle.softmax_scaled(x, s, log=True)
        # a power-of-two scale commutes exactly with the rounding of the input
        if s in (0.125, 1.0):
            assert np.array_equal(p, oracle.softmax(x * s))
        assert np.max(np.abs(p.sum(axis=1) - 1)) < 1e-14
        # shifting x does not matter; scaling the scale is the same as scaling x
        assert np.max(np.abs(oracle.softmax_scaled(x + 5.0, s) - p)) < 1e-13
        assert np.max(np.abs(oracle.softmax_scaled(2.0 * x, s / 2.0) - p)) < 1e-14
        # two entries: a logistic of scale * difference
        two = oracle.softmax_scaled(x[:, :2], s)
        assert np.max(np.abs(two[:, 1] - 1.0 / (1.0 + np.exp(-s * (x[:, 1] - x[:, 0]))))) < 1e-14
        # library second opinion, with and without an (unscaled) additive mask
        tx = torch.from_numpy(x)
        assert np.max(np.abs(p - torch.softmax(s * tx, dim=1).numpy())) < 1e-14
        assert np.max(np.abs(lp - torch.log_softmax(s * tx, dim=1).numpy())) < 1e-13
        a = rng.normal(0, 1, (3, 37))
        a[1, 5] = -np.inf
        pa = oracle.softmax_scaled(x, s, mask=oracle.Mask(additive=a))
        want = torch.softmax(s * tx + torch.from_numpy(a)[torch.arange(9) % 3], dim=1).numpy()
        assert np.max(np.abs(pa - want)) < 1e-14
        # causal rows are the scaled softmax of their prefix
        pc = oracle.softmax_scaled(x, s, mask=oracle.Mask(causal=True, causal_period=4))
        for r in range(9):
            live = r % 4 + 1
            assert np.max(np.abs(pc[r, :live] - oracle.softmax_scaled(x[r:r + 1, :live], s)[0])) < 1e-14
            assert np.all(pc[r, live:] == 0)
    # the limit of a small scale is the uniform row, of a large one the arg-max indicator
    assert np.max(np.abs(oracle.softmax_scaled(x, 1e-12) - 1.0 / 37)) < 1e-12
    hot = oracle.softmax_scaled(x, 1e6)
    assert np.array_equal(hot.argmax(axis=1), x.argmax(axis=1)) and np.all(hot.max(axis=1) == 1.0)
    for bad in (0.0, -1.0, np.inf, np.nan):
        with pytest.raises(ValueError):
            oracle.softmax_scaled(x, bad)


@pytest.mark.parametrize("seed", range(3))
def test_scaled_softmax_brute_force(seed):
    rng = np.random.default_rng(500 + seed)
    rows, cols = int(rng.integers(1, 4)), int(rng.integers(1, 8))
    x = rng.normal(0, 3, (rows, cols))
    a = rng.normal(0, 1, (2, cols))
    s = float(rng.uniform(0.05, 4.0))
    for log in (False, True):
        got = oracle.softmax_scaled(x, s, mask=oracle.Mask(additive=a), log=log)
        want = np.array([[float(v) for v in r] for r in mp_scaled_softmax(x, s, a, log)])
        assert np.max(np.abs(got - want) / np.maximum(1.0, np.abs(want))) < 1e-13
