"""Pins of the oracle's arg-max / arg-min and cumulative sum / product (no GPU): worked examples
recomputed in exact rational arithmetic, closed forms, library second opinions, brute force."""
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from golden_io import _mat, read_records
from paper_2512_23424_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
RECORDS = read_records(os.path.join(GOLDEN, "reduction_examples.txt"))


@pytest.mark.parametrize("rec", [r for r in RECORDS if r["op"] != "colnorm"],
                         ids=[r["name"] for r in RECORDS if r["op"] != "colnorm"])
def test_worked_examples_and_their_derivation(rec):
    x = np.array(_mat(rec["x"]))
    op = rec["op"]
    if op in ("argmax", "argmin"):
        want = np.array([int(v) for v in rec["expect"].split()])
        mine = []
        for row in x:                                      # brute force over Fractions, first index wins
            fr = [Fraction(float(v)) for v in row]
            target = max(fr) if op == "argmax" else min(fr)
            mine.append(fr.index(target))
        assert mine == list(want)
        assert np.array_equal(oracle.argreduce(op, x), want)
    else:
        want = np.array(_mat(rec["expect"]))
        mine = []
        for row in x:
            acc, out = (Fraction(0) if op == "cumsum" else Fraction(1)), []
            for v in row:
                acc = acc + Fraction(float(v)) if op == "cumsum" else acc * Fraction(float(v))
                out.append(float(acc))
            mine.append(out)
        assert np.array_equal(np.array(mine), want)
        assert np.array_equal(oracle.cumulative(op, x), want)


def test_argreduce_against_libraries_and_rules():
    rng = np.random.default_rng(1)
    x = rng.normal(0, 1, (41, 257))
    x[3, 5] = x[3, 200] = 9.0                               # tie at the maximum
    x[4, 7] = x[4, 100] = -9.0                              # tie at the minimum
    x[5, 50] = np.inf
    x[6, 60] = -np.inf
    for op, npf, tf in (("argmax", np.argmax, torch.argmax), ("argmin", np.argmin, torch.argmin)):
        got = oracle.argreduce(op, x)
        assert got.dtype == np.int64
        assert np.array_equal(got, npf(x, axis=1))
        assert np.array_equal(got, tf(torch.from_numpy(x), dim=1).numpy())
    assert oracle.argreduce("argmax", x)[3] == 5 and oracle.argreduce("argmin", x)[4] == 7
    # NaN is the extreme for both, the first NaN wins; numpy and torch agree
    y = x.copy()
    y[7, 30] = y[7, 10] = np.nan
    y[8, 0] = np.nan
    for op, npf in (("argmax", np.argmax), ("argmin", np.argmin)):
        got = oracle.argreduce(op, y)
        assert got[7] == 10 and got[8] == 0
        assert np.array_equal(got, npf(y, axis=1))
    # negating the input swaps the two
    assert np.array_equal(oracle.argreduce("argmax", -x), oracle.argreduce("argmin", x))
    # a permutation of distinct values is recovered
    perm = rng.permutation(1000).astype(np.float64)[None, :]
    assert oracle.argreduce("argmax", perm)[0] == int(np.where(perm[0] == 999)[0][0])
    assert oracle.argreduce("argmin", perm)[0] == int(np.where(perm[0] == 0)[0][0])
    # storage types: comparisons are made on the stored values
    xf = x.astype(np.float32)
    assert np.array_equal(oracle.argreduce("argmax", xf), np.argmax(xf, axis=1))
    xb = wl.f32_to_bf16_bits(xf)
    assert np.array_equal(oracle.argreduce("argmax", xb), np.argmax(wl.bf16_bits_to_f32(xb), axis=1))
    assert np.array_equal(oracle.argreduce("argmin", xb, nthreads=4), np.argmin(wl.bf16_bits_to_f32(xb), axis=1))
    # strides; one column; an empty row is an error
    big = np.zeros((41, 300))
    big[:, :257] = x
    assert np.array_equal(oracle.argreduce("argmax", big[:, :257]), np.argmax(x, axis=1))
    assert np.array_equal(oracle.argreduce("argmin", x[:, :1]), np.zeros(41, dtype=np.int64))
    with pytest.raises(ValueError):
        oracle.argreduce("argmax", np.zeros((3, 0)))


def test_cumulative_closed_forms_and_libraries():
    n = 1000
    ones = np.ones((1, n))
    assert np.array_equal(oracle.cumulative("cumsum", ones)[0], np.arange(1, n + 1))
    k = np.arange(1, n + 1, dtype=np.float64)[None, :]
    assert np.array_equal(oracle.cumulative("cumsum", k)[0], k[0] * (k[0] + 1) / 2)
    # the telescoping product (1 + 1/k) = k + 1
    tele = oracle.cumulative("cumprod", 1.0 + 1.0 / k)[0]
    assert np.max(np.abs(tele - (k[0] + 1)) / (k[0] + 1)) < 1e-12
    # alternating signs: the running product of -1 alternates, of 2 doubles exactly
    assert np.array_equal(oracle.cumulative("cumprod", -np.ones((1, 9)))[0], [-1, 1, -1, 1, -1, 1, -1, 1, -1])
    assert np.array_equal(oracle.cumulative("cumprod", np.full((1, 60), 2.0))[0], 2.0 ** np.arange(1, 61))
    rng = np.random.default_rng(2)
    x = rng.normal(0, 1, (13, 777))
    cs, cp = oracle.cumulative("cumsum", x), oracle.cumulative("cumprod", x[:, :40])
    # differences give the input back; the last column is the row sum
    assert np.max(np.abs(np.diff(cs, axis=1) - x[:, 1:])) < 1e-13 and np.array_equal(cs[:, 0], x[:, 0])
    assert np.max(np.abs(cs[:, -1] - np.array([float(sum(Fraction(v) for v in row)) for row in x]))) < 1e-13
    assert np.max(np.abs(cp[:, 1:] / cp[:, :-1] - x[:, 1:40])) < 1e-12
    # library second opinion
    assert np.max(np.abs(cs - torch.cumsum(torch.from_numpy(x), dim=1).numpy())) < 1e-12
    tp = torch.cumprod(torch.from_numpy(x[:, :40]), dim=1).numpy()
    assert np.max(np.abs(cp - tp) / np.maximum(np.abs(tp), 1e-300)) < 1e-13
    # a cancelling row: the compensated sum keeps what a plain double sum loses
    big = np.array([[1e16, 1.0, -1e16, 1.0]])
    assert np.array_equal(oracle.cumulative("cumsum", big)[0, 2:], [1.0, 2.0])
    # zero and inf / NaN propagate as the arithmetic says
    z = oracle.cumulative("cumprod", np.array([[3.0, 0.0, 5.0, np.inf]]))[0]
    assert z[0] == 3.0 and z[1] == 0.0 and z[2] == 0.0 and np.isnan(z[3])
    s = oracle.cumulative("cumsum", np.array([[1.0, np.inf, 2.0, -np.inf]]))[0]
    assert s[0] == 1.0 and s[1] == np.inf and np.isnan(s[3])
    # storage types, strides, threads
    xf = x.astype(np.float32)
    assert np.array_equal(oracle.cumulative("cumsum", xf), oracle.cumulative("cumsum", xf.astype(np.float64)))
    xb = wl.f32_to_bf16_bits(xf)
    assert np.array_equal(oracle.cumulative("cumsum", xb),
                          oracle.cumulative("cumsum", wl.bf16_bits_to_f32(xb).astype(np.float64)))
    wide = np.zeros((13, 800))
    wide[:, :777] = x
    assert np.array_equal(oracle.cumulative("cumsum", wide[:, :777], nthreads=4), cs)


@pytest.mark.parametrize("seed", range(3))
def test_brute_force_exact_rationals(seed):
    rng = np.random.default_rng(700 + seed)
    rows, cols = int(rng.integers(1, 4)), int(rng.integers(1, 12))
    x = rng.normal(0, 2, (rows, cols))
    cs, cp = oracle.cumulative("cumsum", x), oracle.cumulative("cumprod", x)
    for i in range(rows):
        acc_s, acc_p = Fraction(0), Fraction(1)
        for c in range(cols):
            acc_s += Fraction(float(x[i, c]))
            acc_p *= Fraction(float(x[i, c]))
            assert abs(cs[i, c] - float(acc_s)) <= 1e-15 * max(1.0, abs(float(acc_s)))
            assert abs(cp[i, c] - float(acc_p)) <= 1e-14 * abs(float(acc_p))
        assert oracle.argreduce("argmax", x)[i] == max(range(cols), key=lambda c: (x[i, c], -c))
        assert oracle.argreduce("argmin", x)[i] == min(range(cols), key=lambda c: (x[i, c], c))


# ---- BatchNorm-style column statistics ---------------------------------------------------------

def test_colnorm_worked_example_and_identities():
    from mpmath import mp, mpf, sqrt as mpsqrt
    mp.dps = 40
    rec = [r for r in RECORDS if r["name"] == "colnorm_3x2"][0]
    want0 = np.array([float(v) for v in rec["expect"].split(";")])
    # the file against the closed form at 40 digits
    root = mpsqrt(mpf(3) / 2)
    assert np.max(np.abs(want0 - np.array([float(-root * 2 + mpf("0.5")), 0.5, float(root * 2 + mpf("0.5"))]))) < 4e-16
    x = np.array(_mat(rec["x"]))
    g, b = np.array([2.0, 3.0]), np.array([0.5, -1.0])
    y, mean, var = oracle.colnorm(x, g, b, eps=1e-9)
    assert np.array_equal(mean, [2.0, 10.0]) and abs(var[0] - 2.0 / 3.0) < 1e-16 and var[1] == 0.0
    assert np.max(np.abs(y[:, 0] - want0)) < 1e-8                  # eps = 1e-9 against the eps = 0 closed form
    assert np.array_equal(y[:, 1], [-1.0, -1.0, -1.0])             # a constant column returns beta
    rng = np.random.default_rng(9)
    x = rng.normal(3.0, 2.0, (257, 37))
    g, b = rng.uniform(0.5, 1.5, 37), rng.normal(0, 0.3, 37)
    y, mean, var = oracle.colnorm(x, g, b, eps=1e-5)
    # it is LayerNorm of the transpose with the affine moved to the other side
    yt = oracle.layernorm(np.ascontiguousarray(x.T), eps=1e-5).T * g[None, :] + b[None, :]
    assert np.max(np.abs(y - yt)) < 1e-13
    assert np.max(np.abs(mean - x.mean(axis=0))) < 1e-14 and np.max(np.abs(var - x.var(axis=0))) < 1e-14
    # column moments of the normalised values; a permutation of the rows permutes the output
    z, _, _ = oracle.colnorm(x, eps=1e-5)
    assert np.max(np.abs(z.mean(axis=0))) < 1e-14
    assert np.max(np.abs((z * z).mean(axis=0) - var / (var + 1e-5))) < 1e-13
    perm = rng.permutation(257)
    assert np.max(np.abs(oracle.colnorm(x[perm], g, b, eps=1e-5)[0] - y[perm])) < 1e-13
    # shifting and scaling a column by a positive factor leaves it unchanged at eps = 0
    y0 = oracle.colnorm(x, eps=0.0)[0]
    assert np.max(np.abs(oracle.colnorm(x * 3.0 + 7.0, eps=0.0)[0] - y0)) < 1e-12
    # library second opinion: training-mode batch norm in double
    t = torch.nn.functional.batch_norm(torch.from_numpy(x), None, None, torch.from_numpy(g), torch.from_numpy(b),
                                       training=True, eps=1e-5).numpy()
    assert np.max(np.abs(y - t)) < 1e-12
    # large offset: no cancellation
    off = oracle.colnorm(x + 1e8, eps=0.0)[0]
    assert np.max(np.abs(off - y0)) < 1e-6
    # storage types, strides, threads
    xf = x.astype(np.float32)
    a = oracle.colnorm(xf, g.astype(np.float32), b.astype(np.float32), eps=1e-5)
    c = oracle.colnorm(xf.astype(np.float64), g.astype(np.float32).astype(np.float64), b.astype(np.float32).astype(np.float64), eps=1e-5)
    assert all(np.array_equal(p, q) for p, q in zip(a, c))
    big = np.zeros((257, 50), dtype=np.float32)
    big[:, :37] = xf
    d = oracle.colnorm(big[:, :37], g.astype(np.float32), b.astype(np.float32), eps=1e-5, nthreads=4)
    assert all(np.array_equal(p, q) for p, q in zip(a, d))
    # brute force at 40 digits on a tiny case
    xs = rng.normal(0, 1, (5, 3))
    ys, ms, vs = oracle.colnorm(xs, eps=1e-3)
    for cidx in range(3):
        col = [mpf(float(v)) for v in xs[:, cidx]]
        m = sum(col) / 5
        v = sum((e - m) ** 2 for e in col) / 5
        assert abs(ms[cidx] - float(m)) < 1e-15 and abs(vs[cidx] - float(v)) < 1e-15
        for r in range(5):
            assert abs(ys[r, cidx] - float((col[r] - m) / mpsqrt(v + mpf("0.001")))) < 1e-14
