"""Pins for the fp64 CPU oracle (no GPU needed).

The oracle is checked against things it did not produce: hand-derived worked
examples (tests/golden), closed forms and invariants of the operators, fp64
library routines, and a 40-digit brute force on tiny inputs.  A dropped term, a
wrong sign or index, a transposed operand or a misplaced eps in the oracle
fails at least one test here.
"""
import math
import os

import numpy as np
import pytest
import torch
from mpmath import mp, mpf

import oracle
from golden_io import worked_examples
from paper_2512_23424_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
CASES = worked_examples(GOLDEN)


def _run_case(case):
    x = np.array(case["x"], dtype=np.float64)
    op = case["op"]
    if op in ("softmax", "log_softmax"):
        mask = None
        if "additive" in case or case["causal_period"]:
            add = np.array(case["additive"], dtype=np.float64) if "additive" in case else None
            mask = oracle.Mask(additive=add, causal=bool(case["causal_period"]),
                               causal_period=max(case["causal_period"], 1))
        return getattr(oracle, op)(x, mask=mask)
    if op == "layernorm":
        g = np.array(case["gamma"]) if "gamma" in case else None
        b = np.array(case["beta"]) if "beta" in case else None
        return oracle.layernorm(x, g, b, eps=case["eps"])
    w = np.array(case["weight"]) if "weight" in case else None
    return oracle.rmsnorm(x, w, eps=case["eps"])


@pytest.mark.parametrize("case", CASES, ids=[c["name"] for c in CASES])
def test_worked_examples(case):
    got = _run_case(case)
    want = np.array(case["expect"], dtype=np.float64)
    assert got.shape == want.shape
    for r in range(want.shape[0]):
        if r in case["skip_rows"]:
            continue
        np.testing.assert_allclose(got[r], want[r], rtol=4e-16, atol=1e-300)
        # zeros promised by the contract are +0, bit for bit
        zero = want[r] == 0
        assert not np.signbit(got[r][zero]).any() or case["op"] in ("layernorm", "rmsnorm")


# ---- the fixtures themselves, re-derived at 40 digits -----------------------------

def _mp_softmax(z):
    live = [v for v in z if v != -mp.inf]
    if not live:
        return [mpf(0)] * len(z)
    m = max(live)
    e = [mp.exp(v - m) if v != -mp.inf else mpf(0) for v in z]
    s = mp.fsum(e)
    return [v / s for v in e]


def _mp_eval(case):
    mp.dps = 40
    rows = []
    for r, xr in enumerate(case["x"]):
        x = [mpf(v) for v in xr]
        n = len(x)
        op = case["op"]
        if op in ("softmax", "log_softmax"):
            z = list(x)
            if "additive" in case:
                z = [a + (mpf(b) if math.isfinite(b) else -mp.inf)
                     for a, b in zip(z, case["additive"][r])]
            if case["causal_period"]:
                last = r % case["causal_period"]
                z = [v if c <= last else -mp.inf for c, v in enumerate(z)]
            y = _mp_softmax(z)
            if op == "log_softmax":
                y = [mp.log(v) for v in y]
        elif op == "layernorm":
            mu = mp.fsum(x) / n
            var = mp.fsum([(v - mu) ** 2 for v in x]) / n
            eps = mpf(repr(case["eps"]))
            g = case.get("gamma", [1] * n)
            b = case.get("beta", [0] * n)
            den = mp.sqrt(var + eps)
            y = [((v - mu) / den * mpf(gg) + mpf(bb)) if den != 0 else mpf(0)
                 for v, gg, bb in zip(x, g, b)]
        else:
            ms = mp.fsum([v * v for v in x]) / n
            eps = mpf(repr(case["eps"]))
            w = case.get("weight", [1] * n)
            den = mp.sqrt(ms + eps)
            y = [(v / den * mpf(ww)) if den != 0 else mpf(0) for v, ww in zip(x, w)]
        rows.append(y)
    return rows


@pytest.mark.parametrize("case", CASES, ids=[c["name"] for c in CASES])
def test_golden_file_matches_its_derivation(case):
    ref = _mp_eval(case)
    for r, row in enumerate(case["expect"]):
        if r in case["skip_rows"]:
            continue
        for got, want in zip(row, ref[r]):
            assert abs(mpf(got) - want) <= mpf("3e-16") * max(abs(want), mpf("1e-300"))


# ---- closed forms and invariants -----------------------------------------------------

RNG = np.random.default_rng(12345)


def test_softmax_rows_sum_to_one_and_shift_invariant():
    x = RNG.normal(0, 3, size=(17, 301))
    y = oracle.softmax(x)
    np.testing.assert_allclose(y.sum(axis=1), 1.0, rtol=0, atol=2e-15)
    shift = RNG.normal(0, 50, size=(17, 1))
    np.testing.assert_allclose(oracle.softmax(x + shift), y, rtol=2e-13, atol=0)
    assert (y > 0).all()


def test_softmax_pair_is_logistic():
    d = np.linspace(-30, 30, 41)
    x = np.stack([np.zeros_like(d), d], axis=1)
    y = oracle.softmax(x)
    np.testing.assert_allclose(y[:, 1], 1.0 / (1.0 + np.exp(-d)), rtol=3e-16)
    np.testing.assert_allclose(y[:, 0], 1.0 / (1.0 + np.exp(d)), rtol=3e-16)


def test_uniform_row():
    for n in (1, 2, 8, 64, 1024):
        y = oracle.softmax(np.full((1, n), 7.25))
        assert (y == 1.0 / n).all()
        ly = oracle.log_softmax(np.full((1, n), -3.5))
        np.testing.assert_allclose(ly, -math.log(n), rtol=2e-16, atol=0)


def test_no_overflow_for_large_inputs():
    y = oracle.softmax(np.array([[1e4, 1e4 + 1.0]]))
    np.testing.assert_allclose(y, [[1 / (1 + math.e), math.e / (1 + math.e)]], rtol=3e-16)
    assert oracle.logsumexp_row(np.array([1e4, 1e4])) == pytest.approx(1e4 + math.log(2), rel=1e-16)


def test_log_softmax_is_x_minus_logsumexp():
    x = RNG.normal(0, 4, size=(9, 257))
    ly = oracle.log_softmax(x)
    lse = np.array([oracle.logsumexp_row(r) for r in x])
    assert (lse >= x.max(axis=1)).all()
    np.testing.assert_allclose(ly, x - lse[:, None], rtol=0, atol=2e-14)
    np.testing.assert_allclose(np.exp(ly), oracle.softmax(x), rtol=3e-14)
    # x - lse exactly when the subtraction is exact: powers of two
    lse2 = oracle.logsumexp_row(np.array([0.0, 0.0]))
    assert lse2 == math.log(2.0)


def test_causal_rows_equal_prefix_softmax():
    rows, cols, period = 11, 9, 4
    x = RNG.normal(size=(rows, cols))
    y = oracle.softmax(x, mask=oracle.Mask(causal=True, causal_period=period))
    ly = oracle.log_softmax(x, mask=oracle.Mask(causal=True, causal_period=period))
    for r in range(rows):
        live = r % period + 1
        np.testing.assert_allclose(y[r, :live], oracle.softmax(x[r:r + 1, :live])[0], rtol=1e-15)
        assert (y[r, live:] == 0).all() and not np.signbit(y[r, live:]).any()
        assert (ly[r, live:] == -np.inf).all()
        np.testing.assert_allclose(ly[r, :live], oracle.log_softmax(x[r:r + 1, :live])[0], rtol=1e-14)
    assert (y[::period, 0] == 1.0).all()          # first row of every period: [1, 0, ...]


def test_causal_offset_and_row_ids():
    cols = 6
    x = RNG.normal(size=(3, cols))
    ids = np.array([5, 0, 7])
    y = oracle.softmax(x, mask=oracle.Mask(causal=True, causal_period=4, causal_offset=1),
                       row_ids=ids)
    for i, r in enumerate(ids):
        live = min(cols, r % 4 + 1 + 1)
        assert (y[i, live:] == 0).all()
        np.testing.assert_allclose(y[i, :live], oracle.softmax(x[i:i + 1, :live])[0], rtol=1e-15)


def test_additive_mask_row_modulo_and_stride():
    rows, cols = 7, 5
    x = RNG.normal(size=(rows, cols))
    add_full = RNG.normal(size=(3, cols + 2))         # padded: stride > cols
    add = add_full[:, :cols]
    y = oracle.softmax(x, mask=oracle.Mask(additive=add))
    for r in range(rows):
        np.testing.assert_allclose(y[r], oracle.softmax((x[r] + add[r % 3])[None])[0], rtol=1e-15)


def test_fully_masked_and_non_finite_rows():
    ninf = -np.inf
    x = np.array([[ninf, ninf, ninf], [0.0, ninf, 1.0], [0.0, np.nan, 1.0], [0.0, np.inf, 1.0]])
    y = oracle.softmax(x)
    ly = oracle.log_softmax(x)
    assert (y[0] == 0).all() and not np.signbit(y[0]).any()
    assert (ly[0] == ninf).all()
    assert y[1, 1] == 0 and not np.signbit(y[1, 1]) and ly[1, 1] == ninf
    np.testing.assert_allclose(y[1, [0, 2]], [1 / (1 + math.e), math.e / (1 + math.e)], rtol=3e-16)
    assert np.isnan(y[2]).all() and np.isnan(ly[2]).all()
    assert np.isnan(y[3]).all() and np.isnan(ly[3]).all()
    assert oracle.logsumexp_row(x[0]) == ninf
    # a NaN makes the row NaN even when every other entry is masked
    only = np.array([[np.nan, ninf, ninf], [np.nan, np.nan, np.nan]])
    assert np.isnan(oracle.softmax(only)).all() and np.isnan(oracle.log_softmax(only)).all()


def test_layernorm_moments_and_affine_invariance():
    n, eps = 513, 1e-5
    x = RNG.normal(3, 2, size=(6, n))
    y = oracle.layernorm(x, eps=eps)
    var = x.var(axis=1)
    np.testing.assert_allclose(y.sum(axis=1), 0, atol=1e-12)
    np.testing.assert_allclose((y ** 2).mean(axis=1), var / (var + eps), rtol=1e-13)
    y0 = oracle.layernorm(x, eps=0.0)
    np.testing.assert_allclose(oracle.layernorm(-2.5 * x + 40.0, eps=0.0), -y0, rtol=0, atol=2e-13)
    np.testing.assert_allclose(oracle.layernorm(0.5 * x - 7.0, eps=0.0), y0, rtol=0, atol=2e-13)
    # gamma scales, beta shifts, element by element (not transposed, not swapped)
    g = RNG.uniform(0.5, 1.5, n)
    b = RNG.normal(0, 0.1, n)
    np.testing.assert_allclose(oracle.layernorm(x, g, b, eps=eps), y * g + b, rtol=0, atol=1e-15)
    np.testing.assert_allclose(oracle.layernorm(x, None, b, eps=eps), y + b, rtol=0, atol=1e-15)


def test_layernorm_large_offset_no_cancellation():
    base = RNG.normal(0, 1, size=(1, 1000))
    y = oracle.layernorm(base, eps=0.0)
    y_shift = oracle.layernorm(base + 2.0 ** 30, eps=0.0)      # exact shift for these magnitudes?
    # the shift is not exact in fp64 for every element, so compare loosely but far tighter
    # than an E[x^2] - E[x]^2 formula could manage (that loses all digits at 2^30 offset)
    np.testing.assert_allclose(y_shift, y, rtol=0, atol=5e-6)


def test_rmsnorm_identities():
    n, eps = 300, 1e-6
    x = RNG.normal(0, 1.5, size=(5, n))
    w = RNG.uniform(0.5, 1.5, n)
    y = oracle.rmsnorm(x, w, eps=eps)
    ms = (x ** 2).mean(axis=1)
    np.testing.assert_allclose(((y / w) ** 2).mean(axis=1), ms / (ms + eps), rtol=1e-13)
    y0 = oracle.rmsnorm(x, w, eps=0.0)
    np.testing.assert_allclose(oracle.rmsnorm(-3.0 * x, w, eps=0.0), -y0, rtol=1e-14)
    c = -2.0
    yc = oracle.rmsnorm(np.full((1, n), c), w, eps=eps)
    np.testing.assert_allclose(yc[0], c / math.sqrt(c * c + eps) * w, rtol=3e-16)
    # the mean of squares divides by the row length, not by a fixed constant
    np.testing.assert_allclose(oracle.rmsnorm(np.ones((1, 7)), eps=0.0), 1.0, rtol=2e-16)
    np.testing.assert_allclose(oracle.rmsnorm(2 * np.ones((1, 3)), eps=5.0), 2.0 / 3.0, rtol=2e-16)


def test_layernorm_equals_rmsnorm_of_centred_row():
    x = RNG.normal(3, 2, size=(4, 129))
    eps = 1e-3
    centred = x - x.mean(axis=1, keepdims=True)
    np.testing.assert_allclose(oracle.layernorm(x, eps=eps), oracle.rmsnorm(centred, eps=eps),
                               rtol=0, atol=3e-15)


# ---- fp64 library routines as a second opinion ------------------------------------------

def test_against_torch_float64():
    x = RNG.normal(1, 3, size=(37, 129))
    xt = torch.from_numpy(x)
    g = RNG.uniform(0.5, 1.5, 129)
    b = RNG.normal(0, 0.1, 129)
    np.testing.assert_allclose(oracle.softmax(x), torch.softmax(xt, -1).numpy(), rtol=1e-13, atol=1e-300)
    np.testing.assert_allclose(oracle.log_softmax(x), torch.log_softmax(xt, -1).numpy(), rtol=0, atol=1e-13)
    lse = np.array([oracle.logsumexp_row(r) for r in x])
    np.testing.assert_allclose(lse, torch.logsumexp(xt, -1).numpy(), rtol=1e-14)
    ln = torch.nn.functional.layer_norm(xt, (129,), torch.from_numpy(g), torch.from_numpy(b), 1e-5)
    np.testing.assert_allclose(oracle.layernorm(x, g, b, eps=1e-5), ln.numpy(), rtol=0, atol=1e-13)
    rn = torch.nn.functional.rms_norm(xt, (129,), torch.from_numpy(g), 1e-6)
    np.testing.assert_allclose(oracle.rmsnorm(x, g, eps=1e-6), rn.numpy(), rtol=1e-13, atol=0)


def test_masked_softmax_against_torch_float64():
    rows, cols, period = 13, 10, 5
    x = RNG.normal(size=(rows, cols))
    r = np.arange(rows)[:, None] % period
    c = np.arange(cols)[None, :]
    z = np.where(c > r, -np.inf, x)
    want = torch.softmax(torch.from_numpy(z), -1).numpy()
    got = oracle.softmax(x, mask=oracle.Mask(causal=True, causal_period=period))
    np.testing.assert_allclose(got, want, rtol=1e-14, atol=0)


# ---- storage types --------------------------------------------------------------------------

def test_bf16_and_f32_widening_is_exact():
    vals = RNG.normal(0, 10, size=(3, 64)).astype(np.float32)
    bits = wl.f32_to_bf16_bits(vals)
    as_torch = torch.from_numpy(vals).to(torch.bfloat16)           # library RNE rounding
    assert (torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16) == as_torch).all()
    wide = as_torch.to(torch.float64).numpy()
    np.testing.assert_array_equal(oracle.rmsnorm(bits, eps=1e-6), oracle.rmsnorm(wide, eps=1e-6))
    np.testing.assert_array_equal(oracle.softmax(bits), oracle.softmax(wide))
    np.testing.assert_array_equal(oracle.layernorm(vals, eps=1e-5),
                                  oracle.layernorm(vals.astype(np.float64), eps=1e-5))
    # gamma / weight in bf16 storage are widened the same way
    w = wl.f32_to_bf16_bits(RNG.uniform(0.5, 1.5, 64).astype(np.float32))
    w64 = wl.bf16_bits_to_f32(w).astype(np.float64)
    np.testing.assert_array_equal(oracle.rmsnorm(bits, w, eps=1e-6), oracle.rmsnorm(wide, w64, eps=1e-6))


def test_row_stride_and_threads():
    big = RNG.normal(size=(20, 50))
    view = big[:, :33]                                 # stride 50, cols 33
    np.testing.assert_array_equal(oracle.softmax(view), oracle.softmax(np.ascontiguousarray(view)))
    np.testing.assert_array_equal(oracle.layernorm(view, eps=1e-5, nthreads=4),
                                  oracle.layernorm(np.ascontiguousarray(view), eps=1e-5))
    assert oracle.last_threads() == 1
    oracle.softmax(view, nthreads=3)
    assert oracle.last_threads() == 3


# ---- 40-digit brute force on tiny inputs -----------------------------------------------------

@pytest.mark.parametrize("seed", range(6))
def test_brute_force_mpmath(seed):
    mp.dps = 40
    rng = np.random.default_rng(seed)
    n = int(rng.integers(1, 9))
    x = rng.normal(0, 3, size=(1, n))
    g = rng.uniform(0.5, 1.5, n)
    b = rng.normal(0, 1, n)
    eps = 10.0 ** -int(rng.integers(2, 8))
    xm = [mpf(float(v)) for v in x[0]]
    m = max(xm)
    s = mp.fsum([mp.exp(v - m) for v in xm])
    sm = [mp.exp(v - m) / s for v in xm]
    lsm = [v - m - mp.log(s) for v in xm]
    mu = mp.fsum(xm) / n
    var = mp.fsum([(v - mu) ** 2 for v in xm]) / n
    ln = [(v - mu) / mp.sqrt(var + mpf(eps)) * mpf(float(gg)) + mpf(float(bb))
          for v, gg, bb in zip(xm, g, b)]
    ms = mp.fsum([v * v for v in xm]) / n
    rn = [v / mp.sqrt(ms + mpf(eps)) * mpf(float(gg)) for v, gg in zip(xm, g)]

    def close(got, want, tol):
        for a, w in zip(got, want):
            assert abs(mpf(float(a)) - w) <= tol * max(abs(w), mpf(1)), (a, w)

    close(oracle.softmax(x)[0], sm, mpf("1e-15"))
    close(oracle.log_softmax(x)[0], lsm, mpf("2e-15"))
    close(oracle.layernorm(x, g, b, eps=eps)[0], ln, mpf("1e-13"))
    close(oracle.rmsnorm(x, g, eps=eps)[0], rn, mpf("2e-15"))


# ---- the paper's verifier criterion (Section 3.2.3, Eq. 2-3) ----------------------------------

def test_verifier_fraction():
    ref = np.array([1.0, 2.0, 0.0, -4.0, 100.0])
    gen = np.array([1.0005, 2.004, 0.002, -4.0, 100.2])
    # relative errors 5e-4, 2e-3, (absolute) 2e-3, 0, 2e-3 -> 3 of 5 exceed tau = 1e-3
    assert oracle.verifier_fraction(gen, ref, eps_switch=1e-8, tau=1e-3) == pytest.approx(0.6)
    assert oracle.verifier_fraction(gen, ref, eps_switch=1e-8, tau=4e-3) == 0.0
    assert oracle.verifier_fraction(ref, ref) == 0.0
    # the error is relative to the REFERENCE: |2 - 1| / 1 = 1 > 0.6 (relative to gen it is 0.5)
    assert oracle.verifier_fraction(np.array([2.0]), np.array([1.0]), 1e-8, 0.6) == 1.0
    assert oracle.verifier_fraction(np.array([1.0]), np.array([2.0]), 1e-8, 0.6) == 0.0
    # below the switch the error is absolute: 1e-9 vs 3e-9 is 2e-9 absolute, not 200 % relative
    assert oracle.verifier_fraction(np.array([3e-9]), np.array([1e-9]), 1e-8, 1e-3) == 0.0
    assert oracle.verifier_fraction(np.array([3e-7]), np.array([1e-7]), 1e-8, 1e-3) == 1.0
    nan, inf = np.nan, np.inf
    assert oracle.verifier_fraction(np.array([nan, inf, 1.0, -inf]),
                                    np.array([nan, inf, nan, inf]), 1e-8, 1e-3) == 0.5


# ---- configuration-level sanity of oracle + generators ------------------------------------------

def test_config4_logsumexp_window():
    w = wl.make_config(4, rows=3)
    assert w.x.shape == (3, 262144) and w.extra["outlier_cols"].shape == (3, 26)
    assert ((w.x == np.float32(30.0)).sum(axis=1) >= 26).all()
    for r in range(3):
        lse = oracle.logsumexp_row(w.x[r].astype(np.float64))
        assert 30 + math.log(26) <= lse <= 30 + math.log(27)


def test_config2_and_config5_statistics():
    w2 = wl.make_config(2, rows=8)
    assert abs(w2.x.mean() - 3) < 0.05 and abs(w2.x.std() - 2) < 0.05
    assert 0.5 <= w2.gamma.min() and w2.gamma.max() <= 1.5
    w5 = wl.make_config(5, rows=64)
    y = oracle.softmax(w5.x, mask=oracle.Mask(causal=True, causal_period=4096))
    for r in range(64):
        assert y[r, :r + 1].sum() == pytest.approx(1.0, abs=1e-14)
        assert (y[r, r + 1:] == 0).all()
    assert w5.algorithmic_bytes() == (sum(range(1, 65)) + 64 * 4096) * 2


def test_half_and_bf16_widening_is_exact_for_every_bit_pattern():
    """All 65536 patterns of both 16-bit storage types against numpy's own conversions."""
    bits = np.arange(65536, dtype=np.uint16)
    half = bits.view(np.float16)
    got, want = oracle.widen(half), half.astype(np.float64)
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan], want[~nan]) and np.array_equal(np.signbit(got[~nan]), np.signbit(want[~nan]))
    got = oracle.widen(bits)                                   # uint16 = bf16 bits
    want = (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan], want[~nan]) and np.array_equal(np.signbit(got[~nan]), np.signbit(want[~nan]))
    # the drivers read half through the same conversion
    x = np.random.default_rng(0).normal(0, 2, (5, 33)).astype(np.float16)
    assert np.array_equal(oracle.softmax(x), oracle.softmax(x.astype(np.float64)))
    assert np.array_equal(oracle.rmsnorm(x, x[0], eps=1e-6), oracle.rmsnorm(x.astype(np.float64), x[0].astype(np.float64), eps=1e-6))
