#!/usr/bin/env python3
"""Generates the polynomial coefficients of the normal distribution function used by the
GELU-and-Mul kernel (kernels_act.cuh: normal_cdf).

For x >= 0 the scaled complementary error function erfcx(x) = exp(x^2) erfc(x) behaves like
1 / (x sqrt(pi)) at infinity, so with t = 1 / (1 + x / 2) in (0, 1] the ratio
h(t) = erfcx(x) / t is smooth on the whole interval.  h is fitted by a polynomial in t
(least squares at Chebyshev nodes, weighted for relative error), which gives for a <= 0

    Phi(a) = 0.5 erfc(-a / sqrt 2) = 0.5 exp(-a^2 / 2) t h(t),   x = -a / sqrt 2,

with a relative error that stays small in the far left tail (where 1 + erf cancels).
Reference values come from mpmath at 40 digits.  Prints C initialisers and the measured
error of an fp32 Horner evaluation.  Run by hand when the degrees change; nothing imports it.
"""
import numpy as np
from mpmath import erfc, exp, mp, mpf, sqrt

mp.dps = 40
P = 0.5


def erfcx(x):
    x = mpf(x)
    return erfc(x) * exp(x * x)


def fit(deg, npts=600):
    k = np.arange(npts)
    t = 0.5 * (1 - np.cos(np.pi * (k + 0.5) / npts))
    t = np.concatenate([t, [1.0]])
    x = (1 / t - 1) / P
    h = np.array([float(erfcx(xi) / mpf(ti)) for xi, ti in zip(x, t)])
    v = np.polynomial.chebyshev.chebvander(2 * t - 1, deg)
    c, *_ = np.linalg.lstsq(v / h[:, None], np.ones_like(h), rcond=None)
    mono = np.polynomial.chebyshev.cheb2poly(c)
    return np.polynomial.Polynomial(mono)(np.polynomial.Polynomial([-1.0, 2.0])).coef


def fp32_error(coef, lo=-9.0, n=4001):
    a = np.linspace(lo, 0, n).astype(np.float32)
    x = (np.abs(a) * np.float32(0.70710678118654752)).astype(np.float32)
    t = (np.float32(1) / (np.float32(1) + np.float32(P) * x)).astype(np.float32)
    h = np.full_like(t, np.float32(coef[-1]))
    for c in coef[-2::-1]:
        h = (h * t + np.float32(c)).astype(np.float32)
    e = np.exp2((a * a).astype(np.float32) * np.float32(-0.5 * 1.4426950408889634)).astype(np.float32)
    q = (np.float32(0.5) * t * h * e).astype(np.float64)
    ref = np.array([float(erfc(-mpf(float(v)) / sqrt(2)) / 2) for v in a])
    rel = np.abs(q - ref) / ref
    return rel.max(), rel[a > -1.0].max()


if __name__ == "__main__":
    for deg in (9, 5):
        coef = fit(deg)
        worst, centre = fp32_error(coef)
        print(f"// degree {deg}: max relative error of the fp32 evaluation {worst:.2e} on [-9, 0], {centre:.2e} on [-1, 0]")
        print("{" + ", ".join(f"{np.float32(c):.9e}f" for c in coef) + "}")
