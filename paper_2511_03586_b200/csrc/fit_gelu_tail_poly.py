"""Derives the polynomial used by the GEMM epilogue's GELU.

GELU(z) = z * Phi(z) with Phi the standard normal CDF (the erf form:
Phi(z) = (1 + erf(z / sqrt 2)) / 2).  The epilogue evaluates
    q = 2 ** P(t),  t = min(|z|, T)        (q ~ Phi(-t), the lower tail)
    Phi(z) = q for z < 0, 1 - q otherwise,   q = 0 for |z| > T
where P is the degree-6 polynomial that minimises the maximum absolute error of
log2 Phi(-t) on [0, T] (iteratively re-weighted least squares on Chebyshev
nodes; a Remez exchange would shave a few per cent more).  An absolute error
dP in the exponent is a RELATIVE error ln(2) * dP in q, uniformly over the
tail, so GELU keeps its relative accuracy for negative arguments.

Run:  python fit_gelu_tail_poly.py      (prints the coefficients as C literals)
"""
import math

import numpy as np
from scipy.special import log_ndtr

T = 5.0
DEGREE = 6


def fit(T=T, degree=DEGREE, nodes=8001, iters=200):
    t = np.cos(np.linspace(0.0, np.pi, nodes)) * T / 2 + T / 2
    f = log_ndtr(-t) / math.log(2.0)
    A = np.vander(t / T, degree + 1, increasing=True)
    w = np.ones_like(t)
    for _ in range(iters):
        coef, *_ = np.linalg.lstsq(A * w[:, None], f * w, rcond=None)
        err = A @ coef - f
        w *= 1.0 + 3.0 * np.abs(err) / np.abs(err).max()
        w /= w.max()
    return coef / T ** np.arange(degree + 1), float(np.abs(err).max())


def check_fp32(coef):
    """Maximum relative error of z * Phi(z) evaluated in float32 the way the kernel does."""
    z = np.linspace(-8.0, 8.0, 400001).astype(np.float32)
    t = np.minimum(np.abs(z), np.float32(T))
    c = coef.astype(np.float32)
    p = np.full_like(t, c[-1])
    for k in range(len(c) - 2, -1, -1):
        p = (p * t + c[k]).astype(np.float32)
    q = np.exp2(p.astype(np.float64)).astype(np.float32)
    q = np.where(np.abs(z) > T, np.float32(0), q)
    phi = np.where(z < 0, q, np.float32(1) - q).astype(np.float32)
    got = (z * phi).astype(np.float64)
    zz = z.astype(np.float64)
    ref = zz * np.exp(log_ndtr(zz))
    inside = np.abs(zz) <= T
    rel = np.abs(got - ref)[inside] / np.maximum(np.abs(ref)[inside], 1e-30)
    return float(np.nanmax(rel[np.abs(zz[inside]) > 1e-3])), float(np.abs(got - ref).max())


if __name__ == "__main__":
    coef, e = fit()
    print(f"// degree {DEGREE} fit of log2(Phi(-t)) on [0, {T}]: max |dP| = {e:.3e} (relative error of Phi(-t) <= {e * math.log(2):.2e})")
    for k, c in enumerate(coef):
        print(f"//   c{k} = {c:.9e}f")
    rel, ab = check_fp32(coef)
    print(f"// float32 evaluation: max relative error of GELU on 1e-3 < |z| <= {T}: {rel:.2e}; max absolute error on [-8, 8]: {ab:.2e}")
