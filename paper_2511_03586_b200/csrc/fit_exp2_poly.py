"""Derives the polynomial with which the attention kernel evaluates part of its
exponentials on the FMA pipe instead of the special-function unit.

2^a = 2^n * 2^f with n = round(a) and f = a - n in [-1/2, 1/2].  The kernel
obtains n by adding 1.5 * 2^23 (the sum's low mantissa bits then hold n), takes
2^f ~ P(f), a degree-3 polynomial, and adds n to the exponent field of P(f).
P minimises the maximum RELATIVE error on [-1/2, 1/2] (iteratively re-weighted
least squares on Chebyshev nodes).  Its error, about 1e-4, is far below the
2^-9 rounding of the bf16 probabilities the values are stored as.

Run:  python fit_exp2_poly.py      (prints the coefficients as C literals)
"""
import numpy as np

DEGREE = 3


def fit(degree=DEGREE, nodes=4001, iters=300):
    f = np.cos(np.linspace(0.0, np.pi, nodes)) * 0.5
    y = np.exp2(f)
    A = np.vander(f, degree + 1, increasing=True) / y[:, None]   # relative error: P(f) / 2^f - 1
    one = np.ones_like(f)
    w = np.ones_like(f)
    for _ in range(iters):
        coef, *_ = np.linalg.lstsq(A * w[:, None], one * w, rcond=None)
        err = A @ coef - one
        w *= 1.0 + 3.0 * np.abs(err) / np.abs(err).max()
        w /= w.max()
    return coef, float(np.abs(err).max())


def check_fp32(coef):
    """Maximum relative error of the whole evaluation in float32, the way the kernel does it."""
    a = np.linspace(-125.0, 17.0, 2000001).astype(np.float32)
    magic = np.float32(12582912.0)
    t = (a + magic).astype(np.float32)
    n = (t - magic).astype(np.float32)
    f = (a - n).astype(np.float32)
    c = coef.astype(np.float32)
    p = np.full_like(f, c[-1])
    for k in range(len(c) - 2, -1, -1):
        p = (p * f + c[k]).astype(np.float32)
    bits = p.view(np.int32) + (t.view(np.int32) << 23)
    got = bits.view(np.float32).astype(np.float64)
    ref = np.exp2(a.astype(np.float64))
    return float(np.max(np.abs(got / ref - 1.0)))


if __name__ == "__main__":
    coef, err = fit()
    print(f"// degree-{DEGREE} fit of 2^f on [-1/2, 1/2], max relative error {err:.3e}"
          f" ({check_fp32(coef):.3e} for the whole float32 evaluation on [-125, 17])")
    for k, c in enumerate(coef):
        print(f"constexpr float kExp2C{k} = {np.float32(c):.9e}f;")
