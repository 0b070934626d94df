"""Pins for the CPU oracle's row operators (softmax, layernorm, rmsnorm, bias+GELU+residual, ReLU, SwiGLU).

Nothing here touches the CUDA path.  Every expected value comes from a closed
form, an invariant, an independent series or a textbook table, never from the
oracle's own formula retyped.
"""
import math
import os
from decimal import Decimal, getcontext

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ------------------------------------------------------------------ softmax
def test_softmax_rows_sum_to_one_and_positive():
    rng = np.random.default_rng(1)
    x = rng.normal(0, 4, size=(37, 513))
    y = oracle.softmax(x)
    assert np.all(y > 0)
    np.testing.assert_allclose(y.sum(axis=1), 1.0, rtol=0, atol=513 * 1e-15)


def test_softmax_closed_form_log_weights():
    # x_j = ln w_j  =>  y_j = w_j / sum w
    w = np.arange(1, 41, dtype=np.float64).reshape(2, 20)
    y = oracle.softmax(np.log(w))
    np.testing.assert_allclose(y, w / w.sum(axis=1, keepdims=True), rtol=1e-14)


def test_softmax_shift_invariance_and_no_overflow():
    rng = np.random.default_rng(2)
    x = rng.normal(0, 4, size=(5, 64))
    y = oracle.softmax(x)
    for c in (100.0, -100.0, 700.0):
        np.testing.assert_allclose(oracle.softmax(x + c), y, rtol=1e-12)
    # a row with values near the top of the double range must stay finite
    assert np.all(np.isfinite(oracle.softmax(np.array([[1e308, 1e308, 0.0]]))))


def test_softmax_constant_row_single_column_and_order():
    y = oracle.softmax(np.full((3, 8), -3.25))
    assert np.array_equal(y, np.full((3, 8), 0.125))
    assert np.array_equal(oracle.softmax(np.array([[5.0], [-7.0]])), np.ones((2, 1)))
    rng = np.random.default_rng(3)
    x = rng.normal(size=(4, 33))
    assert np.array_equal(np.argsort(oracle.softmax(x), axis=1), np.argsort(x, axis=1))


def test_softmax_rows_are_independent_and_along_last_dim():
    rng = np.random.default_rng(4)
    x = rng.normal(size=(6, 10))
    y = oracle.softmax(x)
    x2 = x.copy()
    x2[2] += rng.normal(size=10)
    y2 = oracle.softmax(x2)
    keep = [0, 1, 3, 4, 5]
    assert np.array_equal(y[keep], y2[keep])
    assert not np.allclose(y.sum(axis=0), 1.0)  # columns do not sum to one: reduction is over j


def test_softmax_two_point_logistic():
    # softmax([a, 0]) = [1/(1+e^-a), 1/(1+e^a)]
    a = 1.7
    y = oracle.softmax(np.array([[a, 0.0]]))
    np.testing.assert_allclose(y[0], [1 / (1 + math.exp(-a)), 1 / (1 + math.exp(a))], rtol=1e-15)


# ---------------------------------------------------------------- layernorm
def test_layernorm_zero_mean_unit_variance_before_affine():
    rng = np.random.default_rng(5)
    x = rng.normal(1, 2, size=(9, 1000))
    y = oracle.layernorm(x, np.ones(1000), np.zeros(1000), 0.0)
    assert np.max(np.abs(y.mean(axis=1))) < 1e-14
    np.testing.assert_allclose((y * y).mean(axis=1), 1.0, rtol=1e-13)  # biased: divide by M


def test_layernorm_closed_form_ramp():
    # row 0..M-1: mean (M-1)/2, biased variance (M^2-1)/12
    for M in (2, 7, 64):
        x = np.arange(M, dtype=np.float64)[None, :]
        g = np.linspace(0.5, 1.5, M)
        b = np.linspace(-0.1, 0.1, M)
        eps = 1e-5
        expect = (x - (M - 1) / 2) / math.sqrt((M * M - 1) / 12 + eps) * g + b
        np.testing.assert_allclose(oracle.layernorm(x, g, b, eps), expect, rtol=1e-14, atol=1e-15)


def test_layernorm_unbiased_variance_would_fail():
    # guards the 1/M reading: with M = 2 the unbiased estimate is twice the biased one
    y = oracle.layernorm(np.array([[0.0, 2.0]]), np.ones(2), np.zeros(2), 0.0)
    np.testing.assert_allclose(y, [[-1.0, 1.0]], rtol=1e-15)


def test_layernorm_eps_is_inside_the_root():
    # constant-free row with var = 3: y = (x-mu)/sqrt(3+eps), not (x-mu)/(sqrt(3)+eps)
    x = np.array([[-math.sqrt(3.0), math.sqrt(3.0)]])
    eps = 1.0
    y = oracle.layernorm(x, np.ones(2), np.zeros(2), eps)
    np.testing.assert_allclose(y, x / 2.0, rtol=1e-15)


def test_layernorm_invariances():
    rng = np.random.default_rng(6)
    x = rng.normal(size=(4, 50))
    g, b = rng.uniform(0.5, 1.5, 50), rng.normal(0, 0.1, 50)
    y = oracle.layernorm(x, g, b, 0.0)
    np.testing.assert_allclose(oracle.layernorm(x + 3.5, g, b, 0.0), y, rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(oracle.layernorm(x * 7.0, g, b, 0.0), y, rtol=1e-11, atol=1e-12)
    # output minus beta is linear in gamma
    y2 = oracle.layernorm(x, 2 * g, b, 0.0)
    np.testing.assert_allclose(y2 - b, 2 * (y - b), rtol=1e-12, atol=1e-13)
    # gamma and beta are indexed by column, not by row
    gp = g.copy(); gp[7] = 100.0
    yp = oracle.layernorm(x, gp, b, 0.0)
    changed = np.where(np.any(yp != y, axis=0))[0]
    assert list(changed) == [7]


def test_layernorm_constant_row_gives_beta():
    b = np.linspace(-1, 1, 16)
    y = oracle.layernorm(np.full((2, 16), 4.25), np.full(16, 3.0), b, 1e-5)
    assert np.array_equal(y, np.tile(b, (2, 1)))


# ------------------------------------------------------------------ rmsnorm
def test_rmsnorm_closed_forms_and_invariants():
    # constant row c: y = c / sqrt(c^2 + eps) * gamma
    g = np.linspace(0.5, 1.5, 8)
    y = oracle.rmsnorm(np.full((2, 8), -3.0), g, 7.0)
    np.testing.assert_allclose(y, np.tile(-3.0 / 4.0 * g, (2, 1)), rtol=1e-15)
    # row (3, 4): mean square 12.5 -> y = x / sqrt(12.5)
    np.testing.assert_allclose(oracle.rmsnorm(np.array([[3.0, 4.0]]), np.ones(2), 0.0),
                               [[3 / math.sqrt(12.5), 4 / math.sqrt(12.5)]], rtol=1e-15)
    rng = np.random.default_rng(40)
    x = rng.normal(1, 2, size=(5, 33))
    y = oracle.rmsnorm(x, np.ones(33), 0.0)
    np.testing.assert_allclose((y * y).mean(axis=1), 1.0, rtol=1e-13)          # unit mean square
    np.testing.assert_allclose(oracle.rmsnorm(4.0 * x, np.ones(33), 0.0), y, rtol=1e-12)   # scale invariant
    assert not np.allclose(oracle.rmsnorm(x + 1.0, np.ones(33), 0.0), y)       # but not shift invariant
    # on a zero-mean row it coincides with layernorm (beta = 0)
    xc = x - x.mean(axis=1, keepdims=True)
    g = rng.uniform(0.5, 1.5, 33)
    np.testing.assert_allclose(oracle.rmsnorm(xc, g, 1e-5), oracle.layernorm(xc, g, np.zeros(33), 1e-5),
                               rtol=1e-10, atol=1e-12)
    # gamma is indexed by column
    g2 = g.copy(); g2[4] = 9.0
    changed = np.where(np.any(oracle.rmsnorm(x, g2, 1e-5) != oracle.rmsnorm(x, g, 1e-5), axis=0))[0]
    assert list(changed) == [4]


# ------------------------------------------------------- bias + GELU + residual
def _erf_series(x: float) -> float:
    """erf by its Maclaurin series 2/sqrt(pi) * sum (-1)^n x^(2n+1) / (n! (2n+1)),
    in 60-digit decimal arithmetic: independent of libm."""
    getcontext().prec = 60
    xd = Decimal(repr(x))
    term = xd
    total = Decimal(0)
    n = 0
    while True:
        contrib = term / (2 * n + 1)
        total += contrib
        if abs(contrib) < Decimal(10) ** -45:
            break
        n += 1
        term = -term * xd * xd / n
    pi = Decimal("3.14159265358979323846264338327950288419716939937510582097494")
    return float(2 * total / pi.sqrt())


def _gelu_series(z: float) -> float:
    getcontext().prec = 60
    arg = float(Decimal(repr(z)) / Decimal(2).sqrt())
    # erf is evaluated at the rounded argument; its sensitivity there is < 1e-16 relative
    return 0.5 * z * (1.0 + _erf_series(arg))


def _gelu_only(z):
    z = np.atleast_2d(np.asarray(z, dtype=np.float64))
    return oracle.bias_gelu_residual(z, np.zeros(z.shape[1]), None)


def test_gelu_fixed_points_against_series():
    zs = [0.5, 1.0, 2.0, 3.0, -0.5, -1.0, -2.0, -3.0, 0.1, -0.1, 4.0]
    got = _gelu_only(zs)[0]
    expect = np.array([_gelu_series(z) for z in zs])
    np.testing.assert_allclose(got, expect, rtol=2e-13, atol=1e-17)


def test_gelu_matches_normal_cdf_table():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "standard_normal_cdf.txt")) if l[0] not in "#\n"]
    z = np.array([float(r[0]) for r in rows])
    phi = np.array([float(r[1]) for r in rows])
    np.testing.assert_allclose(_gelu_only(z)[0], z * phi, rtol=2e-15 * 10)
    np.testing.assert_allclose(_gelu_only(-z)[0], -z * (1 - phi), rtol=1e-11)


def test_gelu_identities_and_limits():
    assert _gelu_only([0.0])[0, 0] == 0.0
    z = np.linspace(-6, 6, 241)
    g = _gelu_only(z)[0]
    np.testing.assert_allclose(g - _gelu_only(-z)[0], z, rtol=0, atol=1e-15)  # GELU(z) - GELU(-z) = z
    assert _gelu_only([40.0])[0, 0] == 40.0
    assert abs(_gelu_only([-40.0])[0, 0]) == 0.0
    # the tanh approximation differs visibly from the erf form: this must not be it
    tanh_form = 0.5 * 1.5 * (1 + math.tanh(math.sqrt(2 / math.pi) * (1.5 + 0.044715 * 1.5 ** 3)))
    assert abs(_gelu_only([1.5])[0, 0] - tanh_form) > 1e-5


def test_bias_broadcast_residual_and_permutation():
    rng = np.random.default_rng(7)
    x, r = rng.normal(size=(5, 12)), rng.normal(size=(5, 12))
    bias = rng.normal(0, 0.5, 12)
    out = oracle.bias_gelu_residual(x, bias, r)
    # bias is added before the activation, per column; the residual after it
    np.testing.assert_array_equal(out, _gelu_only(x + bias[None, :]) + r)
    np.testing.assert_array_equal(oracle.bias_gelu_residual(x, bias, None), _gelu_only(x + bias[None, :]))
    perm = rng.permutation(12)
    np.testing.assert_array_equal(oracle.bias_gelu_residual(x[:, perm], bias[perm], r[:, perm]), out[:, perm])
    # changing bias[j] changes column j only
    b2 = bias.copy(); b2[3] += 1.0
    changed = np.where(np.any(oracle.bias_gelu_residual(x, b2, r) != out, axis=0))[0]
    assert list(changed) == [3]


# ------------------------------------------------- library cross-check (torch f64)
# --------------------------------------------------------------- reducemean
def test_reducemean_closed_forms_and_invariants():
    # ramp 1..n has mean (n + 1) / 2; a constant row has its constant; integers sum exactly
    for n in (1, 2, 7, 512, 4096):
        x = np.arange(1, n + 1, dtype=np.float64).reshape(1, n)
        np.testing.assert_allclose(oracle.reducemean(x), [(n + 1) / 2], rtol=1e-14)
    assert np.array_equal(oracle.reducemean(np.full((3, 8), 2.5)), np.full(3, 2.5))
    rng = np.random.default_rng(51)
    x = rng.normal(1, 2, size=(6, 333))
    m = oracle.reducemean(x)
    assert m.shape == (6,)
    # rows are independent, the mean is linear, invariant under permutation of a row, shifts with the row
    np.testing.assert_allclose(oracle.reducemean(3 * x + 1), 3 * m + 1, rtol=1e-13)
    np.testing.assert_allclose(oracle.reducemean(x[:, rng.permutation(333)]), m, rtol=1e-13)
    assert np.array_equal(oracle.reducemean(x[2:3]), m[2:3])
    np.testing.assert_allclose(m, [math.fsum(row) / 333 for row in x], rtol=1e-14)
    # it is the first statistic of layernorm: subtracting it centres the row the way layernorm does
    y = oracle.layernorm(x, np.ones(333), np.zeros(333), 0.0)
    c = x - m[:, None]
    np.testing.assert_allclose(y, c / np.sqrt((c * c).mean(axis=1, keepdims=True)), rtol=1e-11, atol=1e-13)


# ------------------------------------------------------------ relu, swiglu
def test_relu_epilogue_special_cases():
    x = np.array([[-2.0, -0.0, 0.0, 3.5], [1e-300, -1e-300, 7.0, -7.0]])
    out = oracle.bias_relu_residual(x)
    assert np.array_equal(out, np.array([[0.0, 0.0, 0.0, 3.5], [1e-300, 0.0, 7.0, 0.0]]))
    # relu(z) - relu(-z) = z and relu(z) + relu(-z) = |z|
    rng = np.random.default_rng(41)
    z = rng.normal(size=(5, 9))
    assert np.array_equal(oracle.bias_relu_residual(z) - oracle.bias_relu_residual(-z), z)
    assert np.array_equal(oracle.bias_relu_residual(z) + oracle.bias_relu_residual(-z), np.abs(z))
    # the bias is added before the kink (broadcast over rows), the residual after it
    bias = rng.normal(size=9)
    r = rng.normal(size=(5, 9))
    got = oracle.bias_relu_residual(z, bias, r)
    for i in range(5):
        for j in range(9):
            t = z[i, j] + bias[j]
            assert got[i, j] == (t if t > 0 else 0.0) + r[i, j]
    # a large negative bias switches everything off and leaves the residual
    assert np.array_equal(oracle.bias_relu_residual(z, np.full(9, -100.0), r), r)


def test_swiglu_closed_forms():
    # SiLU(0) = 0; SiLU(ln 3) = ln 3 * 3/4; SiLU(-ln 3) = -ln 3 / 4
    g = np.array([0.0, math.log(3.0), -math.log(3.0)])
    np.testing.assert_allclose(oracle.swiglu(g, np.ones(3)), [0.0, 0.75 * math.log(3.0), -0.25 * math.log(3.0)],
                               rtol=1e-15, atol=0)
    rng = np.random.default_rng(42)
    g, u = rng.normal(0, 3, size=200), rng.normal(size=200)
    s = oracle.swiglu(g, np.ones_like(g))
    # SiLU(g) - SiLU(-g) = g  and  SiLU(g) + SiLU(-g) = g tanh(g / 2)
    sm = oracle.swiglu(-g, np.ones_like(g))
    np.testing.assert_allclose(s - sm, g, rtol=1e-14, atol=1e-15)
    np.testing.assert_allclose(s + sm, g * np.tanh(g / 2), rtol=1e-13, atol=1e-15)
    # linear in u, and the gate is the FIRST argument: swapping the operands changes the result
    np.testing.assert_allclose(oracle.swiglu(g, u), s * u, rtol=1e-15, atol=0)
    assert not np.allclose(oracle.swiglu(g, u), oracle.swiglu(u, g))
    # limits: SiLU(g) -> g for large g, -> 0 from below for very negative g; minimum value about -0.27846 at g = -1.27846
    np.testing.assert_allclose(oracle.swiglu(np.array([40.0]), np.ones(1)), [40.0], rtol=1e-15)
    assert -1e-15 < oracle.swiglu(np.array([-40.0]), np.ones(1))[0] < 0
    grid = np.linspace(-3, 0, 300001)
    vals = oracle.swiglu(grid, np.ones_like(grid))
    assert abs(vals.min() + 0.27846454276107) < 1e-10 and abs(grid[vals.argmin()] + 1.27846454276107) < 1e-4


def test_relu_swiglu_against_torch_float64():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(43)
    g, u = rng.normal(0, 2, size=(7, 33)), rng.normal(size=(7, 33))
    ref = (torch.nn.functional.silu(torch.from_numpy(g)) * torch.from_numpy(u)).numpy()
    np.testing.assert_allclose(oracle.swiglu(g, u), ref, rtol=1e-14, atol=1e-16)
    bias, r = rng.normal(size=33), rng.normal(size=(7, 33))
    ref = (torch.relu(torch.from_numpy(g) + torch.from_numpy(bias)) + torch.from_numpy(r)).numpy()
    assert np.array_equal(oracle.bias_relu_residual(g, bias, r), ref)


def test_rowops_against_torch_float64():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(8)
    x = rng.normal(0, 4, size=(17, 129))
    xt = torch.from_numpy(x)
    np.testing.assert_allclose(oracle.softmax(x), torch.softmax(xt, dim=-1).numpy(), rtol=1e-12)
    g, b = rng.uniform(0.5, 1.5, 129), rng.normal(0, 0.1, 129)
    ref = torch.nn.functional.layer_norm(xt, (129,), torch.from_numpy(g), torch.from_numpy(b), 1e-5).numpy()
    np.testing.assert_allclose(oracle.layernorm(x, g, b, 1e-5), ref, rtol=1e-11, atol=1e-13)
    r = rng.normal(size=x.shape)
    ref = (torch.nn.functional.gelu(xt + torch.from_numpy(b)) + torch.from_numpy(r)).numpy()
    np.testing.assert_allclose(oracle.bias_gelu_residual(x, b, r), ref, rtol=1e-12, atol=1e-14)


def test_bad_arguments_are_rejected():
    with pytest.raises(ValueError):
        oracle.softmax(np.zeros((2, 0)))
