"""GPU parity of pd_softmax / pd_layernorm / pd_bias_gelu_residual against the
CPU oracle, called through the C ABI.  Tolerance: max relative error 1e-5 (fp32
row operators); for outputs that end in an addition the denominator is floored
at the RMS of the oracle tensor (see parity.max_rel_floored)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_03586_b200 import inputs
from parity import Guarded, dev_f32, host, max_rel, max_rel_floored

pytestmark = pytest.mark.gpu
TOL = 1e-5

ROWS = (1, 3, 33)
COLS = (1, 2, 3, 4, 5, 31, 32, 33, 127, 128, 129, 512, 1000, 1024, 1028, 2048, 4096, 5000, 8192, 8196, 12288, 12292, 16384, 16388, 20480, 20484,
        24576, 24580, 28672, 28676, 40000, 65536, 100000, 131076, 262144, 262148)


@pytest.fixture(scope="module")
def api():
    from paper_2511_03586_b200 import api
    return api


@pytest.mark.parametrize("cols", COLS)
def test_softmax_shapes(api, cols):
    for rows in ROWS:
        x = inputs.softmax_inputs(rows, cols, seed=rows)["x"]
        y = Guarded((rows, cols), torch.float32)
        api.pd_softmax(dev_f32(x), y.t)
        torch.cuda.synchronize()
        y.check()
        assert max_rel(host(y.t), oracle.softmax(x)) < TOL


def test_softmax_configured_and_paper_shapes(api):
    for rows, cols in ((256, 512), (24576, 512)):
        x = inputs.softmax_inputs(rows, cols, seed=0)["x"]
        y = api.pd_softmax(dev_f32(x))
        got = host(y)
        assert max_rel(got, oracle.softmax(x)) < TOL
        assert np.max(np.abs(got.sum(axis=1) - 1)) < 1e-5


def test_softmax_in_place_unaligned_and_deterministic(api):
    x = inputs.softmax_inputs(65, 516, seed=5)["x"]
    xd = dev_f32(x)
    y1 = api.pd_softmax(xd)
    y2 = api.pd_softmax(xd)
    assert torch.equal(y1, y2)
    api.pd_softmax(xd, xd)
    assert torch.equal(xd, y1)
    # a view that starts 4 bytes into an allocation takes the scalar path
    raw = torch.empty(65 * 516 + 1, dtype=torch.float32, device="cuda")
    xu = raw[1:].view(65, 516)
    xu.copy_(torch.from_numpy(x))
    assert max_rel(host(api.pd_softmax(xu)), oracle.softmax(x)) < TOL
    # constant rows give exactly 1/cols when cols is a power of two
    c = torch.full((4, 256), 3.5, device="cuda")
    assert torch.equal(api.pd_softmax(c), torch.full((4, 256), 1 / 256, device="cuda"))


@pytest.mark.parametrize("cols", COLS)
def test_layernorm_shapes(api, cols):
    for rows in ROWS:
        p = inputs.layernorm_inputs(rows, cols, seed=rows)
        y = Guarded((rows, cols), torch.float32)
        api.pd_layernorm(dev_f32(p["x"]), dev_f32(p["gamma"]), dev_f32(p["beta"]), p["eps"], y.t)
        torch.cuda.synchronize()
        y.check()
        ref = oracle.layernorm(p["x"], p["gamma"], p["beta"], np.float32(p["eps"]))
        if cols == 1:
            assert np.allclose(host(y.t), ref, atol=1e-6)
        else:
            assert max_rel_floored(host(y.t), ref) < TOL


# Many rows (several waves of CTAs, a ragged last one) for each kernel family: a warp per row, and CTAs of 64, 128
# and 256 threads per row, with ragged row lengths within them.
@pytest.mark.parametrize("dims", [(5000, 512), (9001, 1024), (4099, 1000), (3001, 2048), (2100, 1540), (1501, 4096),
                                  (1300, 2052), (777, 8192), (700, 4100)])
def test_many_rows(api, dims):
    rows, cols = dims
    p = inputs.layernorm_inputs(rows, cols, seed=cols)
    x, g, b = dev_f32(p["x"]), dev_f32(p["gamma"]), dev_f32(p["beta"])
    y = Guarded((rows, cols), torch.float32)
    api.pd_layernorm(x, g, b, p["eps"], y.t)
    torch.cuda.synchronize()
    y.check()
    assert max_rel_floored(host(y.t), oracle.layernorm(p["x"], p["gamma"], p["beta"], np.float32(p["eps"]))) < TOL
    z = Guarded((rows, cols), torch.float32)
    api.pd_rmsnorm(x, g, p["eps"], z.t)
    torch.cuda.synchronize()
    z.check()
    assert max_rel_floored(host(z.t), oracle.rmsnorm(p["x"], p["gamma"], np.float32(p["eps"]))) < TOL
    # in place, and repeatable
    x2 = x.clone()
    api.pd_layernorm(x2, g, b, p["eps"], x2)
    assert torch.equal(x2, y.t)


def test_layernorm_configured_and_paper_shapes(api):
    for rows, cols in ((4096, 1024), (16384, 1024), (4096, 4096)):
        p = inputs.layernorm_inputs(rows, cols, seed=0)
        xd = dev_f32(p["x"])
        y = api.pd_layernorm(xd, dev_f32(p["gamma"]), dev_f32(p["beta"]), p["eps"])
        ref = oracle.layernorm(p["x"], p["gamma"], p["beta"], np.float32(p["eps"]))
        assert max_rel_floored(host(y), ref) < TOL
        y2 = api.pd_layernorm(xd, dev_f32(p["gamma"]), dev_f32(p["beta"]), p["eps"], xd)   # in place
        assert torch.equal(y, y2)


def test_layernorm_large_mean_is_stable(api):
    # mean >> spread: a one-pass E[x^2] - mu^2 variance would lose every digit here
    rng = np.random.default_rng(9)
    for cols in (1024, 4096, 40000):
        x = (1000.0 + 0.01 * rng.standard_normal((3, cols))).astype(np.float32)
        g, b = np.ones(cols, np.float32), np.zeros(cols, np.float32)
        y = api.pd_layernorm(dev_f32(x), dev_f32(g), dev_f32(b), 0.0)
        assert max_rel_floored(host(y), oracle.layernorm(x, g, b, 0.0)) < 1e-4


@pytest.mark.parametrize("cols", COLS)
def test_rmsnorm_shapes(api, cols):
    for rows in ROWS:
        p = inputs.rmsnorm_inputs(rows, cols, seed=rows)
        y = Guarded((rows, cols), torch.float32)
        api.pd_rmsnorm(dev_f32(p["x"]), dev_f32(p["gamma"]), p["eps"], y.t)
        torch.cuda.synchronize()
        y.check()
        assert max_rel(host(y.t), oracle.rmsnorm(p["x"], p["gamma"], np.float32(p["eps"]))) < TOL


def test_rmsnorm_paper_shape_and_in_place(api):
    rows, cols = 3072, 4096                       # Table "ML operators optimized using PerfLLM": rmsnorm
    p = inputs.rmsnorm_inputs(rows, cols, seed=0)
    xd, gd = dev_f32(p["x"]), dev_f32(p["gamma"])
    y = api.pd_rmsnorm(xd, gd, p["eps"])
    assert max_rel(host(y), oracle.rmsnorm(p["x"], p["gamma"], np.float32(p["eps"]))) < TOL
    api.pd_rmsnorm(xd, gd, p["eps"], xd)
    assert torch.equal(xd, y)


@pytest.mark.parametrize("cols", COLS)
def test_bias_gelu_residual_shapes(api, cols):
    for rows in ROWS:
        p = inputs.bias_gelu_residual_inputs(rows, cols, seed=rows)
        out = Guarded((rows, cols), torch.float32)
        api.pd_bias_gelu_residual(dev_f32(p["x"]), dev_f32(p["bias"]), dev_f32(p["r"]), out.t)
        torch.cuda.synchronize()
        out.check()
        assert max_rel_floored(host(out.t), oracle.bias_gelu_residual(p["x"], p["bias"], p["r"])) < TOL
        out2 = api.pd_bias_gelu_residual(dev_f32(p["x"]), dev_f32(p["bias"]), None)
        assert max_rel_floored(host(out2), oracle.bias_gelu_residual(p["x"], p["bias"], None)) < TOL


def test_bias_gelu_residual_configured_shape_sampled_rows(api):
    rows, cols = 16384, 4096
    p = inputs.bias_gelu_residual_inputs(rows, cols, seed=0)
    xd, rd = dev_f32(p["x"]), dev_f32(p["r"])
    out = api.pd_bias_gelu_residual(xd, dev_f32(p["bias"]), rd)
    pick = np.unique(np.concatenate([[0, 1, rows - 1], np.random.default_rng(0).integers(0, rows, 200)]))
    ref = oracle.bias_gelu_residual(p["x"][pick], p["bias"], p["r"][pick])
    assert max_rel_floored(host(out[torch.from_numpy(pick).cuda()]), ref) < TOL
    # wide range of arguments, including the far tails of erf
    z = np.linspace(-12, 12, 4096 * 4, dtype=np.float32).reshape(4, 4096)
    zero = np.zeros(4096, np.float32)
    got = host(api.pd_bias_gelu_residual(dev_f32(z), dev_f32(zero), None))
    assert np.max(np.abs(got - oracle.bias_gelu_residual(z, zero, None))) < 2e-6
    # in place over x and over r
    o1 = out.clone()
    api.pd_bias_gelu_residual(xd, dev_f32(p["bias"]), rd, rd)
    assert torch.equal(rd, o1)


def test_rowop_errors(api):
    x = torch.zeros(4, 8, device="cuda")
    assert api._lib.pd_softmax(x.data_ptr(), x.data_ptr(), 4, 0, None) == 2        # cols == 0: PD_ERR_BAD_SHAPE
    assert api._lib.pd_softmax(x.data_ptr(), x.data_ptr(), 0, 8, None) == 0        # rows == 0: PD_OK, no launch
    assert api._lib.pd_softmax(x.data_ptr(), None, 4, 8, None) == 1                # PD_ERR_NULL_POINTER
    with pytest.raises(api.PdError, match="PD_ERR_NULL_POINTER"):
        api.pd_softmax(torch.zeros(4, 0, device="cuda"))                           # an empty tensor has no storage
    with pytest.raises(TypeError):
        api.pd_softmax(x.double())
    with pytest.raises(TypeError):
        api.pd_softmax(x.cpu())


# --------------------------------------------------------------- reducemean
@pytest.mark.parametrize("shape", [(4096, 4096), (1, 1), (3, 5), (37, 1024), (1000, 512), (129, 1028), (64, 20000), (5, 70001),
                                   (2, 1 << 20)])
def test_reducemean_against_oracle(api, shape):
    rows, cols = shape
    x = inputs.rmsnorm_inputs(rows, cols, seed=rows + cols)["x"]          # N(1, 2): the mean does not vanish
    y = Guarded((rows,), torch.float32)
    api.pd_reducemean(dev_f32(x), y.t)
    torch.cuda.synchronize()
    y.check()
    assert max_rel_floored(host(y.t), oracle.reducemean(x)) < 1e-5


def test_reducemean_unaligned_rows_and_exact_integers(api):
    # a view that starts 4 bytes into an allocation: the scalar path; integer data sums exactly and 1 / 2048 is exact
    rng = np.random.default_rng(8)
    x = rng.integers(-1000, 1001, size=(40, 2048)).astype(np.float32)
    buf = torch.empty(40 * 2048 + 1, dtype=torch.float32, device="cuda")
    xv = buf[1:].view(40, 2048)
    xv.copy_(torch.from_numpy(x))
    y = torch.empty(40, dtype=torch.float32, device="cuda")
    assert api._lib.pd_reducemean(xv.data_ptr(), y.data_ptr(), 40, 2048, None) == 0
    ref = oracle.reducemean(x)
    assert max_rel_floored(host(y), ref) < 1e-6
    assert np.array_equal(host(api.pd_reducemean(dev_f32(x))), (x.astype(np.float64).sum(axis=1) / 2048).astype(np.float32).astype(np.float64))
