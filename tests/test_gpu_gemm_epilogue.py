"""GPU parity of the contractions with fused epilogues (pd_gemm_bias_act, pd_swiglu_gemm) against the CPU
oracle through the C ABI.

The oracle side composes its plain functions (gemm, then bias + activation + residual, or SiLU(gate) * up) in
float64.  The kernels accumulate and apply the epilogue in fp32 and round once: the bound is the 2e-2 of the
bf16 contractions; fp32 output must agree to 1e-4 (GELU through its fitted tail: 1.5e-5 relative) and bf16
output to one bf16 rounding (2^-8), all relative with the denominator floored at the RMS of the oracle output."""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_03586_b200 import inputs
from parity import Guarded, dev_bf16, dev_f32, host, max_rel_floored

pytestmark = pytest.mark.gpu
TOL = 2e-2
TOL_ONE_ROUNDING = 2.0 ** -8
TOL_F32 = 1e-4


@pytest.fixture(scope="module", params=[1, 2, 0], ids=["single_cta_tiles", "cta_pair_tiles", "auto_tiles"])
def api(request):
    from paper_2511_03586_b200 import api
    api.pd_clear_device_status()
    api.pd_set_gemm_tile_mode(request.param)
    yield api
    api.pd_set_gemm_tile_mode(0)
    assert api.pd_get_device_status() == 0, "a bounded wait expired inside a tensor-core kernel"


def _oracle_bias_act(p, act, use_bias, use_residual):
    s = oracle.gemm(p["a"], p["b"])
    bias = p["bias"] if use_bias else None
    r = p["residual"] if use_residual else None
    if act == 1:
        return oracle.bias_gelu_residual(s, bias if bias is not None else np.zeros(s.shape[1]), r)
    if act == 2:
        return oracle.bias_relu_residual(s, bias, r)
    out = s if bias is None else s + bias.astype(np.float64)
    return out if r is None else out + r.astype(np.float64)


SHAPES = [(128, 256, 64), (1, 8, 8), (130, 264, 72), (300, 72, 136), (257, 1032, 200), (512, 512, 256)]


@pytest.mark.parametrize("c_dtype", [torch.bfloat16, torch.float32], ids=["bf16_out", "f32_out"])
@pytest.mark.parametrize("act", [0, 1, 2], ids=["none", "gelu", "relu"])
@pytest.mark.parametrize("shape", SHAPES)
def test_bias_act_residual_against_oracle(api, shape, act, c_dtype):
    M, N, K = shape
    p = inputs.gemm_layernorm_inputs(M, N, K, seed=M + N + K + act)   # same operand recipe: A, B, bias, residual
    c = Guarded((M, N), c_dtype)
    api.pd_gemm_bias_act(dev_bf16(p["a_bits"]), dev_bf16(p["b_bits"]), dev_f32(p["bias"]),
                         dev_bf16(p["residual_bits"]), act=act, c=c.t)
    torch.cuda.synchronize()
    c.check()
    err = max_rel_floored(host(c.t), _oracle_bias_act(p, act, True, True))
    assert err < TOL
    assert err < (TOL_F32 if c_dtype == torch.float32 else TOL_ONE_ROUNDING)


@pytest.mark.parametrize("use_bias,use_residual", [(False, False), (True, False), (False, True)])
@pytest.mark.parametrize("act", [1, 2], ids=["gelu", "relu"])
def test_optional_operands(api, act, use_bias, use_residual):
    p = inputs.gemm_layernorm_inputs(200, 328, 264, seed=7)
    c = api.pd_gemm_bias_act(dev_bf16(p["a_bits"]), dev_bf16(p["b_bits"]), dev_f32(p["bias"]) if use_bias else None,
                             dev_bf16(p["residual_bits"]) if use_residual else None, act=act, c_dtype=torch.float32)
    assert max_rel_floored(host(c), _oracle_bias_act(p, act, use_bias, use_residual)) < TOL_F32


def test_relu_is_exact_on_integers(api):
    # integer operands: every sum is exact in fp32, so ReLU(A B + bias) + residual must match bit for bit
    M, N, K = 200, 264, 136
    g = inputs.gemm_integer_inputs(M, N, K, seed=3)
    rng = np.random.default_rng(3)
    bias = rng.integers(-50, 51, size=N).astype(np.float32)
    res = rng.integers(-60, 61, size=(M, N)).astype(np.float32)
    c = api.pd_gemm_bias_act(dev_bf16(g["a_bits"][0]), dev_bf16(g["b_bits"][0]), dev_f32(bias),
                             dev_bf16(inputs.f32_to_bf16_bits(res)), act=2, c_dtype=torch.float32)
    ref = oracle.bias_relu_residual(oracle.gemm(g["a"][0], g["b"][0]), bias, res)
    assert np.array_equal(host(c), ref)
    assert (ref == res).any() and (ref != res).any()      # both sides of the kink occur


# (M, N, K): the paper's shape (256 tokens, 4096 -> 448), tiny, ragged in every dimension, and one large
# enough for the 128-column output tiles
SWIGLU_SHAPES = [(256, 448, 4096), (128, 128, 64), (1, 8, 8), (300, 200, 136), (1000, 1032, 64), (4096, 1024, 64)]


@pytest.mark.parametrize("shape", SWIGLU_SHAPES)
def test_swiglu_against_oracle(api, shape):
    M, N, K = shape
    p = inputs.swiglu_inputs(M, N, K, seed=M + N + K)
    y = Guarded((M, N), torch.bfloat16)
    api.pd_swiglu_gemm(dev_bf16(p["x_bits"]), dev_bf16(p["wg_bits"]), dev_bf16(p["wu_bits"]), y=y.t)
    torch.cuda.synchronize()
    y.check()
    ref = oracle.swiglu(oracle.gemm(p["x"], p["wg"]), oracle.gemm(p["x"], p["wu"]))
    err = max_rel_floored(host(y.t), ref)
    assert err < TOL
    assert err < TOL_ONE_ROUNDING


def test_swiglu_gate_and_up_are_not_swapped_and_saturate(api):
    # gate = 8 x (so SiLU(gate) ~ gate where positive, ~ 0 where negative), up = x: Y ~ 8 x^2 or ~ 0
    K = N = 64
    rng = np.random.default_rng(5)
    x = rng.integers(-4, 5, size=(96, K)).astype(np.float32)
    eye = np.eye(K, dtype=np.float32)
    xb = dev_bf16(inputs.f32_to_bf16_bits(x))
    y = host(api.pd_swiglu_gemm(xb, dev_bf16(inputs.f32_to_bf16_bits(8 * eye)), dev_bf16(inputs.f32_to_bf16_bits(eye))))
    ref = oracle.swiglu(8.0 * x, x)
    assert max_rel_floored(y, ref) < TOL_ONE_ROUNDING
    assert np.all(y[x < 0] > -1e-3) and np.all(np.abs(y[x < 0]) < 0.1)
    # gates below -128, where exp(-gate) overflows fp32, give zero, not NaN
    y2 = host(api.pd_swiglu_gemm(xb, dev_bf16(inputs.f32_to_bf16_bits(128 * eye)), dev_bf16(inputs.f32_to_bf16_bits(eye))))
    assert np.isfinite(y2).all() and np.all(y2[x < 0] == 0) and np.array_equal(y2[x > 0], 128.0 * x[x > 0] ** 2)


@pytest.mark.parametrize("shape", [(768, 1024, 2048), (127, 248, 3000), (64, 64, 4096), (1100, 1032, 2048), (512, 264, 8192)])
def test_split_k_over_a_cluster_matches_the_unsplit_kernel(api, shape):
    # few output tiles: under automatic tiles K is split over a cluster of 2, 4 or 8 CTAs; forced off, one CTA per tile
    M, N, K = shape
    p = inputs.gemm_layernorm_inputs(M, N, K, seed=K)
    a, b, bias, r = dev_bf16(p["a_bits"]), dev_bf16(p["b_bits"]), dev_f32(p["bias"]), dev_bf16(p["residual_bits"])
    ref = _oracle_bias_act(p, 1, True, True)
    outs = []
    for mode in (0, 1):
        api.pd_set_gemm_split_k(mode)
        try:
            c = Guarded((M, N), torch.float32)
            api.pd_gemm_bias_act(a, b, bias, r, act=1, c=c.t)
            torch.cuda.synchronize()
            c.check()
            c2 = api.pd_gemm_bias_act(a, b, bias, r, act=1, c_dtype=torch.float32)
            assert torch.equal(c.t, c2)                     # repeatable
            outs.append(host(c.t))
            assert max_rel_floored(outs[-1], ref) < TOL_F32
        finally:
            api.pd_set_gemm_split_k(0)
    assert max_rel_floored(outs[0], outs[1]) < 1e-5


def test_layer_ffn_up_launch_sampled_rows(api):
    # the layer's FFN-up launch at full size (16384 x 4096 x 1024, bias + GELU, bf16 out), under every tile mode of
    # the fixture (the layer itself takes the CTA-pair kernel): sampled rows from every part of the tile walk
    M, K, N = 16384, 1024, 4096
    p = inputs.gemm_layernorm_inputs(M, N, K, seed=11)
    c = api.pd_gemm_bias_act(dev_bf16(p["a_bits"]), dev_bf16(p["b_bits"]), dev_f32(p["bias"]), None, act=api.ACT_GELU)
    pick = np.unique(np.concatenate([[0, 127, 128, 255, 256, M - 257, M - 256, M - 129, M - 128, M - 1],
                                     np.random.default_rng(11).integers(0, M, 60)]))
    ref = oracle.bias_gelu_residual(oracle.gemm(p["a"][pick], p["b"]), p["bias"], None)
    err = max_rel_floored(host(c[torch.from_numpy(pick).cuda()]), ref)
    assert err < TOL
    assert err < TOL_ONE_ROUNDING
    assert bool(torch.isfinite(c.float()).all())


def test_argument_errors(api):
    from paper_2511_03586_b200.api import PdError
    a = torch.zeros(64, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(PdError) as e:
        api.pd_gemm_bias_act(a, a, act=3)
    assert e.value.status == 2          # PD_ERR_BAD_SHAPE
    odd = torch.zeros(64, 60, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(PdError) as e:
        api.pd_swiglu_gemm(a, odd, odd)
    assert e.value.status == 4          # PD_ERR_ALIGNMENT: N not a multiple of 8
    assert api._lib.pd_swiglu_gemm(a.data_ptr(), None, a.data_ptr(), a.data_ptr(), 64, 64, 64, None) == 1
    assert api._lib.pd_swiglu_gemm(a.data_ptr(), a.data_ptr(), a.data_ptr(), a.data_ptr(), 0, 64, 64, None) == 0
