"""GPU parity of pd_gemm_bias_residual_layernorm against the CPU oracle through the C ABI.

The oracle side is the plain composition gemm -> + bias + residual -> layernorm in
float64.  The kernel keeps the sum and the statistics in fp32 and rounds only the
result to bf16, so besides the 2e-2 bound of the bf16 contractions the outputs
must sit within one bf16 rounding (2^-8 relative, denominator floored at the RMS
of the oracle output) of the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_03586_b200 import inputs
from parity import Guarded, dev_bf16, dev_f32, host, max_rel_floored

pytestmark = pytest.mark.gpu
TOL = 2e-2
TOL_ONE_ROUNDING = 2.0 ** -8


@pytest.fixture(scope="module")
def api():
    from paper_2511_03586_b200 import api
    api.pd_clear_device_status()
    yield api
    assert api.pd_get_device_status() == 0, "a bounded wait expired inside a tensor-core kernel"


def _oracle(p, use_bias=True, use_residual=True):
    s = oracle.gemm(p["a"], p["b"])
    if use_bias:
        s = s + p["bias"].astype(np.float64)
    if use_residual:
        s = s + p["residual"].astype(np.float64)
    return oracle.layernorm(s, p["gamma"], p["beta"], np.float32(p["eps"]))


def _run(api, p, use_bias=True, use_residual=True):
    M, N = p["a"].shape[0], p["b"].shape[1]
    y = Guarded((M, N), torch.bfloat16)
    api.pd_gemm_bias_residual_layernorm(dev_bf16(p["a_bits"]), dev_bf16(p["b_bits"]),
                                        dev_f32(p["bias"]) if use_bias else None,
                                        dev_bf16(p["residual_bits"]) if use_residual else None,
                                        dev_f32(p["gamma"]), dev_f32(p["beta"]), p["eps"], y=y.t)
    torch.cuda.synchronize()
    y.check()
    return host(y.t)


# (M, N, K): clusters of 1..8 CTAs, ragged row blocks, one and many k-blocks, ragged k,
# and enough row blocks that every cluster walks several of them
SHAPES = [(128, 256, 64), (1, 256, 8), (300, 512, 136), (1000, 768, 200), (257, 1024, 1024), (77, 2048, 72),
          (130, 1280, 64), (14300, 1024, 64), (9000, 512, 64), (20000, 256, 32)]


@pytest.mark.parametrize("shape", SHAPES)
def test_against_oracle(api, shape):
    M, N, K = shape
    p = inputs.gemm_layernorm_inputs(M, N, K, seed=M + N + K)
    err = max_rel_floored(_run(api, p), _oracle(p))
    assert err < TOL
    assert err < TOL_ONE_ROUNDING


# The layer's two LayerNorm launches at full size: output projection (K = 1024) and FFN down (K = 4096), 16384 rows
# of 1024 columns.  The oracle is run on sampled rows from every part of the walk over the row blocks (first and
# last block, block edges, a random spread): a row's result depends on that row of A and of the residual only.
@pytest.mark.parametrize("K", [1024, 4096])
def test_layer_shapes_sampled_rows(api, K):
    M, N = 16384, 1024
    p = inputs.gemm_layernorm_inputs(M, N, K, seed=K)
    y = api.pd_gemm_bias_residual_layernorm(dev_bf16(p["a_bits"]), dev_bf16(p["b_bits"]), dev_f32(p["bias"]),
                                            dev_bf16(p["residual_bits"]), dev_f32(p["gamma"]), dev_f32(p["beta"]),
                                            p["eps"])
    pick = np.unique(np.concatenate([[0, 31, 32, 127, 128, M - 129, M - 128, M - 33, M - 1],
                                     np.random.default_rng(K).integers(0, M, 60)]))
    s = oracle.gemm(p["a"][pick], p["b"]) + p["bias"].astype(np.float64) + p["residual"][pick].astype(np.float64)
    ref = oracle.layernorm(s, p["gamma"], p["beta"], np.float32(p["eps"]))
    err = max_rel_floored(host(y[torch.from_numpy(pick).cuda()]), ref)
    assert err < TOL
    assert err < TOL_ONE_ROUNDING
    assert bool(torch.isfinite(y.float()).all())


@pytest.mark.parametrize("use_bias,use_residual", [(False, False), (True, False), (False, True)])
def test_optional_operands(api, use_bias, use_residual):
    p = inputs.gemm_layernorm_inputs(333, 768, 264, seed=5)
    err = max_rel_floored(_run(api, p, use_bias, use_residual), _oracle(p, use_bias, use_residual))
    assert err < TOL_ONE_ROUNDING


def test_large_common_offset(api):
    # a row mean 50 standard deviations away from zero must not cost the variance its precision
    p = inputs.gemm_layernorm_inputs(400, 1024, 128, seed=9, bias_mean=70.0)
    err = max_rel_floored(_run(api, p), _oracle(p))
    assert err < TOL_ONE_ROUNDING


def test_constant_rows_give_beta(api):
    # A = 0, no residual, constant bias: every row is constant, the normalised value is 0 and Y = beta
    p = inputs.gemm_layernorm_inputs(200, 512, 64, seed=2)
    p["a_bits"][:] = 0
    p["a"][:] = 0
    p["bias"][:] = 3.25
    got = _run(api, p, use_residual=False)
    expect = inputs.bf16_bits_to_f32(inputs.f32_to_bf16_bits(p["beta"])).astype(np.float64)
    assert np.array_equal(got, np.broadcast_to(expect, got.shape))


def test_repeatable_and_matches_unfused_kernels(api):
    M, N, K = 2000, 1024, 512
    p = inputs.gemm_layernorm_inputs(M, N, K, seed=1)
    a, b, r = dev_bf16(p["a_bits"]), dev_bf16(p["b_bits"]), dev_bf16(p["residual_bits"])
    bias, g, be = dev_f32(p["bias"]), dev_f32(p["gamma"]), dev_f32(p["beta"])
    y1 = api.pd_gemm_bias_residual_layernorm(a, b, bias, r, g, be, p["eps"])
    y2 = api.pd_gemm_bias_residual_layernorm(a, b, bias, r, g, be, p["eps"])
    assert torch.equal(y1, y2)
    # the library's separate kernels (fp32 GEMM output, fp32 LayerNorm) agree to one bf16 rounding
    s = api.pd_gemm_bf16(a, b, c_dtype=torch.float32) + bias + r.float()
    z = api.pd_layernorm(s.contiguous(), g, be, p["eps"])
    assert max_rel_floored(host(y1), host(z)) < TOL_ONE_ROUNDING


def test_graph_replay_and_changing_cluster_sizes(api):
    # Launches of different shapes (clusters of 4, 1, 8 and 2 CTAs) captured into one CUDA graph and replayed give
    # the eager results every time.
    shapes = [(1500, 1024, 128), (700, 256, 64), (520, 2048, 64), (3000, 512, 192)]
    ps = [inputs.gemm_layernorm_inputs(M, N, K, seed=11 + i) for i, (M, N, K) in enumerate(shapes)]
    args = [(dev_bf16(p["a_bits"]), dev_bf16(p["b_bits"]), dev_f32(p["bias"]), dev_bf16(p["residual_bits"]),
             dev_f32(p["gamma"]), dev_f32(p["beta"]), p["eps"]) for p in ps]
    eager = [api.pd_gemm_bias_residual_layernorm(*a) for a in args]
    for p, y in zip(ps, eager):
        assert max_rel_floored(host(y), _oracle(p)) < TOL_ONE_ROUNDING
    outs = [torch.empty_like(y) for y in eager]
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            for a, o in zip(args, outs):
                api.pd_gemm_bias_residual_layernorm(*a, y=o)
    torch.cuda.current_stream().wait_stream(side)
    for _ in range(3):
        for o in outs:
            o.zero_()
        graph.replay()
        torch.cuda.synchronize()
        for y, o in zip(eager, outs):
            assert torch.equal(y, o)


def test_argument_errors(api):
    from paper_2511_03586_b200.api import PdError
    p = inputs.gemm_layernorm_inputs(64, 256, 64, seed=0)
    a, r = dev_bf16(p["a_bits"]), dev_bf16(p["residual_bits"])
    g, be, bias = dev_f32(p["gamma"]), dev_f32(p["beta"]), dev_f32(p["bias"])
    b_bad = torch.zeros(64, 384, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(PdError) as e:
        api.pd_gemm_bias_residual_layernorm(a, b_bad, None, None, dev_f32(np.ones(384)), dev_f32(np.ones(384)), 1e-5)
    assert e.value.status == 3                                          # PD_ERR_UNSUPPORTED
    big = torch.zeros(64, 2304, dtype=torch.bfloat16, device="cuda")      # more than 8 column tiles
    with pytest.raises(PdError) as e:
        api.pd_gemm_bias_residual_layernorm(a, big, None, None, dev_f32(np.ones(2304)), dev_f32(np.ones(2304)), 1e-5)
    assert e.value.status == 3
    # M = 0 is a no-op (raw call: an empty tensor has no address to pass)
    bd = dev_bf16(p["b_bits"])
    st = api._lib.pd_gemm_bias_residual_layernorm(a.data_ptr(), bd.data_ptr(), None, None, g.data_ptr(), be.data_ptr(),
                                                  r.data_ptr(), 0, 256, 64, 1e-5, None)
    assert st == 0
