"""The configured workloads write their distributions as N(a, b) without saying whether b is a standard deviation
or a variance.  Every other test reads b as the standard deviation.  Here each operator is run once on inputs drawn
under the other reading (standard deviation sqrt(b)) and held to the same tolerance, to show that the parity
results do not hinge on that choice.  The encoder layer is run at hidden size 64: with weights of standard
deviation sqrt(0.02) = 0.14 the activations grow with the hidden size (variance 0.02 x hidden), and from hidden
128 on the bf16 storage of Q and K alone moves the attention probabilities by more than the 2e-2 tolerance
(measured: 2.7e-2 at hidden 128), which is why 0.02 is read as a standard deviation in the first place."""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_03586_b200 import inputs
from parity import dev_bf16, dev_f32, host, max_rel, max_rel_floored

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def api():
    from paper_2511_03586_b200 import api
    api.pd_clear_device_status()
    yield api
    assert api.pd_get_device_status() == 0


def test_row_operators_under_the_variance_reading(api):
    x = inputs.softmax_inputs(256, 512, seed=0, sigma=np.sqrt(4.0))["x"]
    assert max_rel(host(api.pd_softmax(dev_f32(x))), oracle.softmax(x)) < 1e-5
    p = inputs.layernorm_inputs(512, 1024, seed=0)
    xv = (1.0 + (p["x"] - 1.0) * (np.sqrt(2.0) / 2.0)).astype(np.float32)
    bv = (p["beta"] * (np.sqrt(0.1) / 0.1)).astype(np.float32)
    y = api.pd_layernorm(dev_f32(xv), dev_f32(p["gamma"]), dev_f32(bv), p["eps"])
    assert max_rel_floored(host(y), oracle.layernorm(xv, p["gamma"], bv, np.float32(p["eps"]))) < 1e-5
    q = inputs.bias_gelu_residual_inputs(256, 4096, seed=0)
    bias = (q["bias"] * (np.sqrt(0.02) / 0.02)).astype(np.float32)
    out = api.pd_bias_gelu_residual(dev_f32(q["x"]), dev_f32(bias), dev_f32(q["r"]))
    assert max_rel_floored(host(out), oracle.bias_gelu_residual(q["x"], bias, q["r"])) < 1e-5


def test_gemm_under_the_variance_reading(api):
    M, N, K = 512, 1024, 1024
    p = inputs.gemm_inputs(M, N, K, seed=0, sigma=K ** -0.25)      # variance 1/sqrt(K)
    a, b = dev_bf16(p["a_bits"][0]), dev_bf16(p["b_bits"][0])
    ref = oracle.gemm(p["a"][0], p["b"][0])
    assert max_rel_floored(host(api.pd_gemm_bf16(a, b, c_dtype=torch.float32)), ref) < 1e-5
    assert max_rel_floored(host(api.pd_gemm_bf16(a, b)), ref) < 2e-2


def test_small_layer_under_the_variance_reading(api):
    shape = inputs.EncoderLayerShape(batch=2, seq=128, hidden=64, heads=1, ffn=128)
    p = inputs.encoder_layer_inputs(shape, seed=0, w_sigma=float(np.sqrt(0.02)))
    mats = ("w_qkv", "w_o", "w_ffn1", "w_ffn2")
    vecs = ("b_qkv", "b_o", "b_ffn1", "b_ffn2", "ln1_gamma", "ln1_beta", "ln2_gamma", "ln2_beta")
    params = api.EncoderLayerParams(**{m: dev_bf16(p[m + "_bits"]) for m in mats}, **{v: dev_f32(p[v]) for v in vecs})
    y = api.pd_encoder_layer_fwd(params, dev_bf16(p["x_bits"]), batch=shape.batch, seq=shape.seq, heads=shape.heads)
    w = {m: inputs.bf16_bits_to_f32(p[m + "_bits"]) for m in mats}
    ref = oracle.encoder_layer(inputs.bf16_bits_to_f32(p["x_bits"]), w["w_qkv"], p["b_qkv"], w["w_o"], p["b_o"],
                               w["w_ffn1"], p["b_ffn1"], w["w_ffn2"], p["b_ffn2"], p["ln1_gamma"], p["ln1_beta"],
                               p["ln2_gamma"], p["ln2_beta"], batch=shape.batch, seq=shape.seq, heads=shape.heads,
                               ln_eps=np.float32(shape.ln_eps))
    assert max_rel_floored(host(y), ref) < 2e-2
