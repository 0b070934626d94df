"""Seeded input generators: determinism, distributions, exact bf16 rounding."""
import numpy as np
import pytest

from paper_2511_03586_b200 import inputs


def test_bf16_round_to_nearest_even_matches_torch():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(0)
    a = np.concatenate([rng.normal(0, 1, 4096), rng.normal(0, 1e-3, 1024), rng.normal(0, 1e4, 1024),
                        [0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895314e38]]).astype(np.float32)
    bits = inputs.f32_to_bf16_bits(a)
    ref = torch.from_numpy(a).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(bits, ref)
    back = inputs.bf16_bits_to_f32(bits)
    assert np.array_equal(back, torch.from_numpy(a).to(torch.bfloat16).float().numpy())
    # ties go to the even mantissa: 1 + 2^-8 -> 1, 1 + 3*2^-8 -> 1 + 2^-6
    assert inputs.bf16_bits_to_f32(inputs.f32_to_bf16_bits(np.float32([1.00390625, 1.01171875]))).tolist() == [1.0, 1.015625]


def test_generators_are_seeded_and_shaped():
    a = inputs.softmax_inputs(8, 512, seed=0)["x"]
    b = inputs.softmax_inputs(8, 512, seed=0)["x"]
    c = inputs.softmax_inputs(8, 512, seed=1)["x"]
    assert a.dtype == np.float32 and a.shape == (8, 512)
    assert np.array_equal(a, b) and not np.array_equal(a, c)
    assert 3.5 < a.std() < 4.5                       # N(0, 4): 4 is the standard deviation
    ln = inputs.layernorm_inputs(64, 1024)
    assert 0.9 < ln["x"].mean() < 1.1 and 1.9 < ln["x"].std() < 2.1
    assert ln["gamma"].min() >= 0.5 and ln["gamma"].max() <= 1.5 and ln["beta"].shape == (1024,)
    g = inputs.gemm_inputs(16, 24, 1024)
    assert g["a_bits"].dtype == np.uint16 and g["a"].shape == (1, 16, 1024) and g["b"].shape == (1, 1024, 24)
    assert abs(g["a"].std() - 1 / 32) < 2e-3
    assert np.array_equal(inputs.f32_to_bf16_bits(g["a"]), g["a_bits"])   # values sit on the bf16 grid
    gi = inputs.gemm_integer_inputs(4, 4, 64, b_is_nk=True)
    assert gi["b"].shape == (1, 4, 64) and np.array_equal(gi["a"], np.round(gi["a"])) and np.abs(gi["a"]).max() <= 8


def test_encoder_layer_inputs():
    shp = inputs.EncoderLayerShape(batch=2, seq=8, hidden=64, heads=4, ffn=128)
    p = inputs.encoder_layer_inputs(shp, seed=3)
    assert p["x_bits"].shape == (16, 64) and p["w_qkv_bits"].shape == (64, 192)
    assert p["w_ffn1_bits"].shape == (64, 128) and p["w_ffn2_bits"].shape == (128, 64)
    assert p["b_qkv"].shape == (192,) and p["ln2_beta"].shape == (64,)
    big = inputs.EncoderLayerShape()
    assert abs(big.gemm_flops() - 446.68e9) < 0.01e9
