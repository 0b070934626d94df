"""Seeded synthetic inputs for the encoder-layer operator kernels.

This module only draws random numbers and casts them; it holds none of the
operators' arithmetic.  Both the CUDA path and the CPU oracle are fed from the
host arrays produced here, so that the two see bit-identical inputs.

Conventions
-----------
* ``numpy.random.Generator(PCG64(seed))``; tensors are drawn in the order the
  functions below list them, in float64, then cast to float32.
* In ``N(a, b)`` the second parameter is the standard deviation.
* bf16 tensors are float32 values rounded to nearest-even onto the bf16 grid
  and returned as ``uint16`` bit patterns (numpy has no bf16 dtype);
  ``bf16_bits_to_f32`` widens them back exactly.
* Shapes follow the paper's operator table (Table "ML operators optimized using
  PerfLLM": softmax 24576x512, layernorm 16384x1024 and 4096x4096,
  matmul/bmm) and BERT-large (hidden 1024, 16 heads of 64, FFN 4096, seq 512).
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


# --------------------------------------------------------------------------
# bf16 <-> fp32 bit casts (round-to-nearest-even); storage format only.
# --------------------------------------------------------------------------
def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32 values to bf16 (nearest-even) and return uint16 bit patterns."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    rounded = u + np.uint32(0x7FFF) + lsb
    out = (rounded >> np.uint32(16)).astype(np.uint16)
    nan = np.isnan(a)
    if nan.any():
        out[nan] = np.uint16(0x7FC0)
    return out


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Widen uint16 bf16 bit patterns to float32 (exact)."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(seed))


def _normal(rng, shape, mean, sigma) -> np.ndarray:
    return (mean + sigma * rng.standard_normal(shape)).astype(np.float32)


def _uniform(rng, shape, lo, hi) -> np.ndarray:
    return rng.uniform(lo, hi, size=shape).astype(np.float32)


# --------------------------------------------------------------------------
# Per-operator inputs
# --------------------------------------------------------------------------
def softmax_inputs(rows: int, cols: int, seed: int = 0, sigma: float = 4.0):
    """X fp32 [rows, cols] ~ N(0, sigma)."""
    rng = _rng(seed)
    return {"x": _normal(rng, (rows, cols), 0.0, sigma)}


def layernorm_inputs(rows: int, cols: int, seed: int = 0):
    """X ~ N(1, 2); gamma ~ U(0.5, 1.5); beta ~ N(0, 0.1); all fp32."""
    rng = _rng(seed)
    x = _normal(rng, (rows, cols), 1.0, 2.0)
    gamma = _uniform(rng, (cols,), 0.5, 1.5)
    beta = _normal(rng, (cols,), 0.0, 0.1)
    return {"x": x, "gamma": gamma, "beta": beta, "eps": 1e-5}


def rmsnorm_inputs(rows: int, cols: int, seed: int = 0):
    """X ~ N(1, 2); gamma ~ U(0.5, 1.5); fp32 (the layernorm recipe without beta)."""
    rng = _rng(seed)
    return {"x": _normal(rng, (rows, cols), 1.0, 2.0), "gamma": _uniform(rng, (cols,), 0.5, 1.5), "eps": 1e-5}


def bias_gelu_residual_inputs(rows: int, cols: int, seed: int = 0):
    """X, R ~ N(0, 1) fp32 [rows, cols]; bias ~ N(0, 0.02) fp32 [cols]."""
    rng = _rng(seed)
    x = _normal(rng, (rows, cols), 0.0, 1.0)
    r = _normal(rng, (rows, cols), 0.0, 1.0)
    bias = _normal(rng, (cols,), 0.0, 0.02)
    return {"x": x, "r": r, "bias": bias}


def gemm_inputs(M: int, N: int, K: int, seed: int = 0, batch: int = 1,
                b_is_nk: bool = False, sigma: float | None = None):
    """A [batch, M, K], B [batch, K, N] (or [batch, N, K] when ``b_is_nk``)
    ~ N(0, 1/sqrt(K)), rounded to bf16.  Returns bit patterns and their exact
    float32 widenings."""
    rng = _rng(seed)
    s = (1.0 / np.sqrt(K)) if sigma is None else sigma
    a = _normal(rng, (batch, M, K), 0.0, s)
    bshape = (batch, N, K) if b_is_nk else (batch, K, N)
    b = _normal(rng, bshape, 0.0, s)
    a_bits, b_bits = f32_to_bf16_bits(a), f32_to_bf16_bits(b)
    return {"a_bits": a_bits, "b_bits": b_bits,
            "a": bf16_bits_to_f32(a_bits), "b": bf16_bits_to_f32(b_bits)}


def gemm_integer_inputs(M: int, N: int, K: int, seed: int = 0, batch: int = 1,
                        b_is_nk: bool = False, lo: int = -8, hi: int = 8):
    """Integer-valued A, B in [lo, hi]: exact in bf16, and every partial sum of
    a K <= 4096 dot product stays below 2**24, so fp32 accumulation is exact."""
    rng = _rng(seed)
    a = rng.integers(lo, hi + 1, size=(batch, M, K)).astype(np.float32)
    bshape = (batch, N, K) if b_is_nk else (batch, K, N)
    b = rng.integers(lo, hi + 1, size=bshape).astype(np.float32)
    return {"a_bits": f32_to_bf16_bits(a), "b_bits": f32_to_bf16_bits(b), "a": a, "b": b}


def gemm_layernorm_inputs(M: int, N: int, K: int, seed: int = 0, bias_mean: float = 0.0):
    """Operands of a projection followed by residual add and LayerNorm: A [M, K], B [K, N] ~ N(0, 1/sqrt(K))
    and residual [M, N] ~ N(0, 1), rounded to bf16; bias ~ N(bias_mean, 0.1), gamma ~ U(0.5, 1.5),
    beta ~ N(0, 0.1) in fp32."""
    rng = _rng(seed)
    s = 1.0 / np.sqrt(K)
    a_bits = f32_to_bf16_bits(_normal(rng, (M, K), 0.0, s))
    b_bits = f32_to_bf16_bits(_normal(rng, (K, N), 0.0, s))
    r_bits = f32_to_bf16_bits(_normal(rng, (M, N), 0.0, 1.0))
    return {"a_bits": a_bits, "b_bits": b_bits, "residual_bits": r_bits,
            "a": bf16_bits_to_f32(a_bits), "b": bf16_bits_to_f32(b_bits), "residual": bf16_bits_to_f32(r_bits),
            "bias": _normal(rng, (N,), bias_mean, 0.1), "gamma": _uniform(rng, (N,), 0.5, 1.5),
            "beta": _normal(rng, (N,), 0.0, 0.1), "eps": 1e-5}


def swiglu_inputs(M: int, N: int, K: int, seed: int = 0):
    """Operands of a SwiGLU projection: X [M, K] ~ N(0, 1), gate and up weights [K, N] ~ N(0, 1/sqrt(K)),
    all rounded to bf16 (bit patterns and their exact float32 widenings)."""
    rng = _rng(seed)
    x_bits = f32_to_bf16_bits(_normal(rng, (M, K), 0.0, 1.0))
    wg_bits = f32_to_bf16_bits(_normal(rng, (K, N), 0.0, 1.0 / np.sqrt(K)))
    wu_bits = f32_to_bf16_bits(_normal(rng, (K, N), 0.0, 1.0 / np.sqrt(K)))
    return {"x_bits": x_bits, "wg_bits": wg_bits, "wu_bits": wu_bits, "x": bf16_bits_to_f32(x_bits),
            "wg": bf16_bits_to_f32(wg_bits), "wu": bf16_bits_to_f32(wu_bits)}


@dataclass(frozen=True)
class EncoderLayerShape:
    batch: int = 32
    seq: int = 512
    hidden: int = 1024
    heads: int = 16
    ffn: int = 4096
    ln_eps: float = 1e-5

    @property
    def tokens(self) -> int:
        return self.batch * self.seq

    @property
    def head_dim(self) -> int:
        return self.hidden // self.heads

    def gemm_flops(self) -> float:
        """Flops of the six dense contractions of one forward pass (2*M*N*K each)."""
        T, H, F, S, d = self.tokens, self.hidden, self.ffn, self.seq, self.head_dim
        qkv = 2.0 * T * H * 3 * H
        attn = 2 * (2.0 * self.batch * self.heads * S * S * d)
        out = 2.0 * T * H * H
        ffn = 2 * (2.0 * T * H * F)
        return qkv + attn + out + ffn


def encoder_layer_inputs(shape: EncoderLayerShape, seed: int = 0, w_sigma: float = 0.02):
    """Post-LN BERT-shaped encoder layer: X bf16 [tokens, hidden] ~ N(0, 1);
    weight matrices bf16 ~ N(0, w_sigma) stored [in, out] row-major, the QKV
    matrix packed as column blocks [Q | K | V] with heads contiguous inside each
    block; biases fp32 ~ N(0, 0.02); gamma ~ U(0.5, 1.5); beta ~ N(0, 0.1)."""
    rng = _rng(seed)
    T, H, F = shape.tokens, shape.hidden, shape.ffn
    out = {}
    out["x_bits"] = f32_to_bf16_bits(_normal(rng, (T, H), 0.0, 1.0))
    for name, shp in (("w_qkv", (H, 3 * H)), ("w_o", (H, H)), ("w_ffn1", (H, F)), ("w_ffn2", (F, H))):
        out[name + "_bits"] = f32_to_bf16_bits(_normal(rng, shp, 0.0, w_sigma))
    for name, n in (("b_qkv", 3 * H), ("b_o", H), ("b_ffn1", F), ("b_ffn2", H)):
        out[name] = _normal(rng, (n,), 0.0, 0.02)
    for i in (1, 2):
        out[f"ln{i}_gamma"] = _uniform(rng, (H,), 0.5, 1.5)
        out[f"ln{i}_beta"] = _normal(rng, (H,), 0.0, 0.1)
    return out
