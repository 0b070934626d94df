"""ctypes front end of the CPU oracle (``pd_oracle.cpp``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by the smoke check and by the
benchmark's CPU-baseline leg.  It imports nothing from the CUDA package.

All functions take numpy arrays (any float dtype; widened to float64 here, which
is exact for float32 and bf16-valued inputs) and return float64 arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pd_oracle.cpp")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None

_D = ctypes.POINTER(ctypes.c_double)
_I64 = ctypes.c_int64


def build(force: bool = False) -> str:
    """Compile the oracle with g++ -O2 (no fast-math) into ``oracle/liboracle.so``."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["g++", "-std=c++17", "-O2", "-fPIC", "-shared", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.oracle_softmax.argtypes = [_D, _D, _I64, _I64]
        lib.oracle_layernorm.argtypes = [_D, _D, _D, _D, _I64, _I64, ctypes.c_double]
        lib.oracle_rmsnorm.argtypes = [_D, _D, _D, _I64, _I64, ctypes.c_double]
        lib.oracle_rmsnorm.restype = ctypes.c_int
        lib.oracle_bias_gelu_residual.argtypes = [_D, _D, _D, _D, _I64, _I64]
        lib.oracle_reducemean.argtypes = [_D, _D, _I64, _I64]
        lib.oracle_reducemean.restype = ctypes.c_int
        lib.oracle_bias_relu_residual.argtypes = [_D, _D, _D, _D, _I64, _I64]
        lib.oracle_bias_relu_residual.restype = ctypes.c_int
        lib.oracle_swiglu.argtypes = [_D, _D, _D, _I64]
        lib.oracle_swiglu.restype = ctypes.c_int
        lib.oracle_gemm.argtypes = [_D, _D, _D, _I64, _I64, _I64]
        lib.oracle_attention.argtypes = [_D, _D, _D, _I64, _I64, _I64, _I64]
        lib.oracle_encoder_layer.argtypes = [_I64] * 5 + [ctypes.c_double] + [_D] * 18
        for name in ("oracle_softmax", "oracle_layernorm", "oracle_bias_gelu_residual", "oracle_gemm",
                     "oracle_attention", "oracle_encoder_layer"):
            getattr(lib, name).restype = ctypes.c_int
        _lib = lib
    return _lib


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float64)


def _p(a):
    return None if a is None else a.ctypes.data_as(_D)


def _check(rc: int, name: str):
    if rc != 0:
        raise ValueError(f"{name} rejected its arguments (code {rc})")


def softmax(x) -> np.ndarray:
    x = _f64(x)
    rows, cols = x.shape
    y = np.empty_like(x)
    _check(_load().oracle_softmax(_p(x), _p(y), rows, cols), "oracle_softmax")
    return y


def layernorm(x, gamma, beta, eps: float) -> np.ndarray:
    x, gamma, beta = _f64(x), _f64(gamma), _f64(beta)
    rows, cols = x.shape
    assert gamma.shape == (cols,) and beta.shape == (cols,)
    y = np.empty_like(x)
    _check(_load().oracle_layernorm(_p(x), _p(gamma), _p(beta), _p(y), rows, cols, float(eps)), "oracle_layernorm")
    return y


def rmsnorm(x, gamma, eps: float) -> np.ndarray:
    x, gamma = _f64(x), _f64(gamma)
    rows, cols = x.shape
    assert gamma.shape == (cols,)
    y = np.empty_like(x)
    _check(_load().oracle_rmsnorm(_p(x), _p(gamma), _p(y), rows, cols, float(eps)), "oracle_rmsnorm")
    return y


def reducemean(x) -> np.ndarray:
    x = _f64(x)
    rows, cols = x.shape
    y = np.empty(rows, dtype=np.float64)
    _check(_load().oracle_reducemean(_p(x), _p(y), rows, cols), "oracle_reducemean")
    return y


def bias_gelu_residual(x, bias, r=None) -> np.ndarray:
    x, bias = _f64(x), _f64(bias)
    rows, cols = x.shape
    assert bias.shape == (cols,)
    r = None if r is None else _f64(r)
    assert r is None or r.shape == x.shape
    out = np.empty_like(x)
    _check(_load().oracle_bias_gelu_residual(_p(x), _p(bias), _p(r), _p(out), rows, cols), "oracle_bias_gelu_residual")
    return out


def bias_relu_residual(x, bias=None, r=None) -> np.ndarray:
    x = _f64(x)
    rows, cols = x.shape
    bias = None if bias is None else _f64(bias)
    r = None if r is None else _f64(r)
    assert bias is None or bias.shape == (cols,)
    assert r is None or r.shape == x.shape
    out = np.empty_like(x)
    _check(_load().oracle_bias_relu_residual(_p(x), _p(bias), _p(r), _p(out), rows, cols), "oracle_bias_relu_residual")
    return out


def swiglu(g, u) -> np.ndarray:
    """SiLU(g) * u element by element."""
    g, u = _f64(g), _f64(u)
    assert g.shape == u.shape
    out = np.empty_like(g)
    _check(_load().oracle_swiglu(_p(g), _p(u), _p(out), g.size), "oracle_swiglu")
    return out


def gemm(a, b) -> np.ndarray:
    """C[M,N] = A[M,K] @ B[K,N]; 3-D inputs are treated as a batch of independent problems."""
    a, b = _f64(a), _f64(b)
    if a.ndim == 3:
        return np.stack([gemm(a[i], b[i]) for i in range(a.shape[0])])
    M, K = a.shape
    K2, N = b.shape
    assert K == K2
    c = np.empty((M, N), dtype=np.float64)
    _check(_load().oracle_gemm(_p(a), _p(b), _p(c), M, N, K), "oracle_gemm")
    return c


def attention(qkv, batch: int, seq: int, heads: int, head_dim: int, return_probs: bool = False):
    qkv = _f64(qkv)
    hidden = heads * head_dim
    assert qkv.shape == (batch * seq, 3 * hidden)
    ctx = np.empty((batch * seq, hidden), dtype=np.float64)
    probs = np.empty((batch, heads, seq, seq), dtype=np.float64) if return_probs else None
    _check(_load().oracle_attention(_p(qkv), _p(ctx), _p(probs), batch, seq, heads, head_dim), "oracle_attention")
    return (ctx, probs) if return_probs else ctx


def encoder_layer(x, w_qkv, b_qkv, w_o, b_o, w_ffn1, b_ffn1, w_ffn2, b_ffn2,
                  ln1_gamma, ln1_beta, ln2_gamma, ln2_beta, *, batch: int, seq: int, heads: int,
                  ln_eps: float = 1e-5, return_intermediates: bool = False):
    x = _f64(x)
    T, H = x.shape
    assert T == batch * seq
    w_qkv, w_o, w_ffn1, w_ffn2 = _f64(w_qkv), _f64(w_o), _f64(w_ffn1), _f64(w_ffn2)
    F = w_ffn1.shape[1]
    assert w_qkv.shape == (H, 3 * H) and w_o.shape == (H, H) and w_ffn1.shape == (H, F) and w_ffn2.shape == (F, H)
    vecs = [_f64(v) for v in (b_qkv, b_o, b_ffn1, b_ffn2, ln1_gamma, ln1_beta, ln2_gamma, ln2_beta)]
    b_qkv, b_o, b_ffn1, b_ffn2, ln1_gamma, ln1_beta, ln2_gamma, ln2_beta = vecs
    assert b_qkv.shape == (3 * H,) and b_o.shape == (H,) and b_ffn1.shape == (F,) and b_ffn2.shape == (H,)
    y = np.empty((T, H), dtype=np.float64)
    inter = {}
    if return_intermediates:
        inter = {"qkv": np.empty((T, 3 * H)), "ctx": np.empty((T, H)), "h1": np.empty((T, H)),
                 "mid": np.empty((T, F))}
    rc = _load().oracle_encoder_layer(
        batch, seq, H, heads, F, float(ln_eps), _p(x), _p(w_qkv), _p(b_qkv), _p(w_o), _p(b_o),
        _p(w_ffn1), _p(b_ffn1), _p(w_ffn2), _p(b_ffn2), _p(ln1_gamma), _p(ln1_beta), _p(ln2_gamma),
        _p(ln2_beta), _p(y), _p(inter.get("qkv")), _p(inter.get("ctx")), _p(inter.get("h1")),
        _p(inter.get("mid")))
    _check(rc, "oracle_encoder_layer")
    return (y, inter) if return_intermediates else y
