"""Pins for the CPU oracle's contraction, attention and encoder-layer functions.

Expected values come from exact integer brute force, selector matrices,
algebraic identities, degenerate cases with a closed form, and float64 library
routines of torch; never from the CUDA path.
"""
import math

import numpy as np
import pytest

import oracle


# --------------------------------------------------------------------- gemm
def test_gemm_exact_integer_brute_force():
    rng = np.random.default_rng(11)
    for (M, N, K) in ((1, 1, 1), (3, 5, 7), (4, 2, 9), (6, 6, 1)):
        a = rng.integers(-8, 9, size=(M, K))
        b = rng.integers(-8, 9, size=(K, N))
        expect = [[sum(int(a[m, k]) * int(b[k, n]) for k in range(K)) for n in range(N)] for m in range(M)]
        got = oracle.gemm(a, b)
        assert got.shape == (M, N)
        assert np.array_equal(got, np.array(expect, dtype=np.float64))


def test_gemm_identity_and_selectors():
    rng = np.random.default_rng(12)
    b = rng.normal(size=(5, 8))
    assert np.array_equal(oracle.gemm(np.eye(5), b), b)
    a = rng.normal(size=(4, 5))
    assert np.array_equal(oracle.gemm(a, np.eye(5)), a)
    # E_ij (single one at row i, col j) picks row j of B into row i of C
    for i, j in ((0, 4), (3, 1)):
        e = np.zeros((4, 5)); e[i, j] = 1.0
        c = oracle.gemm(e, b)
        expect = np.zeros((4, 8)); expect[i] = b[j]
        assert np.array_equal(c, expect)


def test_gemm_is_not_transposed_and_linear():
    rng = np.random.default_rng(13)
    a1, a2 = rng.normal(size=(3, 6)), rng.normal(size=(3, 6))
    b = rng.normal(size=(6, 4))
    np.testing.assert_allclose(oracle.gemm(a1 + a2, b), oracle.gemm(a1, b) + oracle.gemm(a2, b), rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(oracle.gemm(a1, b), (oracle.gemm(b.T.copy(), a1.T.copy())).T, rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(oracle.gemm(a1, b), a1 @ b, rtol=1e-13, atol=1e-15)


def test_gemm_batched_problems_are_independent():
    rng = np.random.default_rng(14)
    a, b = rng.normal(size=(3, 2, 5)), rng.normal(size=(3, 5, 4))
    c = oracle.gemm(a, b)
    for i in range(3):
        assert np.array_equal(c[i], oracle.gemm(a[i], b[i]))


# ---------------------------------------------------------------- attention
def _rand_qkv(rng, batch, seq, heads, d):
    return rng.normal(0, 1, size=(batch * seq, 3 * heads * d))


def test_attention_brute_force_tiny():
    rng = np.random.default_rng(21)
    batch, seq, heads, d = 2, 3, 2, 4
    H = heads * d
    qkv = _rand_qkv(rng, batch, seq, heads, d)
    ctx, probs = oracle.attention(qkv, batch, seq, heads, d, return_probs=True)
    for b in range(batch):
        for h in range(heads):
            for i in range(seq):
                q = qkv[b * seq + i, h * d:(h + 1) * d]
                w = []
                for j in range(seq):
                    k = qkv[b * seq + j, H + h * d:H + (h + 1) * d]
                    w.append(math.exp(sum(float(x) * float(y) for x, y in zip(q, k)) / math.sqrt(d)))
                tot = sum(w)
                for e in range(d):
                    val = sum(w[j] / tot * qkv[b * seq + j, 2 * H + h * d + e] for j in range(seq))
                    assert abs(ctx[b * seq + i, h * d + e] - val) < 1e-13
                np.testing.assert_allclose(probs[b, h, i], np.array(w) / tot, rtol=1e-13)


def test_attention_zero_queries_average_values():
    rng = np.random.default_rng(22)
    batch, seq, heads, d = 2, 5, 3, 4
    H = heads * d
    qkv = _rand_qkv(rng, batch, seq, heads, d)
    qkv[:, :H] = 0.0
    ctx, probs = oracle.attention(qkv, batch, seq, heads, d, return_probs=True)
    assert np.array_equal(probs, np.full_like(probs, 1.0 / seq))
    v = qkv[:, 2 * H:].reshape(batch, seq, H)
    expect = np.repeat(v.mean(axis=1, keepdims=True), seq, axis=1).reshape(batch * seq, H)
    np.testing.assert_allclose(ctx, expect, rtol=1e-13, atol=1e-15)


def test_attention_key_value_permutation_and_head_independence():
    rng = np.random.default_rng(23)
    batch, seq, heads, d = 1, 6, 2, 4
    H = heads * d
    qkv = _rand_qkv(rng, batch, seq, heads, d)
    ctx, probs = oracle.attention(qkv, batch, seq, heads, d, return_probs=True)
    np.testing.assert_allclose(probs.sum(axis=-1), 1.0, rtol=1e-14)
    perm = rng.permutation(seq)
    q2 = qkv.copy()
    q2[:, H:] = qkv[perm, H:]           # permute keys and values together, not queries
    np.testing.assert_allclose(oracle.attention(q2, batch, seq, heads, d), ctx, rtol=1e-12, atol=1e-14)
    # changing head 1's K columns leaves head 0's context untouched
    q3 = qkv.copy()
    q3[:, H + d:H + 2 * d] += rng.normal(size=(seq, d))
    ctx3 = oracle.attention(q3, batch, seq, heads, d)
    assert np.array_equal(ctx3[:, :d], ctx[:, :d])
    assert not np.allclose(ctx3[:, d:], ctx[:, d:])


def test_attention_scale_is_inverse_sqrt_head_dim():
    # one query, two keys: p = logistic((q.k0 - q.k1)/sqrt(d))
    d = 16
    qkv = np.zeros((2, 3 * d))
    qkv[:, :d] = 1.0                      # both queries all-ones
    qkv[0, d:2 * d] = 0.5                 # k0
    qkv[1, d:2 * d] = 0.0                 # k1
    qkv[0, 2 * d:] = 1.0                  # v0 = 1, v1 = 0  -> ctx = p0
    ctx = oracle.attention(qkv, 1, 2, 1, d)
    p0 = 1 / (1 + math.exp(-(0.5 * d) / math.sqrt(d)))
    np.testing.assert_allclose(ctx, np.full((2, d), p0), rtol=1e-14)


# -------------------------------------------------------------------- layer
def _layer_params(rng, T, H, F, scale=0.2):
    p = {
        "x": rng.normal(size=(T, H)),
        "w_qkv": rng.normal(0, scale, size=(H, 3 * H)), "b_qkv": rng.normal(0, 0.1, 3 * H),
        "w_o": rng.normal(0, scale, size=(H, H)), "b_o": rng.normal(0, 0.1, H),
        "w_ffn1": rng.normal(0, scale, size=(H, F)), "b_ffn1": rng.normal(0, 0.1, F),
        "w_ffn2": rng.normal(0, scale, size=(F, H)), "b_ffn2": rng.normal(0, 0.1, H),
        "ln1_gamma": rng.uniform(0.5, 1.5, H), "ln1_beta": rng.normal(0, 0.1, H),
        "ln2_gamma": rng.uniform(0.5, 1.5, H), "ln2_beta": rng.normal(0, 0.1, H),
    }
    return p


def _run(p, batch, seq, heads, **kw):
    return oracle.encoder_layer(p["x"], p["w_qkv"], p["b_qkv"], p["w_o"], p["b_o"], p["w_ffn1"], p["b_ffn1"],
                                p["w_ffn2"], p["b_ffn2"], p["ln1_gamma"], p["ln1_beta"], p["ln2_gamma"],
                                p["ln2_beta"], batch=batch, seq=seq, heads=heads, **kw)


def test_layer_against_torch_float64():
    torch = pytest.importorskip("torch")
    F_ = torch.nn.functional
    rng = np.random.default_rng(31)
    batch, seq, heads, d, F = 2, 7, 3, 4, 20
    H = heads * d
    p = _layer_params(rng, batch * seq, H, F)
    y, inter = _run(p, batch, seq, heads, return_intermediates=True)
    t = {k: torch.from_numpy(np.asarray(v)) for k, v in p.items()}
    qkv = t["x"] @ t["w_qkv"] + t["b_qkv"]
    q, k, v = [z.reshape(batch, seq, heads, d).permute(0, 2, 1, 3) for z in qkv.split(H, dim=1)]
    pr = torch.softmax(q @ k.transpose(-1, -2) / math.sqrt(d), dim=-1)
    ctx = (pr @ v).permute(0, 2, 1, 3).reshape(batch * seq, H)
    h1 = F_.layer_norm(ctx @ t["w_o"] + t["b_o"] + t["x"], (H,), t["ln1_gamma"], t["ln1_beta"], 1e-5)
    mid = F_.gelu(h1 @ t["w_ffn1"] + t["b_ffn1"])
    out = F_.layer_norm(mid @ t["w_ffn2"] + t["b_ffn2"] + h1, (H,), t["ln2_gamma"], t["ln2_beta"], 1e-5)
    np.testing.assert_allclose(inter["qkv"], qkv.numpy(), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(inter["ctx"], ctx.numpy(), rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(inter["h1"], h1.numpy(), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(inter["mid"], mid.numpy(), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(y, out.numpy(), rtol=1e-10, atol=1e-12)


def test_layer_degenerate_projections():
    rng = np.random.default_rng(32)
    batch, seq, heads, d, F = 1, 5, 2, 4, 12
    H = heads * d
    p = _layer_params(rng, batch * seq, H, F)
    p["w_o"][:] = 0.0; p["b_o"][:] = 0.0
    y, inter = _run(p, batch, seq, heads, return_intermediates=True)
    # with a null output projection the first block is LN(X)
    np.testing.assert_allclose(inter["h1"], oracle.layernorm(p["x"], p["ln1_gamma"], p["ln1_beta"], 1e-5), rtol=1e-13, atol=1e-15)
    p["w_ffn2"][:] = 0.0; p["b_ffn2"][:] = 0.0
    y2, inter2 = _run(p, batch, seq, heads, return_intermediates=True)
    np.testing.assert_allclose(y2, oracle.layernorm(inter2["h1"], p["ln2_gamma"], p["ln2_beta"], 1e-5), rtol=1e-13, atol=1e-15)


def test_layer_batch_independence_and_output_statistics():
    rng = np.random.default_rng(33)
    batch, seq, heads, d, F = 3, 4, 2, 4, 16
    H = heads * d
    p = _layer_params(rng, batch * seq, H, F)
    p["ln2_gamma"][:] = 1.0; p["ln2_beta"][:] = 0.0
    y = _run(p, batch, seq, heads)
    assert np.max(np.abs(y.mean(axis=1))) < 1e-13
    np.testing.assert_allclose(y.var(axis=1), 1.0, rtol=1e-3)
    # sequence 1 changes, sequences 0 and 2 must not
    p2 = dict(p); p2["x"] = p["x"].copy(); p2["x"][seq:2 * seq] += 0.5
    y2 = _run(p2, batch, seq, heads)
    assert np.array_equal(y2[:seq], y[:seq]) and np.array_equal(y2[2 * seq:], y[2 * seq:])
    assert not np.allclose(y2[seq:2 * seq], y[seq:2 * seq])
    # one sequence alone gives the same rows as inside the batch
    p1 = dict(p); p1["x"] = p["x"][seq:2 * seq]
    assert np.array_equal(_run(p1, 1, seq, heads), y[seq:2 * seq])


def test_layer_rejects_bad_shapes():
    rng = np.random.default_rng(34)
    p = _layer_params(rng, 4, 6, 8)
    with pytest.raises(ValueError):
        _run(p, 1, 4, 4)   # 6 hidden units do not split into 4 heads
