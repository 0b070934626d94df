"""GPU parity of pd_gemm_bf16 against the CPU oracle through the C ABI.

Integer-valued inputs must match bit for bit with fp32 output (every partial
sum is exactly representable); random bf16 inputs must be within 2e-2 relative
(denominator floored at the RMS of the oracle output), the bound set for bf16
contractions with fp32 accumulation.  In practice fp32 output agrees to ~1e-6
and bf16 output to one bf16 rounding (2^-9)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_03586_b200 import inputs
from parity import Guarded, dev_bf16, host, max_rel_floored

pytestmark = pytest.mark.gpu
TOL = 2e-2


@pytest.fixture(scope="module", params=[1, 2, 0], ids=["single_cta_tiles", "cta_pair_tiles", "auto_tiles"])
def api(request):
    """Every test runs with 128 x BN single-CTA tiles, with 256 x 256 CTA-pair tiles, and with the automatic choice."""
    from paper_2511_03586_b200 import api
    api.pd_clear_device_status()
    api.pd_set_gemm_tile_mode(request.param)
    yield api
    api.pd_set_gemm_tile_mode(0)
    assert api.pd_get_device_status() == 0, "a bounded wait expired inside a tensor-core kernel"


def _oracle(p, b_is_nk):
    b = np.swapaxes(p["b"], -1, -2) if b_is_nk else p["b"]
    return oracle.gemm(p["a"], np.ascontiguousarray(b))


SHAPES = [  # (M, N, K): tile multiples, ragged edges in every dimension, tiny, several k-blocks
    (128, 256, 64), (128, 256, 256), (256, 512, 1024), (8, 8, 8), (1, 8, 8), (130, 264, 72), (127, 248, 1000),
    (300, 72, 136), (64, 64, 4096), (257, 1032, 64), (128, 128, 128), (384, 136, 200), (100, 40, 24),
]


@pytest.mark.parametrize("b_is_nk", [False, True])
@pytest.mark.parametrize("shape", SHAPES)
def test_integer_inputs_are_exact(api, shape, b_is_nk):
    M, N, K = shape
    p = inputs.gemm_integer_inputs(M, N, K, seed=M + N + K, b_is_nk=b_is_nk)
    a, b = dev_bf16(p["a_bits"][0]), dev_bf16(p["b_bits"][0])
    c = Guarded((M, N), torch.float32)
    api.pd_gemm_bf16(a, b, c.t, b_is_nk=b_is_nk)
    torch.cuda.synchronize()
    c.check()
    ref = _oracle(p, b_is_nk)[0]
    assert np.array_equal(host(c.t), ref)
    cb = Guarded((M, N), torch.bfloat16)
    api.pd_gemm_bf16(a, b, cb.t, b_is_nk=b_is_nk)
    torch.cuda.synchronize()
    cb.check()
    ref_bf16 = inputs.bf16_bits_to_f32(inputs.f32_to_bf16_bits(ref.astype(np.float32)))
    assert np.array_equal(host(cb.t), ref_bf16.astype(np.float64))


@pytest.mark.parametrize("b_is_nk", [False, True])
def test_identity_and_selector_matrices(api, b_is_nk):
    K, N = 192, 320
    rng = np.random.default_rng(3)
    bmat = rng.integers(-100, 101, size=(K, N)).astype(np.float32)          # exact in bf16? keep |v| <= 128: yes
    bmat = np.clip(bmat, -128, 128)
    b_store = np.ascontiguousarray(bmat.T) if b_is_nk else bmat
    bd = dev_bf16(inputs.f32_to_bf16_bits(b_store))
    eye = dev_bf16(inputs.f32_to_bf16_bits(np.eye(K, dtype=np.float32)))
    c = api.pd_gemm_bf16(eye, bd, b_is_nk=b_is_nk, c_dtype=torch.float32)
    assert np.array_equal(host(c), bmat.astype(np.float64))
    # E_ij: a single one at (i, j) copies row j of B into row i of C and nothing else
    for i, j in ((0, 0), (5, 77), (130, 191), (191, 64)):
        e = np.zeros((K, K), np.float32); e[i, j] = 1
        c = host(api.pd_gemm_bf16(dev_bf16(inputs.f32_to_bf16_bits(e)), bd, b_is_nk=b_is_nk, c_dtype=torch.float32))
        expect = np.zeros((K, N)); expect[i] = bmat[j]
        assert np.array_equal(c, expect)


@pytest.mark.parametrize("b_is_nk", [False, True])
@pytest.mark.parametrize("shape", [(256, 512, 1024), (130, 264, 520), (512, 64, 512), (512, 512, 64)])
def test_random_inputs_within_tolerance(api, shape, b_is_nk):
    M, N, K = shape
    p = inputs.gemm_inputs(M, N, K, seed=1, b_is_nk=b_is_nk)
    a, b = dev_bf16(p["a_bits"][0]), dev_bf16(p["b_bits"][0])
    ref = _oracle(p, b_is_nk)[0]
    c32 = api.pd_gemm_bf16(a, b, b_is_nk=b_is_nk, c_dtype=torch.float32)
    assert max_rel_floored(host(c32), ref) < 1e-5
    c16 = api.pd_gemm_bf16(a, b, b_is_nk=b_is_nk)
    assert max_rel_floored(host(c16), ref) < TOL
    assert torch.equal(c16, api.pd_gemm_bf16(a, b, b_is_nk=b_is_nk))     # deterministic


@pytest.mark.parametrize("b_is_nk", [False, True])
def test_batched_paper_bmm_shape(api, b_is_nk):
    # Table "ML operators optimized using PerfLLM": bmm 192 x 256 x 128 x 256
    batch, M, K, N = 192, 256, 128, 256
    p = inputs.gemm_integer_inputs(M, N, K, seed=2, batch=batch, b_is_nk=b_is_nk)
    c = api.pd_gemm_bf16(dev_bf16(p["a_bits"]), dev_bf16(p["b_bits"]), b_is_nk=b_is_nk, c_dtype=torch.float32)
    pick = [0, 1, 95, 191]
    sub = {"a": p["a"][pick], "b": p["b"][pick]}
    assert np.array_equal(host(c)[pick], _oracle(sub, b_is_nk))
    # the remaining problems: compare against a float64 matmul (library routine, exact on integers)
    a64 = p["a"].astype(np.float64)
    b64 = (np.swapaxes(p["b"], 1, 2) if b_is_nk else p["b"]).astype(np.float64)
    assert np.array_equal(host(c), a64 @ b64)


@pytest.mark.parametrize("shape", [(2560, 2048, 128), (2500, 1992, 72), (2304, 2304, 64)])
def test_partly_filled_last_round_is_exact(api, shape):
    # 80, 80 and 81 tiles of 256 x 256 on 74 CTA pairs: a second round that only a few pairs take part in, with
    # ragged right and bottom edges in the second shape; integer inputs, so bit equality
    M, N, K = shape
    p = inputs.gemm_integer_inputs(M, N, K, seed=M + N + K, b_is_nk=False)
    a, b = dev_bf16(p["a_bits"][0]), dev_bf16(p["b_bits"][0])
    c = Guarded((M, N), torch.float32)
    api.pd_gemm_bf16(a, b, c.t)
    torch.cuda.synchronize()
    c.check()
    ref = _oracle(p, False)[0]
    assert np.array_equal(host(c.t), ref)
    cb = Guarded((M, N), torch.bfloat16)
    api.pd_gemm_bf16(a, b, cb.t)
    torch.cuda.synchronize()
    cb.check()
    ref_bf16 = inputs.bf16_bits_to_f32(inputs.f32_to_bf16_bits(ref.astype(np.float32)))
    assert np.array_equal(host(cb.t), ref_bf16.astype(np.float64))


def test_layer_qkv_shape_sampled_rows(api):
    # the layer's QKV projection: 768 pair tiles = 10 rounds of 74 and 28 left over
    M, K, N = 16384, 1024, 3072
    p = inputs.gemm_inputs(M, N, K, seed=7)
    a, b = dev_bf16(p["a_bits"][0]), dev_bf16(p["b_bits"][0])
    c32 = api.pd_gemm_bf16(a, b, c_dtype=torch.float32)
    c = api.pd_gemm_bf16(a, b)
    # the last round holds the rows from 15872 on: sample there densely and elsewhere sparsely
    rng = np.random.default_rng(1)
    pick = np.unique(np.concatenate([[0, 255, 256, M - 1, M - 256, M - 257], rng.integers(0, M, 30),
                                     rng.integers(M - 768, M, 50)]))
    ref = oracle.gemm(p["a"][0][pick], p["b"][0])
    idx = torch.from_numpy(pick).cuda()
    assert max_rel_floored(host(c32[idx]), ref) < 1e-5
    assert max_rel_floored(host(c[idx]), ref) < TOL
    assert bool(torch.isfinite(c32).all())
    assert torch.equal(c, c32.to(torch.bfloat16))


def test_paper_matmul_shape(api):
    M, K, N = 768, 1024, 1024
    p = inputs.gemm_inputs(M, N, K, seed=4)
    c = api.pd_gemm_bf16(dev_bf16(p["a_bits"][0]), dev_bf16(p["b_bits"][0]))
    assert max_rel_floored(host(c), _oracle(p, False)[0]) < TOL


def test_configured_shape_sampled_rows(api):
    M, K, N = 16384, 1024, 4096
    p = inputs.gemm_inputs(M, N, K, seed=0)
    a, b = dev_bf16(p["a_bits"][0]), dev_bf16(p["b_bits"][0])
    c = api.pd_gemm_bf16(a, b)
    c32 = api.pd_gemm_bf16(a, b, c_dtype=torch.float32)
    pick = np.unique(np.concatenate([[0, 127, 128, M - 1], np.random.default_rng(0).integers(0, M, 60)]))
    ref = oracle.gemm(p["a"][0][pick], p["b"][0])
    idx = torch.from_numpy(pick).cuda()
    assert max_rel_floored(host(c[idx]), ref) < TOL
    assert max_rel_floored(host(c32[idx]), ref) < 1e-5
    # every output is finite and the bf16 result is the rounding of the fp32 one
    assert bool(torch.isfinite(c32).all())
    assert torch.equal(c, c32.to(torch.bfloat16))


# Row lengths that are not a multiple of eight elements: C sits in a wider matrix (ldc a legal multiple), and every
# column from N on must keep its fill value.  K >= 2048 with few output tiles is the territory of the split-K
# kernel, whose epilogue stores eight columns at a time: such shapes must be routed to the kernels that clip.
@pytest.mark.parametrize("c_dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("b_is_nk", [False, True])
@pytest.mark.parametrize("shape", [(128, 36, 2048), (128, 100, 2048), (200, 250, 4096), (130, 100, 72), (260, 257, 136),
                                   (64, 4, 64), (300, 1001, 264), (130, 100, 100), (64, 72, 2051), (40, 33, 7)])
def test_row_lengths_off_the_vector_width(api, shape, b_is_nk, c_dtype):
    M, N, K = shape
    p = inputs.gemm_integer_inputs(M, N, K, seed=M + N + K, b_is_nk=b_is_nk)
    ref = _oracle(p, b_is_nk)[0]
    if c_dtype == torch.bfloat16:
        ref = inputs.bf16_bits_to_f32(inputs.f32_to_bf16_bits(ref.astype(np.float32))).astype(np.float64)
    unit = 4 if c_dtype == torch.float32 else 8
    # operands in wider matrices whose padding columns hold a large value: nothing beyond K or N may be read as data
    lda = (K + 7) // 8 * 8
    A = torch.full((M, lda), 3.0e4, dtype=torch.bfloat16, device="cuda")
    A[:, :K] = dev_bf16(p["a_bits"][0])
    b_rows, b_cols = (N, K) if b_is_nk else (K, N)
    ldb = (b_cols + 7) // 8 * 8
    B = torch.full((b_rows, ldb), 3.0e4, dtype=torch.bfloat16, device="cuda")
    B[:, :b_cols] = dev_bf16(p["b_bits"][0])
    for ldc in ((N + unit - 1) // unit * unit, (N + unit - 1) // unit * unit + 3 * unit):
        c = Guarded((M, ldc), c_dtype)
        c.t.fill_(-7.0)
        st = api.pd_gemm_bf16_raw(A.data_ptr(), B.data_ptr(), c.t.data_ptr(), M, N, K, lda, ldb, ldc, b_is_nk,
                                  api.PD_F32 if c_dtype == torch.float32 else api.PD_BF16, 1, 0, 0, 0)
        assert st == 0
        torch.cuda.synchronize()
        c.check()
        assert np.array_equal(host(c.t[:, :N]), ref)
        assert bool((c.t[:, N:] == -7.0).all()), "columns outside C were written"


def test_strided_operands_and_errors(api):
    # operands embedded in wider matrices (ld > row length), addressed through the raw entry point
    M, N, K = 96, 80, 72
    p = inputs.gemm_integer_inputs(M, N, K, seed=7)
    A = torch.zeros(M, K + 24, dtype=torch.bfloat16, device="cuda"); A[:, :K] = dev_bf16(p["a_bits"][0])
    B = torch.zeros(K, N + 8, dtype=torch.bfloat16, device="cuda"); B[:, :N] = dev_bf16(p["b_bits"][0])
    Cw = torch.full((M, N + 16), -7.0, dtype=torch.float32, device="cuda")
    st = api.pd_gemm_bf16_raw(A.data_ptr(), B.data_ptr(), Cw.data_ptr(), M, N, K, K + 24, N + 8, N + 16, False,
                              api.PD_F32, 1, 0, 0, 0)
    assert st == 0
    assert np.array_equal(host(Cw[:, :N]), _oracle(p, False)[0])
    assert bool((Cw[:, N:] == -7.0).all())           # columns outside C are untouched
    ptr = A.data_ptr()
    assert api.pd_gemm_bf16_raw(0, ptr, ptr, 8, 8, 8, 8, 8, 8, False, 0, 1, 0, 0, 0) == 1      # null
    assert api.pd_gemm_bf16_raw(ptr, ptr, ptr, 8, 8, 0, 8, 8, 8, False, 0, 1, 0, 0, 0) == 2    # K == 0
    assert api.pd_gemm_bf16_raw(ptr, ptr, ptr, 8, 8, 8, 4, 8, 8, False, 0, 1, 0, 0, 0) == 2    # lda < K
    assert api.pd_gemm_bf16_raw(ptr, ptr, ptr, 8, 8, 8, 12, 8, 8, False, 0, 1, 0, 0, 0) == 4   # lda % 8
    assert api.pd_gemm_bf16_raw(ptr + 2, ptr, ptr, 8, 8, 8, 8, 8, 8, False, 0, 1, 0, 0, 0) == 4
    assert api.pd_gemm_bf16_raw(ptr, ptr, ptr, 0, 8, 8, 8, 8, 8, False, 0, 1, 0, 0, 0) == 0    # empty
