"""Argument checking of every C-ABI entry point, without a GPU.

Each call below is one that the library must turn away (or accept as empty) on the host, before it looks at
the device: null pointers, impossible shapes, misaligned addresses or leading dimensions, unsupported
combinations, and zero outer extents, which are PD_OK with nothing launched.  The pointers are made-up
addresses; none of these calls may ever reach a kernel, on a machine with a GPU or without one.
"""
import ctypes

import pytest

OK, NULLP, SHAPE, UNSUP, ALIGN, WS_SMALL = 0, 1, 2, 3, 4, 5
P = 0x10000          # a 16-byte aligned stand-in for a device address
ODD = P + 2          # not even 4-byte aligned
i64, vp, ci, cf = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int, ctypes.c_float


class Desc(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("seq", ctypes.c_int32), ("hidden", ctypes.c_int32),
                ("heads", ctypes.c_int32), ("ffn", ctypes.c_int32), ("ln_eps", ctypes.c_float)]


class Weights(ctypes.Structure):
    _fields_ = [(n, vp) for n in ("w_qkv", "w_o", "w_ffn1", "w_ffn2", "b_qkv", "b_o", "b_ffn1", "b_ffn2",
                                  "ln1_gamma", "ln1_beta", "ln2_gamma", "ln2_beta")]


@pytest.fixture(scope="module")
def lib():
    from paper_2511_03586_b200 import build
    lib = ctypes.CDLL(build.build())
    lib.pd_softmax.argtypes = [vp, vp, i64, i64, vp]
    lib.pd_layernorm.argtypes = [vp, vp, vp, vp, i64, i64, cf, vp]
    lib.pd_rmsnorm.argtypes = [vp, vp, vp, i64, i64, cf, vp]
    lib.pd_reducemean.argtypes = [vp, vp, i64, i64, vp]
    lib.pd_bias_gelu_residual.argtypes = [vp, vp, vp, vp, i64, i64, vp]
    lib.pd_gemm_bf16.argtypes = [vp, vp, vp, i64, i64, i64, i64, i64, i64, ci, ci, i64, i64, i64, i64, vp]
    lib.pd_gemm_bias_act.argtypes = [vp, vp, vp, vp, vp, i64, i64, i64, ci, ci, vp]
    lib.pd_swiglu_gemm.argtypes = [vp, vp, vp, vp, i64, i64, i64, vp]
    lib.pd_gemm_bias_residual_layernorm.argtypes = [vp, vp, vp, vp, vp, vp, vp, i64, i64, i64, cf, vp]
    lib.pd_attention_fwd.argtypes = [vp, vp, i64, i64, i64, vp]
    lib.pd_encoder_layer_workspace_bytes.argtypes = [ctypes.POINTER(Desc)]
    lib.pd_encoder_layer_workspace_bytes.restype = ctypes.c_size_t
    lib.pd_encoder_layer_fwd.argtypes = [ctypes.POINTER(Desc), ctypes.POINTER(Weights), vp, vp, vp, ctypes.c_size_t, vp]
    lib.pd_encoder_layer_fwd_static.argtypes = [ctypes.POINTER(Desc), ctypes.POINTER(Weights), vp, vp, vp]
    lib.pd_encoder_layer_static_scratch_bytes.restype = ctypes.c_size_t
    return lib


def test_row_operators(lib):
    assert lib.pd_layernorm(None, P, P, P, 4, 8, 1e-5, None) == NULLP
    assert lib.pd_layernorm(P, P, None, P, 4, 8, 1e-5, None) == NULLP
    assert lib.pd_layernorm(P, P, P, P, -1, 8, 1e-5, None) == SHAPE
    assert lib.pd_layernorm(P, P, P, P, 4, 0, 1e-5, None) == SHAPE
    assert lib.pd_layernorm(P, P, P, P, 4, 8, -1.0, None) == SHAPE
    assert lib.pd_layernorm(P, P, P, P, 4, 8, float("nan"), None) == SHAPE
    assert lib.pd_layernorm(P, ODD, P, P, 4, 8, 1e-5, None) == ALIGN
    assert lib.pd_layernorm(P, P, P, P, 0, 8, 1e-5, None) == OK

    assert lib.pd_rmsnorm(P, None, P, 4, 8, 1e-5, None) == NULLP
    assert lib.pd_rmsnorm(P, P, P, 4, -3, 1e-5, None) == SHAPE
    assert lib.pd_rmsnorm(P, P, P, 4, 8, -1e-5, None) == SHAPE
    assert lib.pd_rmsnorm(ODD, P, P, 4, 8, 1e-5, None) == ALIGN
    assert lib.pd_rmsnorm(P, P, P, 0, 8, 1e-5, None) == OK

    assert lib.pd_reducemean(P, None, 4, 8, None) == NULLP
    assert lib.pd_reducemean(P, P, 4, 0, None) == SHAPE
    assert lib.pd_reducemean(P, ODD, 4, 8, None) == ALIGN
    assert lib.pd_reducemean(P, P, 0, 8, None) == OK

    assert lib.pd_bias_gelu_residual(P, None, P, P, 4, 8, None) == NULLP
    assert lib.pd_bias_gelu_residual(P, P, None, P, -4, 8, None) == SHAPE       # the residual may be absent
    assert lib.pd_bias_gelu_residual(P, P, ODD, P, 4, 8, None) == ALIGN
    assert lib.pd_bias_gelu_residual(P, P, None, P, 0, 8, None) == OK

    assert lib.pd_softmax(P, P, -1, 8, None) == SHAPE


def test_gemm(lib):
    def gemm(A=P, B=P, C=P, M=64, N=64, K=64, lda=64, ldb=64, ldc=64, nk=0, dt=0, batch=1, sa=0, sb=0, sc=0):
        return lib.pd_gemm_bf16(A, B, C, M, N, K, lda, ldb, ldc, nk, dt, batch, sa, sb, sc, None)
    assert gemm(A=None) == NULLP
    assert gemm(K=0) == SHAPE
    assert gemm(M=-1) == SHAPE
    assert gemm(dt=5) == SHAPE
    assert gemm(M=1 << 31) == SHAPE
    assert gemm(lda=56) == SHAPE                      # shorter than a row
    assert gemm(N=80, ldb=64, ldc=80) == SHAPE        # B [K, N]: ldb below N
    assert gemm(lda=68) == ALIGN                      # not a multiple of 8 elements
    assert gemm(dt=1, ldc=66) == ALIGN                # fp32 C: multiples of 4 elements
    assert gemm(B=P + 8) == ALIGN
    assert gemm(batch=2, sa=4096, sb=4096, sc=-8) == SHAPE
    assert gemm(batch=2, sa=4100, sb=4096, sc=4096) == ALIGN
    assert gemm(batch=2, sa=4096, sb=0, sc=4096) == UNSUP     # broadcast operand
    assert gemm(M=0) == OK
    assert gemm(N=0, ldb=64, ldc=64) == OK
    assert gemm(batch=0) == OK

    def act(A=P, B=P, bias=P, res=None, C=P, M=64, N=64, K=64, a=1, dt=0):
        return lib.pd_gemm_bias_act(A, B, bias, res, C, M, N, K, a, dt, None)
    assert act(C=None) == NULLP
    assert act(a=3) == SHAPE
    assert act(K=-8) == SHAPE
    assert act(dt=2) == SHAPE
    assert act(bias=P + 4) == ALIGN
    assert act(res=P + 2) == ALIGN
    assert act(K=60) == ALIGN
    assert act(N=68) == ALIGN
    assert act(M=0) == OK
    assert act(bias=None, M=0) == OK                  # bias and residual are optional

    assert lib.pd_swiglu_gemm(P, None, P, P, 64, 64, 64, None) == NULLP
    assert lib.pd_swiglu_gemm(P, P, P, P, 64, 64, 0, None) == SHAPE
    assert lib.pd_swiglu_gemm(P, P, P, P, 64, 60, 64, None) == ALIGN
    assert lib.pd_swiglu_gemm(P, P, P + 8, P, 64, 64, 64, None) == ALIGN
    assert lib.pd_swiglu_gemm(P, P, P, P, 0, 64, 64, None) == OK

    def ln(A=P, B=P, bias=P, res=P, g=P, b=P, Y=P, M=128, N=256, K=64, eps=1e-5):
        return lib.pd_gemm_bias_residual_layernorm(A, B, bias, res, g, b, Y, M, N, K, eps, None)
    assert ln(g=None) == NULLP
    assert ln(N=0) == SHAPE
    assert ln(eps=-1.0) == SHAPE
    assert ln(N=320) == UNSUP                         # not a multiple of 256 columns
    assert ln(N=4096) == UNSUP                        # more than eight CTAs to a row block
    assert ln(K=60) == ALIGN
    assert ln(res=P + 8) == ALIGN
    assert ln(M=0) == OK
    assert ln(bias=None, res=None, M=0) == OK

    for mode, want in ((-1, SHAPE), (3, SHAPE), (0, OK)):
        assert lib.pd_set_gemm_tile_mode(mode) == want
    for mode, want in ((-1, SHAPE), (2, SHAPE), (0, OK)):
        assert lib.pd_set_gemm_split_k(mode) == want


def test_attention_and_layer(lib):
    assert lib.pd_attention_fwd(None, P, 1, 128, 4, None) == NULLP
    assert lib.pd_attention_fwd(P, P, -1, 128, 4, None) == SHAPE
    assert lib.pd_attention_fwd(P, P, 1, 0, 4, None) == SHAPE
    assert lib.pd_attention_fwd(P, P, 1, 128, 0, None) == SHAPE
    assert lib.pd_attention_fwd(P, P, 1, 513, 4, None) == UNSUP
    assert lib.pd_attention_fwd(P + 8, P, 1, 128, 4, None) == ALIGN
    assert lib.pd_attention_fwd(P, P, 0, 128, 4, None) == OK

    w = Weights(*([P] * 12))
    good = Desc(2, 128, 256, 4, 512, 1e-5)
    need = lib.pd_encoder_layer_workspace_bytes(ctypes.byref(good))
    assert need > 0
    assert lib.pd_encoder_layer_fwd(None, ctypes.byref(w), P, P, P, need, None) == NULLP
    assert lib.pd_encoder_layer_fwd(ctypes.byref(good), None, P, P, P, need, None) == NULLP
    assert lib.pd_encoder_layer_fwd(ctypes.byref(good), ctypes.byref(w), None, P, P, need, None) == NULLP
    assert lib.pd_encoder_layer_fwd(ctypes.byref(good), ctypes.byref(w), P, P, P, need - 1, None) == WS_SMALL
    assert lib.pd_encoder_layer_fwd(ctypes.byref(Desc(2, 128, 256, 3, 512, 1e-5)), ctypes.byref(w), P, P, P, need,
                                    None) in (SHAPE, UNSUP)     # 256 hidden does not split into 3 heads of 64
    assert lib.pd_encoder_layer_fwd(ctypes.byref(Desc(2, 0, 256, 4, 512, 1e-5)), ctypes.byref(w), P, P, P, need,
                                    None) == SHAPE
    missing = Weights(*([P] * 12))
    missing.ln2_beta = None
    assert lib.pd_encoder_layer_fwd(ctypes.byref(good), ctypes.byref(missing), P, P, P, need, None) == NULLP

    # the allocation-free variant turns away what its fixed array cannot hold, before anything else happens
    big = Desc(32, 512, 1024, 16, 4096, 1e-5)
    assert lib.pd_encoder_layer_workspace_bytes(ctypes.byref(big)) > lib.pd_encoder_layer_static_scratch_bytes()
    assert lib.pd_encoder_layer_fwd_static(ctypes.byref(big), ctypes.byref(w), P, P, None) == WS_SMALL
    assert lib.pd_encoder_layer_fwd_static(None, ctypes.byref(w), P, P, None) == NULLP
    # faults are reported in the same order as by pd_encoder_layer_fwd: a null or misaligned x before the size
    assert lib.pd_encoder_layer_fwd_static(ctypes.byref(big), ctypes.byref(w), None, P, None) == NULLP
    assert lib.pd_encoder_layer_fwd_static(ctypes.byref(big), ctypes.byref(w), P + 8, P, None) == ALIGN
    assert lib.pd_encoder_layer_fwd_static(ctypes.byref(big), ctypes.byref(missing), P, P, None) == NULLP
    # more tokens than an int can index
    huge = Desc(1 << 23, 512, 256, 4, 512, 1e-5)
    assert lib.pd_encoder_layer_fwd(ctypes.byref(huge), ctypes.byref(w), P, P, P, need, None) == SHAPE
    assert lib.pd_encoder_layer_workspace_bytes(ctypes.byref(huge)) == 0

    # where the intermediates sit inside the workspace: consecutive, 256-byte aligned, adding up to the total
    n = 7
    off, size = (ctypes.c_size_t * n)(), (ctypes.c_size_t * n)()
    lib.pd_encoder_layer_workspace_layout.argtypes = [ctypes.POINTER(Desc), ctypes.POINTER(ctypes.c_size_t),
                                                      ctypes.POINTER(ctypes.c_size_t)]
    assert lib.pd_encoder_layer_workspace_layout(ctypes.byref(good), off, size) == OK
    assert off[0] == 0 and all(off[i] + size[i] == off[i + 1] for i in range(n - 1)) and off[n - 1] + size[n - 1] == need
    assert all(o % 256 == 0 for o in off)
    T, H, F = 2 * 128, 256, 512
    assert size[0] == T * 3 * H * 2 and size[3] == T * H * 2 and size[5] == T * H * 2 and size[6] == T * F * 2
    assert size[1] == 0 and size[2] == 0          # fused attention keeps scores and probabilities on the SM
    assert lib.pd_encoder_layer_workspace_layout(None, off, size) == NULLP
    assert lib.pd_encoder_layer_workspace_layout(ctypes.byref(good), None, size) == NULLP
    assert lib.pd_encoder_layer_workspace_layout(ctypes.byref(Desc(2, 0, 256, 4, 512, 1e-5)), off, size) == SHAPE
