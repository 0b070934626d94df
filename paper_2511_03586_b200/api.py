"""Thin ctypes binding of ``libpd.so``: argument marshalling only.

Every function mirrors one entry point of ``include/pd.h`` under the same name,
takes CUDA ``torch.Tensor`` arguments (torch supplies device memory and the
stream, nothing else), and raises :class:`PdError` on a non-zero status.  There
is no fallback: if the library is missing or cannot be loaded, importing this
module fails.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libpd.so")

PD_OK = 0
PD_BF16, PD_F32 = 0, 1

EXPORTS = (
    "pd_status_string", "pd_last_cuda_error", "pd_get_device_status", "pd_clear_device_status",
    "pd_softmax", "pd_layernorm", "pd_rmsnorm", "pd_bias_gelu_residual", "pd_gemm_bf16", "pd_set_gemm_tile_mode", "pd_attention_fwd",
    "pd_encoder_layer_workspace_bytes", "pd_encoder_layer_workspace_layout", "pd_encoder_layer_fwd", "pd_encoder_layer_stage_count",
    "pd_encoder_layer_stage_name", "pd_encoder_layer_fwd_profiled", "pd_encoder_layer_static_scratch_bytes",
    "pd_encoder_layer_fwd_static",
)


class PdError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        name = _lib.pd_status_string(status).decode()
        extra = f" (cudaError {_lib.pd_last_cuda_error()})" if name == "PD_ERR_CUDA" else ""
        super().__init__(f"{where}: {name}{extra}")


class EncoderLayerDesc(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("seq", ctypes.c_int32), ("hidden", ctypes.c_int32),
                ("heads", ctypes.c_int32), ("ffn", ctypes.c_int32), ("ln_eps", ctypes.c_float)]


class EncoderLayerWeights(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in (
        "w_qkv", "w_o", "w_ffn1", "w_ffn2", "b_qkv", "b_o", "b_ffn1", "b_ffn2",
        "ln1_gamma", "ln1_beta", "ln2_gamma", "ln2_beta")]


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2511_03586_b200.build` (needs nvcc)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i64, st = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int
    lib.pd_status_string.argtypes = [st]; lib.pd_status_string.restype = ctypes.c_char_p
    lib.pd_last_cuda_error.argtypes = []; lib.pd_last_cuda_error.restype = ctypes.c_int
    lib.pd_get_device_status.argtypes = [ctypes.POINTER(ctypes.c_int)]; lib.pd_get_device_status.restype = st
    lib.pd_clear_device_status.argtypes = []; lib.pd_clear_device_status.restype = st
    lib.pd_debug_set_wait_limit_ns.argtypes = [ctypes.c_uint64]; lib.pd_debug_set_wait_limit_ns.restype = st
    lib.pd_debug_withhold_loads.argtypes = [ctypes.c_int]; lib.pd_debug_withhold_loads.restype = st
    lib.pd_softmax.argtypes = [vp, vp, i64, i64, vp]; lib.pd_softmax.restype = st
    lib.pd_layernorm.argtypes = [vp, vp, vp, vp, i64, i64, ctypes.c_float, vp]; lib.pd_layernorm.restype = st
    lib.pd_rmsnorm.argtypes = [vp, vp, vp, i64, i64, ctypes.c_float, vp]; lib.pd_rmsnorm.restype = st
    lib.pd_reducemean.argtypes = [vp, vp, i64, i64, vp]; lib.pd_reducemean.restype = st
    lib.pd_bias_gelu_residual.argtypes = [vp, vp, vp, vp, i64, i64, vp]; lib.pd_bias_gelu_residual.restype = st
    lib.pd_gemm_bf16.argtypes = [vp, vp, vp, i64, i64, i64, i64, i64, i64, ctypes.c_int, ctypes.c_int,
                                 i64, i64, i64, i64, vp]
    lib.pd_gemm_bf16.restype = st
    lib.pd_set_gemm_tile_mode.argtypes = [ctypes.c_int]; lib.pd_set_gemm_tile_mode.restype = st
    lib.pd_gemm_bias_act.argtypes = [vp, vp, vp, vp, vp, i64, i64, i64, ctypes.c_int, ctypes.c_int, vp]
    lib.pd_gemm_bias_act.restype = st
    lib.pd_swiglu_gemm.argtypes = [vp, vp, vp, vp, i64, i64, i64, vp]; lib.pd_swiglu_gemm.restype = st
    lib.pd_set_gemm_split_k.argtypes = [ctypes.c_int]; lib.pd_set_gemm_split_k.restype = st
    lib.pd_set_layernorm_fusion.argtypes = [ctypes.c_int]; lib.pd_set_layernorm_fusion.restype = st
    lib.pd_gemm_bias_residual_layernorm.argtypes = [vp, vp, vp, vp, vp, vp, vp, i64, i64, i64, ctypes.c_float, vp]
    lib.pd_gemm_bias_residual_layernorm.restype = st
    lib.pd_attention_fwd.argtypes = [vp, vp, i64, i64, i64, vp]; lib.pd_attention_fwd.restype = st
    lib.pd_encoder_layer_workspace_bytes.argtypes = [ctypes.POINTER(EncoderLayerDesc)]
    lib.pd_encoder_layer_workspace_bytes.restype = ctypes.c_size_t
    lib.pd_encoder_layer_workspace_layout.argtypes = [ctypes.POINTER(EncoderLayerDesc),
                                                      ctypes.POINTER(ctypes.c_size_t), ctypes.POINTER(ctypes.c_size_t)]
    lib.pd_encoder_layer_workspace_layout.restype = st
    lib.pd_encoder_layer_fwd.argtypes = [ctypes.POINTER(EncoderLayerDesc), ctypes.POINTER(EncoderLayerWeights),
                                         vp, vp, vp, ctypes.c_size_t, vp]
    lib.pd_encoder_layer_fwd.restype = st
    lib.pd_encoder_stack_workspace_bytes.argtypes = [ctypes.POINTER(EncoderLayerDesc), ctypes.c_int]
    lib.pd_encoder_stack_workspace_bytes.restype = ctypes.c_size_t
    lib.pd_encoder_stack_fwd.argtypes = [ctypes.POINTER(EncoderLayerDesc), ctypes.POINTER(EncoderLayerWeights),
                                         ctypes.c_int, vp, vp, vp, ctypes.c_size_t, vp]
    lib.pd_encoder_stack_fwd.restype = st
    lib.pd_encoder_layer_static_scratch_bytes.argtypes = []
    lib.pd_encoder_layer_static_scratch_bytes.restype = ctypes.c_size_t
    lib.pd_encoder_layer_fwd_static.argtypes = [ctypes.POINTER(EncoderLayerDesc), ctypes.POINTER(EncoderLayerWeights),
                                                vp, vp, vp]
    lib.pd_encoder_layer_fwd_static.restype = st
    lib.pd_encoder_layer_kernel_count.argtypes = [ctypes.POINTER(EncoderLayerDesc)]
    lib.pd_encoder_layer_kernel_count.restype = ctypes.c_int
    lib.pd_encoder_layer_stage_count.argtypes = []; lib.pd_encoder_layer_stage_count.restype = ctypes.c_int
    lib.pd_encoder_layer_stage_name.argtypes = [ctypes.c_int]
    lib.pd_encoder_layer_stage_name.restype = ctypes.c_char_p
    lib.pd_encoder_layer_fwd_profiled.argtypes = lib.pd_encoder_layer_fwd.argtypes + [ctypes.POINTER(ctypes.c_float)]
    lib.pd_encoder_layer_fwd_profiled.restype = st
    return lib


_lib = _load()


def _check(status: int, where: str):
    if status != PD_OK:
        raise PdError(status, where)


def _stream(stream) -> int:
    return (stream if stream is not None else torch.cuda.current_stream()).cuda_stream


def _dev(t: torch.Tensor, dtype, name: str) -> int:
    if not (isinstance(t, torch.Tensor) and t.is_cuda):
        raise TypeError(f"{name} must be a CUDA tensor")
    if t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}, got {t.dtype}")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    return t.data_ptr()


def pd_softmax(x: torch.Tensor, y: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    rows, cols = x.shape
    if y is None:
        y = torch.empty_like(x)
    _check(_lib.pd_softmax(_dev(x, torch.float32, "x"), _dev(y, torch.float32, "y"), rows, cols, _stream(stream)),
           "pd_softmax")
    return y


def pd_layernorm(x, gamma, beta, eps: float, y=None, stream=None) -> torch.Tensor:
    rows, cols = x.shape
    if y is None:
        y = torch.empty_like(x)
    _check(_lib.pd_layernorm(_dev(x, torch.float32, "x"), _dev(gamma, torch.float32, "gamma"),
                             _dev(beta, torch.float32, "beta"), _dev(y, torch.float32, "y"), rows, cols,
                             float(eps), _stream(stream)), "pd_layernorm")
    return y


def pd_rmsnorm(x, gamma, eps: float, y=None, stream=None) -> torch.Tensor:
    rows, cols = x.shape
    if y is None:
        y = torch.empty_like(x)
    _check(_lib.pd_rmsnorm(_dev(x, torch.float32, "x"), _dev(gamma, torch.float32, "gamma"),
                           _dev(y, torch.float32, "y"), rows, cols, float(eps), _stream(stream)), "pd_rmsnorm")
    return y


def pd_reducemean(x, y=None, stream=None) -> torch.Tensor:
    rows, cols = x.shape
    if y is None:
        y = torch.empty(rows, dtype=torch.float32, device=x.device)
    _check(_lib.pd_reducemean(_dev(x, torch.float32, "x"), _dev(y, torch.float32, "y"), rows, cols, _stream(stream)),
           "pd_reducemean")
    return y


def pd_bias_gelu_residual(x, bias, r=None, out=None, stream=None) -> torch.Tensor:
    rows, cols = x.shape
    if out is None:
        out = torch.empty_like(x)
    rp = None if r is None else _dev(r, torch.float32, "r")
    _check(_lib.pd_bias_gelu_residual(_dev(x, torch.float32, "x"), _dev(bias, torch.float32, "bias"), rp,
                                      _dev(out, torch.float32, "out"), rows, cols, _stream(stream)),
           "pd_bias_gelu_residual")
    return out


def pd_gemm_bf16(a: torch.Tensor, b: torch.Tensor, c: torch.Tensor | None = None, *, b_is_nk: bool = False,
                 c_dtype=torch.bfloat16, stream=None) -> torch.Tensor:
    """C = A @ B for bf16 A [M,K] (or [batch,M,K]) and B [K,N] (or [N,K] when
    ``b_is_nk``; batched likewise).  Inputs must be dense."""
    batched = a.dim() == 3
    if batched:
        batch, M, K = a.shape
    else:
        (M, K), batch = a.shape, 1
    N = b.shape[-2] if b_is_nk else b.shape[-1]
    if c is None:
        c = torch.empty(((batch, M, N) if batched else (M, N)), dtype=c_dtype, device=a.device)
    ldb = b.shape[-1]
    _check(_lib.pd_gemm_bf16(_dev(a, torch.bfloat16, "a"), _dev(b, torch.bfloat16, "b"), _dev(c, c.dtype, "c"),
                             M, N, K, K, ldb, N, int(b_is_nk), PD_F32 if c.dtype == torch.float32 else PD_BF16,
                             batch, M * K, b.shape[-2] * b.shape[-1], M * N, _stream(stream)), "pd_gemm_bf16")
    return c


def pd_set_gemm_tile_mode(mode: int) -> None:
    """0: automatic; 1: single-CTA tiles only; 2: CTA-pair (cta_group::2) tiles for every shape."""
    _check(_lib.pd_set_gemm_tile_mode(int(mode)), "pd_set_gemm_tile_mode")


def pd_gemm_bf16_raw(a_ptr, b_ptr, c_ptr, M, N, K, lda, ldb, ldc, b_is_nk, c_dtype, batch, strideA, strideB,
                     strideC, stream=None) -> int:
    """Direct call with explicit pointers and strides; returns the status instead of raising."""
    return _lib.pd_gemm_bf16(a_ptr, b_ptr, c_ptr, M, N, K, lda, ldb, ldc, int(b_is_nk), int(c_dtype), batch,
                             strideA, strideB, strideC, _stream(stream))


ACT_NONE, ACT_GELU, ACT_RELU = 0, 1, 2


def pd_gemm_bias_act(a, b, bias=None, residual=None, *, act: int = ACT_NONE, c_dtype=torch.bfloat16, c=None,
                     stream=None) -> torch.Tensor:
    """C = act(A @ B + bias) + residual for bf16 A [M,K], B [K,N], residual [M,N]; fp32 bias [N]."""
    M, K = a.shape
    N = b.shape[1]
    if c is None:
        c = torch.empty(M, N, dtype=c_dtype, device=a.device)
    _check(_lib.pd_gemm_bias_act(_dev(a, torch.bfloat16, "a"), _dev(b, torch.bfloat16, "b"),
                                 None if bias is None else _dev(bias, torch.float32, "bias"),
                                 None if residual is None else _dev(residual, torch.bfloat16, "residual"),
                                 _dev(c, c.dtype, "c"), M, N, K, int(act),
                                 PD_F32 if c.dtype == torch.float32 else PD_BF16, _stream(stream)), "pd_gemm_bias_act")
    return c


def pd_swiglu_gemm(x, wg, wu, y=None, stream=None) -> torch.Tensor:
    """Y = SiLU(X @ Wg) * (X @ Wu) for bf16 X [M,K], Wg, Wu [K,N]; bf16 Y."""
    M, K = x.shape
    N = wg.shape[1]
    if y is None:
        y = torch.empty(M, N, dtype=torch.bfloat16, device=x.device)
    _check(_lib.pd_swiglu_gemm(_dev(x, torch.bfloat16, "x"), _dev(wg, torch.bfloat16, "wg"),
                               _dev(wu, torch.bfloat16, "wu"), _dev(y, torch.bfloat16, "y"), M, N, K,
                               _stream(stream)), "pd_swiglu_gemm")
    return y


def pd_set_gemm_split_k(mode: int) -> None:
    """0: split K over a thread-block cluster when a contraction has few output tiles; 1: never."""
    _check(_lib.pd_set_gemm_split_k(int(mode)), "pd_set_gemm_split_k")


def pd_set_layernorm_fusion(mode: int) -> None:
    """0: LayerNorm inside the feeding contraction's epilogue where the shape allows; 1: separate row kernel."""
    _check(_lib.pd_set_layernorm_fusion(int(mode)), "pd_set_layernorm_fusion")


def pd_gemm_bias_residual_layernorm(a, b, bias, residual, gamma, beta, eps: float, y=None, stream=None) -> torch.Tensor:
    """Y = LayerNorm(A @ B + bias + residual) for bf16 A [M,K], B [K,N], residual [M,N] (or None),
    fp32 bias (or None), gamma, beta [N]; bf16 Y."""
    M, K = a.shape
    N = b.shape[1]
    if y is None:
        y = torch.empty(M, N, dtype=torch.bfloat16, device=a.device)
    _check(_lib.pd_gemm_bias_residual_layernorm(
        _dev(a, torch.bfloat16, "a"), _dev(b, torch.bfloat16, "b"),
        None if bias is None else _dev(bias, torch.float32, "bias"),
        None if residual is None else _dev(residual, torch.bfloat16, "residual"),
        _dev(gamma, torch.float32, "gamma"), _dev(beta, torch.float32, "beta"), _dev(y, torch.bfloat16, "y"),
        M, N, K, float(eps), _stream(stream)), "pd_gemm_bias_residual_layernorm")
    return y


def pd_attention_fwd(qkv: torch.Tensor, *, batch: int, seq: int, heads: int, ctx: torch.Tensor | None = None,
                     stream=None) -> torch.Tensor:
    """qkv bf16 [batch*seq, 3*heads*64] -> ctx bf16 [batch*seq, heads*64]."""
    if tuple(qkv.shape) != (batch * seq, 3 * heads * 64):
        raise ValueError("qkv must be [batch*seq, 3*heads*64]")
    if ctx is None:
        ctx = torch.empty(batch * seq, heads * 64, dtype=torch.bfloat16, device=qkv.device)
    _check(_lib.pd_attention_fwd(_dev(qkv, torch.bfloat16, "qkv"), _dev(ctx, torch.bfloat16, "ctx"), batch, seq,
                                 heads, _stream(stream)), "pd_attention_fwd")
    return ctx


@dataclass
class EncoderLayerParams:
    """Device tensors of one layer (bf16 matrices [in, out], fp32 vectors)."""
    w_qkv: torch.Tensor
    w_o: torch.Tensor
    w_ffn1: torch.Tensor
    w_ffn2: torch.Tensor
    b_qkv: torch.Tensor
    b_o: torch.Tensor
    b_ffn1: torch.Tensor
    b_ffn2: torch.Tensor
    ln1_gamma: torch.Tensor
    ln1_beta: torch.Tensor
    ln2_gamma: torch.Tensor
    ln2_beta: torch.Tensor

    def as_struct(self) -> EncoderLayerWeights:
        s = EncoderLayerWeights()
        for name in ("w_qkv", "w_o", "w_ffn1", "w_ffn2"):
            setattr(s, name, _dev(getattr(self, name), torch.bfloat16, name))
        for name in ("b_qkv", "b_o", "b_ffn1", "b_ffn2", "ln1_gamma", "ln1_beta", "ln2_gamma", "ln2_beta"):
            setattr(s, name, _dev(getattr(self, name), torch.float32, name))
        return s


def pd_encoder_layer_workspace_bytes(batch: int, seq: int, hidden: int, heads: int, ffn: int,
                                     ln_eps: float = 1e-5) -> int:
    d = EncoderLayerDesc(batch, seq, hidden, heads, ffn, ln_eps)
    return int(_lib.pd_encoder_layer_workspace_bytes(ctypes.byref(d)))


LAYER_BUFFERS = ("qkv", "scores", "probs", "ctx", "pre", "h1", "mid")


def pd_encoder_layer_workspace_layout(batch: int, seq: int, hidden: int, heads: int, ffn: int,
                                      ln_eps: float = 1e-5) -> dict:
    """{buffer name: (byte offset, byte size)} of the layer's intermediates inside its workspace."""
    d = EncoderLayerDesc(batch, seq, hidden, heads, ffn, ln_eps)
    n = len(LAYER_BUFFERS)
    off, size = (ctypes.c_size_t * n)(), (ctypes.c_size_t * n)()
    _check(_lib.pd_encoder_layer_workspace_layout(ctypes.byref(d), off, size), "pd_encoder_layer_workspace_layout")
    return {name: (int(off[i]), int(size[i])) for i, name in enumerate(LAYER_BUFFERS)}


def pd_encoder_layer_fwd(params: EncoderLayerParams, x: torch.Tensor, *, batch: int, seq: int, heads: int,
                         ln_eps: float = 1e-5, y: torch.Tensor | None = None,
                         workspace: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    T, hidden = x.shape
    if T != batch * seq:
        raise ValueError("x must be [batch*seq, hidden]")
    ffn = params.w_ffn1.shape[1]
    d = EncoderLayerDesc(batch, seq, hidden, heads, ffn, ln_eps)
    if y is None:
        y = torch.empty_like(x)
    if workspace is None:
        nbytes = int(_lib.pd_encoder_layer_workspace_bytes(ctypes.byref(d)))
        workspace = torch.empty(max(nbytes, 1), dtype=torch.uint8, device=x.device)
    w = params.as_struct()
    _check(_lib.pd_encoder_layer_fwd(ctypes.byref(d), ctypes.byref(w), _dev(x, torch.bfloat16, "x"),
                                     _dev(y, torch.bfloat16, "y"), workspace.data_ptr(), workspace.numel(),
                                     _stream(stream)), "pd_encoder_layer_fwd")
    return y


def pd_encoder_stack_fwd(layers, x: torch.Tensor, *, batch: int, seq: int, heads: int, ln_eps: float = 1e-5,
                         y: torch.Tensor | None = None, workspace: torch.Tensor | None = None, stream=None):
    """Runs ``layers`` (a list of EncoderLayerParams of one shape) one after the other on x [batch*seq, hidden]."""
    T, hidden = x.shape
    if T != batch * seq:
        raise ValueError("x must be [batch*seq, hidden]")
    d = EncoderLayerDesc(batch, seq, hidden, heads, layers[0].w_ffn1.shape[1], ln_eps)
    if y is None:
        y = torch.empty_like(x)
    if workspace is None:
        nbytes = int(_lib.pd_encoder_stack_workspace_bytes(ctypes.byref(d), len(layers)))
        workspace = torch.empty(max(nbytes, 1), dtype=torch.uint8, device=x.device)
    w = (EncoderLayerWeights * len(layers))(*[p.as_struct() for p in layers])
    _check(_lib.pd_encoder_stack_fwd(ctypes.byref(d), w, len(layers), _dev(x, torch.bfloat16, "x"),
                                     _dev(y, torch.bfloat16, "y"), workspace.data_ptr(), workspace.numel(),
                                     _stream(stream)), "pd_encoder_stack_fwd")
    return y


def pd_encoder_layer_static_scratch_bytes() -> int:
    return int(_lib.pd_encoder_layer_static_scratch_bytes())


def pd_encoder_layer_fwd_static(params: EncoderLayerParams, x: torch.Tensor, y: torch.Tensor, *, batch: int,
                                seq: int, heads: int, ln_eps: float = 1e-5, stream=None) -> torch.Tensor:
    """The layer for callers that cannot allocate: intermediates live in the
    library's fixed 32 MiB device array, and the caller passes the output tensor
    too, so neither this binding nor the library allocates anything."""
    T, hidden = x.shape
    if T != batch * seq:
        raise ValueError("x must be [batch*seq, hidden]")
    d = EncoderLayerDesc(batch, seq, hidden, heads, params.w_ffn1.shape[1], ln_eps)
    w = params.as_struct()
    _check(_lib.pd_encoder_layer_fwd_static(ctypes.byref(d), ctypes.byref(w), _dev(x, torch.bfloat16, "x"),
                                            _dev(y, torch.bfloat16, "y"), _stream(stream)),
           "pd_encoder_layer_fwd_static")
    return y


def pd_encoder_layer_kernel_count(batch: int, seq: int, hidden: int, heads: int, ffn: int) -> int:
    d = EncoderLayerDesc(batch, seq, hidden, heads, ffn, 1e-5)
    return int(_lib.pd_encoder_layer_kernel_count(ctypes.byref(d)))


def pd_encoder_layer_stage_names() -> list[str]:
    return [_lib.pd_encoder_layer_stage_name(i).decode() for i in range(_lib.pd_encoder_layer_stage_count())]


def pd_encoder_layer_fwd_profiled(params: EncoderLayerParams, x: torch.Tensor, *, batch: int, seq: int, heads: int,
                                  ln_eps: float = 1e-5, y: torch.Tensor | None = None,
                                  workspace: torch.Tensor | None = None, stream=None):
    """Runs the layer with per-stage CUDA events; returns (y, {stage name: ms})."""
    T, hidden = x.shape
    if T != batch * seq:
        raise ValueError("x must be [batch*seq, hidden]")
    d = EncoderLayerDesc(batch, seq, hidden, heads, params.w_ffn1.shape[1], ln_eps)
    if y is None:
        y = torch.empty_like(x)
    if workspace is None:
        nbytes = int(_lib.pd_encoder_layer_workspace_bytes(ctypes.byref(d)))
        workspace = torch.empty(max(nbytes, 1), dtype=torch.uint8, device=x.device)
    w = params.as_struct()
    n = _lib.pd_encoder_layer_stage_count()
    ms = (ctypes.c_float * n)()
    _check(_lib.pd_encoder_layer_fwd_profiled(ctypes.byref(d), ctypes.byref(w), _dev(x, torch.bfloat16, "x"),
                                              _dev(y, torch.bfloat16, "y"), workspace.data_ptr(),
                                              workspace.numel(), _stream(stream), ms), "pd_encoder_layer_fwd_profiled")
    return y, dict(zip(pd_encoder_layer_stage_names(), [float(v) for v in ms]))


def pd_get_device_status() -> int:
    code = ctypes.c_int(0)
    st = _lib.pd_get_device_status(ctypes.byref(code))
    if st not in (PD_OK, 7):
        raise PdError(st, "pd_get_device_status")
    return code.value


def pd_clear_device_status() -> None:
    _check(_lib.pd_clear_device_status(), "pd_clear_device_status")


def pd_debug_set_wait_limit_ns(limit_ns: int) -> None:
    """Time after which a wait inside the single-CTA contraction kernel gives up (default 2 s)."""
    _check(_lib.pd_debug_set_wait_limit_ns(int(limit_ns)), "pd_debug_set_wait_limit_ns")


def pd_debug_withhold_loads(on: bool) -> None:
    """Test switch: the single-CTA contraction kernel's producer issues no load, so a bounded wait runs out."""
    _check(_lib.pd_debug_withhold_loads(int(bool(on))), "pd_debug_withhold_loads")
