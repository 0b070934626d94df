// Forward pass of one post-LN transformer encoder layer: a host-side driver that
// chains the library's kernels on one stream with no host synchronisation.
//
//   QKV = X Wqkv + bqkv                                   (GEMM, bias epilogue)
//   Ctx = softmax(Q K^T / 8) V  per (batch, head)         (fused attention kernel for seq <= 512;
//                                                          otherwise batched GEMM, softmax, batched GEMM)
//   H1  = LayerNorm(Ctx Wo + bo + X)                      (GEMM with bias + residual + LayerNorm epilogue)
//   Mid = GELU(H1 W1 + b1)                                (GEMM, bias + GELU epilogue)
//   Y   = LayerNorm(Mid W2 + b2 + H1)                     (GEMM with bias + residual + LayerNorm epilogue)
// When the hidden size does not suit the fused LayerNorm epilogue (or it is switched off), the two
// LayerNorm GEMMs write their fp32 sum to a scratch tensor and the LayerNorm row kernel follows.
#include <atomic>

#include <nvtx3/nvToolsExt.h>

#include "pd_common.cuh"

namespace pd {
namespace {

constexpr int kHeadDim = 64;
constexpr size_t kAlign = 256;

inline size_t round_up(size_t v) { return (v + kAlign - 1) / kAlign * kAlign; }

struct Workspace {
  size_t qkv, scores, probs, ctx, pre, h1, mid, total;
};

bool valid_desc(const pd_encoder_layer_desc* d) {
  if (!d) return false;
  if (d->batch < 0 || d->seq <= 0 || d->hidden <= 0 || d->heads <= 0 || d->ffn <= 0) return false;
  if ((int64_t)d->batch * d->seq > 0x7fffffff) return false;  // the launchers index tokens with int
  if (!(d->ln_eps >= 0.f)) return false;
  return true;
}

bool supported_desc(const pd_encoder_layer_desc* d) {
  if (d->hidden != d->heads * kHeadDim || d->ffn % 8 != 0) return false;
  return fused_attention_supported(d->seq, kHeadDim) || d->seq % 8 == 0;
}

bool use_fused_attention(const pd_encoder_layer_desc* d) { return fused_attention_supported(d->seq, kHeadDim); }

int g_layernorm_fusion = 0;  // 0: fuse LayerNorm into the GEMM where the shape allows, 1: always separate kernels

bool use_fused_layernorm(const pd_encoder_layer_desc* d) {
  if (g_layernorm_fusion == 1) return false;
  GemmProblem g;
  g.M = (int64_t)d->batch * d->seq; g.N = d->hidden; g.K = d->hidden;
  return gemm_layernorm_supported(g);
}

Workspace plan(const pd_encoder_layer_desc* d) {
  const size_t T = (size_t)d->batch * d->seq, H = d->hidden, F = d->ffn, S = d->seq;
  // scores and probabilities are materialised only on the unfused attention path
  const size_t score_elems = use_fused_attention(d) ? 0 : (size_t)d->batch * d->heads * S * S;
  Workspace w{};
  size_t off = 0;
  w.qkv = off; off += round_up(T * 3 * H * 2);
  w.scores = off; off += round_up(score_elems * 4);
  w.probs = off; off += round_up(score_elems * 2);
  w.ctx = off; off += round_up(T * H * 2);
  // fp32 pre-LayerNorm sums: not materialised when the LayerNorm runs inside the GEMM
  w.pre = off; off += round_up(use_fused_layernorm(d) ? 0 : T * H * 4);
  w.h1 = off; off += round_up(T * H * 2);
  w.mid = off; off += round_up(T * F * 2);
  w.total = off;
  return w;
}

}  // namespace
}  // namespace pd

extern "C" size_t pd_encoder_layer_workspace_bytes(const pd_encoder_layer_desc* desc) {
  if (!pd::valid_desc(desc) || !pd::supported_desc(desc)) return 0;
  return pd::plan(desc).total;
}

extern "C" pd_status pd_encoder_layer_workspace_layout(const pd_encoder_layer_desc* desc, size_t* offsets,
                                                       size_t* sizes) {
  if (!desc || !offsets || !sizes) return PD_ERR_NULL_POINTER;
  if (!pd::valid_desc(desc)) return PD_ERR_BAD_SHAPE;
  if (!pd::supported_desc(desc)) return PD_ERR_UNSUPPORTED;
  const pd::Workspace w = pd::plan(desc);
  const size_t off[PD_LAYER_BUFFER_COUNT + 1] = {w.qkv, w.scores, w.probs, w.ctx, w.pre, w.h1, w.mid, w.total};
  for (int i = 0; i < PD_LAYER_BUFFER_COUNT; ++i) {
    offsets[i] = off[i];
    sizes[i] = off[i + 1] - off[i];  // the buffers follow one another in this order
  }
  return PD_OK;
}

namespace pd {
namespace {

constexpr int kStages = 7;
const char* const kStageNames[kStages] = {"qkv_gemm", "attention", "out_proj_gemm", "layernorm1",
                                          "ffn_up_gemm", "ffn_down_gemm", "layernorm2"};
const char* const kStageRangeNames[kStages] = {"pd.qkv_gemm", "pd.attention", "pd.out_proj_gemm", "pd.layernorm1",
                                               "pd.ffn_up_gemm", "pd.ffn_down_gemm", "pd.layernorm2"};

// Argument checks shared by every layer entry point: null pointers, then the shape, then alignment.
pd_status check_layer_args(const pd_encoder_layer_desc* desc, const pd_encoder_layer_weights* w, const void* x,
                           const void* y) {
  if (!desc || !w || !x || !y) return PD_ERR_NULL_POINTER;
  if (!w->w_qkv || !w->w_o || !w->w_ffn1 || !w->w_ffn2 || !w->b_qkv || !w->b_o || !w->b_ffn1 || !w->b_ffn2 ||
      !w->ln1_gamma || !w->ln1_beta || !w->ln2_gamma || !w->ln2_beta)
    return PD_ERR_NULL_POINTER;
  if (!valid_desc(desc)) return PD_ERR_BAD_SHAPE;
  if (!supported_desc(desc)) return PD_ERR_UNSUPPORTED;
  const void* ptrs[] = {x, y, w->w_qkv, w->w_o, w->w_ffn1, w->w_ffn2, w->b_qkv, w->b_o, w->b_ffn1, w->b_ffn2,
                        w->ln1_gamma, w->ln1_beta, w->ln2_gamma, w->ln2_beta};
  for (const void* p : ptrs)
    if (!aligned16(p)) return PD_ERR_ALIGNMENT;
  return PD_OK;
}

// Enqueues the whole layer.  When `ev` is not null it holds kStages + 1 events:
// ev[i] is recorded before stage i and ev[kStages] after the last one.
pd_status run_layer(const pd_encoder_layer_desc* desc, const pd_encoder_layer_weights* w, const void* x, void* y,
                    void* workspace, size_t workspace_bytes, cudaStream_t stream, cudaEvent_t* ev) {
  // Every stage is bracketed by an NVTX range named after it (host side, around the enqueueing calls), so that a
  // timeline tool shows the layer's structure; without a tool attached the calls do nothing.
  int stage = 0;
  bool range_open = false;
  auto mark = [&]() {
    if (range_open) nvtxRangePop();
    range_open = stage < kStages;
    if (range_open) nvtxRangePushA(kStageRangeNames[stage]);
    if (ev) cudaEventRecord(ev[stage], stream);
    ++stage;
  };
  struct RangeGuard {  // closes the open range on every return path
    bool& open;
    ~RangeGuard() {
      if (open) nvtxRangePop();
    }
  } guard{range_open};
  if (pd_status st0 = check_layer_args(desc, w, x, y); st0 != PD_OK) return st0;
  if (desc->batch == 0) return PD_OK;
  const Workspace ws = plan(desc);
  if (!workspace) return PD_ERR_NULL_POINTER;
  if (reinterpret_cast<uintptr_t>(workspace) % kAlign) return PD_ERR_ALIGNMENT;
  if (workspace_bytes < ws.total) return PD_ERR_WORKSPACE_TOO_SMALL;
  pd_status st = require_sm100();
  if (st != PD_OK) return st;

  const int64_t B = desc->batch, S = desc->seq, H = desc->hidden, NH = desc->heads, F = desc->ffn, T = B * S;
  logf("encoder layer batch %lld seq %lld hidden %lld heads %lld ffn %lld: attention %s, LayerNorms %s", (long long)B,
       (long long)S, (long long)H, (long long)NH, (long long)F, use_fused_attention(desc) ? "fused" : "as three launches",
       use_fused_layernorm(desc) ? "in the contractions' epilogues" : "as row kernels");
  uint8_t* base = static_cast<uint8_t*>(workspace);
  auto* qkv = reinterpret_cast<__nv_bfloat16*>(base + ws.qkv);
  auto* scores = reinterpret_cast<float*>(base + ws.scores);
  auto* probs = reinterpret_cast<__nv_bfloat16*>(base + ws.probs);
  auto* ctx = reinterpret_cast<__nv_bfloat16*>(base + ws.ctx);
  auto* pre = reinterpret_cast<float*>(base + ws.pre);
  auto* h1 = reinterpret_cast<__nv_bfloat16*>(base + ws.h1);
  auto* mid = reinterpret_cast<__nv_bfloat16*>(base + ws.mid);
  const auto* xb = static_cast<const __nv_bfloat16*>(x);

  mark();
  {  // QKV projection
    GemmProblem g;
    g.A = x; g.B = w->w_qkv; g.C = qkv; g.M = T; g.N = 3 * H; g.K = H; g.lda = H; g.ldb = 3 * H; g.ldc = 3 * H;
    g.bias = w->b_qkv;
    if ((st = launch_gemm(g, stream)) != PD_OK) return st;
  }
  mark();
  if (use_fused_attention(desc)) {
    if ((st = launch_fused_attention(qkv, ctx, B, S, NH, stream)) != PD_OK) return st;
  } else {
    {  // scores = Q K^T / sqrt(64), fp32, one [S, S] block per (batch, head)
      GemmProblem g;
      g.A = qkv; g.B = qkv + H; g.C = scores; g.M = S; g.N = S; g.K = kHeadDim; g.lda = 3 * H; g.ldb = 3 * H; g.ldc = S;
      g.b_is_nk = true; g.c_dtype = PD_F32; g.alpha = 0.125f;
      g.batch_inner = NH; g.batch_outer = B;
      g.strideA_inner = kHeadDim; g.strideA_outer = S * 3 * H;
      g.strideB_inner = kHeadDim; g.strideB_outer = S * 3 * H;
      g.strideC_inner = S * S; g.strideC_outer = NH * S * S;
      if ((st = launch_gemm(g, stream)) != PD_OK) return st;
    }
    if ((st = launch_softmax(scores, probs, true, B * NH * S, S, stream)) != PD_OK) return st;
    {  // Ctx = P V, heads written back to their column blocks
      GemmProblem g;
      g.A = probs; g.B = qkv + 2 * H; g.C = ctx; g.M = S; g.N = kHeadDim; g.K = S; g.lda = S; g.ldb = 3 * H; g.ldc = H;
      g.batch_inner = NH; g.batch_outer = B;
      g.strideA_inner = S * S; g.strideA_outer = NH * S * S;
      g.strideB_inner = kHeadDim; g.strideB_outer = S * 3 * H;
      g.strideC_inner = kHeadDim; g.strideC_outer = S * H;
      if ((st = launch_gemm(g, stream)) != PD_OK) return st;
    }
  }
  const bool fuse_ln = use_fused_layernorm(desc);
  mark();
  {  // output projection + bias + residual, then LayerNorm (in the epilogue, or from the fp32 sum)
    GemmProblem g;
    g.A = ctx; g.B = w->w_o; g.M = T; g.N = H; g.K = H; g.lda = H; g.ldb = H; g.ldc = H;
    g.bias = w->b_o; g.residual = xb; g.ldr = H;
    if (fuse_ln) {
      g.C = h1;
      if ((st = launch_gemm_layernorm(g, w->ln1_gamma, w->ln1_beta, desc->ln_eps, stream)) != PD_OK) return st;
      mark();
    } else {
      g.C = pre; g.c_dtype = PD_F32;
      if ((st = launch_gemm(g, stream)) != PD_OK) return st;
      mark();
      if ((st = launch_layernorm(pre, w->ln1_gamma, w->ln1_beta, h1, true, T, H, desc->ln_eps, stream)) != PD_OK)
        return st;
    }
  }
  mark();
  {  // FFN up + bias + GELU
    GemmProblem g;
    g.A = h1; g.B = w->w_ffn1; g.C = mid; g.M = T; g.N = F; g.K = H; g.lda = H; g.ldb = F; g.ldc = F;
    g.bias = w->b_ffn1; g.act = 1;
    if ((st = launch_gemm(g, stream)) != PD_OK) return st;
  }
  mark();
  {  // FFN down + bias + residual, then LayerNorm
    GemmProblem g;
    g.A = mid; g.B = w->w_ffn2; g.M = T; g.N = H; g.K = F; g.lda = F; g.ldb = H; g.ldc = H;
    g.bias = w->b_ffn2; g.residual = h1; g.ldr = H;
    if (fuse_ln) {
      g.C = y;
      // Mid (T x F bf16) exceeds L2 at the configured size and FFN-up wrote it first row first
      g.rows_descending = true;
      st = launch_gemm_layernorm(g, w->ln2_gamma, w->ln2_beta, desc->ln_eps, stream);
      mark();
    } else {
      g.C = pre; g.c_dtype = PD_F32;
      if ((st = launch_gemm(g, stream)) != PD_OK) return st;
      mark();
      st = launch_layernorm(pre, w->ln2_gamma, w->ln2_beta, y, true, T, H, desc->ln_eps, stream);
    }
  }
  mark();
  return st;
}

}  // namespace
}  // namespace pd

extern "C" pd_status pd_encoder_layer_fwd(const pd_encoder_layer_desc* desc, const pd_encoder_layer_weights* w,
                                          const void* x, void* y, void* workspace, size_t workspace_bytes,
                                          cudaStream_t stream) {
  return pd::run_layer(desc, w, x, y, workspace, workspace_bytes, stream, nullptr);
}

// ---- a stack of layers ---------------------------------------------------------
extern "C" size_t pd_encoder_stack_workspace_bytes(const pd_encoder_layer_desc* desc, int n_layers) {
  if (!pd::valid_desc(desc) || !pd::supported_desc(desc) || n_layers < 1) return 0;
  const size_t act = pd::round_up((size_t)desc->batch * desc->seq * desc->hidden * 2);
  return pd::plan(desc).total + (n_layers > 1 ? 2 * act : 0);
}

extern "C" pd_status pd_encoder_stack_fwd(const pd_encoder_layer_desc* desc, const pd_encoder_layer_weights* weights,
                                          int n_layers, const void* x, void* y, void* workspace,
                                          size_t workspace_bytes, cudaStream_t stream) {
  using namespace pd;
  if (!desc || !weights || !x || !y) return PD_ERR_NULL_POINTER;
  if (!valid_desc(desc) || n_layers < 1) return PD_ERR_BAD_SHAPE;
  if (!supported_desc(desc)) return PD_ERR_UNSUPPORTED;
  if (desc->batch == 0) return PD_OK;
  if (!workspace) return PD_ERR_NULL_POINTER;
  if (reinterpret_cast<uintptr_t>(workspace) % kAlign) return PD_ERR_ALIGNMENT;
  if (workspace_bytes < pd_encoder_stack_workspace_bytes(desc, n_layers)) return PD_ERR_WORKSPACE_TOO_SMALL;
  // layout: the layer's own workspace, then two activation tensors the layers alternate between
  const size_t layer_bytes = plan(desc).total;
  const size_t act = round_up((size_t)desc->batch * desc->seq * desc->hidden * 2);
  uint8_t* base = static_cast<uint8_t*>(workspace);
  void* pong[2] = {base + layer_bytes, base + layer_bytes + act};
  const void* in = x;
  for (int l = 0; l < n_layers; ++l) {
    void* out = l == n_layers - 1 ? y : pong[l & 1];
    const pd_status st = run_layer(desc, weights + l, in, out, workspace, layer_bytes, stream, nullptr);
    if (st != PD_OK) return st;
    in = out;
  }
  return PD_OK;
}

extern "C" pd_status pd_set_layernorm_fusion(int mode) {
  if (mode < 0 || mode > 1) return PD_ERR_BAD_SHAPE;
  pd::g_layernorm_fusion = mode;
  return PD_OK;
}

extern "C" int pd_encoder_layer_kernel_count(const pd_encoder_layer_desc* desc) {
  if (!pd::valid_desc(desc) || !pd::supported_desc(desc) || desc->batch == 0) return 0;
  return 1 + (pd::use_fused_attention(desc) ? 1 : 3) + 1 + (pd::use_fused_layernorm(desc) ? 2 : 4);
}

extern "C" int pd_encoder_layer_stage_count(void) { return pd::kStages; }

extern "C" const char* pd_encoder_layer_stage_name(int stage) {
  return (stage >= 0 && stage < pd::kStages) ? pd::kStageNames[stage] : "";
}

extern "C" pd_status pd_encoder_layer_fwd_profiled(const pd_encoder_layer_desc* desc,
                                                   const pd_encoder_layer_weights* w, const void* x, void* y,
                                                   void* workspace, size_t workspace_bytes, cudaStream_t stream,
                                                   float* stage_ms) {
  using namespace pd;
  if (!stage_ms) return PD_ERR_NULL_POINTER;
  cudaEvent_t ev[kStages + 1];
  int created = 0;
  cudaError_t e = cudaSuccess;
  for (; created <= kStages; ++created)
    if ((e = cudaEventCreate(&ev[created])) != cudaSuccess) break;
  pd_status st = e == cudaSuccess ? PD_OK : record_cuda_error(e);
  if (st == PD_OK) st = run_layer(desc, w, x, y, workspace, workspace_bytes, stream, ev);
  if (st == PD_OK) {
    // an empty batch records nothing: report zeros
    const bool ran = desc->batch > 0;
    if (ran && (e = cudaEventSynchronize(ev[kStages])) != cudaSuccess) st = record_cuda_error(e);
    for (int i = 0; i < kStages && st == PD_OK; ++i) {
      stage_ms[i] = 0.f;
      if (ran && (e = cudaEventElapsedTime(&stage_ms[i], ev[i], ev[i + 1])) != cudaSuccess) st = record_cuda_error(e);
    }
  }
  for (int i = 0; i < created; ++i) cudaEventDestroy(ev[i]);
  return st;
}

extern "C" pd_status pd_attention_fwd(const void* qkv, void* ctx, int64_t batch, int64_t seq, int64_t heads,
                                      cudaStream_t stream) {
  using namespace pd;
  if (!qkv || !ctx) return PD_ERR_NULL_POINTER;
  if (batch < 0 || seq <= 0 || heads <= 0 || batch > 0x7fffffff || heads > 0x7fffffff) return PD_ERR_BAD_SHAPE;
  if (!fused_attention_supported(seq, kHeadDim)) return PD_ERR_UNSUPPORTED;
  if (!aligned16(qkv) || !aligned16(ctx)) return PD_ERR_ALIGNMENT;
  if (batch == 0) return PD_OK;
  pd_status st = require_sm100();
  if (st != PD_OK) return st;
  return launch_fused_attention(static_cast<const __nv_bfloat16*>(qkv), static_cast<__nv_bfloat16*>(ctx), batch, seq,
                                heads, stream);
}

// ---- allocation-free variant ---------------------------------------------------
// Scratch for callers that cannot hand the library a workspace of their own.
// The array lives in the library's device image: every GPU that loads the
// library carries these bytes until the process exits.
#define PD_STATIC_SCRATCH_BYTES (32u << 20)
static __device__ __align__(256) unsigned char g_layer_scratch[PD_STATIC_SCRATCH_BYTES];

namespace pd {
namespace {

// Device address of g_layer_scratch on the current device.  In host code the
// symbol's name is only a handle, never an address a kernel may be given, so
// the address is looked up once per device (with that device current).
pd_status static_scratch_ptr(void** out) {
  constexpr int kMaxDevices = 64;
  static std::atomic<void*> cached[kMaxDevices];  // two threads making the first call store the same address
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return record_cuda_error(e);
  if (dev < 0 || dev >= kMaxDevices) return PD_ERR_UNSUPPORTED;
  void* ptr = cached[dev].load(std::memory_order_acquire);
  if (!ptr) {
    e = cudaGetSymbolAddress(&ptr, g_layer_scratch);
    if (e != cudaSuccess) return record_cuda_error(e);
    if (!ptr) return PD_ERR_CUDA;
    cached[dev].store(ptr, std::memory_order_release);
  }
  *out = ptr;
  return PD_OK;
}

}  // namespace
}  // namespace pd

extern "C" size_t pd_encoder_layer_static_scratch_bytes(void) { return PD_STATIC_SCRATCH_BYTES; }

extern "C" pd_status pd_encoder_layer_fwd_static(const pd_encoder_layer_desc* desc,
                                                 const pd_encoder_layer_weights* w, const void* x, void* y,
                                                 cudaStream_t stream) {
  using namespace pd;
  // the same checks in the same order as pd_encoder_layer_fwd, so that an argument with several faults is
  // reported alike by both; the size check comes where that call checks its workspace
  if (pd_status st = check_layer_args(desc, w, x, y); st != PD_OK) return st;
  if (desc->batch == 0) return PD_OK;
  if (plan(desc).total > PD_STATIC_SCRATCH_BYTES) return PD_ERR_WORKSPACE_TOO_SMALL;
  void* scratch = nullptr;
  pd_status st = static_scratch_ptr(&scratch);
  if (st != PD_OK) return st;
  return run_layer(desc, w, x, y, scratch, PD_STATIC_SCRATCH_BYTES, stream, nullptr);
}
