/* pd.h - C ABI of the B200 (sm_100a) encoder-layer operator library.
 *
 * The operators are the ones the paper's search system exists to generate
 * (Table "ML operators optimized using PerfLLM": softmax, layernorm, matmul,
 * bmm, add), written in the loop-nest notation of Section 2.1
 * "Representation" / Table "Supported representation features in PerfDojo",
 * and chained into the forward pass of one post-LN transformer encoder layer.
 *
 * Conventions common to every entry point
 *  - Pointers are DEVICE pointers unless a comment says "host".  The caller owns
 *    every buffer (workspace included); the library allocates no device memory
 *    and keeps no pointer after it returns.
 *  - Tensors are dense and row-major.  Sizes are in elements, strides (ld*) too.
 *  - Calls validate their arguments on the host, enqueue work on `stream` and
 *    return without synchronising.  On an argument error (every status but
 *    PD_ERR_CUDA) nothing has been enqueued.  The single-kernel entry points
 *    enqueue nothing on PD_ERR_CUDA either; the chained ones
 *    (pd_encoder_layer_fwd and its variants, pd_encoder_stack_fwd) stop at the
 *    launch that failed, with earlier kernels already on the stream: after
 *    PD_ERR_CUDA from them, y and the workspace hold unspecified values.
 *  - PD_OK means "enqueued".  The tensor-core entry points (pd_gemm_*,
 *    pd_swiglu_gemm, pd_attention_fwd, the layer and stack calls) bound every
 *    wait inside their kernels; a kernel whose wait ran out returns early and
 *    leaves a code in the device status word, so their results are valid only
 *    if pd_get_device_status reports 0 after the stream has been synchronised.
 *    The word is shared by all streams of the device.
 *  - A zero outer extent (rows == 0, M == 0, N == 0, batch == 0) is PD_OK and
 *    launches nothing; a zero reduction extent (cols == 0, K == 0) is
 *    PD_ERR_BAD_SHAPE.
 *  - Results are deterministic: no atomics, fixed reduction trees.
 *  - The current device must be compute capability 10.x, else PD_ERR_UNSUPPORTED.
 *  - There is no CPU fallback of any kind.
 */
#ifndef PD_H_
#define PD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef PD_NO_CUDA_HEADERS
typedef struct CUstream_st* cudaStream_t;
#else
#include <cuda_runtime_api.h>
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  PD_OK = 0,
  PD_ERR_NULL_POINTER = 1,
  PD_ERR_BAD_SHAPE = 2,
  PD_ERR_UNSUPPORTED = 3,
  PD_ERR_ALIGNMENT = 4,
  PD_ERR_WORKSPACE_TOO_SMALL = 5,
  PD_ERR_CUDA = 6,
  PD_ERR_DEVICE_TIMEOUT = 7
} pd_status;

typedef enum { PD_BF16 = 0, PD_F32 = 1 } pd_dtype;

/* Human-readable name of a status; static storage, never null. */
const char* pd_status_string(pd_status status);

/* cudaError_t (as int) behind the calling thread's most recent PD_ERR_CUDA. */
int pd_last_cuda_error(void);

/* Every bounded wait inside the tensor-core kernels records a non-zero code in
 * a device status word when it gives up (the kernel then drains and returns
 * instead of hanging).  This call synchronises the current device, copies the
 * word to *code (host pointer; 0 = no timeout since the last clear), and
 * returns PD_ERR_DEVICE_TIMEOUT if it is non-zero.  pd_clear_device_status
 * resets it. */
pd_status pd_get_device_status(int* code);
pd_status pd_clear_device_status(void);

/* Test aids for the bounded waits (the analogue of the run and compile
 * time-outs of the paper's search loop, Sections 4.2.3 "Performance on x86" and
 * 4.3 "Search with PerfLLM": a candidate that does not finish is cut off and
 * reported, it does not take the system down).
 * pd_debug_set_wait_limit_ns: the time after which a wait inside the single-CTA
 * and the CTA-pair contraction kernels (pd_set_gemm_tile_mode(1) / (2)) gives
 * up, 1 us to 10 s (else PD_ERR_BAD_SHAPE); default 2 s.
 * pd_debug_withhold_loads(1): those kernels' producers issue no load, so the
 * warp that feeds the tensor core waits for its first operand stage in vain,
 * gives up after the limit, records code 102 in the device status word, and
 * every role of the kernel drains and returns (in the pair kernel the partner
 * CTA's epilogue warps give up on their own wait for the accumulator, code
 * 104 if they are first; nothing faults, traps or stays behind; the output is
 * not written).
 * pd_debug_withhold_loads(0) restores normal operation.  Both settings are
 * process-wide and apply to launches enqueued after the call. */
pd_status pd_debug_set_wait_limit_ns(uint64_t limit_ns);
pd_status pd_debug_withhold_loads(int on);

/* Row-wise softmax over the last dimension (operator "softmax" of the paper's
 * operator table; reduction, broadcast and element-wise features):
 *   y[i,j] = exp(x[i,j] - m_i) / sum_j exp(x[i,j] - m_i),  m_i = max_j x[i,j].
 * x, y: fp32 [rows, cols], contiguous rows (ld == cols).  y may alias x.
 * Fast paths need 16-byte aligned pointers and cols % 4 == 0; other shapes take
 * a slower GPU path.  fp32 arithmetic, full-precision expf. */
pd_status pd_softmax(const float* x, float* y, int64_t rows, int64_t cols, cudaStream_t stream);

/* Layer normalisation over the last dimension (operators "layernorm 1/2"):
 *   mu_i = mean_j x[i,j];  var_i = mean_j (x[i,j] - mu_i)^2   (biased, 1/cols)
 *   y[i,j] = (x[i,j] - mu_i) / sqrt(var_i + eps) * gamma[j] + beta[j].
 * x, y: fp32 [rows, cols]; gamma, beta: fp32 [cols].  y may alias x. */
pd_status pd_layernorm(const float* x, const float* gamma, const float* beta, float* y,
                       int64_t rows, int64_t cols, float eps, cudaStream_t stream);

/* Root-mean-square normalisation over the last dimension (operator "rmsnorm" of
 * the paper's table, 3072 x 4096):
 *   y[i,j] = x[i,j] / sqrt(mean_j x[i,j]^2 + eps) * gamma[j].
 * x, y: fp32 [rows, cols]; gamma: fp32 [cols].  y may alias x. */
pd_status pd_rmsnorm(const float* x, const float* gamma, float* y, int64_t rows, int64_t cols, float eps,
                     cudaStream_t stream);

/* Fused bias + GELU(erf) + residual in one pass over HBM (element-wise and
 * broadcast features; nearest paper operators "add" and "relu"):
 *   out[i,j] = GELU(x[i,j] + bias[j]) + r[i,j],  GELU(z) = z/2 * (1 + erf(z/sqrt 2)).
 * x, out: fp32 [rows, cols]; bias: fp32 [cols]; r: fp32 [rows, cols] or NULL
 * (no residual term).  out may alias x or r. */
pd_status pd_bias_gelu_residual(const float* x, const float* bias, const float* r, float* out,
                                int64_t rows, int64_t cols, cudaStream_t stream);

/* bf16 matrix product with fp32 accumulation on the tcgen05 tensor cores
 * (operators "matmul" and, with batch > 1, "bmm"):
 *   C[b][m,n] = sum_k A[b][m,k] * B[b][k,n].
 * A: bf16 [M, K], row stride lda.  B: bf16, either [K, N] with row stride ldb
 * (b_is_nk == 0) or stored transposed as [N, K] with row stride ldb
 * (b_is_nk == 1).  C: [M, N], row stride ldc, bf16 (round-to-nearest-even) or
 * fp32 per c_dtype.  Problem b starts strideA/strideB/strideC elements after
 * problem b-1 (ignored when batch == 1).
 * Requirements: 16-byte aligned base pointers; lda, ldb, strideA, strideB
 * multiples of 8 elements; ldc * sizeof(C element) and strideC * sizeof(C
 * element) multiples of 16 bytes (else PD_ERR_ALIGNMENT); ld* at least the
 * row length; M, N, K otherwise arbitrary (ragged edges are zero-filled on load
 * and clipped on store: nothing beyond column N - 1 of a row of C is written,
 * also when ldc > N; a row end that does not fall on a 16-byte boundary is
 * written with plain stores instead of a bulk tensor store).  C must not
 * overlap A or B. */
pd_status pd_gemm_bf16(const void* A, const void* B, void* C, int64_t M, int64_t N, int64_t K,
                       int64_t lda, int64_t ldb, int64_t ldc, int b_is_nk, pd_dtype c_dtype,
                       int64_t batch, int64_t strideA, int64_t strideB, int64_t strideC,
                       cudaStream_t stream);

/* Tuning and testing aid for every contraction the library launches (it has no
 * counterpart in the paper).  mode 0 (default): choose automatically between
 * 128 x BN tiles computed by one CTA and 256 x 256 tiles computed by a pair of
 * CTAs (tcgen05 cta_group::2); mode 1: single-CTA tiles only; mode 2: CTA-pair
 * tiles for every shape.  Results do not depend on the mode beyond fp32
 * summation order inside the tensor core (identical here: both walk k in
 * ascending 16-element steps).  Process-wide, not thread-safe against
 * concurrent launches.  Other values: PD_ERR_BAD_SHAPE. */
pd_status pd_set_gemm_tile_mode(int mode);

/* Mean over the last dimension (operator "reducemean" of the paper's table,
 * 4096 x 4096; the reduction LayerNorm's first statistic also takes):
 *   y[i] = (1 / cols) * sum_j x[i,j].
 * x: fp32 [rows, cols], contiguous rows; y: fp32 [rows]; device pointers, 4-byte
 * aligned (else PD_ERR_ALIGNMENT; 16-byte aligned x with cols % 4 == 0 takes the
 * vector path).  fp32 arithmetic, tree-shaped summation.  rows = 0 is a no-op. */
pd_status pd_reducemean(const float* x, float* y, int64_t rows, int64_t cols, cudaStream_t stream);

/* Contraction with the fused epilogue the encoder layer's projections use
 * (operators "matmul", "add" and "relu" of the paper's table "ML operators
 * optimized using PerfLLM" in one kernel; GELU is the activation of the
 * layer's feed-forward block):
 *   C = act(A B + bias) + residual
 * A: bf16 [M, K]; B: bf16 [K, N]; bias: fp32 [N] or NULL; residual: bf16 [M, N]
 * or NULL; C: bf16 or fp32 [M, N] (c_dtype); all row-major, contiguous, device
 * pointers, 16-byte aligned, K and N multiples of 8 (else PD_ERR_ALIGNMENT).
 * act: 0 none, 1 GELU in its erf form z Phi(z), 2 ReLU max(z, 0); other values
 * PD_ERR_BAD_SHAPE.  Accumulation and the epilogue are fp32; the result is
 * rounded once, to c_dtype.  M = 0 or N = 0 is a no-op.  The caller owns every
 * buffer; C must not overlap an input. */
pd_status pd_gemm_bias_act(const void* A, const void* B, const float* bias, const void* residual, void* C,
                           int64_t M, int64_t N, int64_t K, int act, pd_dtype c_dtype, cudaStream_t stream);

/* SwiGLU feed-forward projection (operator "swiglu", 1 x 256 x 4096 x 448, of
 * the same table, read as 256 tokens, 4096 inputs, 448 outputs):
 *   Y = SiLU(X Wg) * (X Wu),   SiLU(g) = g / (1 + exp(-g)),
 * the two contractions and the element-wise product in one kernel: each
 * accumulator tile holds the gate and the up product of the same output
 * columns.  X: bf16 [M, K]; Wg, Wu: bf16 [K, N]; Y: bf16 [M, N]; row-major,
 * contiguous, device pointers, 16-byte aligned, K and N multiples of 8 (else
 * PD_ERR_ALIGNMENT).  Accumulation and the activation are fp32; Y is rounded
 * once, to bf16.  M = 0 or N = 0 is a no-op.  The caller owns every buffer; Y
 * must not overlap an input. */
pd_status pd_swiglu_gemm(const void* X, const void* Wg, const void* Wu, void* Y, int64_t M, int64_t N, int64_t K,
                         cudaStream_t stream);

/* Contraction with a LayerNorm epilogue: operators "matmul"/"bmm", "add" and
 * "layernorm" of the paper's table "ML operators optimized using PerfLLM" as
 * one kernel (its Section on fusing operators motivates keeping intermediates
 * out of memory):
 *   S[m, :] = A[m, :] B + bias + residual[m, :]              (fp32)
 *   Y[m, :] = (S[m, :] - mean_m) / sqrt(var_m + eps) * gamma + beta
 * with mean_m and the biased variance var_m taken over the N columns of row m.
 * A: bf16 [M, K]; B: bf16 [K, N]; bias: fp32 [N] or NULL; residual: bf16 [M, N]
 * or NULL; gamma, beta: fp32 [N]; Y: bf16 [M, N]; all row-major, contiguous,
 * device pointers, 16-byte aligned, K a multiple of 8 (else PD_ERR_ALIGNMENT).
 * N must be a multiple of 256 and at most 2048 (the N / 256 CTAs holding one
 * row block form a thread-block cluster and exchange row statistics through
 * distributed shared memory), else PD_ERR_UNSUPPORTED.  The caller owns every
 * buffer; Y must not overlap an input.  M = 0 is a no-op.  Accumulation, the
 * sum S and the statistics are fp32; only Y is rounded to bf16. */
pd_status pd_gemm_bias_residual_layernorm(const void* A, const void* B, const float* bias, const void* residual,
                                          const float* gamma, const float* beta, void* Y, int64_t M, int64_t N,
                                          int64_t K, float eps, cudaStream_t stream);

/* Tuning and testing aid (no counterpart in the paper).  mode 0 (default): a
 * contraction with K >= 2048 whose output tiles would cover less than half of
 * the SMs (the paper's swiglu 256 x 448 x 4096 is such a problem) is split
 * along K over a thread-block cluster of 2, 4 or 8 CTAs
 * that add their partial sums through distributed shared memory before the
 * epilogue; results differ from the unsplit kernels only by fp32 summation
 * order.  mode 1: never split.  Splitting applies only under
 * pd_set_gemm_tile_mode(0).  Process-wide, not thread-safe against concurrent
 * launches.  Other values: PD_ERR_BAD_SHAPE. */
pd_status pd_set_gemm_split_k(int mode);

/* Fused multi-head scaled-dot-product attention (operators "bmm", "softmax",
 * "bmm" of the paper's table chained per head; scores and probabilities stay
 * on the SM).  qkv: bf16 [batch*seq, 3*heads*64] = column blocks [Q | K | V],
 * head h in columns 64h..64h+63 of each block, token t = b*seq + s.
 *   ctx[b, :, 64h..64h+63] = softmax(Q[b,h] K[b,h]^T / 8) V[b,h]
 * ctx: bf16 [batch*seq, heads*64]; must not overlap qkv.  Head dimension is 64
 * and 1 <= seq <= 512 (else PD_ERR_UNSUPPORTED).  Softmax is exact for any
 * finite input and computed in fp32: every row is referred to a running
 * reference exponent that is raised, with what has been accumulated rescaled,
 * before an exponential could overflow.  Probabilities are rounded to bf16 for
 * the second product, which accumulates in fp32. */
pd_status pd_attention_fwd(const void* qkv, void* ctx, int64_t batch, int64_t seq, int64_t heads,
                           cudaStream_t stream);

/* Shape of one post-LN encoder layer (BERT-large: 32 x 512 tokens, hidden 1024,
 * 16 heads of 64, FFN 4096).  hidden must equal heads * 64 and ffn must be a
 * multiple of 8; seq must be at most 512 or a multiple of 8 (longer sequences
 * take an unfused attention path that materialises scores in the workspace);
 * anything else is PD_ERR_UNSUPPORTED. */
typedef struct {
  int32_t batch, seq, hidden, heads, ffn;
  float ln_eps;
} pd_encoder_layer_desc;

/* Weights of one layer.  Matrices are bf16 [in, out] row-major: w_qkv
 * [hidden, 3*hidden] with column blocks [Q | K | V] and head h in columns
 * 64h..64h+63 of each block; w_o [hidden, hidden]; w_ffn1 [hidden, ffn];
 * w_ffn2 [ffn, hidden].  Biases and LayerNorm parameters are fp32 vectors. */
typedef struct {
  const void *w_qkv, *w_o, *w_ffn1, *w_ffn2;
  const float *b_qkv, *b_o, *b_ffn1, *b_ffn2;
  const float *ln1_gamma, *ln1_beta, *ln2_gamma, *ln2_beta;
} pd_encoder_layer_weights;

/* Bytes of caller-provided device workspace pd_encoder_layer_fwd needs for
 * `desc` (0 if desc is NULL or invalid). */
size_t pd_encoder_layer_workspace_bytes(const pd_encoder_layer_desc* desc);

/* Where the intermediates of pd_encoder_layer_fwd live inside its workspace, for
 * callers that want to inspect them (the stage-by-stage validation of the
 * paper's Section 2.2 "Transformations": every transformed program is compared
 * with the original).  offsets[i] and sizes[i] (host arrays of
 * PD_LAYER_BUFFER_COUNT entries, bytes) describe buffer i under the current
 * fusion mode; a buffer the layer does not materialise for `desc` has size 0.
 *   PD_LAYER_BUF_QKV    bf16 [tokens, 3*hidden]     PD_LAYER_BUF_CTX  bf16 [tokens, hidden]
 *   PD_LAYER_BUF_SCORES fp32 [batch*heads*seq, seq] PD_LAYER_BUF_PRE  fp32 [tokens, hidden]
 *   PD_LAYER_BUF_PROBS  bf16 [batch*heads*seq, seq] PD_LAYER_BUF_H1   bf16 [tokens, hidden]
 *                                                   PD_LAYER_BUF_MID  bf16 [tokens, ffn]
 * NULL arguments: PD_ERR_NULL_POINTER; desc as for pd_encoder_layer_fwd. */
enum { PD_LAYER_BUF_QKV = 0, PD_LAYER_BUF_SCORES, PD_LAYER_BUF_PROBS, PD_LAYER_BUF_CTX, PD_LAYER_BUF_PRE,
       PD_LAYER_BUF_H1, PD_LAYER_BUF_MID, PD_LAYER_BUFFER_COUNT };
pd_status pd_encoder_layer_workspace_layout(const pd_encoder_layer_desc* desc, size_t* offsets, size_t* sizes);

/* Forward pass of one encoder layer, no dropout, no mask, token t = b*seq + s:
 *   QKV = X Wqkv + bqkv
 *   Ctx[b,h] = softmax(Q[b,h] K[b,h]^T / sqrt(64)) V[b,h]
 *   H1  = LayerNorm(Ctx Wo + bo + X; gamma1, beta1)
 *   Mid = GELU(H1 W1 + b1)
 *   Y   = LayerNorm(Mid W2 + b2 + H1; gamma2, beta2)
 * desc, weights: host structs (device pointers inside).  x, y: bf16
 * [batch*seq, hidden]; y must not overlap x or the workspace.  workspace: 256-
 * byte aligned, at least pd_encoder_layer_workspace_bytes(desc) bytes, else
 * PD_ERR_WORKSPACE_TOO_SMALL.  Contractions accumulate in fp32; softmax,
 * LayerNorm statistics and the pre-LayerNorm sums are fp32; Q, K, V, the
 * attention probabilities, Ctx, H1, Mid and Y are stored as bf16. */
pd_status pd_encoder_layer_fwd(const pd_encoder_layer_desc* desc, const pd_encoder_layer_weights* weights,
                               const void* x, void* y, void* workspace, size_t workspace_bytes,
                               cudaStream_t stream);

/* A stack of n_layers encoder layers of the same shape, each with its own
 * weights (weights: host array of n_layers structs), layer l + 1 reading what
 * layer l wrote (the paper's kernels come from whole models: its Section
 * "Search with PerfLLM" evaluates operators "in existing models"):
 *   X_0 = x,  X_{l+1} = layer_l(X_l),  y = X_{n_layers}.
 * Every layer is pd_encoder_layer_fwd; all of them are enqueued on `stream`
 * without host synchronisation, the activations between layers (bf16) alternate
 * between two tensors inside the workspace.  workspace: 256-byte aligned, at
 * least pd_encoder_stack_workspace_bytes(desc, n_layers) bytes (0 for an invalid
 * desc or n_layers < 1), else PD_ERR_WORKSPACE_TOO_SMALL.  Other arguments and
 * errors as for pd_encoder_layer_fwd; n_layers < 1 is PD_ERR_BAD_SHAPE. */
size_t pd_encoder_stack_workspace_bytes(const pd_encoder_layer_desc* desc, int n_layers);
pd_status pd_encoder_stack_fwd(const pd_encoder_layer_desc* desc, const pd_encoder_layer_weights* weights,
                               int n_layers, const void* x, void* y, void* workspace, size_t workspace_bytes,
                               cudaStream_t stream);

/* Tuning and testing aid for the layer entry points (no counterpart in the
 * paper, whose table lists "layernorm" as an operator of its own).  mode 0
 * (default): when hidden is a multiple of 256 and at most 2048, each of the two
 * LayerNorms runs inside the epilogue of the contraction that feeds it (the
 * CTAs that hold one row block's column tiles form a thread-block cluster and
 * exchange per-row means and centred second moments through distributed shared
 * memory), so the fp32 pre-LayerNorm tensor is never written; other hidden sizes use the separate row kernel.
 * mode 1: always the separate row kernel (the contraction writes the fp32 sum
 * to the workspace).  Both forms compute the statistics in fp32 from the same
 * fp32 sums and differ only in summation order.  The mode also decides how much
 * workspace pd_encoder_layer_workspace_bytes reports: set it before asking.
 * Process-wide, not thread-safe against concurrent calls.  Other values:
 * PD_ERR_BAD_SHAPE. */
pd_status pd_set_layernorm_fusion(int mode);

/* Allocation-free variant of pd_encoder_layer_fwd (the paper has no counterpart:
 * this entry point exists for integration reasons only).  Some callers cannot
 * obtain device memory at the point where they need a layer: a serving process
 * whose memory pool already owns the whole GPU, code running where a
 * cudaMalloc (which synchronises the device) is not acceptable, or a plug-in
 * that is handed inputs and outputs but no allocator.  For them the layer's
 * intermediates go into a fixed array of pd_encoder_layer_static_scratch_bytes()
 * = 32 MiB inside the library's device image (held by every GPU that loads the
 * library, until the process exits) instead of a caller-provided workspace.
 *  - Same arguments, results and error codes as pd_encoder_layer_fwd, minus the
 *    workspace, checked in the same order (the size check below stands where
 *    that call checks its workspace).  A shape whose intermediates need more than the array holds
 *    (pd_encoder_layer_workspace_bytes(desc) > 32 MiB; BERT-large fits up to
 *    about 1800 tokens, 1400 with the LayerNorms unfused) is rejected with
 *    PD_ERR_WORKSPACE_TOO_SMALL and nothing is enqueued.
 *  - The call allocates nothing: no cudaMalloc/cudaFree and no allocating
 *    library routine, on any call.
 *  - The first call on each device looks up the array's device address
 *    (cudaGetSymbolAddress, with that device current).  Make that first call
 *    before starting any stream capture.  Several host threads may make it at
 *    once (they store the same address).
 *  - All calls share the one array and it keeps whatever the previous call left
 *    there (every intermediate is fully rewritten before it is read, so nothing
 *    needs clearing).  Two calls that overlap on the GPU - different streams, or
 *    different host threads - race on it: serialise them. */
size_t pd_encoder_layer_static_scratch_bytes(void);
pd_status pd_encoder_layer_fwd_static(const pd_encoder_layer_desc* desc, const pd_encoder_layer_weights* weights,
                                      const void* x, void* y, cudaStream_t stream);

/* Measurement aid: the same forward pass with a CUDA event recorded around
 * every stage the driver enqueues (the paper's evaluation likewise times each
 * operator on its own, Section "Search with PerfLLM").  After enqueueing, the
 * call WAITS for the layer to finish and writes the device time of stage i, in
 * milliseconds, to stage_ms[i] (host pointer, pd_encoder_layer_stage_count()
 * floats).  pd_encoder_layer_stage_name(i) names stage i (static storage, ""
 * when out of range).  Results in y are identical to pd_encoder_layer_fwd.
 * A LayerNorm that runs inside its contraction's epilogue is timed with that
 * contraction, and its own stage reports (nearly) zero. */
int pd_encoder_layer_stage_count(void);
/* Number of kernels one pd_encoder_layer_fwd call enqueues for `desc` under the
 * current fusion mode (0 for an invalid, unsupported or empty desc): five for
 * BERT-large (QKV GEMM, attention, output projection + LayerNorm, FFN up + GELU,
 * FFN down + LayerNorm). */
int pd_encoder_layer_kernel_count(const pd_encoder_layer_desc* desc);
const char* pd_encoder_layer_stage_name(int stage);
pd_status pd_encoder_layer_fwd_profiled(const pd_encoder_layer_desc* desc,
                                        const pd_encoder_layer_weights* weights, const void* x, void* y,
                                        void* workspace, size_t workspace_bytes, cudaStream_t stream,
                                        float* stage_ms);

#ifdef __cplusplus
}
#endif
#endif /* PD_H_ */
