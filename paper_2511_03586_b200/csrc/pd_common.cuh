// Shared host/device helpers of the pd library (internal; not part of the C ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "pd.h"

namespace pd {

constexpr int kWarp = 32;

// ---- host side -----------------------------------------------------------
// Records `e` for pd_last_cuda_error() and maps it to a status.
pd_status record_cuda_error(cudaError_t e);
// cudaGetLastError() after a launch, mapped to a status.
inline pd_status check_launch() { return record_cuda_error(cudaGetLastError()); }
// PD_OK when the current device is compute capability 10.x.
pd_status require_sm100();
// Number of SMs of the current device (cached per device).
int sm_count();
// Device address of the status word the bounded waits report to (nullptr on failure).
int* device_status_ptr();
// Test aids behind pd_debug_set_wait_limit_ns / pd_debug_withhold_loads: the time after which a wait inside the
// single-CTA contraction kernel gives up (default 2 s), and whether that kernel's producer skips its loads, so
// that the wait for them runs out.
uint64_t debug_wait_limit_ns();
int debug_withhold_loads();
// Variant-selection log: with PD_LOG=1 in the environment every launcher writes one line to stderr naming the
// kernel variant it chose (read once per process; costs one branch otherwise).
bool log_enabled();
void logf(const char* fmt, ...) __attribute__((format(printf, 1, 2)));

// Raises the dynamic shared-memory limit of `kernel` on the current device, once per device (the attribute belongs
// to the device's context, and one process may drive several devices).  `done` is the caller's per-kernel record.
constexpr int kMaxDevicesPerProcess = 64;
struct PerDeviceFlag {
  std::atomic<bool> set[kMaxDevicesPerProcess] = {};  // concurrent first launches both set the attribute: harmless
};
template <typename Kernel>
inline pd_status allow_dynamic_smem(Kernel kernel, int bytes, PerDeviceFlag& done) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return record_cuda_error(e);
  if (dev < 0 || dev >= kMaxDevicesPerProcess) return PD_ERR_UNSUPPORTED;
  if (!done.set[dev].load(std::memory_order_acquire)) {
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e != cudaSuccess) return record_cuda_error(e);
    done.set[dev].store(true, std::memory_order_release);
  }
  return PD_OK;
}

// Launch with programmatic stream serialisation: the kernel may become resident and run its prologue while the
// previous kernel of the stream is still draining; it must call griddep_wait() before it touches global memory
// that an earlier kernel may still read or write.  Kernels call griddep_launch_dependents() to let their own
// successor do the same.
template <typename... KArgs, typename... Args>
inline void launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                       Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// The same with the CTAs grouped into thread-block clusters of `cluster` along x (grid.x a multiple of it).
template <typename... KArgs, typename... Args>
inline void launch_pdl_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, unsigned cluster, size_t smem,
                               cudaStream_t stream, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = cluster;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// ---- device side ---------------------------------------------------------
// Blocks until every kernel this one depends on has completed and its writes are visible (no-op when the
// kernel was launched without programmatic serialisation).
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// Allows the next kernel of the stream to be scheduled as soon as resources free up.
__device__ __forceinline__ void griddep_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Block-wide reductions over NWARPS warps through a small shared array; every
// thread receives the result.  `slot` selects one of two scratch rows so that
// back-to-back reductions need only one barrier each.
template <int NWARPS, bool IS_MAX>
__device__ __forceinline__ float block_reduce(float v, float (*scratch)[NWARPS], int slot) {
  v = IS_MAX ? warp_max(v) : warp_sum(v);
  if constexpr (NWARPS == 1) return v;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) scratch[slot][warp] = v;
  __syncthreads();
  float r = scratch[slot][0];
#pragma unroll
  for (int w = 1; w < NWARPS; ++w) r = IS_MAX ? fmaxf(r, scratch[slot][w]) : r + scratch[slot][w];
  return r;
}

// ---- rows shared by the CTAs of a thread-block cluster ----------------------------
// Rows too long for one CTA's registers are held by a cluster: CTA r keeps columns [r * chunk, (r + 1) * chunk)
// and the row statistics are combined through distributed shared memory.
__device__ __forceinline__ unsigned cluster_rank() {
  unsigned r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ unsigned cluster_size() {
  unsigned r;
  asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
  return r;
}
// All-reduce over the cluster of one value per CTA (`v`, identical in all threads of the CTA): thread k writes it
// into slot [own rank] of CTA k's exchange array, a cluster barrier (release / acquire) publishes the writes,
// and everyone combines the slots in rank order.  `xchg`: 8 floats of shared memory used by no other reduction.
template <bool IS_MAX>
__device__ __forceinline__ float cluster_allreduce(float v, float* xchg) {
  const unsigned n = cluster_size(), rank = cluster_rank();
  if (threadIdx.x < n) {
    const unsigned local = static_cast<unsigned>(__cvta_generic_to_shared(xchg + rank));
    unsigned remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(threadIdx.x));
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(remote), "f"(v) : "memory");
  }
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
  float r = xchg[0];
  for (unsigned k = 1; k < n; ++k) r = IS_MAX ? fmaxf(r, xchg[k]) : r + xchg[k];
  return r;
}

// Two sums at once (one barrier): `xchg` holds 16 floats.
__device__ __forceinline__ float2 cluster_allreduce_sum2(float a, float b, float* xchg) {
  const unsigned n = cluster_size(), rank = cluster_rank();
  if (threadIdx.x < n) {
    const unsigned local = static_cast<unsigned>(__cvta_generic_to_shared(xchg + 2 * rank));
    unsigned remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(threadIdx.x));
    asm volatile("st.shared::cluster.v2.f32 [%0], {%1, %2};" ::"r"(remote), "f"(a), "f"(b) : "memory");
  }
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
  float2 r = make_float2(xchg[0], xchg[1]);
  for (unsigned k = 1; k < n; ++k) {
    r.x += xchg[2 * k];
    r.y += xchg[2 * k + 1];
  }
  return r;
}

// Streaming 128-bit global accesses: inputs are read once and outputs written
// once, so neither should displace reusable lines.
__device__ __forceinline__ float4 ld_stream(const float4* p) { return __ldcs(p); }
__device__ __forceinline__ void st_stream(float4* p, float4 v) { __stcs(p, v); }

__device__ __forceinline__ void store_out4(float* base, int64_t idx4, float4 v) {
  st_stream(reinterpret_cast<float4*>(base) + idx4, v);
}
__device__ __forceinline__ void store_out4(__nv_bfloat16* base, int64_t idx4, float4 v) {
  __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
  uint2 u;
  u.x = *reinterpret_cast<uint32_t*>(&lo);
  u.y = *reinterpret_cast<uint32_t*>(&hi);
  __stcs(reinterpret_cast<uint2*>(base) + idx4, u);
}
__device__ __forceinline__ void store_out1(float* base, int64_t idx, float v) { base[idx] = v; }
__device__ __forceinline__ void store_out1(__nv_bfloat16* base, int64_t idx, float v) {
  base[idx] = __float2bfloat16_rn(v);
}

// ---- internal launchers (defined in the per-operator .cu files) ------------
// Softmax with fp32 or bf16 output; x fp32 [rows, cols].
pd_status launch_softmax(const float* x, void* y, bool y_is_bf16, int64_t rows, int64_t cols, cudaStream_t s);
// LayerNorm with fp32 or bf16 output.
pd_status launch_layernorm(const float* x, const float* gamma, const float* beta, void* y, bool y_is_bf16,
                           int64_t rows, int64_t cols, float eps, cudaStream_t s);
pd_status launch_rmsnorm(const float* x, const float* gamma, float* y, int64_t rows, int64_t cols, float eps,
                         cudaStream_t s);
pd_status launch_reducemean(const float* x, float* y, int64_t rows, int64_t cols, cudaStream_t s);
pd_status launch_bias_gelu_residual(const float* x, const float* bias, const float* r, float* out,
                                    int64_t rows, int64_t cols, cudaStream_t s);


// One (optionally batched) bf16 contraction with a fused epilogue:
//   C[bo][bi][m,n] = epilogue(alpha * sum_k A[bo][bi][m,k] * B[bo][bi][k,n])
//   epilogue(v)    = act(v + bias[n]) + residual[m,n]
// or, in gated form (B2 set), with G = A B and U = A B2:  C = SiLU(G) * U  (no bias, activation or residual).
// The batch index has two levels (outer, inner) so that the per-head operands
// of attention can be addressed inside the packed [tokens, 3*hidden] tensor.
struct GemmProblem {
  const void* A = nullptr;  // bf16 [M, K], row stride lda
  const void* B = nullptr;  // bf16 [K, N] (b_is_nk false) or [N, K] (true), row stride ldb
  void* C = nullptr;        // c_dtype [M, N], row stride ldc
  int64_t M = 0, N = 0, K = 0, lda = 0, ldb = 0, ldc = 0;
  bool b_is_nk = false;
  pd_dtype c_dtype = PD_BF16;
  int64_t batch_inner = 1, batch_outer = 1;
  int64_t strideA_inner = 0, strideA_outer = 0, strideB_inner = 0, strideB_outer = 0;
  int64_t strideC_inner = 0, strideC_outer = 0;
  float alpha = 1.0f;
  const float* bias = nullptr;               // fp32 [N] or null
  int act = 0;                               // after the bias: 0 nothing, 1 erf-form GELU, 2 ReLU
  const void* B2 = nullptr;                  // bf16 [K, N], row stride ldb: second weight of the gated form, or null
  const __nv_bfloat16* residual = nullptr;   // bf16 [M, N], row stride ldr, or null (unbatched only)
  int64_t ldr = 0;
  // Walk the row blocks of C from the last to the first (LayerNorm GEMM only).  A consumer whose A operand is
  // larger than L2 and was written first row first by the launch before it finds the most recently written
  // rows still in L2 when it starts at the far end; results do not depend on the order.
  bool rows_descending = false;
};
pd_status launch_gemm(const GemmProblem& p, cudaStream_t s);
// The same contraction on 256 x 256 tiles computed by pairs of CTAs (cta_group::2).
bool gemm_pair_tiles_profitable(const GemmProblem& p);
void set_gemm_tile_mode(int mode);
void set_gemm_split_k_mode(int mode);
pd_status launch_gemm_pair(const GemmProblem& p, cudaStream_t s);
// Split-K over a thread-block cluster for problems with few output tiles: the cluster size to use (0: none) and
// the launcher (128 x 256 accumulator tiles, reduce-scatter through distributed shared memory).
int gemm_split_k_factor(const GemmProblem& p);
pd_status launch_gemm_split_k(const GemmProblem& p, int split, cudaStream_t s);
// C = LayerNorm(alpha A B + bias + residual; gamma, beta, eps) over the N columns of each row, bf16 out, in one
// kernel: the CTAs that hold the column tiles of a row block form a cluster and exchange row statistics.
// N must be a multiple of 256, at most 2048.
bool gemm_layernorm_supported(const GemmProblem& p);
pd_status launch_gemm_layernorm(const GemmProblem& p, const float* gamma, const float* beta, float eps,
                                cudaStream_t s);

// Fused attention on qkv[batch*seq, 3*heads*64] -> ctx[batch*seq, heads*64] (both bf16).
bool fused_attention_supported(int64_t seq, int64_t head_dim);
pd_status launch_fused_attention(const __nv_bfloat16* qkv, __nv_bfloat16* ctx, int64_t batch, int64_t seq,
                                 int64_t heads, cudaStream_t s);

}  // namespace pd
