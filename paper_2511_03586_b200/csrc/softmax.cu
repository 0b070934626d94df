// Row-wise softmax, fp32 in, fp32 or bf16 out.
//
//   y[i,j] = exp(x[i,j] - m_i) / sum_j exp(x[i,j] - m_i),  m_i = max_j x[i,j]
//
// HBM-bound: 8 bytes per element (4 when writing bf16).  Each row is read from
// global memory exactly once into registers with 128-bit loads, reduced with
// warp shuffles, and written once.
//   * cols <= 1024            : one warp per row (up to 8 float4 per lane), two rows per CTA
//   * cols <= 8192            : one CTA of 64 to 256 threads per row (8 float4 per thread)
//   * cols <= 28672           : one CTA of 256 threads per row, 12 to 28 float4 per thread at 85 or 128
//                               registers (three or two rows in flight per SM)
//   * cols <= 262144          : one cluster of 2 to 8 CTAs per row, ceil(cols / 16384) CTAs of 512 threads up
//                               to 131072 columns and ceil(cols / 32768) of 1024 beyond (statistics combined
//                               through distributed shared memory)
//   * longer, 16-byte aligned : one CTA per row, online (max, sum) pass from HBM, normalising pass from L2
//   * anything else / ragged  : one CTA per row, three scalar passes from global/L2
#include "pd_common.cuh"

namespace pd {
namespace {

#define kNegInf (-INFINITY)

constexpr int64_t kFatRowCols = 28672;  // columns one 256-thread CTA holds at 28 float4 per thread

// One row held by THREADS_PER_ROW threads, VPT float4 each; threads of a row are
// consecutive lanes.  THREADS_PER_ROW == 32: one warp per row, several rows per
// CTA.  THREADS_PER_ROW == blockDim.x: one row per CTA.
template <int VPT, int THREADS_PER_ROW, int THREADS_PER_CTA, typename OutT>
__global__ void __launch_bounds__(THREADS_PER_CTA, VPT > 12 ? 2 : VPT > 8 ? 3 : (THREADS_PER_CTA >= 1024 ? 1 : (THREADS_PER_CTA == 128 ? 5 : 1024 / THREADS_PER_CTA)))  // at most 64 registers (1024 threads resident per SM); 96 for the 128-thread CTAs of 4096-column rows, where five CTAs with the compiler free to keep more loads apart measured 3 % faster than eight; 85 / 128 for the 256-thread CTAs that hold 12 / 16 to 28 float4 per thread (rows of 8196 to 28672 columns, three / two of them in flight per SM)
softmax_rows_in_registers(const float* __restrict__ x, OutT* __restrict__ y, int64_t rows, int cols) {
  constexpr int ROWS_PER_CTA = THREADS_PER_CTA / THREADS_PER_ROW;
  constexpr int NWARPS = THREADS_PER_ROW / 32;
  __shared__ float scratch[2][NWARPS];
  const int t = threadIdx.x % THREADS_PER_ROW;
  const int cols4 = cols >> 2;
  griddep_wait();
  griddep_launch_dependents();
  for (int64_t row = (int64_t)blockIdx.x * ROWS_PER_CTA + threadIdx.x / THREADS_PER_ROW; row < rows;
       row += (int64_t)gridDim.x * ROWS_PER_CTA) {
    const float4* xr = reinterpret_cast<const float4*>(x + row * cols);
    float4 v[VPT];
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
      const int c = t + i * THREADS_PER_ROW;
      v[i] = (c < cols4) ? ld_stream(xr + c) : make_float4(kNegInf, kNegInf, kNegInf, kNegInf);
    }
    float m = kNegInf;
#pragma unroll
    for (int i = 0; i < VPT; ++i) m = fmaxf(m, fmaxf(fmaxf(v[i].x, v[i].y), fmaxf(v[i].z, v[i].w)));
    m = block_reduce<NWARPS, true>(m, scratch, 0);
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
      v[i].x = expf(v[i].x - m);
      v[i].y = expf(v[i].y - m);
      v[i].z = expf(v[i].z - m);
      v[i].w = expf(v[i].w - m);
      s += (v[i].x + v[i].y) + (v[i].z + v[i].w);
    }
    s = block_reduce<NWARPS, false>(s, scratch, 1);
    const float inv = 1.0f / s;
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
      const int c = t + i * THREADS_PER_ROW;
      if (c < cols4)
        store_out4(y, row * cols4 + c, make_float4(v[i].x * inv, v[i].y * inv, v[i].z * inv, v[i].w * inv));
    }
    if constexpr (NWARPS > 1) __syncthreads();  // scratch is reused by the next row
  }
}

// Rows of 32768 < cols <= 262144: one cluster of up to 8 CTAs per row, the columns dealt evenly, each CTA keeping
// its share (at most 32 per thread) in registers; 512-thread CTAs, two per SM, up to 131072 columns; maximum and sum are combined over the cluster through distributed shared memory,
// so the row is still read once and written once.
template <int THREADS, typename OutT>
__global__ void __launch_bounds__(THREADS, 1024 / THREADS)
softmax_rows_cluster(const float* __restrict__ x, OutT* __restrict__ y, int64_t rows, int cols) {
  constexpr int VPT = 8, NWARPS = THREADS / 32;
  __shared__ float scratch[2][NWARPS];
  __shared__ float xchg[2][8];
  const int cols4 = cols >> 2;
  const int64_t row = blockIdx.x / cluster_size();
  const int chunk4 = (cols4 + (int)cluster_size() - 1) / (int)cluster_size();  // float4 per CTA, at most VPT * THREADS
  const int base = (int)cluster_rank() * chunk4;
  const int end = min(base + chunk4, cols4);
  griddep_wait();
  griddep_launch_dependents();
  const float4* xr = reinterpret_cast<const float4*>(x + row * cols);
  float4 v[VPT];
#pragma unroll
  for (int i = 0; i < VPT; ++i) {
    const int c = base + threadIdx.x + i * THREADS;
    v[i] = (c < end) ? ld_stream(xr + c) : make_float4(kNegInf, kNegInf, kNegInf, kNegInf);
  }
  float m = kNegInf;
#pragma unroll
  for (int i = 0; i < VPT; ++i) m = fmaxf(m, fmaxf(fmaxf(v[i].x, v[i].y), fmaxf(v[i].z, v[i].w)));
  m = cluster_allreduce<true>(block_reduce<NWARPS, true>(m, scratch, 0), xchg[0]);
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < VPT; ++i) {
    v[i].x = expf(v[i].x - m);
    v[i].y = expf(v[i].y - m);
    v[i].z = expf(v[i].z - m);
    v[i].w = expf(v[i].w - m);
    s += (v[i].x + v[i].y) + (v[i].z + v[i].w);
  }
  s = cluster_allreduce<false>(block_reduce<NWARPS, false>(s, scratch, 1), xchg[1]);
  const float inv = 1.0f / s;
#pragma unroll
  for (int i = 0; i < VPT; ++i) {
    const int c = base + threadIdx.x + i * THREADS;
    if (c < end)
      store_out4(y, row * cols4 + c, make_float4(v[i].x * inv, v[i].y * inv, v[i].z * inv, v[i].w * inv));
  }
}

// Any cols, any alignment: one CTA per row, scalar coalesced accesses, the row
// is re-read from L2 for the second and third pass.
template <typename OutT>
__global__ void __launch_bounds__(256)
softmax_rows_generic(const float* __restrict__ x, OutT* __restrict__ y, int64_t rows, int64_t cols) {
  __shared__ float scratch[2][8];
  for (int64_t row = blockIdx.x; row < rows; row += gridDim.x) {
    const float* xr = x + row * cols;
    float m = kNegInf;
    for (int64_t j = threadIdx.x; j < cols; j += 256) m = fmaxf(m, xr[j]);
    m = block_reduce<8, true>(m, scratch, 0);
    float s = 0.f;
    for (int64_t j = threadIdx.x; j < cols; j += 256) s += expf(xr[j] - m);
    s = block_reduce<8, false>(s, scratch, 1);
    const float inv = 1.0f / s;
    for (int64_t j = threadIdx.x; j < cols; j += 256) store_out1(y, row * cols + j, expf(xr[j] - m) * inv);
    __syncthreads();
  }
}

// Rows too long for registers (cols > 32768), 16-byte aligned: one CTA of 512 threads per row, two passes.
// Pass 1 streams the row from HBM with 128-bit loads and keeps an online (max, sum) pair per thread (the sum is
// rescaled whenever the running max grows), merged across the CTA; pass 2 re-reads the row, by then in L2,
// and writes exp(x - max) / sum.
template <typename OutT>
__global__ void __launch_bounds__(512)
softmax_rows_streaming(const float* __restrict__ x, OutT* __restrict__ y, int64_t rows, int64_t cols) {
  __shared__ float scratch[2][16];
  const int64_t cols4 = cols >> 2;
  for (int64_t row = blockIdx.x; row < rows; row += gridDim.x) {
    const float4* xr = reinterpret_cast<const float4*>(x + row * cols);
    float m = kNegInf, s = 0.f;
    for (int64_t c = threadIdx.x; c < cols4; c += 512) {
      const float4 v = __ldg(xr + c);
      const float m4 = fmaxf(fmaxf(v.x, v.y), fmaxf(v.z, v.w));
      if (m4 > m) {
        s *= expf(m - m4);  // exp(-inf) = 0 on the first visit
        m = m4;
      }
      s += (expf(v.x - m) + expf(v.y - m)) + (expf(v.z - m) + expf(v.w - m));
    }
    const float M = block_reduce<16, true>(m, scratch, 0);
    s = (m == kNegInf) ? 0.f : s * expf(m - M);
    const float inv = 1.0f / block_reduce<16, false>(s, scratch, 1);
    for (int64_t c = threadIdx.x; c < cols4; c += 512) {
      const float4 v = __ldg(xr + c);
      store_out4(y, row * cols4 + c,
                 make_float4(expf(v.x - M) * inv, expf(v.y - M) * inv, expf(v.z - M) * inv, expf(v.w - M) * inv));
    }
    __syncthreads();
  }
}

template <int VPT, typename OutT>
void launch_warp_rows(const float* x, OutT* y, int64_t rows, int cols, cudaStream_t s) {
  constexpr int kThreads = 64, kRowsPerCta = kThreads / 32;  // two rows per CTA: the finest grain for the last, partly filled wave
  auto kernel = softmax_rows_in_registers<VPT, 32, kThreads, OutT>;
  // one CTA per two rows, all launched: the hardware scheduler balances many short CTAs better than a
  // grid-stride loop over a resident set does
  const int64_t ctas = (rows + kRowsPerCta - 1) / kRowsPerCta;
  const int grid = (int)(ctas < 0x7fffffff ? ctas : 0x7fffffff);
  launch_pdl(kernel, dim3(grid), dim3(kThreads), 0, s, x, y, rows, cols);
}

// One CTA of THREADS threads per row, up to VPT float4 per thread.
template <int THREADS, typename OutT, int VPT = 8>
void launch_cta_rows(const float* x, OutT* y, int64_t rows, int cols, cudaStream_t s) {
  auto kernel = softmax_rows_in_registers<VPT, THREADS, THREADS, OutT>;
  const int grid = (int)(rows < 0x7fffffff ? rows : 0x7fffffff);
  launch_pdl(kernel, dim3(grid), dim3(THREADS), 0, s, x, y, rows, cols);
}

template <typename OutT>
pd_status dispatch(const float* x, OutT* y, int64_t rows, int64_t cols, cudaStream_t s) {
  const bool vec_ok = (cols % 4 == 0) && aligned16(x) && ((reinterpret_cast<uintptr_t>(y) & (sizeof(OutT) * 4 - 1)) == 0);
  logf("%s %lld x %lld: %s", "softmax", (long long)rows, (long long)cols,
       !vec_ok ? "scalar three-pass path (unaligned or ragged rows)"
       : cols <= 1024 ? "one warp per row, row in registers"
       : cols <= kFatRowCols ? "one CTA per row, row in registers"
       : cols <= 262144 ? "one cluster per row, row in registers" : "one CTA per row, streaming passes");
  if (vec_ok && cols <= 1024) {
    const int c = (int)cols;
    if (c <= 128) launch_warp_rows<1>(x, y, rows, c, s);
    else if (c <= 256) launch_warp_rows<2>(x, y, rows, c, s);
    else if (c <= 512) launch_warp_rows<4>(x, y, rows, c, s);
    else launch_warp_rows<8>(x, y, rows, c, s);
  } else if (vec_ok && cols <= kFatRowCols) {
    const int c = (int)cols;
    if (c <= 2048) launch_cta_rows<64>(x, y, rows, c, s);
    else if (c <= 4096) launch_cta_rows<128>(x, y, rows, c, s);
    else if (c <= 8192) launch_cta_rows<256>(x, y, rows, c, s);
    // from 8196 columns on: 256 threads with 12 float4 each (85 registers, three rows in flight per SM) or 16 to 28
    // (128 registers, two rows in flight); a CTA of 512 or 1024 threads with 8 float4 each leaves the memory pipe idle
    // while its row is reduced (LayerNorm: 5.7 -> 6.4 TB/s at 12288 columns, 4.0 -> 5.8 at 20480)
    else if (c <= 12288) launch_cta_rows<256, OutT, 12>(x, y, rows, c, s);
    else if (c <= 16384) launch_cta_rows<256, OutT, 16>(x, y, rows, c, s);
    else if (c <= 20480) launch_cta_rows<256, OutT, 20>(x, y, rows, c, s);
    else if (c <= 24576) launch_cta_rows<256, OutT, 24>(x, y, rows, c, s);
    else launch_cta_rows<256, OutT, 28>(x, y, rows, c, s);
  } else if (vec_ok && cols <= 262144 && rows * 8 <= 0x7fffffff) {
    // (clusters of the 256-thread CTAs above are slower than these: LayerNorm at 65536 columns 3.0 against 4.2 TB/s)
    if (cols <= 131072) {
      const unsigned cl = (unsigned)((cols + 16383) / 16384);
      launch_pdl_cluster(softmax_rows_cluster<512, OutT>, dim3((unsigned)rows * cl), dim3(512), cl, 0, s, x, y, rows, (int)cols);
    } else {
      const unsigned cl = (unsigned)((cols + 32767) / 32768);
      launch_pdl_cluster(softmax_rows_cluster<1024, OutT>, dim3((unsigned)rows * cl), dim3(1024), cl, 0, s, x, y, rows, (int)cols);
    }
  } else if (vec_ok && x != reinterpret_cast<const float*>(y)) {
    const int grid = (int)(rows < (int64_t)sm_count() * 4 ? rows : (int64_t)sm_count() * 4);
    softmax_rows_streaming<OutT><<<grid, 512, 0, s>>>(x, y, rows, cols);
  } else {
    const int grid = (int)(rows < (int64_t)sm_count() * 16 ? rows : (int64_t)sm_count() * 16);
    softmax_rows_generic<OutT><<<grid, 256, 0, s>>>(x, y, rows, cols);
  }
  return check_launch();
}

}  // namespace

pd_status launch_softmax(const float* x, void* y, bool y_is_bf16, int64_t rows, int64_t cols, cudaStream_t s) {
  if (y_is_bf16) return dispatch(x, static_cast<__nv_bfloat16*>(y), rows, cols, s);
  return dispatch(x, static_cast<float*>(y), rows, cols, s);
}

}  // namespace pd

extern "C" pd_status pd_softmax(const float* x, float* y, int64_t rows, int64_t cols, cudaStream_t stream) {
  if (!x || !y) return PD_ERR_NULL_POINTER;
  if (rows < 0 || cols <= 0) return PD_ERR_BAD_SHAPE;
  if ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(y)) & 3u) return PD_ERR_ALIGNMENT;
  if (rows == 0) return PD_OK;
  pd_status st = pd::require_sm100();
  if (st != PD_OK) return st;
  return pd::launch_softmax(x, y, false, rows, cols, stream);
}
