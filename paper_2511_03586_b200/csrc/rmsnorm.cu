// Root-mean-square normalisation over the last dimension, fp32 in, fp32 out
// (operator "rmsnorm" of the paper's operator table, 3072 x 4096):
//
//   y[i,j] = x[i,j] * rsqrt(mean_j x[i,j]^2 + eps) * gamma[j]
//
// HBM-bound, 8 bytes per element: the row is read once into registers with
// 128-bit streaming loads, the sum of squares is reduced with warp shuffles (and
// through shared memory when several warps share a row), and the row is written
// once.  Same paths as the LayerNorm kernel: a warp (cols <= 1024), a CTA (<= 28672) or a cluster of 2 to 8
// CTAs (<= 262144) per row, by row length.
#include "pd_common.cuh"

namespace pd {
namespace {

template <int VPT, int THREADS_PER_ROW, int THREADS_PER_CTA>
__global__ void __launch_bounds__(THREADS_PER_CTA, VPT > 12 ? 2 : VPT > 8 ? 3 : (THREADS_PER_CTA >= 1024 ? 1 : (THREADS_PER_CTA == 128 ? 5 : 1024 / THREADS_PER_CTA)))  // at most 64 registers (1024 threads resident per SM); 96 for the 128-thread CTAs of 4096-column rows, where five CTAs with the compiler free to keep more loads apart measured 3 % faster than eight; 85 / 128 for the 256-thread CTAs that hold 12 / 16 to 28 float4 per thread (rows of 8196 to 28672 columns, three / two of them in flight per SM)
rmsnorm_rows_in_registers(const float* __restrict__ x, const float* __restrict__ gamma, float* __restrict__ y,
                          int64_t rows, int cols, float eps) {
  constexpr int ROWS_PER_CTA = THREADS_PER_CTA / THREADS_PER_ROW;
  constexpr int NWARPS = THREADS_PER_ROW / 32;
  __shared__ float scratch[2][NWARPS];
  const int t = threadIdx.x % THREADS_PER_ROW;
  const int cols4 = cols >> 2;
  const float inv_cols = 1.0f / (float)cols;
  const float4* g4 = reinterpret_cast<const float4*>(gamma);
  griddep_wait();
  griddep_launch_dependents();
  int slot = 0;
  for (int64_t row = (int64_t)blockIdx.x * ROWS_PER_CTA + threadIdx.x / THREADS_PER_ROW; row < rows;
       row += (int64_t)gridDim.x * ROWS_PER_CTA, slot ^= 1) {
    const float4* xr = reinterpret_cast<const float4*>(x + row * cols);
    float4 v[VPT];
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
      const int c = t + i * THREADS_PER_ROW;
      v[i] = (c < cols4) ? ld_stream(xr + c) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    float q = 0.f;
#pragma unroll
    for (int i = 0; i < VPT; ++i) q += (v[i].x * v[i].x + v[i].y * v[i].y) + (v[i].z * v[i].z + v[i].w * v[i].w);
    const float rstd = rsqrtf(block_reduce<NWARPS, false>(q, scratch, slot) * inv_cols + eps);
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
      const int c = t + i * THREADS_PER_ROW;
      if (c < cols4) {
        const float4 g = __ldg(g4 + c);
        store_out4(y, row * cols4 + c,
                   make_float4(v[i].x * rstd * g.x, v[i].y * rstd * g.y, v[i].z * rstd * g.z, v[i].w * rstd * g.w));
      }
    }
  }
}

// Rows of 32768 < cols <= 262144: one cluster of up to 8 CTAs per row, the columns dealt evenly, each CTA keeping
// its share (at most 32 per thread) in registers; 512-thread CTAs, two per SM, up to 131072 columns; the sum of squares is combined over the cluster through distributed shared memory.
template <int THREADS>
__global__ void __launch_bounds__(THREADS, 1024 / THREADS)
rmsnorm_rows_cluster(const float* __restrict__ x, const float* __restrict__ gamma, float* __restrict__ y, int64_t rows,
                     int cols, float eps) {
  constexpr int VPT = 8, NWARPS = THREADS / 32;
  __shared__ float scratch[2][NWARPS];
  __shared__ float xchg[8];
  const int cols4 = cols >> 2;
  const float4* g4 = reinterpret_cast<const float4*>(gamma);
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
    v[i] = (c < end) ? ld_stream(xr + c) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  float q = 0.f;
#pragma unroll
  for (int i = 0; i < VPT; ++i) q += (v[i].x * v[i].x + v[i].y * v[i].y) + (v[i].z * v[i].z + v[i].w * v[i].w);
  q = cluster_allreduce<false>(block_reduce<NWARPS, false>(q, scratch, 0), xchg);
  const float rstd = rsqrtf(q / (float)cols + eps);
#pragma unroll
  for (int i = 0; i < VPT; ++i) {
    const int c = base + threadIdx.x + i * THREADS;
    if (c < end) {
      const float4 g = __ldg(g4 + c);
      store_out4(y, row * cols4 + c,
                 make_float4(v[i].x * rstd * g.x, v[i].y * rstd * g.y, v[i].z * rstd * g.z, v[i].w * rstd * g.w));
    }
  }
}

__global__ void __launch_bounds__(256)
rmsnorm_rows_generic(const float* __restrict__ x, const float* __restrict__ gamma, float* __restrict__ y,
                     int64_t rows, int64_t cols, float eps) {
  __shared__ float scratch[2][8];
  int slot = 0;
  for (int64_t row = blockIdx.x; row < rows; row += gridDim.x, slot ^= 1) {
    const float* xr = x + row * cols;
    float q = 0.f;
    for (int64_t j = threadIdx.x; j < cols; j += 256) q += xr[j] * xr[j];
    const float rstd = rsqrtf(block_reduce<8, false>(q, scratch, slot) / (float)cols + eps);
    for (int64_t j = threadIdx.x; j < cols; j += 256) y[row * cols + j] = xr[j] * rstd * gamma[j];
  }
}

template <int VPT>
void launch_warp_rows(const float* x, const float* g, float* y, int64_t rows, int cols, float eps, cudaStream_t s) {
  constexpr int kThreads = 64, kRowsPerCta = kThreads / 32;  // two rows per CTA: the finest grain for the last, partly filled wave
  const int64_t ctas = (rows + kRowsPerCta - 1) / kRowsPerCta;
  const int grid = (int)(ctas < 0x7fffffff ? ctas : 0x7fffffff);
  launch_pdl(rmsnorm_rows_in_registers<VPT, 32, kThreads>, dim3(grid), dim3(kThreads), 0, s, x, g, y, rows, cols, eps);
}

template <int THREADS, int VPT = 8>
void launch_cta_rows(const float* x, const float* g, float* y, int64_t rows, int cols, float eps, cudaStream_t s) {
  const int grid = (int)(rows < 0x7fffffff ? rows : 0x7fffffff);
  launch_pdl(rmsnorm_rows_in_registers<VPT, THREADS, THREADS>, dim3(grid), dim3(THREADS), 0, s, x, g, y, rows, cols, eps);
}

constexpr int64_t kFatRowCols = 28672;  // columns one 256-thread CTA holds at 28 float4 per thread

}  // namespace

pd_status launch_rmsnorm(const float* x, const float* g, float* y, int64_t rows, int64_t cols, float eps,
                         cudaStream_t s) {
  const bool vec_ok = (cols % 4 == 0) && aligned16(x) && aligned16(g) && aligned16(y);
  const int c = (int)cols;
  logf("rmsnorm %lld x %lld: %s", (long long)rows, (long long)cols,
       !vec_ok ? "scalar path (unaligned or ragged rows)" : cols <= 1024 ? "one warp per row, row in registers"
       : cols <= 28672 ? "one CTA per row, row in registers" : cols <= 262144 ? "one cluster per row, row in registers" : "scalar path");
  if (vec_ok && cols <= 1024) {
    if (c <= 128) launch_warp_rows<1>(x, g, y, rows, c, eps, s);
    else if (c <= 256) launch_warp_rows<2>(x, g, y, rows, c, eps, s);
    else if (c <= 512) launch_warp_rows<4>(x, g, y, rows, c, eps, s);
    else launch_warp_rows<8>(x, g, y, rows, c, eps, s);
  } else if (vec_ok && cols <= kFatRowCols) {
    if (c <= 2048) launch_cta_rows<64>(x, g, y, rows, c, eps, s);
    else if (c <= 4096) launch_cta_rows<128>(x, g, y, rows, c, eps, s);
    else if (c <= 8192) launch_cta_rows<256>(x, g, y, rows, c, eps, s);
    // from 8196 columns on: 256 threads with 12 float4 each (85 registers, three rows in flight per SM) or 16 to 28
    // (128 registers, two rows in flight); a CTA of 512 or 1024 threads with 8 float4 each leaves the memory pipe idle
    // while its row is reduced (LayerNorm: 5.7 -> 6.4 TB/s at 12288 columns, 4.0 -> 5.8 at 20480)
    else if (c <= 12288) launch_cta_rows<256, 12>(x, g, y, rows, c, eps, s);
    else if (c <= 16384) launch_cta_rows<256, 16>(x, g, y, rows, c, eps, s);
    else if (c <= 20480) launch_cta_rows<256, 20>(x, g, y, rows, c, eps, s);
    else if (c <= 24576) launch_cta_rows<256, 24>(x, g, y, rows, c, eps, s);
    else launch_cta_rows<256, 28>(x, g, y, rows, c, eps, s);
  } else if (vec_ok && cols <= 262144 && rows * 8 <= 0x7fffffff) {
    // (clusters of the 256-thread CTAs above are slower than these: LayerNorm at 65536 columns 3.0 against 4.2 TB/s)
    if (cols <= 131072) {
      const unsigned cl = (unsigned)((cols + 16383) / 16384);
      launch_pdl_cluster(rmsnorm_rows_cluster<512>, dim3((unsigned)rows * cl), dim3(512), cl, 0, s, x, g, y, rows, c, eps);
    } else {
      const unsigned cl = (unsigned)((cols + 32767) / 32768);
      launch_pdl_cluster(rmsnorm_rows_cluster<1024>, dim3((unsigned)rows * cl), dim3(1024), cl, 0, s, x, g, y, rows, c, eps);
    }
  } else {
    const int grid = (int)(rows < (int64_t)sm_count() * 16 ? rows : (int64_t)sm_count() * 16);
    rmsnorm_rows_generic<<<grid, 256, 0, s>>>(x, g, y, rows, cols, eps);
  }
  return check_launch();
}

}  // namespace pd

extern "C" pd_status pd_rmsnorm(const float* x, const float* gamma, float* y, int64_t rows, int64_t cols, float eps,
                                cudaStream_t stream) {
  if (!x || !gamma || !y) return PD_ERR_NULL_POINTER;
  if (rows < 0 || cols <= 0 || !(eps >= 0.f)) return PD_ERR_BAD_SHAPE;
  if ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(y) | reinterpret_cast<uintptr_t>(gamma)) & 3u)
    return PD_ERR_ALIGNMENT;
  if (rows == 0) return PD_OK;
  pd_status st = pd::require_sm100();
  if (st != PD_OK) return st;
  return pd::launch_rmsnorm(x, gamma, y, rows, cols, eps, stream);
}
