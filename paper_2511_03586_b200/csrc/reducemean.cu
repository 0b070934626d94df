// Mean over the last dimension, fp32 in, fp32 out (operator "reducemean" of the
// paper's operator table, 4096 x 4096):
//
//   y[i] = (1 / cols) * sum_j x[i,j]
//
// HBM-bound, 4 bytes per element (the output is negligible): each row is read
// once with 128-bit streaming loads.  A warp takes a row of up to 1024 columns,
// a CTA of 128 threads a longer one (grid-striding over the row, so any length
// works); partial sums are kept in four independent accumulators per thread and
// combined with warp shuffles (and through shared memory for a CTA), i.e. as a
// tree, which keeps the fp32 rounding error near that of pairwise summation.
#include "pd_common.cuh"

namespace pd {
namespace {

__device__ __forceinline__ float sum4(float4 v) { return (v.x + v.y) + (v.z + v.w); }

// One warp per row: cols4 = cols / 4 <= 256 float4 per row.
__global__ void __launch_bounds__(256)
reducemean_warp_rows(const float* __restrict__ x, float* __restrict__ y, int64_t rows, int cols) {
  const int lane = threadIdx.x & 31;
  const int cols4 = cols >> 2;
  const float inv = 1.0f / (float)cols;
  griddep_wait();
  griddep_launch_dependents();
  for (int64_t row = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5); row < rows; row += (int64_t)gridDim.x * 8) {
    const float4* xr = reinterpret_cast<const float4*>(x + row * cols);
    float a[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int c = lane + 32 * i;
      if (c < cols4) a[i & 3] += sum4(ld_stream(xr + c));
    }
    const float s = warp_sum((a[0] + a[1]) + (a[2] + a[3]));
    if (lane == 0) y[row] = s * inv;
  }
}

// One CTA of 128 threads per row of any length; `vec` = rows are 16-byte aligned and cols % 4 == 0.
template <bool VEC>
__global__ void __launch_bounds__(128)
reducemean_cta_rows(const float* __restrict__ x, float* __restrict__ y, int64_t rows, int64_t cols) {
  __shared__ float scratch[2][4];
  const float inv = 1.0f / (float)cols;
  griddep_wait();
  griddep_launch_dependents();
  int slot = 0;
  for (int64_t row = blockIdx.x; row < rows; row += gridDim.x, slot ^= 1) {
    float a[4] = {0.f, 0.f, 0.f, 0.f};
    if (VEC) {
      const float4* xr = reinterpret_cast<const float4*>(x + row * cols);
      const int64_t cols4 = cols >> 2;
      int64_t c = threadIdx.x;
      for (; c + 3 * 128 < cols4; c += 4 * 128) {
        const float4 v0 = ld_stream(xr + c), v1 = ld_stream(xr + c + 128), v2 = ld_stream(xr + c + 256),
                     v3 = ld_stream(xr + c + 384);
        a[0] += sum4(v0); a[1] += sum4(v1); a[2] += sum4(v2); a[3] += sum4(v3);
      }
      for (; c < cols4; c += 128) a[0] += sum4(ld_stream(xr + c));
    } else {
      const float* xr = x + row * cols;
      int k = 0;
      for (int64_t j = threadIdx.x; j < cols; j += 128, k = (k + 1) & 3) a[k] += xr[j];
    }
    const float s = block_reduce<4, false>((a[0] + a[1]) + (a[2] + a[3]), scratch, slot);
    if (threadIdx.x == 0) y[row] = s * inv;
  }
}

}  // namespace

pd_status launch_reducemean(const float* x, float* y, int64_t rows, int64_t cols, cudaStream_t s) {
  const bool vec_ok = (cols % 4 == 0) && aligned16(x);
  if (vec_ok && cols <= 1024) {
    const int64_t ctas = (rows + 7) / 8;
    launch_pdl(reducemean_warp_rows, dim3((unsigned)(ctas < 0x7fffffff ? ctas : 0x7fffffff)), dim3(256), 0, s, x, y, rows,
               (int)cols);
  } else {
    const unsigned grid = (unsigned)(rows < 0x7fffffff ? rows : 0x7fffffff);
    if (vec_ok) launch_pdl(reducemean_cta_rows<true>, dim3(grid), dim3(128), 0, s, x, y, rows, cols);
    else launch_pdl(reducemean_cta_rows<false>, dim3(grid), dim3(128), 0, s, x, y, rows, cols);
  }
  return check_launch();
}

}  // namespace pd

extern "C" pd_status pd_reducemean(const float* x, float* y, int64_t rows, int64_t cols, cudaStream_t stream) {
  if (!x || !y) return PD_ERR_NULL_POINTER;
  if (rows < 0 || cols <= 0) return PD_ERR_BAD_SHAPE;
  if ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(y)) & 3u) return PD_ERR_ALIGNMENT;
  if (rows == 0) return PD_OK;
  pd_status st = pd::require_sm100();
  if (st != PD_OK) return st;
  return pd::launch_reducemean(x, y, rows, cols, stream);
}
