// out[i,j] = GELU(x[i,j] + bias[j]) + r[i,j]   (r optional), GELU in its erf form.
//
// One pass over HBM: 12 bytes per element with a residual, 8 without.  Every
// thread streams UNROLL float4 of x (and r) with 128-bit loads that are all
// issued before the arithmetic, takes its bias float4 through the read-only
// path (the bias vector stays in L1/L2), and writes one float4 per input float4.
#include "pd_common.cuh"

namespace pd {
namespace {

__device__ __forceinline__ float gelu_erf(float z) {
  return 0.5f * z * (1.0f + erff(z * 0.70710678118654752440f));
}

template <bool HAS_R, int UNROLL>
__global__ void __launch_bounds__(256)
bias_gelu_residual_vec4(const float* __restrict__ x, const float* __restrict__ bias, const float* __restrict__ r,
                        float* __restrict__ out, int64_t n4, int cols4) {
  const float4* x4 = reinterpret_cast<const float4*>(x);
  const float4* r4 = reinterpret_cast<const float4*>(r);
  const float4* b4 = reinterpret_cast<const float4*>(bias);
  float4* o4 = reinterpret_cast<float4*>(out);
  const int64_t base = (int64_t)blockIdx.x * (256 * UNROLL) + threadIdx.x;
  float4 xv[UNROLL], rv[UNROLL];
#pragma unroll
  for (int u = 0; u < UNROLL; ++u) {
    const int64_t i = base + u * 256;
    if (i < n4) {
      xv[u] = ld_stream(x4 + i);
      if (HAS_R) rv[u] = ld_stream(r4 + i);
    }
  }
#pragma unroll
  for (int u = 0; u < UNROLL; ++u) {
    const int64_t i = base + u * 256;
    if (i < n4) {
      const float4 b = __ldg(b4 + (int)(i % cols4));
      float4 o;
      o.x = gelu_erf(xv[u].x + b.x);
      o.y = gelu_erf(xv[u].y + b.y);
      o.z = gelu_erf(xv[u].z + b.z);
      o.w = gelu_erf(xv[u].w + b.w);
      if (HAS_R) { o.x += rv[u].x; o.y += rv[u].y; o.z += rv[u].z; o.w += rv[u].w; }
      st_stream(o4 + i, o);
    }
  }
}

template <bool HAS_R>
__global__ void __launch_bounds__(256)
bias_gelu_residual_scalar(const float* __restrict__ x, const float* __restrict__ bias, const float* __restrict__ r,
                          float* __restrict__ out, int64_t n, int64_t cols) {
  for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < n; i += (int64_t)gridDim.x * 256) {
    float o = gelu_erf(x[i] + bias[i % cols]);
    if (HAS_R) o += r[i];
    out[i] = o;
  }
}

}  // namespace

pd_status launch_bias_gelu_residual(const float* x, const float* bias, const float* r, float* out, int64_t rows,
                                    int64_t cols, cudaStream_t s) {
  const int64_t n = rows * cols;
  const bool vec_ok = (cols % 4 == 0) && aligned16(x) && aligned16(bias) && aligned16(out) && (!r || aligned16(r));
  if (vec_ok) {
    constexpr int kUnroll = 4;
    const int64_t n4 = n / 4;
    const int64_t grid = (n4 + 256 * kUnroll - 1) / (256 * kUnroll);
    if (grid > 0x7fffffff) return PD_ERR_BAD_SHAPE;
    if (r) bias_gelu_residual_vec4<true, kUnroll><<<(int)grid, 256, 0, s>>>(x, bias, r, out, n4, (int)(cols / 4));
    else bias_gelu_residual_vec4<false, kUnroll><<<(int)grid, 256, 0, s>>>(x, bias, r, out, n4, (int)(cols / 4));
  } else {
    int64_t grid = (n + 255) / 256;
    const int64_t cap = (int64_t)sm_count() * 32;
    if (grid > cap) grid = cap;
    if (r) bias_gelu_residual_scalar<true><<<(int)grid, 256, 0, s>>>(x, bias, r, out, n, cols);
    else bias_gelu_residual_scalar<false><<<(int)grid, 256, 0, s>>>(x, bias, r, out, n, cols);
  }
  return check_launch();
}

}  // namespace pd

extern "C" pd_status pd_bias_gelu_residual(const float* x, const float* bias, const float* r, float* out,
                                           int64_t rows, int64_t cols, cudaStream_t stream) {
  if (!x || !bias || !out) return PD_ERR_NULL_POINTER;
  if (rows < 0 || cols <= 0) return PD_ERR_BAD_SHAPE;
  if ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(out) | reinterpret_cast<uintptr_t>(bias) |
       reinterpret_cast<uintptr_t>(r)) & 3u)
    return PD_ERR_ALIGNMENT;
  if (rows == 0) return PD_OK;
  pd_status st = pd::require_sm100();
  if (st != PD_OK) return st;
  return pd::launch_bias_gelu_residual(x, bias, r, out, rows, cols, stream);
}
