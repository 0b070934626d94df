// Layer normalisation over the last dimension, fp32 in, fp32 or bf16 out.
//
//   mu_i = mean_j x[i,j];  var_i = mean_j (x[i,j] - mu_i)^2  (biased)
//   y[i,j] = (x[i,j] - mu_i) * rsqrt(var_i + eps) * gamma[j] + beta[j]
//
// HBM-bound: 8 bytes per element.  The row is read once into registers with
// 128-bit loads; the mean and the centred second moment are then passes over
// registers (data centred before squaring, mean refined by the mean of the
// residuals: no E[x^2] - mu^2 cancellation), reduced with warp shuffles.
//   * cols <= 1024   : one warp per row, two rows per CTA
//   * cols <= 8192   : one CTA of 64 to 256 threads per row, 8 float4 per thread
//   * cols <= 28672  : one CTA of 256 threads per row, 12 to 28 float4 per thread at 85 or 128 registers (three
//                      or two rows in flight per SM)
//   * cols <= 262144 : one cluster of 2 to 8 CTAs per row, ceil(cols / 16384) CTAs of 512 threads up to
//                      131072 columns and ceil(cols / 32768) of 1024 beyond (partial statistics merged
//                      through distributed shared memory)
//   * longer, aligned: one CTA per row, three 128-bit passes (mean from HBM; centred
//                      second moment and normalisation from L2)
//   * otherwise      : one CTA per row, three scalar passes from global/L2; partial
//                      statistics are merged pairwise (Chan/Welford form)
#include "pd_common.cuh"

namespace pd {
namespace {

constexpr int64_t kFatRowCols = 28672;  // columns one 256-thread CTA holds at 28 float4 per thread

template <int VPT, int THREADS_PER_ROW, int THREADS_PER_CTA, typename OutT>
__global__ void __launch_bounds__(THREADS_PER_CTA, VPT > 12 ? 2 : VPT > 8 ? 3 : (THREADS_PER_CTA >= 1024 ? 1 : (THREADS_PER_CTA == 128 ? 5 : 1024 / THREADS_PER_CTA)))  // at most 64 registers (1024 threads resident per SM); 96 for the 128-thread CTAs of 4096-column rows, where five CTAs with the compiler free to keep more loads apart measured 3 % faster than eight; 85 / 128 for the 256-thread CTAs that hold 12 / 16 to 28 float4 per thread (rows of 8196 to 28672 columns, three / two of them in flight per SM)
layernorm_rows_in_registers(const float* __restrict__ x, const float* __restrict__ gamma,
                            const float* __restrict__ beta, OutT* __restrict__ y, int64_t rows, int cols,
                            float eps) {
  constexpr int ROWS_PER_CTA = THREADS_PER_CTA / THREADS_PER_ROW;
  constexpr int NWARPS = THREADS_PER_ROW / 32;
  __shared__ float scratch[3][NWARPS];
  const int t = threadIdx.x % THREADS_PER_ROW;
  const int cols4 = cols >> 2;
  const float inv_cols = 1.0f / (float)cols;
  const float4* g4 = reinterpret_cast<const float4*>(gamma);
  const float4* b4 = reinterpret_cast<const float4*>(beta);
  griddep_wait();
  griddep_launch_dependents();
  for (int64_t row = (int64_t)blockIdx.x * ROWS_PER_CTA + threadIdx.x / THREADS_PER_ROW; row < rows;
       row += (int64_t)gridDim.x * ROWS_PER_CTA) {
    const float4* xr = reinterpret_cast<const float4*>(x + row * cols);
    float4 v[VPT];
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
      const int c = t + i * THREADS_PER_ROW;
      v[i] = (c < cols4) ? ld_stream(xr + c) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < VPT; ++i) s += (v[i].x + v[i].y) + (v[i].z + v[i].w);
    const float mu0 = block_reduce<NWARPS, false>(s, scratch, 0) * inv_cols;
    // Centre on the first estimate, then refine it with the mean of the
    // residuals: the fp32 sum above loses digits when |mean| >> spread, the sum
    // of the (small) residuals does not.
    float d1 = 0.f, d2 = 0.f;
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
      const int c = t + i * THREADS_PER_ROW;
      if (c < cols4) {
        v[i].x -= mu0; v[i].y -= mu0; v[i].z -= mu0; v[i].w -= mu0;
        d1 += (v[i].x + v[i].y) + (v[i].z + v[i].w);
        d2 += (v[i].x * v[i].x + v[i].y * v[i].y) + (v[i].z * v[i].z + v[i].w * v[i].w);
      }
    }
    const float delta = block_reduce<NWARPS, false>(d1, scratch, 1) * inv_cols;
    const float var = fmaxf(block_reduce<NWARPS, false>(d2, scratch, 2) * inv_cols - delta * delta, 0.f);
    const float rstd = rsqrtf(var + eps);
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
      const int c = t + i * THREADS_PER_ROW;
      if (c < cols4) {
        const float4 g = __ldg(g4 + c), b = __ldg(b4 + c);
        store_out4(y, row * cols4 + c,
                   make_float4((v[i].x - delta) * rstd * g.x + b.x, (v[i].y - delta) * rstd * g.y + b.y,
                               (v[i].z - delta) * rstd * g.z + b.z, (v[i].w - delta) * rstd * g.w + b.w));
      }
    }
    if constexpr (NWARPS > 1) __syncthreads();
  }
}

// Rows of 32768 < cols <= 262144: one cluster of up to 8 CTAs per row, the columns dealt evenly, each CTA keeping
// its share (at most 32 per thread) in registers; 512-thread CTAs, two per SM, up to 131072 columns; the three sums are combined over the cluster through distributed shared memory.
template <int THREADS, typename OutT>
__global__ void __launch_bounds__(THREADS, 1024 / THREADS)
layernorm_rows_cluster(const float* __restrict__ x, const float* __restrict__ gamma, const float* __restrict__ beta,
                       OutT* __restrict__ y, int64_t rows, int cols, float eps) {
  constexpr int VPT = 8, NWARPS = THREADS / 32;
  __shared__ float scratch[3][NWARPS];
  __shared__ float xchg[8];
  __shared__ __align__(8) float xchg2[16];
  const int cols4 = cols >> 2;
  const float inv_cols = 1.0f / (float)cols;
  const float4* g4 = reinterpret_cast<const float4*>(gamma);
  const float4* b4 = reinterpret_cast<const float4*>(beta);
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
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < VPT; ++i) s += (v[i].x + v[i].y) + (v[i].z + v[i].w);
  const float mu0 = cluster_allreduce<false>(block_reduce<NWARPS, false>(s, scratch, 0), xchg) * inv_cols;
  // centre on the first estimate and refine it with the mean of the residuals, as in the single-CTA kernel
  float d1 = 0.f, d2 = 0.f;
#pragma unroll
  for (int i = 0; i < VPT; ++i) {
    const int c = base + threadIdx.x + i * THREADS;
    if (c < end) {
      v[i].x -= mu0; v[i].y -= mu0; v[i].z -= mu0; v[i].w -= mu0;
      d1 += (v[i].x + v[i].y) + (v[i].z + v[i].w);
      d2 += (v[i].x * v[i].x + v[i].y * v[i].y) + (v[i].z * v[i].z + v[i].w * v[i].w);
    }
  }
  d1 = block_reduce<NWARPS, false>(d1, scratch, 1);
  d2 = block_reduce<NWARPS, false>(d2, scratch, 2);
  const float2 dd = cluster_allreduce_sum2(d1, d2, xchg2);
  const float delta = dd.x * inv_cols;
  const float var = fmaxf(dd.y * inv_cols - delta * delta, 0.f);
  const float rstd = rsqrtf(var + eps);
#pragma unroll
  for (int i = 0; i < VPT; ++i) {
    const int c = base + threadIdx.x + i * THREADS;
    if (c < end) {
      const float4 g = __ldg(g4 + c), b = __ldg(b4 + c);
      store_out4(y, row * cols4 + c,
                 make_float4((v[i].x - delta) * rstd * g.x + b.x, (v[i].y - delta) * rstd * g.y + b.y,
                             (v[i].z - delta) * rstd * g.z + b.z, (v[i].w - delta) * rstd * g.w + b.w));
    }
  }
}

// (count, mean, M2) partial statistics and their pairwise merge.
struct Moments {
  float n, mean, m2;
};
__device__ __forceinline__ Moments merge(Moments a, Moments b) {
  const float n = a.n + b.n;
  if (n == 0.f) return a;
  const float d = b.mean - a.mean, w = b.n / n;
  return Moments{n, a.mean + d * w, a.m2 + b.m2 + d * d * a.n * w};
}

template <typename OutT>
__global__ void __launch_bounds__(256)
layernorm_rows_generic(const float* __restrict__ x, const float* __restrict__ gamma,
                       const float* __restrict__ beta, OutT* __restrict__ y, int64_t rows, int64_t cols,
                       float eps) {
  __shared__ Moments part[8];
  __shared__ float stat[2];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int64_t row = blockIdx.x; row < rows; row += gridDim.x) {
    const float* xr = x + row * cols;
    // per-thread Welford over a strided slice of the row, on data shifted by the
    // row's first element so that a large common offset costs no precision
    const float shift = xr[0];
    Moments m{0.f, 0.f, 0.f};
    for (int64_t j = threadIdx.x; j < cols; j += 256) {
      const float v = xr[j] - shift;
      m.n += 1.f;
      const float d = v - m.mean;
      m.mean += d / m.n;
      m.m2 += d * (v - m.mean);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      Moments other{__shfl_xor_sync(0xffffffffu, m.n, o), __shfl_xor_sync(0xffffffffu, m.mean, o),
                    __shfl_xor_sync(0xffffffffu, m.m2, o)};
      // merge in a lane-independent order so that every lane ends with the same bits
      m = (lane & o) ? merge(other, m) : merge(m, other);
    }
    if (lane == 0) part[warp] = m;
    __syncthreads();
    if (threadIdx.x == 0) {
      Moments tot = part[0];
      for (int w = 1; w < 8; ++w) tot = merge(tot, part[w]);
      stat[0] = tot.mean;
      stat[1] = rsqrtf(tot.m2 / (float)cols + eps);
    }
    __syncthreads();
    const float mu = stat[0], rstd = stat[1];
    for (int64_t j = threadIdx.x; j < cols; j += 256)
      store_out1(y, row * cols + j, ((xr[j] - shift) - mu) * rstd * gamma[j] + beta[j]);
    __syncthreads();
  }
}

// Rows too long for registers (cols > 32768), 16-byte aligned: one CTA of 512 threads per row, three passes with
// 128-bit accesses: mean (from HBM), centred second moment and normalisation (both from L2, where the row still is).
template <typename OutT>
__global__ void __launch_bounds__(512)
layernorm_rows_streaming(const float* __restrict__ x, const float* __restrict__ gamma,
                         const float* __restrict__ beta, OutT* __restrict__ y, int64_t rows, int64_t cols,
                         float eps) {
  __shared__ float scratch[3][16];
  const int64_t cols4 = cols >> 2;
  const float inv_cols = 1.0f / (float)cols;
  const float4* g4 = reinterpret_cast<const float4*>(gamma);
  const float4* b4 = reinterpret_cast<const float4*>(beta);
  for (int64_t row = blockIdx.x; row < rows; row += gridDim.x) {
    const float4* xr = reinterpret_cast<const float4*>(x + row * cols);
    const float shift = __ldg(reinterpret_cast<const float*>(xr));  // keeps the first sum small when |mean| >> spread
    float s = 0.f;
    for (int64_t c = threadIdx.x; c < cols4; c += 512) {
      const float4 v = __ldg(xr + c);
      s += ((v.x - shift) + (v.y - shift)) + ((v.z - shift) + (v.w - shift));
    }
    const float mu = shift + block_reduce<16, false>(s, scratch, 0) * inv_cols;
    float q = 0.f, d1 = 0.f;
    for (int64_t c = threadIdx.x; c < cols4; c += 512) {
      const float4 v = __ldg(xr + c);
      const float a = v.x - mu, b = v.y - mu, cc = v.z - mu, d = v.w - mu;
      d1 += (a + b) + (cc + d);
      q += (a * a + b * b) + (cc * cc + d * d);
    }
    const float delta = block_reduce<16, false>(d1, scratch, 1) * inv_cols;  // residual of the mean
    const float var = fmaxf(block_reduce<16, false>(q, scratch, 2) * inv_cols - delta * delta, 0.f);
    const float rstd = rsqrtf(var + eps);  // (v - mu) - delta below: adding delta to mu would round it away
    for (int64_t c = threadIdx.x; c < cols4; c += 512) {
      const float4 v = __ldg(xr + c), g = __ldg(g4 + c), b = __ldg(b4 + c);
      store_out4(y, row * cols4 + c,
                 make_float4(((v.x - mu) - delta) * rstd * g.x + b.x, ((v.y - mu) - delta) * rstd * g.y + b.y,
                             ((v.z - mu) - delta) * rstd * g.z + b.z, ((v.w - mu) - delta) * rstd * g.w + b.w));
    }
    __syncthreads();
  }
}

template <int VPT, typename OutT>
void launch_warp_rows(const float* x, const float* g, const float* b, OutT* y, int64_t rows, int cols, float eps,
                      cudaStream_t s) {
  constexpr int kThreads = 64, kRowsPerCta = kThreads / 32;  // two rows per CTA: the finest grain for the last, partly filled wave
  auto kernel = layernorm_rows_in_registers<VPT, 32, kThreads, OutT>;
  // one CTA per two rows, all launched: the hardware scheduler balances many short CTAs better than a
  // grid-stride loop over a resident set does
  const int64_t ctas = (rows + kRowsPerCta - 1) / kRowsPerCta;
  const int grid = (int)(ctas < 0x7fffffff ? ctas : 0x7fffffff);
  launch_pdl(kernel, dim3(grid), dim3(kThreads), 0, s, x, g, b, y, rows, cols, eps);
}

// One CTA of THREADS threads per row, up to VPT float4 per thread.
template <int THREADS, typename OutT, int VPT = 8>
void launch_cta_rows(const float* x, const float* g, const float* b, OutT* y, int64_t rows, int cols, float eps,
                     cudaStream_t s) {
  auto kernel = layernorm_rows_in_registers<VPT, THREADS, THREADS, OutT>;
  const int grid = (int)(rows < 0x7fffffff ? rows : 0x7fffffff);
  launch_pdl(kernel, dim3(grid), dim3(THREADS), 0, s, x, g, b, y, rows, cols, eps);
}

template <typename OutT>
pd_status dispatch(const float* x, const float* g, const float* b, OutT* y, int64_t rows, int64_t cols, float eps,
                   cudaStream_t s) {
  const bool vec_ok = (cols % 4 == 0) && aligned16(x) && aligned16(g) && aligned16(b) &&
                      ((reinterpret_cast<uintptr_t>(y) & (sizeof(OutT) * 4 - 1)) == 0);
  logf("%s %lld x %lld: %s", "layernorm", (long long)rows, (long long)cols,
       !vec_ok ? "scalar three-pass path (unaligned or ragged rows)"
       : cols <= 1024 ? "one warp per row, row in registers"
       : cols <= kFatRowCols ? "one CTA per row, row in registers"
       : cols <= 262144 ? "one cluster per row, row in registers" : "one CTA per row, streaming passes");
  if (vec_ok && cols <= 1024) {
    const int c = (int)cols;
    if (c <= 128) launch_warp_rows<1>(x, g, b, y, rows, c, eps, s);
    else if (c <= 256) launch_warp_rows<2>(x, g, b, y, rows, c, eps, s);
    else if (c <= 512) launch_warp_rows<4>(x, g, b, y, rows, c, eps, s);
    else launch_warp_rows<8>(x, g, b, y, rows, c, eps, s);
  } else if (vec_ok && cols <= kFatRowCols) {
    const int c = (int)cols;
    if (c <= 2048) launch_cta_rows<64>(x, g, b, y, rows, c, eps, s);
    else if (c <= 4096) launch_cta_rows<128>(x, g, b, y, rows, c, eps, s);
    else if (c <= 8192) launch_cta_rows<256>(x, g, b, y, rows, c, eps, s);
    // from 8196 columns on: 256 threads with 12 float4 each (85 registers, three rows in flight per SM) or 16 to 28
    // (128 registers, two rows in flight); a CTA of 512 or 1024 threads with 8 float4 each leaves the memory pipe idle
    // while its row is reduced (LayerNorm: 5.7 -> 6.4 TB/s at 12288 columns, 4.0 -> 5.8 at 20480)
    else if (c <= 12288) launch_cta_rows<256, OutT, 12>(x, g, b, y, rows, c, eps, s);
    else if (c <= 16384) launch_cta_rows<256, OutT, 16>(x, g, b, y, rows, c, eps, s);
    else if (c <= 20480) launch_cta_rows<256, OutT, 20>(x, g, b, y, rows, c, eps, s);
    else if (c <= 24576) launch_cta_rows<256, OutT, 24>(x, g, b, y, rows, c, eps, s);
    else launch_cta_rows<256, OutT, 28>(x, g, b, y, rows, c, eps, s);
  } else if (vec_ok && cols <= 262144 && rows * 8 <= 0x7fffffff) {
    // (clusters of the 256-thread CTAs above are slower than these: LayerNorm at 65536 columns 3.0 against 4.2 TB/s)
    if (cols <= 131072) {
      const unsigned cl = (unsigned)((cols + 16383) / 16384);
      launch_pdl_cluster(layernorm_rows_cluster<512, OutT>, dim3((unsigned)rows * cl), dim3(512), cl, 0, s, x, g, b, y, rows,
                         (int)cols, eps);
    } else {
      const unsigned cl = (unsigned)((cols + 32767) / 32768);
      launch_pdl_cluster(layernorm_rows_cluster<1024, OutT>, dim3((unsigned)rows * cl), dim3(1024), cl, 0, s, x, g, b, y, rows,
                         (int)cols, eps);
    }
  } else if (vec_ok && x != reinterpret_cast<const float*>(y)) {
    const int grid = (int)(rows < (int64_t)sm_count() * 4 ? rows : (int64_t)sm_count() * 4);
    layernorm_rows_streaming<OutT><<<grid, 512, 0, s>>>(x, g, b, y, rows, cols, eps);
  } else {
    const int grid = (int)(rows < (int64_t)sm_count() * 16 ? rows : (int64_t)sm_count() * 16);
    layernorm_rows_generic<OutT><<<grid, 256, 0, s>>>(x, g, b, y, rows, cols, eps);
  }
  return check_launch();
}

}  // namespace

pd_status launch_layernorm(const float* x, const float* gamma, const float* beta, void* y, bool y_is_bf16,
                           int64_t rows, int64_t cols, float eps, cudaStream_t s) {
  if (y_is_bf16) return dispatch(x, gamma, beta, static_cast<__nv_bfloat16*>(y), rows, cols, eps, s);
  return dispatch(x, gamma, beta, static_cast<float*>(y), rows, cols, eps, s);
}

}  // namespace pd

extern "C" pd_status pd_layernorm(const float* x, const float* gamma, const float* beta, float* y, int64_t rows,
                                  int64_t cols, float eps, cudaStream_t stream) {
  if (!x || !gamma || !beta || !y) return PD_ERR_NULL_POINTER;
  if (rows < 0 || cols <= 0 || !(eps >= 0.f)) return PD_ERR_BAD_SHAPE;
  if ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(y) | reinterpret_cast<uintptr_t>(gamma) |
       reinterpret_cast<uintptr_t>(beta)) & 3u)
    return PD_ERR_ALIGNMENT;
  if (rows == 0) return PD_OK;
  pd_status st = pd::require_sm100();
  if (st != PD_OK) return st;
  return pd::launch_layernorm(x, gamma, beta, y, false, rows, cols, eps, stream);
}
