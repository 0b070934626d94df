// Pieces shared by the tcgen05 GEMM kernels (1-CTA and 2-CTA tiles): tile
// constants, kernel parameters, the fused epilogue and the tensor-map helpers.
// Internal to the library.
#pragma once

#include "pd_common.cuh"
#include "sm100_ptx.cuh"

namespace pd {
namespace gemm {

constexpr int BM = 128;       // tile rows = TMEM lanes
constexpr int BK = 64;        // k-block: 64 bf16 = one 128-byte swizzle row
constexpr int UMMA_K = 16;    // k extent of one tcgen05.mma for 16-bit inputs
constexpr int kEpilogueWarps = 8;
constexpr int kThreads = 64 + 32 * kEpilogueWarps;
constexpr int kEpilogueThreads = 32 * kEpilogueWarps;
constexpr int kSmemLimit = 227 * 1024;

constexpr int kEpilogueBytes = kEpilogueWarps * 4096;  // one 32-row x 128-byte staging buffer per warp

struct KernelParams {
  void* C;
  const float* bias;
  const __nv_bfloat16* residual;
  int* status;
  int64_t ldc, strideC_inner, strideC_outer, ldr;
  int M, N, K;
  int tiles_m, tiles_n, batch_inner, num_tiles;  // num_tiles = batch_outer * batch_inner * tiles_m * tiles_n
  float alpha;
  int c_is_f32, act;  // act: 0 nothing, 1 erf-form GELU, 2 ReLU
  // Single-CTA and CTA-pair kernels only (zero elsewhere): the time after which their waits give up (0: the default
  // of 2 s), and the test switch that makes their producers skip every load, so that the wait for the first stage
  // runs out.
  unsigned long long wait_limit_ns;
  int withhold_loads;
};

__device__ __forceinline__ uint64_t wait_limit(const KernelParams& p) {
  return p.wait_limit_ns != 0 ? (uint64_t)p.wait_limit_ns : 2000000000ull;
}

// Codes left in the device status word by an expired wait.
enum : int { kTimeoutProducer = 101, kTimeoutMmaFull = 102, kTimeoutMmaAcc = 103, kTimeoutEpilogue = 104 };

// GELU in its erf form, z * Phi(z), with the normal tail evaluated as
//   q = 2^P(t) ~ Phi(-t),  t = min(|z|, 5),  Phi(z) = z < 0 ? q : 1 - q,  q = 0 beyond 5.
// P is the degree-6 minimax fit of log2 Phi(-t) on [0, 5] produced by
// fit_gelu_tail_poly.py (max |dP| = 1.8e-5, i.e. a relative error of 1.2e-5 in the
// tail; in fp32 the whole function stays within 1.5e-5 relative, 2e-6 absolute).
// One exponential and ten FP32 operations per value instead of erff's branches.
__device__ __forceinline__ float gelu_erf(float z) {
  const float a = fabsf(z);
  const float t = fminf(a, 5.0f);
  float p = 2.945814984e-05f;
  p = fmaf(p, t, -7.087827801e-04f);
  p = fmaf(p, t, 7.746013990e-03f);
  p = fmaf(p, t, -5.260629289e-02f);
  p = fmaf(p, t, -4.596254617e-01f);
  p = fmaf(p, t, -1.150867236e+00f);
  p = fmaf(p, t, -1.000017644e+00f);
  float q;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(q) : "f"(p));
  q = a > 5.0f ? 0.0f : q;
  return z * (z < 0.0f ? q : 1.0f - q);
}

// The same function for two values at once, in the form  max(z, 0) + u * q  with  u = -t = max(-|z|, -5)
// (equal to z * Phi(z) on both sides of zero), the polynomial written in u and, like the last step,
// evaluated as packed fp32 pairs: the epilogue that applies it is bound by instruction issue, and this form
// needs one instruction per value for u and none for the sign or the cut-off.  Beyond |z| = 5 the tail stays
// at Phi(-5) = 2.9e-7 instead of dropping to zero: an absolute error of at most 1.5e-6 there.
// u (not -|z|) multiplies q, so an infinite z stays infinite instead of becoming 0 * inf.
__device__ __forceinline__ uint64_t gelu_erf_x2(uint64_t z2) {
  using namespace sm100;
  float z0, z1;
  unpack_f32x2(z2, z0, z1);
  const uint64_t u2 = pack_f32x2(fmaxf(-fabsf(z0), -5.0f), fmaxf(-fabsf(z1), -5.0f));
  uint64_t p2 = pack_f32x2(2.945814984e-05f, 2.945814984e-05f);
  p2 = fma_f32x2(p2, u2, pack_f32x2(7.087827801e-04f, 7.087827801e-04f));
  p2 = fma_f32x2(p2, u2, pack_f32x2(7.746013990e-03f, 7.746013990e-03f));
  p2 = fma_f32x2(p2, u2, pack_f32x2(5.260629289e-02f, 5.260629289e-02f));
  p2 = fma_f32x2(p2, u2, pack_f32x2(-4.596254617e-01f, -4.596254617e-01f));
  p2 = fma_f32x2(p2, u2, pack_f32x2(1.150867236e+00f, 1.150867236e+00f));
  p2 = fma_f32x2(p2, u2, pack_f32x2(-1.000017644e+00f, -1.000017644e+00f));
  float p0, p1, q0, q1;
  unpack_f32x2(p2, p0, p1);
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(q0) : "f"(p0));
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(q1) : "f"(p1));
  return fma_f32x2(u2, pack_f32x2(q0, q1), pack_f32x2(fmaxf(z0, 0.0f), fmaxf(z1, 0.0f)));
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// The bf16 residual values of 32 consecutive columns of one row, fetched one
// step ahead of their use; out-of-range parts are zero.
struct ResidualRegs {
  uint4 q[4];
  __device__ __forceinline__ void load(const KernelParams& p, int m, int n0, bool row_ok) {
    if (p.residual == nullptr) return;
    const __nv_bfloat16* rr = p.residual + (int64_t)m * p.ldr + n0;
    if (row_ok && n0 + 32 <= p.N) {
#pragma unroll
      for (int j = 0; j < 4; ++j) q[j] = __ldg(reinterpret_cast<const uint4*>(rr) + j);
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        uint32_t w[4] = {0u, 0u, 0u, 0u};
#pragma unroll
        for (int t = 0; t < 8; ++t)
          if (row_ok && n0 + j * 8 + t < p.N)
            w[t >> 1] |= (uint32_t)__bfloat16_as_ushort(rr[j * 8 + t]) << (16 * (t & 1));
        q[j] = make_uint4(w[0], w[1], w[2], w[3]);
      }
    }
  }
};

// Epilogue role of one warp (warps 2..9 of the CTA): for every tile this CTA
// owns, wait for its accumulator, drain this warp's share of it and release it.
// The accumulator is drained 32 columns at a time; one TMA store carries 128
// bytes of each of the warp's 32 rows: a chunk of 64 bf16 columns (two steps)
// or 32 fp32 columns (one step).  The two warps of a lane group take alternate
// chunks.  `first_tile`/`tile_stride` enumerate the tiles, `row_block` maps a
// tile's m index to the first of the 128 rows held in this CTA's tensor memory,
// `release` is called once per tile by one lane, after the whole warp's last tensor-memory read.
template <int BN, bool C_F32, typename RowBlockFn, typename ReleaseFn>
__device__ __forceinline__ void epilogue_warp(const KernelParams& p, const CUtensorMap* tmap_c, uint32_t tmem_base,
                                              uint32_t epi_base, uint32_t acc_full_bar0, volatile int* abort_flag,
                                              int first_tile, int tile_stride, RowBlockFn row_block,
                                              ReleaseFn release) {
  using namespace sm100;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr int STEPS = C_F32 ? 1 : 2;
  constexpr int CW = 32 * STEPS;       // chunk width in columns
  constexpr int NCHUNK = BN / CW;
  const int quarter = warp & 3;         // TMEM lanes 32*quarter .. 32*quarter+31 belong to this warp
  const int group = (warp - 2) >> 2;    // 0: even chunks, 1: odd chunks
  const uint32_t buf = epi_base + (uint32_t)(warp - 2) * 4096u;
  const uint32_t row_addr = buf + (uint32_t)lane * 128u;
  const uint32_t sw = (uint32_t)(lane & 7);  // 128-byte swizzle: 16-byte unit index ^= row % 8
  const int my_steps = ((NCHUNK - group + 1) / 2) * STEPS;
  auto col_of = [&](int i) { return ((i / STEPS) * 2 + group) * CW + (i % STEPS) * 32; };
  int local = 0;
  // A TMA store clips at the row's end only in whole 16-byte units.  When N elements are not a whole number of
  // them, the chunk that holds the end of the row is written with plain stores instead.
  const bool ragged_n = ((int64_t)p.N * (C_F32 ? 4 : 2)) % 16 != 0;
  if (lane == 0) prefetch_tensormap(tmap_c);
  for (int tile = first_tile; tile < p.num_tiles; tile += tile_stride, ++local) {
    const int nt = tile % p.tiles_n;
    const int mt = (tile / p.tiles_n) % p.tiles_m;
    const int b = tile / (p.tiles_n * p.tiles_m);
    const int bi = b % p.batch_inner, bo = b / p.batch_inner;
    const int acc = local & 1;
    const uint32_t acc_ph = (local >> 1) & 1u;
    const int m_warp = row_block(mt) + quarter * 32;  // first row of this warp
    const int m = m_warp + lane;
    const bool row_ok = m < p.M;
    const int n_tile = nt * BN;
    ResidualRegs cur, nxt;
    if (my_steps > 0 && n_tile + col_of(0) < p.N)
      cur.load(p, m, n_tile + col_of(0), row_ok);  // independent of the accumulator: issued before the wait
    if (!mbar_wait(acc_full_bar0 + 8u * acc, acc_ph, abort_flag, p.status, kTimeoutEpilogue, wait_limit(p))) break;
    tcgen05_fence_after_sync();
    const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * BN;
#pragma unroll 1
    for (int i = 0; i < my_steps; ++i) {
      const int c0 = col_of(i);
      const int n0 = n_tile + c0;
      if (n0 >= p.N) break;  // uniform over the warp; columns grow with i
      const int step = i % STEPS;
      const bool has_next = (i + 1 < my_steps) && (n_tile + col_of(i + 1) < p.N);
      uint32_t r[32];
      tmem_ld_32x32b_x32(t_row + c0, r);
      if (has_next) nxt.load(p, m, n_tile + col_of(i + 1), row_ok);
      tmem_ld_wait();
      // two fp32 values per instruction wherever the operation exists in packed form
      uint64_t v2[16];
      {
        const uint64_t alpha2 = pack_f32x2(p.alpha, p.alpha);
        if (p.bias != nullptr && n0 + 32 <= p.N) {
#pragma unroll
          for (int j = 0; j < 32; j += 4) {
            const float4 bv = __ldg(reinterpret_cast<const float4*>(p.bias + n0 + j));
            v2[j / 2] = fma_f32x2(pack_b32x2(r[j], r[j + 1]), alpha2, pack_f32x2(bv.x, bv.y));
            v2[j / 2 + 1] = fma_f32x2(pack_b32x2(r[j + 2], r[j + 3]), alpha2, pack_f32x2(bv.z, bv.w));
          }
        } else {
#pragma unroll
          for (int j = 0; j < 32; j += 2) {
            float b0 = 0.f, b1 = 0.f;
            if (p.bias != nullptr) {
              if (n0 + j < p.N) b0 = __ldg(p.bias + n0 + j);
              if (n0 + j + 1 < p.N) b1 = __ldg(p.bias + n0 + j + 1);
            }
            v2[j / 2] = fma_f32x2(pack_b32x2(r[j], r[j + 1]), alpha2, pack_f32x2(b0, b1));
          }
        }
      }
      if (p.act == 1) {
#pragma unroll
        for (int j = 0; j < 16; ++j) v2[j] = gelu_erf_x2(v2[j]);
      } else if (p.act == 2) {
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          float z0, z1;
          unpack_f32x2(v2[j], z0, z1);
          v2[j] = pack_f32x2(fmaxf(z0, 0.0f), fmaxf(z1, 0.0f));
        }
      }
      if (p.residual != nullptr) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const uint32_t w[4] = {cur.q[j].x, cur.q[j].y, cur.q[j].z, cur.q[j].w};
#pragma unroll
          for (int t = 0; t < 4; ++t) v2[4 * j + t] = add_f32x2(v2[4 * j + t], pack_b32x2(w[t] << 16, w[t] & 0xffff0000u));
        }
      }
      float v[32];
#pragma unroll
      for (int j = 0; j < 16; ++j) unpack_f32x2(v2[j], v[2 * j], v[2 * j + 1]);
      if (ragged_n && n0 - step * 32 + CW > p.N) {
        if (row_ok) {
          const int64_t off = (int64_t)bo * p.strideC_outer + (int64_t)bi * p.strideC_inner + (int64_t)m * p.ldc + n0;
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            if (n0 + j < p.N) {
              if constexpr (C_F32) static_cast<float*>(p.C)[off + j] = v[j];
              else static_cast<__nv_bfloat16*>(p.C)[off + j] = __float2bfloat16_rn(v[j]);
            }
          }
        }
        cur = nxt;
        continue;
      }
      if (step == 0) {
        // the previous store of this warp must have finished reading the buffer
        if (lane == 0) tma_store_wait_read<0>();
        __syncwarp();
      }
      if constexpr (C_F32) {
#pragma unroll
        for (int u = 0; u < 8; ++u)
          st_shared_v4(row_addr + (((uint32_t)u ^ sw) << 4),
                       make_uint4(__float_as_uint(v[4 * u]), __float_as_uint(v[4 * u + 1]),
                                  __float_as_uint(v[4 * u + 2]), __float_as_uint(v[4 * u + 3])));
      } else {
#pragma unroll
        for (int u = 0; u < 4; ++u)
          st_shared_v4(row_addr + (((uint32_t)(step * 4 + u) ^ sw) << 4),
                       make_uint4(pack_bf16(v[8 * u], v[8 * u + 1]), pack_bf16(v[8 * u + 2], v[8 * u + 3]),
                                  pack_bf16(v[8 * u + 4], v[8 * u + 5]), pack_bf16(v[8 * u + 6], v[8 * u + 7])));
      }
      if (step == STEPS - 1 || n0 + 32 >= p.N) {
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          tma_store_4d(tmap_c, buf, n0 - step * 32, m_warp, bi, bo);
          tma_store_commit();
        }
      }
      cur = nxt;
    }
    tcgen05_fence_before_sync();
    __syncwarp();
    if (lane == 0) release(acc);  // one arrival per warp
  }
  // Shared memory must outlive every store that still reads it (the writes themselves are complete, and visible to
  // whatever follows in the stream, when the grid has finished).
  if (lane == 0) tma_store_wait_read<0>();
  __syncwarp();
}

// Epilogue of the gated form.  The accumulator holds G = A Wg in columns [0, BN/2) and U = A Wu in columns
// [BN/2, BN) for the same BN/2 output columns; the warp writes SiLU(G) * U = G * U / (1 + exp(-G)) as bf16.
// The two warps of a lane group take alternate steps of 32 output columns; each step goes out through one
// half of the warp's staging buffer (32 rows x 64 bytes, 64-byte swizzle) and its own TMA store, so that a
// step is staged while the previous one is still being read.
template <int BN, typename ReleaseFn>
__device__ __forceinline__ void epilogue_warp_gated(const KernelParams& p, const CUtensorMap* tmap_c, uint32_t tmem_base,
                                                    uint32_t epi_base, uint32_t acc_full_bar0, volatile int* abort_flag,
                                                    int first_tile, int tile_stride, ReleaseFn release) {
  using namespace sm100;
  constexpr int OC = BN / 2;            // output columns per tile
  constexpr int STEPS = OC / 64;        // steps of 32 columns per warp and tile
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int quarter = warp & 3;
  const int group = (warp - 2) >> 2;
  const uint32_t buf = epi_base + (uint32_t)(warp - 2) * 4096u;
  const uint32_t sw = (uint32_t)((lane >> 1) & 3);  // 64-byte swizzle: 16-byte unit index ^= (row / 2) % 4
  const uint64_t nlog2e2 = pack_f32x2(-1.4426950408889634f, -1.4426950408889634f), one2 = pack_f32x2(1.0f, 1.0f);
  int local = 0;
  uint32_t stores = 0;
  if (lane == 0) prefetch_tensormap(tmap_c);
  for (int tile = first_tile; tile < p.num_tiles; tile += tile_stride, ++local) {
    const int nt = tile % p.tiles_n;
    const int mt = tile / p.tiles_n;
    const int acc = local & 1;
    const uint32_t acc_ph = (local >> 1) & 1u;
    const int m_warp = mt * BM + quarter * 32;
    if (!mbar_wait(acc_full_bar0 + 8u * acc, acc_ph, abort_flag, p.status, kTimeoutEpilogue, wait_limit(p))) break;
    tcgen05_fence_after_sync();
    const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * BN;
#pragma unroll 1
    for (int i = 0; i < STEPS; ++i) {
      const int c0 = (2 * i + group) * 32;
      if (nt * OC + c0 >= p.N) break;  // uniform over the warp
      uint32_t rg[32], ru[32];
      tmem_ld_32x32b_x32(t_row + c0, rg);
      tmem_ld_32x32b_x32(t_row + OC + c0, ru);
      tmem_ld_wait();
      uint32_t packed[16];
#pragma unroll
      for (int j = 0; j < 32; j += 2) {
        const uint64_t g2 = pack_b32x2(rg[j], rg[j + 1]);
        float x0, x1;
        unpack_f32x2(mul_f32x2(g2, nlog2e2), x0, x1);
        float e0, e1;
        asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e0) : "f"(x0));
        asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e1) : "f"(x1));
        float d0, d1;
        unpack_f32x2(add_f32x2(pack_f32x2(e0, e1), one2), d0, d1);
        float r0, r1;
        asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r0) : "f"(d0));
        asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r1) : "f"(d1));
        // (g * sigmoid(g)) * u, in this order: g * u alone could overflow where the product with sigmoid does not
        float y0, y1;
        unpack_f32x2(mul_f32x2(mul_f32x2(g2, pack_f32x2(r0, r1)), pack_b32x2(ru[j], ru[j + 1])), y0, y1);
        packed[j / 2] = pack_bf16(y0, y1);
      }
      const uint32_t half = buf + (stores & 1u) * 2048u;
      if (lane == 0) tma_store_wait_read<1>();  // the store before the previous one has finished reading this half
      __syncwarp();
#pragma unroll
      for (int u = 0; u < 4; ++u)
        st_shared_v4(half + (uint32_t)lane * 64u + (((uint32_t)u ^ sw) << 4),
                     make_uint4(packed[4 * u], packed[4 * u + 1], packed[4 * u + 2], packed[4 * u + 3]));
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) {
        tma_store_4d(tmap_c, half, nt * OC + c0, m_warp, 0, 0);
        tma_store_commit();
      }
      ++stores;
    }
    tcgen05_fence_before_sync();
    __syncwarp();
    if (lane == 0) release(acc);  // one arrival per warp
  }
  if (lane == 0) tma_store_wait_read<0>();
  __syncwarp();
}

// ---- host side -----------------------------------------------------------------
using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = [] {
    void* f = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      f = nullptr;
    return reinterpret_cast<EncodeTiledFn>(f);
  }();
  return fn;
}

// Tensor [outer][inner][rows][cols] of bf16 (or fp32 when `f32`) with cols
// contiguous, 128-byte swizzle unless another is named, zero fill outside the extents.  Strides in elements.
inline bool make_map(CUtensorMap* map, bool f32, const void* base, int64_t cols, int64_t rows, int64_t ld, int64_t n_inner,
              int64_t stride_inner, int64_t n_outer, int64_t stride_outer, int box_cols, int box_rows,
              CUtensorMapSwizzle swizzle = CU_TENSOR_MAP_SWIZZLE_128B) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  const cuuint64_t esize = f32 ? 4 : 2;
  // Unit batch extents still need a legal (16-byte multiple) stride.
  if (n_inner == 1) stride_inner = ld * rows;
  if (n_outer == 1) stride_outer = (n_inner == 1 ? ld * rows : stride_inner * n_inner);
  const cuuint64_t dims[4] = {(cuuint64_t)cols, (cuuint64_t)rows, (cuuint64_t)n_inner, (cuuint64_t)n_outer};
  const cuuint64_t strides[3] = {(cuuint64_t)ld * esize, (cuuint64_t)stride_inner * esize,
                                 (cuuint64_t)stride_outer * esize};
  const cuuint32_t box[4] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows, 1, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  return fn(map, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4,
            const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}


}  // namespace gemm
}  // namespace pd
