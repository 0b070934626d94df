// bf16 x bf16 -> fp32 contraction on the tcgen05 tensor cores with a fused epilogue.
//
//   C[m,n] = act(alpha * sum_k A[m,k] B[k,n] + bias[n]) + residual[m,n]
//
// Persistent, warp-specialised kernel, one CTA of 320 threads per SM:
//   warp 0, one lane : TMA producer.  Streams 128 x 64 tiles of A and BN x 64
//                      tiles of B (128-byte swizzle) into a ring of shared-memory
//                      stages; a "full" mbarrier per stage counts the bytes.
//   warp 1, one lane : MMA issuer.  Four tcgen05.mma (128 x BN x 16) per stage
//                      accumulate into one of two TMEM accumulators; a
//                      tcgen05.commit hands the stage back ("empty" barrier) and,
//                      after the last k-block, publishes the accumulator.
//   warps 2-9        : epilogue.  Two warps share each group of 32 TMEM lanes (32
//                      rows of the tile) and take alternate chunks of 128 output
//                      bytes per row.  A warp drains its chunk 32 columns at a
//                      time (tcgen05.ld), applies the epilogue in fp32, stages
//                      the chunk in its swizzled 4 KiB shared-memory buffer and
//                      hands it to a TMA store, while its sibling works on the
//                      next chunk and the MMA warp already fills the other
//                      accumulator with the next tile.  Residual values are
//                      fetched one step ahead.
// B is taken either as [K, N] (N contiguous: an "MN-major" MMA operand, loaded
// as BN/64 boxes of 64 x 64) or as [N, K] (K contiguous, "K-major").  Ragged M,
// N, K edges are zero-filled by TMA on load and clipped by TMA on store.
// Every mbarrier wait is bounded: on expiry the kernel records a code in the
// device status word, all roles drain, tensor memory is freed and the kernel
// returns.
#include "pd_common.cuh"
#include "sm100_ptx.cuh"

namespace pd {
namespace {

using namespace sm100;

constexpr int BM = 128;       // tile rows = TMEM lanes
constexpr int BK = 64;        // k-block: 64 bf16 = one 128-byte swizzle row
constexpr int UMMA_K = 16;    // k extent of one tcgen05.mma for 16-bit inputs
constexpr int kEpilogueWarps = 8;
constexpr int kThreads = 64 + 32 * kEpilogueWarps;
constexpr int kEpilogueThreads = 32 * kEpilogueWarps;
constexpr int kSmemLimit = 227 * 1024;

template <int BN>
struct Cfg {
  static constexpr int kStageA = BM * BK * 2;
  static constexpr int kStageB = BN * BK * 2;
  static constexpr int kStage = kStageA + kStageB;
  static constexpr int kBarrierBytes = 1024;
  static constexpr int kEpilogueBytes = kEpilogueWarps * 4096;  // one 32-row x 128-byte staging buffer per warp
  static constexpr int kStagesMax = (kSmemLimit - 1024 /*alignment slack*/ - kBarrierBytes - kEpilogueBytes) / kStage;
  static constexpr int kStages = kStagesMax > 8 ? 8 : kStagesMax;
  static constexpr int kSmemBytes = kStages * kStage + kEpilogueBytes + kBarrierBytes + 1024;
  static constexpr int kTmemCols = 2 * BN;  // two accumulators; 128, 256 or 512: a power of two
};

struct KernelParams {
  void* C;
  const float* bias;
  const __nv_bfloat16* residual;
  int* status;
  int64_t ldc, strideC_inner, strideC_outer, ldr;
  int M, N, K;
  int tiles_m, tiles_n, batch_inner, num_tiles;  // num_tiles = batch_outer * batch_inner * tiles_m * tiles_n
  float alpha;
  int c_is_f32, gelu;
};

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

template <int BN, bool B_NK, bool C_F32>
__global__ void __launch_bounds__(kThreads, 1)
gemm_bf16_tcgen05_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                         const __grid_constant__ CUtensorMap tmap_c, const KernelParams p) {
  using C = Cfg<BN>;
  constexpr int kStages = C::kStages;
  extern __shared__ uint8_t smem_raw[];
  // 128-byte swizzled tiles must start on a 1024-byte boundary.
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t epi_base = smem_base + kStages * C::kStage;  // 1024-byte aligned: kStage is a multiple of 1024
  const uint32_t bar_base = epi_base + C::kEpilogueBytes;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (kStages + s); };
  auto acc_full_bar = [&](int a) { return bar_base + 8u * (2 * kStages + a); };
  auto acc_empty_bar = [&](int a) { return bar_base + 8u * (2 * kStages + 2 + a); };
  const uint32_t drain_bar = bar_base + 8u * (2 * kStages + 4);
  uint8_t* ctrl = smem_gen + kStages * C::kStage + C::kEpilogueBytes + 8 * (2 * kStages + 5);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(ctrl);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(ctrl + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_kb = (p.K + BK - 1) / BK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(acc_full_bar(a), 1);
      mbar_init(acc_empty_bar(a), kEpilogueThreads);
    }
    mbar_init(drain_bar, 1);
    *abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async_smem();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), C::kTmemCols);
    tmem_relinquish_alloc_permit();
  }
  tcgen05_fence_before_sync();
  __syncthreads();
  tcgen05_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------- TMA producer
    if (lane == 0) {
      prefetch_tensormap(&tmap_a);
      prefetch_tensormap(&tmap_b);
      uint32_t it = 0;  // k-blocks issued so far, over all tiles
      bool ok = true;
      for (int tile = blockIdx.x; tile < p.num_tiles && ok; tile += gridDim.x) {
        const int nt = tile % p.tiles_n;
        const int mt = (tile / p.tiles_n) % p.tiles_m;
        const int b = tile / (p.tiles_n * p.tiles_m);
        const int bi = b % p.batch_inner, bo = b / p.batch_inner;
        for (int kb = 0; kb < num_kb; ++kb, ++it) {
          const int s = it % kStages;
          const uint32_t ph = (it / kStages) & 1u;
          if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, p.status, kTimeoutProducer)) { ok = false; break; }
          const uint32_t sa = smem_base + s * C::kStage, sb = sa + C::kStageA;
          mbar_arrive_expect_tx(full_bar(s), C::kStage);
          tma_load_4d(sa, &tmap_a, full_bar(s), kb * BK, mt * BM, bi, bo);
          if (B_NK) {
            tma_load_4d(sb, &tmap_b, full_bar(s), kb * BK, nt * BN, bi, bo);
          } else {
#pragma unroll
            for (int j = 0; j < BN / 64; ++j)
              tma_load_4d(sb + j * (64 * BK * 2), &tmap_b, full_bar(s), nt * BN + j * 64, kb * BK, bi, bo);
          }
        }
      }
      if (!ok) {
        // Leave no copy in flight: wait (briefly) for every stage last armed.
        const uint32_t issued = it;
        for (int s = 0; s < kStages; ++s) {
          if ((uint32_t)s >= issued) break;
          const uint32_t last = ((issued - 1 - s) / kStages) * kStages + s;
          volatile int never = 0;
          mbar_wait(full_bar(s), (last / kStages) & 1u, &never, nullptr, 0, 20000000ull);
        }
      }
    }
  } else if (warp == 1) {
    // --------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc_bf16(BM, BN, false, !B_NK);
      uint32_t it = 0;
      int local = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < p.num_tiles && ok; tile += gridDim.x, ++local) {
        const int acc = local & 1;
        const uint32_t acc_ph = (local >> 1) & 1u;
        if (!mbar_wait(acc_empty_bar(acc), acc_ph ^ 1u, abort_flag, p.status, kTimeoutMmaAcc)) { ok = false; break; }
        tcgen05_fence_after_sync();
        const uint32_t d_tmem = tmem_base + acc * BN;
        for (int kb = 0; kb < num_kb; ++kb, ++it) {
          const int s = it % kStages;
          const uint32_t ph = (it / kStages) & 1u;
          if (!mbar_wait(full_bar(s), ph, abort_flag, p.status, kTimeoutMmaFull)) { ok = false; break; }
          tcgen05_fence_after_sync();
          const uint32_t sa = smem_base + s * C::kStage, sb = sa + C::kStageA;
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            const uint64_t a_desc = make_smem_desc(sa + k * (UMMA_K * 2), 0, 1024);
            const uint64_t b_desc = B_NK ? make_smem_desc(sb + k * (UMMA_K * 2), 0, 1024)
                                         : make_smem_desc(sb + k * (UMMA_K * 128), 64 * BK * 2, 1024);
            mma_bf16_ss(d_tmem, a_desc, b_desc, idesc, (kb | k) != 0 ? 1u : 0u);
          }
          mma_commit(empty_bar(s));
        }
        if (ok) mma_commit(acc_full_bar(acc));
      }
      if (!ok) {
        // Let every MMA already issued finish before tensor memory is freed.
        mma_commit(drain_bar);
        volatile int never = 0;
        mbar_wait(drain_bar, 0, &never, nullptr, 0, 20000000ull);
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    // The accumulator is drained 32 columns at a time; one TMA store carries 128
    // bytes of each of the warp's 32 rows: a chunk of 64 bf16 columns (two
    // steps) or 32 fp32 columns (one step).  The two warps of a lane group take
    // alternate chunks.
    constexpr int STEPS = C_F32 ? 1 : 2;
    constexpr int CW = 32 * STEPS;       // chunk width in columns
    constexpr int NCHUNK = BN / CW;
    const int quarter = warp & 3;         // TMEM lanes 32*quarter .. 32*quarter+31 belong to this warp
    const int group = (warp - 2) >> 2;    // 0: even chunks, 1: odd chunks
    const int row_in_tile = quarter * 32 + lane;
    const uint32_t buf = epi_base + (uint32_t)(warp - 2) * 4096u;
    const uint32_t row_addr = buf + (uint32_t)lane * 128u;
    const uint32_t sw = (uint32_t)(lane & 7);  // 128-byte swizzle: 16-byte unit index ^= row % 8
    const int my_steps = ((NCHUNK - group + 1) / 2) * STEPS;
    auto col_of = [&](int i) { return ((i / STEPS) * 2 + group) * CW + (i % STEPS) * 32; };
    int local = 0;
    bool ok = true;
    if (lane == 0) prefetch_tensormap(&tmap_c);
    for (int tile = blockIdx.x; tile < p.num_tiles && ok; tile += gridDim.x, ++local) {
      const int nt = tile % p.tiles_n;
      const int mt = (tile / p.tiles_n) % p.tiles_m;
      const int b = tile / (p.tiles_n * p.tiles_m);
      const int bi = b % p.batch_inner, bo = b / p.batch_inner;
      const int acc = local & 1;
      const uint32_t acc_ph = (local >> 1) & 1u;
      const int m = mt * BM + row_in_tile;
      const bool row_ok = m < p.M;
      const int n_tile = nt * BN;
      ResidualRegs cur, nxt;
      if (my_steps > 0 && n_tile + col_of(0) < p.N)
        cur.load(p, m, n_tile + col_of(0), row_ok);  // independent of the accumulator: issued before the wait
      if (!mbar_wait(acc_full_bar(acc), acc_ph, abort_flag, p.status, kTimeoutEpilogue)) { ok = false; break; }
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
        float v[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]) * p.alpha;
        if (p.bias != nullptr) {
          if (n0 + 32 <= p.N) {
#pragma unroll
            for (int j = 0; j < 32; j += 4) {
              const float4 bv = __ldg(reinterpret_cast<const float4*>(p.bias + n0 + j));
              v[j] += bv.x; v[j + 1] += bv.y; v[j + 2] += bv.z; v[j + 3] += bv.w;
            }
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j)
              if (n0 + j < p.N) v[j] += __ldg(p.bias + n0 + j);
          }
        }
        if (p.gelu) {
#pragma unroll
          for (int j = 0; j < 32; ++j) v[j] = gelu_erf(v[j]);
        }
        if (p.residual != nullptr) {
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const uint32_t w[4] = {cur.q[j].x, cur.q[j].y, cur.q[j].z, cur.q[j].w};
#pragma unroll
            for (int t = 0; t < 4; ++t) {
              v[8 * j + 2 * t] += __uint_as_float(w[t] << 16);
              v[8 * j + 2 * t + 1] += __uint_as_float(w[t] & 0xffff0000u);
            }
          }
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
            tma_store_4d(&tmap_c, buf, n0 - step * 32, mt * BM + quarter * 32, bi, bo);
            tma_store_commit();
          }
        }
        cur = nxt;
      }
      tcgen05_fence_before_sync();
      mbar_arrive(acc_empty_bar(acc));
    }
    // Shared memory must outlive every store that still reads it.
    if (lane == 0) tma_store_wait_all<0>();
    __syncwarp();
  }

  // ------------------------------------------------------------------- teardown
  __syncwarp();
  tcgen05_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tcgen05_fence_after_sync();
    tmem_dealloc(tmem_base, C::kTmemCols);
  }
}

// ---- host side -----------------------------------------------------------------
using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
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
// contiguous, 128-byte swizzle, zero fill outside the extents.  Strides in elements.
bool make_map(CUtensorMap* map, bool f32, const void* base, int64_t cols, int64_t rows, int64_t ld, int64_t n_inner,
              int64_t stride_inner, int64_t n_outer, int64_t stride_outer, int box_cols, int box_rows) {
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
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int BN, bool B_NK, bool C_F32>
pd_status launch_variant(const GemmProblem& g, cudaStream_t s) {
  using C = Cfg<BN>;
  CUtensorMap ta, tb, tc;
  if (!make_map(&ta, false, g.A, g.K, g.M, g.lda, g.batch_inner, g.strideA_inner, g.batch_outer, g.strideA_outer, BK, BM))
    return PD_ERR_UNSUPPORTED;
  const bool okb = B_NK ? make_map(&tb, false, g.B, g.K, g.N, g.ldb, g.batch_inner, g.strideB_inner, g.batch_outer,
                                   g.strideB_outer, BK, BN)
                        : make_map(&tb, false, g.B, g.N, g.K, g.ldb, g.batch_inner, g.strideB_inner, g.batch_outer,
                                   g.strideB_outer, 64, BK);
  if (!okb) return PD_ERR_UNSUPPORTED;
  // C is written in boxes of 32 rows x 128 bytes (one epilogue warp, one chunk).
  if (!make_map(&tc, C_F32, g.C, g.N, g.M, g.ldc, g.batch_inner, g.strideC_inner, g.batch_outer, g.strideC_outer,
                C_F32 ? 32 : 64, 32))
    return PD_ERR_UNSUPPORTED;

  KernelParams p{};
  p.C = g.C; p.bias = g.bias; p.residual = g.residual; p.status = device_status_ptr();
  if (!p.status) return PD_ERR_CUDA;
  p.ldc = g.ldc; p.strideC_inner = g.strideC_inner; p.strideC_outer = g.strideC_outer; p.ldr = g.ldr;
  p.M = (int)g.M; p.N = (int)g.N; p.K = (int)g.K;
  p.tiles_m = (int)((g.M + BM - 1) / BM);
  p.tiles_n = (int)((g.N + BN - 1) / BN);
  p.batch_inner = (int)g.batch_inner;
  const int64_t tiles = (int64_t)p.tiles_m * p.tiles_n * g.batch_inner * g.batch_outer;
  if (tiles > 0x7fffffff) return PD_ERR_BAD_SHAPE;
  p.num_tiles = (int)tiles;
  p.alpha = g.alpha; p.c_is_f32 = g.c_dtype == PD_F32; p.gelu = g.gelu;

  auto kernel = gemm_bf16_tcgen05_kernel<BN, B_NK, C_F32>;
  static bool attr_set = false;  // per template instantiation
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes);
    if (e != cudaSuccess) return record_cuda_error(e);
    attr_set = true;
  }
  const int grid = p.num_tiles < sm_count() ? p.num_tiles : sm_count();
  kernel<<<grid, kThreads, C::kSmemBytes, s>>>(ta, tb, tc, p);
  return check_launch();
}

template <int BN>
pd_status launch_bn(const GemmProblem& g, cudaStream_t s) {
  if (g.b_is_nk)
    return g.c_dtype == PD_F32 ? launch_variant<BN, true, true>(g, s) : launch_variant<BN, true, false>(g, s);
  return g.c_dtype == PD_F32 ? launch_variant<BN, false, true>(g, s) : launch_variant<BN, false, false>(g, s);
}

}  // namespace

pd_status launch_gemm(const GemmProblem& g, cudaStream_t s) {
  // 128 x 256 tiles reuse operands best (the 128 x 128 main loop runs at about
  // two thirds of their rate); narrower tiles are used when N is small or when
  // they fill the last wave of SMs so much better that it pays.
  const int sms = sm_count();
  auto cost = [&](int bn, double rate) {
    const int64_t tiles = ((g.M + BM - 1) / BM) * ((g.N + bn - 1) / bn) * g.batch_inner * g.batch_outer;
    const int64_t waves = (tiles + sms - 1) / sms;
    return (double)waves * bn / rate;  // time ~ waves x tile width / main-loop rate
  };
  int bn = 256;
  if (g.N <= 64) bn = 64;
  else if (g.N <= 128) bn = 128;
  else if (cost(128, 0.66) < cost(256, 1.0)) bn = 128;
  if (bn == 256) return launch_bn<256>(g, s);
  if (bn == 128) return launch_bn<128>(g, s);
  return launch_bn<64>(g, s);
}

}  // namespace pd

extern "C" pd_status pd_gemm_bf16(const void* A, const void* B, void* C, int64_t M, int64_t N, int64_t K,
                                  int64_t lda, int64_t ldb, int64_t ldc, int b_is_nk, pd_dtype c_dtype,
                                  int64_t batch, int64_t strideA, int64_t strideB, int64_t strideC,
                                  cudaStream_t stream) {
  if (!A || !B || !C) return PD_ERR_NULL_POINTER;
  if (M < 0 || N < 0 || K <= 0 || batch < 0) return PD_ERR_BAD_SHAPE;
  if (c_dtype != PD_BF16 && c_dtype != PD_F32) return PD_ERR_BAD_SHAPE;
  if (M > 0x7fffffff || N > 0x7fffffff || K > 0x7fffffff || batch > 0x7fffffff) return PD_ERR_BAD_SHAPE;
  const int64_t b_cols = b_is_nk ? K : N;
  if (lda < K || ldb < b_cols || ldc < N) return PD_ERR_BAD_SHAPE;
  const int64_t c_elems_per_16B = c_dtype == PD_F32 ? 4 : 8;
  if (!pd::aligned16(A) || !pd::aligned16(B) || !pd::aligned16(C) || lda % 8 || ldb % 8 || ldc % c_elems_per_16B)
    return PD_ERR_ALIGNMENT;
  if (batch > 1) {
    if (strideA < 0 || strideB < 0 || strideC < 0) return PD_ERR_BAD_SHAPE;
    if (strideA % 8 || strideB % 8 || strideC % c_elems_per_16B) return PD_ERR_ALIGNMENT;
    if (strideA == 0 || strideB == 0) return PD_ERR_UNSUPPORTED;  // broadcast operands: not supported
  }
  if (M == 0 || N == 0 || batch == 0) return PD_OK;
  pd_status st = pd::require_sm100();
  if (st != PD_OK) return st;
  pd::GemmProblem g;
  g.A = A; g.B = B; g.C = C; g.M = M; g.N = N; g.K = K; g.lda = lda; g.ldb = ldb; g.ldc = ldc;
  g.b_is_nk = b_is_nk != 0; g.c_dtype = c_dtype;
  g.batch_inner = batch; g.batch_outer = 1;
  g.strideA_inner = strideA; g.strideB_inner = strideB; g.strideC_inner = strideC;
  return pd::launch_gemm(g, stream);
}
