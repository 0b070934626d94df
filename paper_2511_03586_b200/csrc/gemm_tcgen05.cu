// bf16 x bf16 -> fp32 contraction on the tcgen05 tensor cores with a fused epilogue.
//
//   C[m,n] = act(alpha * sum_k A[m,k] B[k,n] + bias[n]) + residual[m,n]
//
// Persistent, warp-specialised kernel, one CTA of 320 threads per SM:
//   warp 0           : TMA producer (the warp walks the loop, one elected lane issues).  Streams 128 x 64 tiles of A and BN x 64
//                      tiles of B (128-byte swizzle) into a ring of shared-memory
//                      stages; a "full" mbarrier per stage counts the bytes.
//   warp 1           : MMA issuer (likewise).  Four tcgen05.mma (128 x BN x 16) per stage
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
#include "gemm_common.cuh"

namespace pd {
namespace {

using namespace sm100;
using namespace gemm;

template <int BN>
struct Cfg {
  static constexpr int kStageA = BM * BK * 2;
  static constexpr int kStageB = BN * BK * 2;
  static constexpr int kStage = kStageA + kStageB;
  static constexpr int kBarrierBytes = 1024;
  static constexpr int kStagesMax = (kSmemLimit - 1024 /*alignment slack*/ - kBarrierBytes - kEpilogueBytes) / kStage;
  static constexpr int kStages = kStagesMax > 8 ? 8 : kStagesMax;
  static constexpr int kSmemBytes = kStages * kStage + kEpilogueBytes + kBarrierBytes + 1024;
  static constexpr int kTmemCols = 2 * BN;  // two accumulators; 128, 256 or 512: a power of two
};

// GATED: the tile's B operand is BN/2 columns of the first weight followed by the same BN/2 columns of a
// second one (tmap_b2), and the epilogue writes SiLU(first product) * second product, BN/2 columns wide.
template <int BN, bool B_NK, bool C_F32, bool GATED>
__global__ void __launch_bounds__(kThreads, 1)
gemm_bf16_tcgen05_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                         const __grid_constant__ CUtensorMap tmap_b2, const __grid_constant__ CUtensorMap tmap_c,
                         const KernelParams p) {
  static_assert(!GATED || (!B_NK && !C_F32 && BN >= 128), "gated form: B as [K, N], bf16 out, 64-column boxes");
  using C = Cfg<BN>;
  constexpr int kStages = C::kStages;
  extern __shared__ uint8_t smem_raw[];
  // 128-byte swizzled tiles must start on a 1024-byte boundary.
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t epi_base = smem_base + kStages * C::kStage;  // 1024-byte aligned: kStage is a multiple of 1024
  const uint32_t bar_base = epi_base + kEpilogueBytes;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (kStages + s); };
  auto acc_full_bar = [&](int a) { return bar_base + 8u * (2 * kStages + a); };
  auto acc_empty_bar = [&](int a) { return bar_base + 8u * (2 * kStages + 2 + a); };
  const uint32_t drain_bar = bar_base + 8u * (2 * kStages + 4);
  uint8_t* ctrl = smem_gen + kStages * C::kStage + kEpilogueBytes + 8 * (2 * kStages + 5);
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
      mbar_init(acc_empty_bar(a), kEpilogueThreads / 32);  // one arrival per epilogue warp
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
  // everything above is independent of other kernels' data; from here on global memory is touched
  griddep_wait();
  griddep_launch_dependents();

  if (warp == 0) {
    // ------------------------------------------------------------- TMA producer
    {
      // The whole warp walks the loop and waits; one elected lane issues the copies.
      if (lane == 0) {
        prefetch_tensormap(&tmap_a);
        prefetch_tensormap(&tmap_b);
        if (GATED) prefetch_tensormap(&tmap_b2);
      }
      uint32_t it = 0;  // k-blocks issued so far, over all tiles
      bool ok = true;
      // (test switch: with withhold_loads set the producer issues nothing, and the wait for the first stage runs out)
      for (int tile = blockIdx.x; tile < p.num_tiles && ok && !p.withhold_loads; tile += gridDim.x) {
        const int nt = tile % p.tiles_n;
        const int mt = (tile / p.tiles_n) % p.tiles_m;
        const int b = tile / (p.tiles_n * p.tiles_m);
        const int bi = b % p.batch_inner, bo = b / p.batch_inner;
        for (int kb = 0; kb < num_kb; ++kb, ++it) {
          const int s = it % kStages;
          const uint32_t ph = (it / kStages) & 1u;
          if (!mbar_wait_warp(empty_bar(s), ph ^ 1u, abort_flag, p.status, kTimeoutProducer, wait_limit(p))) { ok = false; break; }
          const uint32_t sa = smem_base + s * C::kStage, sb = sa + C::kStageA;
          if (elect_one()) {
            mbar_arrive_expect_tx(full_bar(s), C::kStage);
            tma_load_4d(sa, &tmap_a, full_bar(s), kb * BK, mt * BM, bi, bo);
            if constexpr (GATED) {
#pragma unroll
              for (int j = 0; j < BN / 64; ++j)
                tma_load_4d(sb + j * (64 * BK * 2), j < BN / 128 ? &tmap_b : &tmap_b2, full_bar(s),
                            nt * (BN / 2) + (j % (BN / 128)) * 64, kb * BK, 0, 0);
            } else if (B_NK) {
              tma_load_4d(sb, &tmap_b, full_bar(s), kb * BK, nt * BN, bi, bo);
            } else {
#pragma unroll
              for (int j = 0; j < BN / 64; ++j)
                tma_load_4d(sb + j * (64 * BK * 2), &tmap_b, full_bar(s), nt * BN + j * 64, kb * BK, bi, bo);
            }
          }
          __syncwarp();
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
    {
      // The whole warp walks the loop and waits; one elected lane issues.
      constexpr uint32_t idesc = make_idesc_bf16(BM, BN, false, !B_NK);
      uint32_t it = 0;
      int local = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < p.num_tiles && ok; tile += gridDim.x, ++local) {
        const int acc = local & 1;
        const uint32_t acc_ph = (local >> 1) & 1u;
        if (!mbar_wait_warp(acc_empty_bar(acc), acc_ph ^ 1u, abort_flag, p.status, kTimeoutMmaAcc, wait_limit(p))) { ok = false; break; }
        tcgen05_fence_after_sync();
        const uint32_t d_tmem = tmem_base + acc * BN;
        for (int kb = 0; kb < num_kb; ++kb, ++it) {
          const int s = it % kStages;
          const uint32_t ph = (it / kStages) & 1u;
          if (!mbar_wait_warp(full_bar(s), ph, abort_flag, p.status, kTimeoutMmaFull, wait_limit(p))) { ok = false; break; }
          tcgen05_fence_after_sync();
          const uint32_t sa = smem_base + s * C::kStage, sb = sa + C::kStageA;
          if (elect_one()) {
#pragma unroll
            for (int k = 0; k < BK / UMMA_K; ++k) {
              const uint64_t a_desc = make_smem_desc(sa + k * (UMMA_K * 2), 0, 1024);
              const uint64_t b_desc = B_NK ? make_smem_desc(sb + k * (UMMA_K * 2), 0, 1024)
                                           : make_smem_desc(sb + k * (UMMA_K * 128), 64 * BK * 2, 1024);
              mma_bf16_ss(d_tmem, a_desc, b_desc, idesc, (kb | k) != 0 ? 1u : 0u);
            }
            mma_commit(empty_bar(s));
          }
          __syncwarp();
        }
        if (ok && elect_one()) mma_commit(acc_full_bar(acc));
        __syncwarp();
      }
      if (!ok) {
        // Let every MMA already issued finish before tensor memory is freed.
        if (lane == 0) mma_commit(drain_bar);
        __syncwarp();
        volatile int never = 0;
        mbar_wait(drain_bar, 0, &never, nullptr, 0, 20000000ull);
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    if constexpr (GATED)
      epilogue_warp_gated<BN>(p, &tmap_c, tmem_base, epi_base, acc_full_bar(0), abort_flag, blockIdx.x, gridDim.x,
                              [&](int acc) { mbar_arrive(acc_empty_bar(acc)); });
    else
      epilogue_warp<BN, C_F32>(
          p, &tmap_c, tmem_base, epi_base, acc_full_bar(0), abort_flag, blockIdx.x, gridDim.x,
          [](int mt) { return mt * BM; }, [&](int acc) { mbar_arrive(acc_empty_bar(acc)); });
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

template <int BN, bool B_NK, bool C_F32, bool GATED = false>
pd_status launch_variant(const GemmProblem& g, cudaStream_t s) {
  using C = Cfg<BN>;
  constexpr int OC = GATED ? BN / 2 : BN;  // output columns per tile
  CUtensorMap ta, tb, tb2, tc;
  if (!make_map(&ta, false, g.A, g.K, g.M, g.lda, g.batch_inner, g.strideA_inner, g.batch_outer, g.strideA_outer, BK, BM))
    return PD_ERR_UNSUPPORTED;
  const bool okb = B_NK ? make_map(&tb, false, g.B, g.K, g.N, g.ldb, g.batch_inner, g.strideB_inner, g.batch_outer,
                                   g.strideB_outer, BK, BN)
                        : make_map(&tb, false, g.B, g.N, g.K, g.ldb, g.batch_inner, g.strideB_inner, g.batch_outer,
                                   g.strideB_outer, 64, BK);
  if (!okb) return PD_ERR_UNSUPPORTED;
  tb2 = tb;
  if (GATED && !make_map(&tb2, false, g.B2, g.N, g.K, g.ldb, 1, 0, 1, 0, 64, BK)) return PD_ERR_UNSUPPORTED;
  // C is written in boxes of 32 rows x 128 bytes (one epilogue warp, one chunk); the gated epilogue writes
  // boxes of 32 rows x 64 bytes.
  const bool okc = GATED ? make_map(&tc, false, g.C, g.N, g.M, g.ldc, 1, 0, 1, 0, 32, 32, CU_TENSOR_MAP_SWIZZLE_64B)
                         : make_map(&tc, C_F32, g.C, g.N, g.M, g.ldc, g.batch_inner, g.strideC_inner, g.batch_outer,
                                    g.strideC_outer, C_F32 ? 32 : 64, 32);
  if (!okc) return PD_ERR_UNSUPPORTED;

  KernelParams p{};
  p.C = g.C; p.bias = g.bias; p.residual = g.residual; p.status = device_status_ptr();
  if (!p.status) return PD_ERR_CUDA;
  p.ldc = g.ldc; p.strideC_inner = g.strideC_inner; p.strideC_outer = g.strideC_outer; p.ldr = g.ldr;
  p.M = (int)g.M; p.N = (int)g.N; p.K = (int)g.K;
  p.tiles_m = (int)((g.M + BM - 1) / BM);
  p.tiles_n = (int)((g.N + OC - 1) / OC);
  p.batch_inner = (int)g.batch_inner;
  const int64_t tiles = (int64_t)p.tiles_m * p.tiles_n * g.batch_inner * g.batch_outer;
  if (tiles > 0x7fffffff) return PD_ERR_BAD_SHAPE;
  p.num_tiles = (int)tiles;
  p.alpha = g.alpha; p.c_is_f32 = g.c_dtype == PD_F32; p.act = g.act;
  p.wait_limit_ns = debug_wait_limit_ns();
  p.withhold_loads = debug_withhold_loads();

  auto kernel = gemm_bf16_tcgen05_kernel<BN, B_NK, C_F32, GATED>;
  static PerDeviceFlag smem_allowed;  // one per kernel (template instantiation)
  if (pd_status st = allow_dynamic_smem(kernel, C::kSmemBytes, smem_allowed); st != PD_OK) return st;
  const int grid = p.num_tiles < sm_count() ? p.num_tiles : sm_count();
  launch_pdl(kernel, dim3(grid), dim3(kThreads), C::kSmemBytes, s, ta, tb, tb2, tc, p);
  return check_launch();
}

template <int BN>
pd_status launch_bn(const GemmProblem& g, cudaStream_t s) {
  if (g.b_is_nk)
    return g.c_dtype == PD_F32 ? launch_variant<BN, true, true>(g, s) : launch_variant<BN, true, false>(g, s);
  return g.c_dtype == PD_F32 ? launch_variant<BN, false, true>(g, s) : launch_variant<BN, false, false>(g, s);
}

}  // namespace

namespace {
int g_tile_mode = 0;  // 0: automatic, 1: single-CTA tiles only, 2: CTA-pair tiles whenever the shape allows
}
void set_gemm_tile_mode(int mode) { g_tile_mode = mode; }
namespace {
int g_split_k_mode = 0;  // 0: split K over a cluster when the problem has few tiles, 1: never
}
void set_gemm_split_k_mode(int mode) { g_split_k_mode = mode; }

pd_status launch_gemm(const GemmProblem& g, cudaStream_t s) {
  if (g_tile_mode == 0 && g_split_k_mode != 1) {
    const int split = gemm_split_k_factor(g);
    if (split > 0 && (g.B2 == nullptr || (!g.bias && !g.residual && !g.act))) {
      logf("gemm %lld x %lld x %lld%s: 128 x 256 tiles, K split over clusters of %d CTAs", (long long)g.M, (long long)g.N,
           (long long)g.K, g.B2 ? " (gated)" : "", split);
      return launch_gemm_split_k(g, split, s);
    }
  }
  if (g.B2 != nullptr) {
    // gated form: 128 x 128 output tiles, or 128 x 64 when those fill the SMs' last wave better
    if (g.b_is_nk || g.c_dtype != PD_BF16 || g.batch_inner != 1 || g.batch_outer != 1 || g.bias || g.residual || g.act)
      return PD_ERR_UNSUPPORTED;
    const int64_t tiles_m = (g.M + BM - 1) / BM, sms = sm_count();
    const int64_t t128 = tiles_m * ((g.N + 127) / 128), t64 = tiles_m * ((g.N + 63) / 64);
    const double c128 = (double)((t128 + sms - 1) / sms) * 256.0, c64 = (double)((t64 + sms - 1) / sms) * 128.0 / 0.66;
    logf("gemm %lld x %lld x %lld (gated): 128 x %d output tiles, one CTA each", (long long)g.M, (long long)g.N,
         (long long)g.K, c64 < c128 ? 64 : 128);
    return c64 < c128 ? launch_variant<128, false, false, true>(g, s) : launch_variant<256, false, false, true>(g, s);
  }
  if (g_tile_mode == 2 || (g_tile_mode == 0 && gemm_pair_tiles_profitable(g))) {
    logf("gemm %lld x %lld x %lld batch %lld: 256 x 256 tiles on CTA pairs", (long long)g.M, (long long)g.N, (long long)g.K,
         (long long)(g.batch_inner * g.batch_outer));
    return launch_gemm_pair(g, s);
  }
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
  logf("gemm %lld x %lld x %lld batch %lld: 128 x %d tiles, one CTA each", (long long)g.M, (long long)g.N, (long long)g.K,
       (long long)(g.batch_inner * g.batch_outer), bn);
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

extern "C" pd_status pd_set_gemm_tile_mode(int mode) {
  if (mode < 0 || mode > 2) return PD_ERR_BAD_SHAPE;
  pd::set_gemm_tile_mode(mode);
  return PD_OK;
}

extern "C" pd_status pd_gemm_bias_act(const void* A, const void* B, const float* bias, const void* residual, void* C,
                                      int64_t M, int64_t N, int64_t K, int act, pd_dtype c_dtype,
                                      cudaStream_t stream) {
  if (!A || !B || !C) return PD_ERR_NULL_POINTER;
  if (M < 0 || N < 0 || K <= 0 || act < 0 || act > 2) return PD_ERR_BAD_SHAPE;
  if (c_dtype != PD_BF16 && c_dtype != PD_F32) return PD_ERR_BAD_SHAPE;
  if (M > 0x7fffffff || N > 0x7fffffff || K > 0x7fffffff) return PD_ERR_BAD_SHAPE;
  if (!pd::aligned16(A) || !pd::aligned16(B) || !pd::aligned16(C) || !pd::aligned16(bias) || !pd::aligned16(residual) ||
      K % 8 || N % 8)
    return PD_ERR_ALIGNMENT;
  if (M == 0 || N == 0) return PD_OK;
  pd_status st = pd::require_sm100();
  if (st != PD_OK) return st;
  pd::GemmProblem g;
  g.A = A; g.B = B; g.C = C; g.M = M; g.N = N; g.K = K; g.lda = K; g.ldb = N; g.ldc = N;
  g.c_dtype = c_dtype; g.bias = bias; g.act = act;
  g.residual = static_cast<const __nv_bfloat16*>(residual); g.ldr = N;
  return pd::launch_gemm(g, stream);
}

extern "C" pd_status pd_swiglu_gemm(const void* X, const void* Wg, const void* Wu, void* Y, int64_t M, int64_t N,
                                    int64_t K, cudaStream_t stream) {
  if (!X || !Wg || !Wu || !Y) return PD_ERR_NULL_POINTER;
  if (M < 0 || N < 0 || K <= 0) return PD_ERR_BAD_SHAPE;
  if (M > 0x7fffffff || N > 0x7fffffff || K > 0x7fffffff) return PD_ERR_BAD_SHAPE;
  if (!pd::aligned16(X) || !pd::aligned16(Wg) || !pd::aligned16(Wu) || !pd::aligned16(Y) || K % 8 || N % 8)
    return PD_ERR_ALIGNMENT;
  if (M == 0 || N == 0) return PD_OK;
  pd_status st = pd::require_sm100();
  if (st != PD_OK) return st;
  pd::GemmProblem g;
  g.A = X; g.B = Wg; g.B2 = Wu; g.C = Y; g.M = M; g.N = N; g.K = K; g.lda = K; g.ldb = N; g.ldc = N;
  return pd::launch_gemm(g, stream);
}

extern "C" pd_status pd_set_gemm_split_k(int mode) {
  if (mode < 0 || mode > 1) return PD_ERR_BAD_SHAPE;
  pd::set_gemm_split_k_mode(mode);
  return PD_OK;
}
