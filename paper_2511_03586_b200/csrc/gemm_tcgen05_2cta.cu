// bf16 GEMM with 256 x 256 output tiles computed by a pair of CTAs (a cluster of
// two SMs) with one tcgen05.mma.cta_group::2 per k-step.
//
// Why: with one CTA per 128 x 256 tile every MMA reads 12 KiB of operands from
// shared memory while TMA writes as much, which saturates the shared-memory
// port before the tensor pipe.  In a pair each CTA holds its own 128 rows of A
// but only HALF of the B tile (128 of the 256 columns); the MMA reads both
// halves, so per CTA the shared-memory traffic per k-step drops by a third and
// six 32 KiB stages fit instead of four 48 KiB ones.
//
// Roles per CTA (320 threads, same as the single-CTA kernel):
//   warp 0           : TMA producer (one elected lane issues) for this CTA's A rows and B half.  All byte
//                      counts are signalled on the EVEN CTA's "full" barrier,
//                      which the even CTA arms for both (no load is multicast).
//   warp 1           : in the even CTA only, the MMA issuer: the warp walks the
//                      loop, one elected lane issues (M = 256, N = 256,
//                      K = 16 per instruction; accumulator rows 0-127 in its own
//                      tensor memory, rows 128-255 in the partner's).  Its
//                      commits arrive on the "empty" / "accumulator full"
//                      barriers of both CTAs.
//   warps 2-9        : epilogue over the CTA's own 128 x 256 half of the tile
//                      (shared with the single-CTA kernel); the partner's
//                      epilogue threads release the accumulator by arriving on
//                      the even CTA's barrier through the cluster address space.
// Every wait is bounded as in the single-CTA kernel.
#include "gemm_common.cuh"

namespace pd {
namespace {

using namespace sm100;
using namespace gemm;

constexpr int kPairN = 256;                 // tile columns per pair
constexpr int kHalfN = kPairN / 2;          // B columns held by each CTA
constexpr int kStageA = BM * BK * 2;        // 16 KiB
constexpr int kStageB = kHalfN * BK * 2;    // 16 KiB
constexpr int kStage = kStageA + kStageB;
constexpr int kBarrierBytes = 1024;
constexpr int kStages = (kSmemLimit - 1024 - kBarrierBytes - kEpilogueBytes) / kStage;  // 6
constexpr int kSmemBytes = kStages * kStage + kEpilogueBytes + kBarrierBytes + 1024;
constexpr int kTmemCols = 2 * kPairN;       // two accumulators of 256 columns
static_assert(kStages >= 4, "pipeline too shallow");

template <bool B_NK, bool C_F32>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
gemm_bf16_tcgen05_pair_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                              const __grid_constant__ CUtensorMap tmap_c, const KernelParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;  // identical offset in both CTAs
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t epi_base = smem_base + kStages * kStage;
  const uint32_t bar_base = epi_base + kEpilogueBytes;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (kStages + s); };
  auto acc_full_bar = [&](int a) { return bar_base + 8u * (2 * kStages + a); };
  auto acc_empty_bar = [&](int a) { return bar_base + 8u * (2 * kStages + 2 + a); };
  const uint32_t drain_bar = bar_base + 8u * (2 * kStages + 4);
  uint8_t* ctrl = smem_gen + kStages * kStage + kEpilogueBytes + 8 * (2 * kStages + 5);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(ctrl);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(ctrl + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();  // 0: even CTA (issues the MMAs), 1: its partner
  const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
  const int num_kb = (p.K + BK - 1) / BK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(full_bar(s), 1);   // used in the even CTA only
      mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(acc_full_bar(a), 1);
      mbar_init(acc_empty_bar(a), 2 * kEpilogueThreads / 32);  // both CTAs' epilogue warps; used in the even CTA only
    }
    mbar_init(drain_bar, 1);
    *abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async_smem();
  }
  if (warp == 1) {
    tmem_alloc_pair(smem_u32(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
    tmem_relinquish_alloc_permit_pair();
  }
  tcgen05_fence_before_sync();
  cluster_sync_all();  // barriers of both CTAs are initialised before anyone signals them
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
      }
      uint32_t it = 0;
      bool ok = true;
      // (test switch: with withhold_loads set the producer issues nothing, and the wait for the first stage runs out)
      for (int tile = pair; tile < p.num_tiles && ok && !p.withhold_loads; tile += num_pairs) {
        const int nt = tile % p.tiles_n;
        const int mt = (tile / p.tiles_n) % p.tiles_m;
        const int b = tile / (p.tiles_n * p.tiles_m);
        const int bi = b % p.batch_inner, bo = b / p.batch_inner;
        const int m0 = mt * (2 * BM) + (int)rank * BM;
        const int n0 = nt * kPairN + (int)rank * kHalfN;
        for (int kb = 0; kb < num_kb; ++kb, ++it) {
          const int s = it % kStages;
          const uint32_t ph = (it / kStages) & 1u;
          if (!mbar_wait_warp(empty_bar(s), ph ^ 1u, abort_flag, p.status, kTimeoutProducer, wait_limit(p))) { ok = false; break; }
          const uint32_t sa = smem_base + s * kStage, sb = sa + kStageA;
          const uint32_t full0 = map_to_cta(full_bar(s), 0);
          if (elect_one()) {
            if (rank == 0) mbar_arrive_expect_tx(full_bar(s), 2 * kStage);  // bytes of both CTAs
            tma_load_4d_pair(sa, &tmap_a, full0, kb * BK, m0, bi, bo);
            if (B_NK) {
              tma_load_4d_pair(sb, &tmap_b, full0, kb * BK, n0, bi, bo);
            } else {
#pragma unroll
              for (int j = 0; j < kHalfN / 64; ++j)
                tma_load_4d_pair(sb + j * (64 * BK * 2), &tmap_b, full0, n0 + j * 64, kb * BK, bi, bo);
            }
          }
          __syncwarp();
        }
      }
      if (!ok) {
        // Leave no copy in flight: the loads signal the even CTA's barrier, so just
        // give them time to land before this CTA's shared memory can go away.
        const uint64_t t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 1000000ull) {
        }
      }
    }
  } else if (warp == 1) {
    // --------------------------------------------------------------- MMA issuer
    if (rank == 0) {
      // The whole warp walks the loop and waits; one elected lane issues.
      constexpr uint32_t idesc = make_idesc_bf16(2 * BM, kPairN, false, !B_NK);
      uint32_t it = 0;
      int local = 0;
      bool ok = true;
      for (int tile = pair; tile < p.num_tiles && ok; tile += num_pairs, ++local) {
        const int acc = local & 1;
        const uint32_t acc_ph = (local >> 1) & 1u;
        if (!mbar_wait_warp(acc_empty_bar(acc), acc_ph ^ 1u, abort_flag, p.status, kTimeoutMmaAcc, wait_limit(p))) { ok = false; break; }
        tcgen05_fence_after_sync();
        const uint32_t d_tmem = tmem_base + acc * kPairN;
        for (int kb = 0; kb < num_kb; ++kb, ++it) {
          const int s = it % kStages;
          const uint32_t ph = (it / kStages) & 1u;
          if (!mbar_wait_warp(full_bar(s), ph, abort_flag, p.status, kTimeoutMmaFull, wait_limit(p))) { ok = false; break; }
          tcgen05_fence_after_sync();
          const uint32_t sa = smem_base + s * kStage, sb = sa + kStageA;
          if (elect_one()) {
#pragma unroll
            for (int k = 0; k < BK / UMMA_K; ++k) {
              const uint64_t a_desc = make_smem_desc(sa + k * (UMMA_K * 2), 0, 1024);
              const uint64_t b_desc = B_NK ? make_smem_desc(sb + k * (UMMA_K * 2), 0, 1024)
                                           : make_smem_desc(sb + k * (UMMA_K * 128), 64 * BK * 2, 1024);
              mma_bf16_ss_pair(d_tmem, a_desc, b_desc, idesc, (kb | k) != 0 ? 1u : 0u);
            }
            mma_commit_pair(empty_bar(s), 0x3);  // the stage is free in both CTAs
          }
          __syncwarp();
        }
        if (ok && elect_one()) mma_commit_pair(acc_full_bar(acc), 0x3);
        __syncwarp();
      }
      if (!ok) {
        // Let every MMA already issued finish before tensor memory is freed.
        if (lane == 0) mma_commit_pair(drain_bar, 0x1);
        __syncwarp();
        volatile int never = 0;
        mbar_wait(drain_bar, 0, &never, nullptr, 0, 20000000ull);
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    const uint32_t rel0 = map_to_cta(acc_empty_bar(0), 0), rel1 = map_to_cta(acc_empty_bar(1), 0);
    epilogue_warp<kPairN, C_F32>(
        p, &tmap_c, tmem_base, epi_base, acc_full_bar(0), abort_flag, pair, num_pairs,
        [&](int mt) { return mt * (2 * BM) + (int)rank * BM; },
        // The warp's tensor-memory loads have completed (tcgen05.wait::ld) and are ordered before this signal by
        // the tcgen05 fence; the signal publishes no memory of its own, so it carries no release ordering: a
        // cluster-scope release here waited some 2400 clk per tile for the warp's bulk stores to drain.
        [&](int acc) { mbar_arrive_cluster_relaxed(acc ? rel1 : rel0); });
  }

  // ------------------------------------------------------------------- teardown
  // Neither CTA may leave while its partner can still signal its barriers, read
  // its shared memory through the MMA, or write its tensor memory.
  __syncwarp();
  tcgen05_fence_before_sync();
  cluster_sync_all();
  if (warp == 1) {
    tcgen05_fence_after_sync();
    tmem_dealloc_pair(tmem_base, kTmemCols);
  }
}

template <bool B_NK, bool C_F32>
pd_status launch_pair_variant(const GemmProblem& g, cudaStream_t s) {
  CUtensorMap ta, tb, tc;
  if (!make_map(&ta, false, g.A, g.K, g.M, g.lda, g.batch_inner, g.strideA_inner, g.batch_outer, g.strideA_outer, BK, BM))
    return PD_ERR_UNSUPPORTED;
  const bool okb = B_NK ? make_map(&tb, false, g.B, g.K, g.N, g.ldb, g.batch_inner, g.strideB_inner, g.batch_outer,
                                   g.strideB_outer, BK, kHalfN)
                        : make_map(&tb, false, g.B, g.N, g.K, g.ldb, g.batch_inner, g.strideB_inner, g.batch_outer,
                                   g.strideB_outer, 64, BK);
  if (!okb) return PD_ERR_UNSUPPORTED;
  if (!make_map(&tc, C_F32, g.C, g.N, g.M, g.ldc, g.batch_inner, g.strideC_inner, g.batch_outer, g.strideC_outer,
                C_F32 ? 32 : 64, 32))
    return PD_ERR_UNSUPPORTED;

  KernelParams p{};
  p.C = g.C; p.bias = g.bias; p.residual = g.residual; p.status = device_status_ptr();
  if (!p.status) return PD_ERR_CUDA;
  p.ldc = g.ldc; p.strideC_inner = g.strideC_inner; p.strideC_outer = g.strideC_outer; p.ldr = g.ldr;
  p.M = (int)g.M; p.N = (int)g.N; p.K = (int)g.K;
  p.tiles_m = (int)((g.M + 2 * BM - 1) / (2 * BM));
  p.tiles_n = (int)((g.N + kPairN - 1) / kPairN);
  p.batch_inner = (int)g.batch_inner;
  const int64_t tiles = (int64_t)p.tiles_m * p.tiles_n * g.batch_inner * g.batch_outer;
  if (tiles > 0x7fffffff) return PD_ERR_BAD_SHAPE;
  p.num_tiles = (int)tiles;
  p.alpha = g.alpha; p.c_is_f32 = C_F32; p.act = g.act;
  p.wait_limit_ns = debug_wait_limit_ns();
  p.withhold_loads = debug_withhold_loads();

  auto kernel = gemm_bf16_tcgen05_pair_kernel<B_NK, C_F32>;
  static PerDeviceFlag smem_allowed;  // one per kernel (template instantiation)
  if (pd_status st = allow_dynamic_smem(kernel, kSmemBytes, smem_allowed); st != PD_OK) return st;
  const int pairs = (int)(tiles < sm_count() / 2 ? tiles : sm_count() / 2);
  launch_pdl(kernel, dim3(2 * pairs), dim3(kThreads), kSmemBytes, s, ta, tb, tc, p);
  return check_launch();
}

}  // namespace

bool gemm_pair_tiles_profitable(const GemmProblem& g) {
  // 256 x 256 pair tiles pay off when there are enough of them to fill the SM
  // pairs and enough k-blocks to amortise the deeper pipeline.
  const int64_t tiles = ((g.M + 255) / 256) * ((g.N + 255) / 256) * g.batch_inner * g.batch_outer;
  return g.M >= 256 && g.N >= 256 && g.K >= 256 && tiles >= sm_count() / 2;
}

pd_status launch_gemm_pair(const GemmProblem& g, cudaStream_t s) {
  if (g.b_is_nk)
    return g.c_dtype == PD_F32 ? launch_pair_variant<true, true>(g, s) : launch_pair_variant<true, false>(g, s);
  return g.c_dtype == PD_F32 ? launch_pair_variant<false, true>(g, s) : launch_pair_variant<false, false>(g, s);
}

}  // namespace pd
