// Contractions with fewer output tiles than SMs: split-K over a thread-block cluster.
//
// A problem such as 256 x 448 x 4096 has a handful of 128 x 256 output tiles; one
// CTA per tile would leave most of the GPU idle and stream its whole K extent
// through a single SM's TMA pipeline, which is bound by latency, not bandwidth.
// Here the S CTAs of a cluster (S = 2, 4 or 8) share one output tile:
//   1. CTA r contracts k-blocks [r nkb / S, (r + 1) nkb / S) into its own
//      tensor-memory accumulator (same TMA producer / MMA issuer roles and
//      shared-memory ring as the persistent kernel);
//   2. cluster barrier: every accumulator is complete and every ring is idle;
//   3. reduce-scatter through distributed shared memory: the accumulator columns
//      are dealt to the S CTAs; every CTA writes its partial sums of the columns
//      it does not own into the owner's (idle) ring, 16 bytes per store;
//   4. cluster barrier (release / acquire): the partial sums have landed;
//   5. every CTA adds the S - 1 received partials to its own, applies the epilogue
//      (scale, bias, activation, residual; or SiLU(gate) * up in the gated form)
//      and stores its columns, 8 consecutive values of a row per thread.
// The sums are formed in a fixed order (own partial, then ranks ascending), so
// results are repeatable; they differ from the unsplit kernel only by fp32
// summation order.  Every mbarrier wait is bounded; the cluster barriers are
// reached by every thread on every path.
#include "gemm_common.cuh"

namespace pd {
namespace {

using namespace sm100;
using namespace gemm;

template <int BN>
struct SplitCfg {
  static constexpr int kStageA = BM * BK * 2;
  static constexpr int kStageB = BN * BK * 2;
  static constexpr int kStage = kStageA + kStageB;
  static constexpr int kStages = (kSmemLimit - 2048) / kStage > 8 ? 8 : (kSmemLimit - 2048) / kStage;
  static constexpr int kRecvBytes = BN * 512;  // S senders x (BN / S columns) x 128 rows x 4 bytes
  static_assert(kRecvBytes <= kStages * kStage, "the reduction buffer lives in the idle ring");
  static constexpr int kSmemBytes = kStages * kStage + 1024 /*barriers*/ + 1024 /*alignment slack*/;
};

struct SplitParams {
  int c_is_f32;
  const __nv_bfloat16* residual;
};

template <int BN, bool B_NK, bool GATED, int S>
__global__ void __launch_bounds__(kThreads, 1)
gemm_bf16_splitk_cluster_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                                const __grid_constant__ CUtensorMap tmap_b2, const KernelParams p, const SplitParams sp) {
  static_assert(!GATED || (!B_NK && BN == 256), "gated form: B as [K, N], 128 output columns per tile");
  using C = SplitCfg<BN>;
  constexpr int kStages = C::kStages;
  constexpr int OC = GATED ? BN / 2 : BN;  // output columns per tile
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t bar_base = smem_base + kStages * C::kStage;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (kStages + s); };
  const uint32_t acc_full_bar = bar_base + 8u * (2 * kStages);
  const uint32_t drain_bar = bar_base + 8u * (2 * kStages + 1);
  uint8_t* ctrl = smem_gen + kStages * C::kStage + 8 * (2 * kStages + 2);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(ctrl);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(ctrl + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = (int)cluster_ctarank();
  const int tile = blockIdx.x / S;
  const int nt = tile % p.tiles_n, mt = tile / p.tiles_n;
  const int num_kb = (p.K + BK - 1) / BK;
  const int kb0 = (int)((int64_t)rank * num_kb / S), kb1 = (int)((int64_t)(rank + 1) * num_kb / S);  // not empty: num_kb >= S

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    mbar_init(acc_full_bar, 1);
    mbar_init(drain_bar, 1);
    *abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async_smem();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), BN);
    tmem_relinquish_alloc_permit();
  }
  tcgen05_fence_before_sync();
  __syncthreads();
  tcgen05_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  griddep_wait();
  griddep_launch_dependents();

  bool acc_ok = true;  // epilogue warps: this CTA's accumulator is complete
  if (warp == 0) {
    // ------------------------------------------------------------- TMA producer
    {
      // The whole warp walks the loop and waits; one elected lane issues the copies.
      if (lane == 0) {
        prefetch_tensormap(&tmap_a);
        prefetch_tensormap(&tmap_b);
        if (GATED) prefetch_tensormap(&tmap_b2);
      }
      uint32_t it = 0;
      bool ok = true;
      for (int kb = kb0; kb < kb1; ++kb, ++it) {
        const int s = it % kStages;
        const uint32_t ph = (it / kStages) & 1u;
        if (!mbar_wait_warp(empty_bar(s), ph ^ 1u, abort_flag, p.status, kTimeoutProducer)) { ok = false; break; }
        const uint32_t sa = smem_base + s * C::kStage, sb = sa + C::kStageA;
        if (elect_one()) {
          mbar_arrive_expect_tx(full_bar(s), C::kStage);
          tma_load_4d(sa, &tmap_a, full_bar(s), kb * BK, mt * BM, 0, 0);
          if constexpr (GATED) {
#pragma unroll
            for (int j = 0; j < BN / 64; ++j)
              tma_load_4d(sb + j * (64 * BK * 2), j < BN / 128 ? &tmap_b : &tmap_b2, full_bar(s),
                          nt * OC + (j % (BN / 128)) * 64, kb * BK, 0, 0);
          } else if (B_NK) {
            tma_load_4d(sb, &tmap_b, full_bar(s), kb * BK, nt * BN, 0, 0);
          } else {
#pragma unroll
            for (int j = 0; j < BN / 64; ++j)
              tma_load_4d(sb + j * (64 * BK * 2), &tmap_b, full_bar(s), nt * BN + j * 64, kb * BK, 0, 0);
          }
        }
        __syncwarp();
      }
      if (!ok) {
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
      bool ok = true;
      for (int kb = kb0; kb < kb1; ++kb, ++it) {
        const int s = it % kStages;
        const uint32_t ph = (it / kStages) & 1u;
        if (!mbar_wait_warp(full_bar(s), ph, abort_flag, p.status, kTimeoutMmaFull)) { ok = false; break; }
        tcgen05_fence_after_sync();
        const uint32_t sa = smem_base + s * C::kStage, sb = sa + C::kStageA;
        if (elect_one()) {
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            const uint64_t a_desc = make_smem_desc(sa + k * (UMMA_K * 2), 0, 1024);
            const uint64_t b_desc = B_NK ? make_smem_desc(sb + k * (UMMA_K * 2), 0, 1024)
                                         : make_smem_desc(sb + k * (UMMA_K * 128), 64 * BK * 2, 1024);
            mma_bf16_ss(tmem_base, a_desc, b_desc, idesc, (kb > kb0 || k > 0) ? 1u : 0u);
          }
          mma_commit(empty_bar(s));
        }
        __syncwarp();
      }
      if (ok) {
        if (elect_one()) mma_commit(acc_full_bar);
        __syncwarp();
      } else {
        if (lane == 0) mma_commit(drain_bar);
        __syncwarp();
        volatile int never = 0;
        mbar_wait(drain_bar, 0, &never, nullptr, 0, 20000000ull);
      }
    }
  } else {
    acc_ok = mbar_wait(acc_full_bar, 0, abort_flag, p.status, kTimeoutEpilogue);
    acc_ok = __all_sync(0xffffffffu, acc_ok);  // the tensor-memory loads below need the whole warp
    tcgen05_fence_after_sync();
  }

  // ---- 2. every accumulator of the cluster is complete, every ring idle (also reached after an expired wait)
  __syncwarp();
  cluster_sync_all();

  // Accumulator columns are dealt to the ranks in chunks of 8.  Rank d, column half g (the two warps of a lane
  // group), chunk j of NCH:  plain: d W + g W/2 + 8 j;  gated (W/2 gate columns and the W/2 up columns of the same
  // outputs): (j < NCH/2 ? 0 : BN/2) + d W/2 + g W/4 + 8 (j mod NCH/2).
  constexpr int W = BN / S;    // accumulator columns owned by one rank
  constexpr int NCH = W / 16;  // chunks of 8 columns per thread
  static_assert(NCH >= (GATED ? 2 : 1), "cluster too large for this tile");
  auto chunk_col = [&](int d, int g, int j) {
    if (GATED) {
      constexpr int h = NCH / 2 > 0 ? NCH / 2 : 1;
      return (j < h ? 0 : BN / 2) + d * (W / 2) + g * (W / 4) + 8 * (j % h);
    }
    return d * W + g * (W / 2) + 8 * j;
  };
  const int quarter = warp & 3, group = (warp - 2) >> 2;
  const int row = quarter * 32 + lane;
  const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16);
  // receive buffer of a CTA, at the start of its ring: [sender][g][j][half][row] x 16 bytes, so that the 32 lanes
  // of a warp (32 consecutive rows) write and read 512 consecutive bytes per instruction
  auto recv_off = [&](int src, int g, int j, int half) {
    return (uint32_t)((((((src * 2 + g) * NCH + j) * 2 + half) * BM) + row) * 16);
  };

  // ---- 3. partial sums of columns owned elsewhere go to their owners
  if (warp >= 2 && acc_ok) {
#pragma unroll 1
    for (int dd = 1; dd < S; ++dd) {
      const int d = (rank + dd) % S;  // every rank starts with a different owner
      uint32_t r[NCH][8];
#pragma unroll
      for (int j = 0; j < NCH; ++j) tmem_ld_32x32b_x8(t_row + chunk_col(d, group, j), r[j]);
      tmem_ld_wait();
#pragma unroll
      for (int j = 0; j < NCH; ++j) {
        st_cluster_v4_b32(map_to_cta(smem_base + recv_off(rank, group, j, 0), (uint32_t)d), r[j][0], r[j][1], r[j][2], r[j][3]);
        st_cluster_v4_b32(map_to_cta(smem_base + recv_off(rank, group, j, 1), (uint32_t)d), r[j][4], r[j][5], r[j][6], r[j][7]);
      }
    }
  }
  // ---- 4. the partial sums have landed
  __syncwarp();
  cluster_sync_all();

  // ---- 5. own columns: sum, epilogue, store
  if (warp >= 2 && acc_ok) {
    const int m = mt * BM + row;
    uint32_t own[NCH][8];  // this CTA's own partial sums of its columns
#pragma unroll
    for (int j = 0; j < NCH; ++j) tmem_ld_32x32b_x8(t_row + chunk_col(rank, group, j), own[j]);
    tmem_ld_wait();
    auto reduced_chunk = [&](int j, float (&v)[8]) {
#pragma unroll
      for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(own[j][i]);
#pragma unroll
      for (int src = 0; src < S; ++src) {
        if (src == rank) continue;
        const float4 lo = ld_shared_v4_f32(smem_base + recv_off(src, group, j, 0));
        const float4 hi = ld_shared_v4_f32(smem_base + recv_off(src, group, j, 1));
        v[0] += lo.x; v[1] += lo.y; v[2] += lo.z; v[3] += lo.w;
        v[4] += hi.x; v[5] += hi.y; v[6] += hi.z; v[7] += hi.w;
      }
    };
    auto store8 = [&](int n0, const float (&v)[8]) {
      if (m >= p.M || n0 >= p.N) return;  // N is a multiple of 8: a chunk is inside or outside as a whole
      if (sp.c_is_f32) {
        float4* dst = reinterpret_cast<float4*>(static_cast<float*>(p.C) + (int64_t)m * p.ldc + n0);
        dst[0] = make_float4(v[0], v[1], v[2], v[3]);
        dst[1] = make_float4(v[4], v[5], v[6], v[7]);
      } else {
        *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(p.C) + (int64_t)m * p.ldc + n0) =
            make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
      }
    };
    if constexpr (GATED) {
#pragma unroll
      for (int j = 0; j < NCH / 2; ++j) {
        float g8[8], u8[8], y[8];
        reduced_chunk(j, g8);
        reduced_chunk(j + NCH / 2, u8);
#pragma unroll
        for (int i = 0; i < 8; ++i) y[i] = g8[i] * (1.0f / (1.0f + exp2f(-1.4426950408889634f * g8[i]))) * u8[i];
        store8(nt * OC + chunk_col(rank, group, j), y);
      }
    } else {
#pragma unroll
      for (int j = 0; j < NCH; ++j) {
        float v[8];
        reduced_chunk(j, v);
        const int n0 = nt * BN + chunk_col(rank, group, j);
        if (n0 < p.N) {
          float bv[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
          if (p.bias != nullptr) {
            const float4 b0 = __ldg(reinterpret_cast<const float4*>(p.bias + n0));
            const float4 b1 = __ldg(reinterpret_cast<const float4*>(p.bias + n0) + 1);
            bv[0] = b0.x; bv[1] = b0.y; bv[2] = b0.z; bv[3] = b0.w;
            bv[4] = b1.x; bv[5] = b1.y; bv[6] = b1.z; bv[7] = b1.w;
          }
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            float z = fmaf(v[i], p.alpha, bv[i]);
            if (p.act == 1) z = gelu_erf(z);
            else if (p.act == 2) z = fmaxf(z, 0.0f);
            v[i] = z;
          }
          if (sp.residual != nullptr && m < p.M) {
            const uint4 q = __ldg(reinterpret_cast<const uint4*>(sp.residual + (int64_t)m * p.ldr + n0));
            const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
            for (int t = 0; t < 4; ++t) {
              v[2 * t] += __uint_as_float(w[t] << 16);
              v[2 * t + 1] += __uint_as_float(w[t] & 0xffff0000u);
            }
          }
        }
        store8(n0, v);
      }
    }
  }

  // ------------------------------------------------------------------- teardown
  __syncwarp();
  tcgen05_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tcgen05_fence_after_sync();
    tmem_dealloc(tmem_base, BN);
  }
}

template <int BN, bool B_NK, bool GATED, int S>
pd_status launch_split_variant(const GemmProblem& g, cudaStream_t s) {
  constexpr int split = S;
  using C = SplitCfg<BN>;
  constexpr int OC = GATED ? BN / 2 : BN;
  CUtensorMap ta, tb, tb2;
  if (!make_map(&ta, false, g.A, g.K, g.M, g.lda, 1, 0, 1, 0, BK, BM)) return PD_ERR_UNSUPPORTED;
  const bool okb = B_NK ? make_map(&tb, false, g.B, g.K, g.N, g.ldb, 1, 0, 1, 0, BK, BN)
                        : make_map(&tb, false, g.B, g.N, g.K, g.ldb, 1, 0, 1, 0, 64, BK);
  if (!okb) return PD_ERR_UNSUPPORTED;
  tb2 = tb;
  if (GATED && !make_map(&tb2, false, g.B2, g.N, g.K, g.ldb, 1, 0, 1, 0, 64, BK)) return PD_ERR_UNSUPPORTED;

  KernelParams p{};
  p.C = g.C; p.bias = g.bias; p.residual = g.residual; p.status = device_status_ptr();
  if (!p.status) return PD_ERR_CUDA;
  p.ldc = g.ldc; p.ldr = g.ldr;
  p.M = (int)g.M; p.N = (int)g.N; p.K = (int)g.K;
  p.tiles_m = (int)((g.M + BM - 1) / BM);
  p.tiles_n = (int)((g.N + OC - 1) / OC);
  p.batch_inner = 1;
  p.num_tiles = p.tiles_m * p.tiles_n;
  p.alpha = g.alpha; p.c_is_f32 = g.c_dtype == PD_F32; p.act = g.act;
  SplitParams sp{p.c_is_f32, g.residual};

  auto kernel = gemm_bf16_splitk_cluster_kernel<BN, B_NK, GATED, S>;
  static PerDeviceFlag smem_allowed;  // one per kernel (template instantiation)
  if (pd_status st = allow_dynamic_smem(kernel, C::kSmemBytes, smem_allowed); st != PD_OK) return st;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(p.num_tiles * split);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = C::kSmemBytes;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = split;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  cudaLaunchKernelEx(&cfg, kernel, ta, tb, tb2, p, sp);
  return check_launch();
}

}  // namespace

// Cluster size to split K over (0: do not split).  Worth it when the tiles of the problem cover less than half
// of the SMs and every CTA still gets at least two k-blocks.
int gemm_split_k_factor(const GemmProblem& g) {
  if (g.batch_inner != 1 || g.batch_outer != 1) return 0;
  if (g.B2 != nullptr && (g.b_is_nk || g.c_dtype != PD_BF16)) return 0;
  // The epilogue of the split kernel stores, and reads bias and residual, eight whole columns at a time: a row
  // whose length is not a multiple of eight is left to the kernels whose TMA stores clip the edge.
  if (g.N % 8 != 0 || g.ldc % (g.c_dtype == PD_F32 ? 4 : 8) != 0 || (g.residual != nullptr && g.ldr % 8 != 0)) return 0;
  if (g.bias != nullptr && !aligned16(g.bias)) return 0;
  const int64_t oc = g.B2 != nullptr ? 128 : 256;
  const int64_t tiles = ((g.M + BM - 1) / BM) * ((g.N + oc - 1) / oc);
  const int64_t num_kb = (g.K + BK - 1) / BK;
  // Shorter K extents finish within the fixed cost of the two cluster barriers and the exchange (measured:
  // 768 x 1024 x 1024 ties, 256 x 448 x 4096 halves its time).
  if (num_kb < 32) return 0;
  int split = 8;
  while (split > 1 && (tiles * split > sm_count() || num_kb < 4 * split)) split /= 2;
  return split >= 2 ? split : 0;
}

namespace {
template <bool B_NK, bool GATED>
pd_status launch_split(const GemmProblem& g, int split, cudaStream_t s) {
  switch (split) {
    case 2: return launch_split_variant<256, B_NK, GATED, 2>(g, s);
    case 4: return launch_split_variant<256, B_NK, GATED, 4>(g, s);
    case 8: return launch_split_variant<256, B_NK, GATED, 8>(g, s);
  }
  return PD_ERR_UNSUPPORTED;
}
}  // namespace

pd_status launch_gemm_split_k(const GemmProblem& g, int split, cudaStream_t s) {
  if (g.B2 != nullptr) return launch_split<false, true>(g, split, s);
  return g.b_is_nk ? launch_split<true, false>(g, split, s) : launch_split<false, false>(g, split, s);
}

}  // namespace pd
