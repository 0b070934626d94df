// Y = LayerNorm(A B + bias + residual; gamma, beta): the projection, the residual
// add and the LayerNorm that closes each half of an encoder layer in one kernel.
//
// LayerNorm needs whole rows, a 128 x 256 accumulator tile holds a quarter of a
// 1024-wide row.  So the N / 256 CTAs that own the tiles of the same 128 rows
// form a thread-block cluster and run in lockstep over the row blocks:
//   * main loop: as in the single-CTA GEMM (TMA producer warp, MMA issuer warp,
//     one elected lane of each issuing; two TMEM accumulators, four 48 KiB stages);
//   * epilogue pass 1 (sixteen warps, so that four per scheduler hide each
//     other's latencies): every epilogue thread owns 64 columns of one row.  It
//     forms v = acc + bias + residual in fp32, writes v back over the
//     accumulator in tensor memory, and computes the mean and centred second
//     moment of its 64 values (accumulated around the first value, so a large
//     common offset costs no precision).  The four warps that share a row
//     combine their parts through shared memory;
//   * exchange: the combined (mean, second moment) of each row goes to every CTA
//     of the cluster with asynchronous distributed-shared-memory stores that
//     credit the receiver's mbarrier, so nobody waits on a fence; a second
//     cluster-wide mbarrier tells the senders that the previous tile's values
//     have been read before they are overwritten.  Each CTA merges the N / 256
//     partial statistics pairwise in the same fixed order;
//   * epilogue pass 2 reads v back from tensor memory, normalises, applies gamma
//     and beta, and stores bf16 through swizzled shared memory and TMA, while the
//     MMA warp fills the other accumulator.
// bias, gamma and beta of the CTA's 256 columns sit in shared memory.  The fp32
// pre-LayerNorm tensor never exists in global memory.
// Requirements: N a multiple of 256 and at most 2048 (cluster of up to 8 CTAs),
// bf16 A [M, K], bf16 B [K, N], bf16 residual and output [M, N].
// Every wait is bounded as in the other tensor-core kernels.
#include "gemm_common.cuh"

namespace pd {
namespace {

using namespace sm100;
using namespace gemm;

constexpr int BN = 256;
constexpr int kMaxCluster = 8;
constexpr int kStageA = BM * BK * 2, kStageB = BN * BK * 2, kStage = kStageA + kStageB;
constexpr int kStages = 4;
constexpr int kLnEpilogueWarps = 16;                             // four per TMEM lane quarter: 64 columns each
constexpr int kLnEpilogueThreads = 32 * kLnEpilogueWarps;
constexpr int kLnThreads = 64 + kLnEpilogueThreads;
constexpr int kStep = 16;                                        // columns per epilogue step
constexpr int kStagingPerWarp = 32 * kStep * 2;                  // 32 rows x 16 bf16 columns
constexpr int kStagingBytes = kLnEpilogueWarps * kStagingPerWarp;
constexpr int kStatsBytes = kMaxCluster * BM * 8;                // one (mean, M2) per source CTA and row
constexpr int kPairBytes = 3 * BM * 8;                           // hand-over from the three other warps of a row
constexpr int kParamBytes = 3 * BN * 4;                          // bias, gamma, beta of this CTA's columns
constexpr int kBarrierBytes = 256;
constexpr int kSmemBytes =
    kStages * kStage + kStagingBytes + kStatsBytes + kPairBytes + kParamBytes + kBarrierBytes + 1024;
static_assert(kSmemBytes <= kSmemLimit, "shared memory budget");
constexpr int kTmemCols = 2 * BN;

struct LnParams {
  const float* gamma;
  const float* beta;
  float eps;
  int cluster;  // CTAs per cluster = N / 256
  int descending;  // walk the row blocks from the last to the first (GemmProblem::rows_descending)
};

enum : int { kTimeoutLnStats = 105, kTimeoutLnPair = 106, kTimeoutLnConsumed = 107 };

template <bool B_NK>
__global__ void __launch_bounds__(kLnThreads, 1)
gemm_bias_residual_layernorm_kernel(const __grid_constant__ CUtensorMap tmap_a,
                                    const __grid_constant__ CUtensorMap tmap_b,
                                    const __grid_constant__ CUtensorMap tmap_c, const KernelParams p,
                                    const LnParams ln) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t staging_base = smem_base + kStages * kStage;
  const uint32_t stats_base = staging_base + kStagingBytes;
  const uint32_t pair_base = stats_base + kStatsBytes;
  const uint32_t param_base = pair_base + kPairBytes;
  const uint32_t bar_base = param_base + kParamBytes;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (kStages + s); };
  auto acc_full_bar = [&](int a) { return bar_base + 8u * (2 * kStages + a); };
  auto acc_empty_bar = [&](int a) { return bar_base + 8u * (2 * kStages + 2 + a); };
  const uint32_t drain_bar = bar_base + 8u * (2 * kStages + 4);
  const uint32_t stats_bar = bar_base + 8u * (2 * kStages + 5);     // this tile's statistics have all landed here
  const uint32_t consumed_bar = bar_base + 8u * (2 * kStages + 6);  // every CTA has read the statistics sent from here
  auto pair_bar = [&](int q) { return bar_base + 8u * (2 * kStages + 7 + q); };
  uint8_t* ctrl = smem_gen + (bar_base - smem_base) + 8 * (2 * kStages + 11);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(ctrl);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(ctrl + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_kb = (p.K + BK - 1) / BK;
  const int nt = (int)cluster_ctarank();            // this CTA's column tile
  const int cluster_id = blockIdx.x / ln.cluster;
  const int num_clusters = gridDim.x / ln.cluster;  // row blocks are dealt round-robin to clusters
  // step i of a cluster works on row block phys(cluster_id + i * num_clusters)
  auto phys = [&](int lt) { return ln.descending ? p.tiles_m - 1 - lt : lt; };

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(acc_full_bar(a), 1);
      mbar_init(acc_empty_bar(a), kLnEpilogueThreads);
    }
    mbar_init(drain_bar, 1);
    mbar_init(stats_bar, 1);                               // armed once per tile with the expected byte count
    mbar_init(consumed_bar, ln.cluster * kLnEpilogueWarps);  // one arrival per epilogue warp of every CTA
    for (int q = 0; q < 4; ++q) mbar_init(pair_bar(q), 3);
    *abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async_smem();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
    tmem_relinquish_alloc_permit();
  }
  tcgen05_fence_before_sync();
  cluster_sync_all();  // every CTA's barriers exist before anyone signals them
  tcgen05_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
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
      for (int lt = cluster_id; lt < p.tiles_m && ok; lt += num_clusters) {
        const int mt = phys(lt);
        for (int kb = 0; kb < num_kb; ++kb, ++it) {
          const int s = it % kStages;
          const uint32_t ph = (it / kStages) & 1u;
          if (!mbar_wait_warp(empty_bar(s), ph ^ 1u, abort_flag, p.status, kTimeoutProducer)) { ok = false; break; }
          const uint32_t sa = smem_base + s * kStage, sb = sa + kStageA;
          if (elect_one()) {
            mbar_arrive_expect_tx(full_bar(s), kStage);
            tma_load_4d(sa, &tmap_a, full_bar(s), kb * BK, mt * BM, 0, 0);
            if (B_NK) {
              tma_load_4d(sb, &tmap_b, full_bar(s), kb * BK, nt * BN, 0, 0);
            } else {
#pragma unroll
              for (int j = 0; j < BN / 64; ++j)
                tma_load_4d(sb + j * (64 * BK * 2), &tmap_b, full_bar(s), nt * BN + j * 64, kb * BK, 0, 0);
            }
          }
          __syncwarp();
        }
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
      int local = 0;
      bool ok = true;
      for (int lt = cluster_id; lt < p.tiles_m && ok; lt += num_clusters, ++local) {
        const int acc = local & 1;
        const uint32_t acc_ph = (local >> 1) & 1u;
        if (!mbar_wait_warp(acc_empty_bar(acc), acc_ph ^ 1u, abort_flag, p.status, kTimeoutMmaAcc)) { ok = false; break; }
        tcgen05_fence_after_sync();
        const uint32_t d_tmem = tmem_base + acc * BN;
        for (int kb = 0; kb < num_kb; ++kb, ++it) {
          const int s = it % kStages;
          const uint32_t ph = (it / kStages) & 1u;
          if (!mbar_wait_warp(full_bar(s), ph, abort_flag, p.status, kTimeoutMmaFull)) { ok = false; break; }
          tcgen05_fence_after_sync();
          const uint32_t sa = smem_base + s * kStage, sb = sa + kStageA;
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
        if (lane == 0) mma_commit(drain_bar);
        __syncwarp();
        volatile int never = 0;
        mbar_wait(drain_bar, 0, &never, nullptr, 0, 20000000ull);
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    const int quarter = warp & 3;        // TMEM lanes 32*quarter .. +31
    const int group = (warp - 2) >> 2;   // columns [64*group, +64); group 0 also talks to the cluster
    const int row = quarter * 32 + lane;
    const uint32_t buf = staging_base + (uint32_t)(warp - 2) * kStagingPerWarp;
    const uint32_t row_addr = buf + (uint32_t)lane * 32u;
    const uint32_t sw = (uint32_t)((lane >> 2) & 1);  // 32-byte swizzle: 16-byte unit index ^= (row / 4) % 2
    const int n_tile = nt * BN;
    const int c_base = 64 * group;       // this thread's first column inside the tile

    // bias, gamma and beta of this CTA's columns: shared memory copies (zeros for a missing bias)
    {
      float* prm = reinterpret_cast<float*>(smem_gen + (param_base - smem_base));
      for (int t = threadIdx.x - 64; t < 3 * BN; t += kLnEpilogueThreads) {
        const int c = n_tile + (t & (BN - 1));
        prm[t] = t < BN ? (p.bias != nullptr ? __ldg(p.bias + c) : 0.f) : (t < 2 * BN ? __ldg(ln.gamma + c) : __ldg(ln.beta + c));
      }
      asm volatile("bar.sync 1, %0;" ::"n"(kLnEpilogueThreads) : "memory");
    }

    // The residual of this thread's 64 columns of one row, fetched one tile ahead of its use.
    uint4 res[4][2];
    auto load_residual = [&](int lt) {
      const int m = phys(lt) * BM + row;
      if (p.residual == nullptr || lt >= p.tiles_m || m >= p.M) return;
      const uint4* rr = reinterpret_cast<const uint4*>(p.residual + (int64_t)m * p.ldr + n_tile + c_base);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        res[i][0] = __ldg(rr + 2 * i);
        res[i][1] = __ldg(rr + 2 * i + 1);
      }
    };
#pragma unroll
    for (int i = 0; i < 4; ++i) res[i][0] = res[i][1] = make_uint4(0u, 0u, 0u, 0u);
    int local = 0;
    if (lane == 0) prefetch_tensormap(&tmap_c);
    load_residual(cluster_id);
    for (int lt = cluster_id; lt < p.tiles_m; lt += num_clusters, ++local) {
      const int mt = phys(lt);
      const int acc = local & 1;
      const uint32_t acc_ph = (local >> 1) & 1u;
      const uint32_t tile_ph = local & 1u;  // phase parity of the once-per-tile barriers
      const int m_warp = mt * BM + quarter * 32;
      // the previous tile's phase of stats_bar is complete (this warp waited for it): expect this tile's bytes
      if (warp == 2 && lane == 0) mbar_arrive_expect_tx(stats_bar, (uint32_t)ln.cluster * BM * 8u);
      // the next tile's residual (one 128-byte line per thread) starts its way from DRAM into L2 a tile ahead
      if (p.residual != nullptr && lt + num_clusters < p.tiles_m && phys(lt + num_clusters) * BM + row < p.M)
        asm volatile("prefetch.global.L2 [%0];" ::"l"(p.residual + ((int64_t)phys(lt + num_clusters) * BM + row) * p.ldr +
                                                      n_tile + c_base));
      if (!mbar_wait(acc_full_bar(acc), acc_ph, abort_flag, p.status, kTimeoutEpilogue)) break;
      tcgen05_fence_after_sync();
      const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * BN + c_base;
      // ---- pass 1: v = alpha acc + bias + residual goes back into tensor memory; statistics of the 64 values
      // (two fp32 values per instruction throughout: the epilogue is bound by instruction issue)
      float shift = 0.f;
      uint64_t nshift2 = 0, a1[2] = {0, 0}, a2[2] = {0, 0};
      const uint64_t alpha2 = pack_f32x2(p.alpha, p.alpha);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        uint32_t r[kStep];
        tmem_ld_32x32b_x16(t_row + i * kStep, r);
        tmem_ld_wait();
        uint64_t v[kStep / 2];
#pragma unroll
        for (int j = 0; j < kStep; j += 4) {
          const float4 bv = ld_shared_v4_f32(param_base + (uint32_t)(c_base + i * kStep + j) * 4u);
          v[j / 2] = fma_f32x2(pack_b32x2(r[j], r[j + 1]), alpha2, pack_f32x2(bv.x, bv.y));
          v[j / 2 + 1] = fma_f32x2(pack_b32x2(r[j + 2], r[j + 3]), alpha2, pack_f32x2(bv.z, bv.w));
        }
        if (p.residual != nullptr) {
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            const uint32_t w[4] = {res[i][j].x, res[i][j].y, res[i][j].z, res[i][j].w};
#pragma unroll
            for (int t = 0; t < 4; ++t)
              v[4 * j + t] = add_f32x2(v[4 * j + t], pack_b32x2(w[t] << 16, w[t] & 0xffff0000u));
          }
        }
#pragma unroll
        for (int j = 0; j < kStep / 2; ++j) unpack_b32x2(v[j], r[2 * j], r[2 * j + 1]);
        tmem_st_32x32b_x16(t_row + i * kStep, r);
        if (i == 0) {
          shift = __uint_as_float(r[0]);
          nshift2 = pack_f32x2(-shift, -shift);
        }
#pragma unroll
        for (int j = 0; j < kStep / 2; ++j) {
          const uint64_t d = add_f32x2(v[j], nshift2);
          a1[j & 1] = add_f32x2(a1[j & 1], d);
          a2[j & 1] = fma_f32x2(d, d, a2[j & 1]);
        }
      }
      load_residual(lt + num_clusters);  // the next tile's residual travels during the exchange and pass 2
      float mean_p, m2_p;  // of this thread's 64 values
      {
        float s1a, s1b, s2a, s2b;
        unpack_f32x2(add_f32x2(a1[0], a1[1]), s1a, s1b);
        unpack_f32x2(add_f32x2(a2[0], a2[1]), s2a, s2b);
        const float s1 = s1a + s1b, s2 = s2a + s2b;
        const float mean_d = s1 * (1.0f / 64.0f);
        mean_p = shift + mean_d;
        m2_p = fmaxf(s2 - s1 * mean_d, 0.f);
      }
      // ---- the four warps of a row combine their parts; group 0 sends the result to every CTA of the cluster
      if (group != 0) {
        st_shared_v2_f32(pair_base + (uint32_t)((group - 1) * BM + row) * 8u, mean_p, m2_p);
        __syncwarp();
        if (lane == 0) mbar_arrive(pair_bar(quarter));
      } else {
        if (!mbar_wait(pair_bar(quarter), tile_ph, abort_flag, p.status, kTimeoutLnPair)) break;
        float mean_c = mean_p, m2_c = m2_p;
#pragma unroll
        for (int g = 1; g < 4; ++g) {  // counts 64 g and 64: the merge weights are g / (g + 1) and 1 / (g + 1)
          const float2 other = ld_shared_v2_f32(pair_base + (uint32_t)((g - 1) * BM + row) * 8u);
          const float d = other.x - mean_c;
          m2_c += other.y + d * d * (64.0f * (float)g / (float)(g + 1));
          mean_c = fmaf(d, 1.0f / (float)(g + 1), mean_c);
        }
        // the values sent for the previous tile must have been read everywhere before they are overwritten
        if (local > 0 && !mbar_wait(consumed_bar, tile_ph ^ 1u, abort_flag, p.status, kTimeoutLnConsumed)) break;
        const uint32_t dst = stats_base + (uint32_t)(nt * BM + row) * 8u;
#pragma unroll
        for (int rk = 0; rk < kMaxCluster; ++rk)
          if (rk < ln.cluster) st_async_v2_f32(map_to_cta(dst, rk), mean_c, m2_c, map_to_cta(stats_bar, rk));
      }
      tmem_st_wait();
      if (!mbar_wait(stats_bar, tile_ph, abort_flag, p.status, kTimeoutLnStats)) break;
      // ---- merge the row's partial statistics (fixed order: identical in every CTA)
      float mean = 0.f, m2 = 0.f;
      {
        float2 st[kMaxCluster];
#pragma unroll
        for (int q = 0; q < kMaxCluster; ++q)
          st[q] = q < ln.cluster ? ld_shared_v2_f32(stats_base + (uint32_t)(q * BM + row) * 8u) : make_float2(0.f, 0.f);
        mean = st[0].x;
        m2 = st[0].y;
#pragma unroll
        for (int q = 1; q < kMaxCluster; ++q) {  // counts 256 q and 256
          if (q < ln.cluster) {
            const float d = st[q].x - mean;
            m2 += st[q].y + d * d * (256.0f * (float)q / (float)(q + 1));
            mean = fmaf(d, 1.0f / (float)(q + 1), mean);
          }
        }
      }
      const float rstd = rsqrtf(m2 / (float)p.N + ln.eps);
      const uint64_t nmean2 = pack_f32x2(-mean, -mean), rstd2 = pack_f32x2(rstd, rstd);
      // ---- pass 2: normalise and store, 16 columns per TMA store
#pragma unroll 1
      for (int i = 0; i < 4; ++i) {
        const int c0 = c_base + i * kStep;
        uint32_t r[kStep];
        tmem_ld_32x32b_x16(t_row + i * kStep, r);
        tmem_ld_wait();
        uint32_t packed[kStep / 2];
#pragma unroll
        for (int j = 0; j < kStep; j += 4) {
          const float4 g = ld_shared_v4_f32(param_base + (uint32_t)(BN + c0 + j) * 4u);
          const float4 b = ld_shared_v4_f32(param_base + (uint32_t)(2 * BN + c0 + j) * 4u);
          const uint64_t t0 = mul_f32x2(add_f32x2(pack_b32x2(r[j], r[j + 1]), nmean2), rstd2);
          const uint64_t t1 = mul_f32x2(add_f32x2(pack_b32x2(r[j + 2], r[j + 3]), nmean2), rstd2);
          float y0, y1, y2, y3;
          unpack_f32x2(fma_f32x2(t0, pack_f32x2(g.x, g.y), pack_f32x2(b.x, b.y)), y0, y1);
          unpack_f32x2(fma_f32x2(t1, pack_f32x2(g.z, g.w), pack_f32x2(b.z, b.w)), y2, y3);
          packed[j / 2] = pack_bf16(y0, y1);
          packed[j / 2 + 1] = pack_bf16(y2, y3);
        }
        if (lane == 0) tma_store_wait_read<0>();  // the previous store of this warp has finished reading the buffer
        __syncwarp();
#pragma unroll
        for (int u = 0; u < 2; ++u)
          st_shared_v4(row_addr + (((uint32_t)u ^ sw) << 4),
                       make_uint4(packed[4 * u], packed[4 * u + 1], packed[4 * u + 2], packed[4 * u + 3]));
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          tma_store_4d(&tmap_c, buf, n_tile + c0, m_warp, 0, 0);
          tma_store_commit();
        }
      }
      tcgen05_fence_before_sync();
      mbar_arrive(acc_empty_bar(acc));
      // Every lane of this warp has read the tile's statistics: their values went into rstd long ago, so the
      // loads have been performed and the signal needs no release fence (which would stall the warp here).
      __syncwarp();
      if (lane < ln.cluster) mbar_arrive_cluster_relaxed(map_to_cta(consumed_bar, (uint32_t)lane));
    }
    if (lane == 0) tma_store_wait_read<0>();
    __syncwarp();
  }

  // ------------------------------------------------------------------- teardown
  // No CTA may leave while a partner can still write its shared memory or signal its barriers.
  __syncwarp();
  tcgen05_fence_before_sync();
  cluster_sync_all();
  if (warp == 1) {
    tcgen05_fence_after_sync();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

template <bool B_NK>
pd_status launch_ln_variant(const GemmProblem& g, const float* gamma, const float* beta, float eps, cudaStream_t s) {
  CUtensorMap ta, tb, tc;
  if (!make_map(&ta, false, g.A, g.K, g.M, g.lda, 1, 0, 1, 0, BK, BM)) return PD_ERR_UNSUPPORTED;
  const bool okb = B_NK ? make_map(&tb, false, g.B, g.K, g.N, g.ldb, 1, 0, 1, 0, BK, BN)
                        : make_map(&tb, false, g.B, g.N, g.K, g.ldb, 1, 0, 1, 0, 64, BK);
  if (!okb) return PD_ERR_UNSUPPORTED;
  if (!make_map(&tc, false, g.C, g.N, g.M, g.ldc, 1, 0, 1, 0, kStep, 32, CU_TENSOR_MAP_SWIZZLE_32B))
    return PD_ERR_UNSUPPORTED;

  KernelParams p{};
  p.C = g.C; p.bias = g.bias; p.residual = g.residual; p.status = device_status_ptr();
  if (!p.status) return PD_ERR_CUDA;
  p.ldc = g.ldc; p.ldr = g.ldr;
  p.M = (int)g.M; p.N = (int)g.N; p.K = (int)g.K;
  p.tiles_m = (int)((g.M + BM - 1) / BM);
  p.tiles_n = (int)(g.N / BN);
  p.batch_inner = 1;
  p.num_tiles = p.tiles_m * p.tiles_n;
  p.alpha = g.alpha; p.c_is_f32 = 0; p.act = 0;
  LnParams ln{gamma, beta, eps, p.tiles_n, g.rows_descending ? 1 : 0};

  auto kernel = gemm_bias_residual_layernorm_kernel<B_NK>;
  static PerDeviceFlag smem_allowed;  // one per kernel (template instantiation)
  if (pd_status st = allow_dynamic_smem(kernel, kSmemBytes, smem_allowed); st != PD_OK) return st;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((sm_count() / ln.cluster) * ln.cluster);
  cfg.blockDim = dim3(kLnThreads);
  cfg.dynamicSmemBytes = kSmemBytes;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = ln.cluster;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  // Row blocks are dealt statically to the clusters, so launch only as many clusters as can be resident at once
  // (a cluster has to fit inside one GPC, which can leave a few SMs without one).
  static std::atomic<int> resident[kMaxDevicesPerProcess][kMaxCluster + 1];  // per device and cluster size, 0 = not queried yet
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevicesPerProcess) return PD_ERR_UNSUPPORTED;
  int clusters = resident[dev][ln.cluster].load(std::memory_order_relaxed);
  if (clusters == 0) {
    if (cudaOccupancyMaxActiveClusters(&clusters, kernel, &cfg) != cudaSuccess || clusters < 1) {
      (void)cudaGetLastError();
      clusters = 1;
    }
    resident[dev][ln.cluster].store(clusters, std::memory_order_relaxed);
  }
  if (clusters > sm_count() / ln.cluster) clusters = sm_count() / ln.cluster;
  if (clusters > p.tiles_m) clusters = p.tiles_m;
  if (clusters < 1) clusters = 1;
  cfg.gridDim = dim3(clusters * ln.cluster);
  logf("gemm + layernorm %lld x %lld x %lld: %d clusters of %d CTAs, rows %s", (long long)g.M, (long long)g.N, (long long)g.K,
       clusters, ln.cluster, g.rows_descending ? "last first" : "first first");
  cudaLaunchKernelEx(&cfg, kernel, ta, tb, tc, p, ln);
  return check_launch();
}

}  // namespace

bool gemm_layernorm_supported(const GemmProblem& g) {
  return g.N % BN == 0 && g.N / BN <= kMaxCluster && g.batch_inner == 1 && g.batch_outer == 1 && g.c_dtype == PD_BF16 &&
         g.M >= 1 && g.act == 0 && g.B2 == nullptr;
}

pd_status launch_gemm_layernorm(const GemmProblem& g, const float* gamma, const float* beta, float eps,
                                cudaStream_t s) {
  if (!gemm_layernorm_supported(g)) return PD_ERR_UNSUPPORTED;
  return g.b_is_nk ? launch_ln_variant<true>(g, gamma, beta, eps, s) : launch_ln_variant<false>(g, gamma, beta, eps, s);
}

}  // namespace pd

extern "C" pd_status pd_gemm_bias_residual_layernorm(const void* A, const void* B, const float* bias,
                                                     const void* residual, const float* gamma, const float* beta,
                                                     void* Y, int64_t M, int64_t N, int64_t K, float eps,
                                                     cudaStream_t stream) {
  if (!A || !B || !gamma || !beta || !Y) return PD_ERR_NULL_POINTER;
  if (M < 0 || N <= 0 || K <= 0 || !(eps >= 0.f)) return PD_ERR_BAD_SHAPE;
  if (M > 0x7fffffff || N > 0x7fffffff || K > 0x7fffffff) return PD_ERR_BAD_SHAPE;
  if (N % pd::BN != 0 || N / pd::BN > pd::kMaxCluster) return PD_ERR_UNSUPPORTED;
  if (K % 8) return PD_ERR_ALIGNMENT;
  const void* ptrs[] = {A, B, bias, residual, gamma, beta, Y};
  for (const void* q : ptrs)
    if (!pd::aligned16(q)) return PD_ERR_ALIGNMENT;
  if (M == 0) return PD_OK;
  pd_status st = pd::require_sm100();
  if (st != PD_OK) return st;
  pd::GemmProblem g;
  g.A = A; g.B = B; g.C = Y; g.M = M; g.N = N; g.K = K; g.lda = K; g.ldb = N; g.ldc = N;
  g.bias = bias; g.residual = static_cast<const __nv_bfloat16*>(residual); g.ldr = N;
  return pd::launch_gemm_layernorm(g, gamma, beta, eps, stream);
}
