// Fused multi-head attention for sequences of up to 512 keys, head dimension 64:
//
//   Ctx[b,h] = softmax(Q[b,h] K[b,h]^T / sqrt(64)) V[b,h]
//
// on the packed projection qkv[tokens, 3*hidden] = [Q | K | V].  Scores and
// probabilities never leave the SM.
//
// One persistent CTA of 320 threads per SM walks over work units of
// (batch, head, pair of 128-query blocks):
//   warp 8, one lane : TMA producer.  K and V of the head (up to 512 x 64 each)
//                      are loaded once per unit, Q once per query block.
//   warp 9, one lane : MMA issuer.  S = Q K^T as one 128 x 128 x 64 product per
//                      block of 128 keys into tensor memory (all 512 columns
//                      hold the fp32 scores of the 128 queries), then, as the
//                      softmax warps publish blocks of probabilities,
//                      O += P_j V_j (128 x 64 x 128) into columns 0-63, which
//                      the scores of block 0 no longer need by then.
//   warps 0-7        : softmax, two threads per query row (warps 0-3 take the even
//                      key blocks, warps 4-7 the odd ones).  Pass 1 reads the
//                      scores from tensor memory and takes the row maximum
//                      (the two halves exchange theirs through shared memory);
//                      pass 2 re-reads them block by block, forms
//                      p = 2^((s - max) * log2(e) / 8) (exact softmax: the maximum is
//                      known before the first exponential, nothing is ever
//                      rescaled), accumulates the fp32 row sum and writes P as
//                      bf16 into the half's swizzled shared-memory tile, which
//                      the MMA reads as its A operand.  Tensor-memory loads are
//                      issued one chunk ahead of the arithmetic.  Finally each
//                      thread reads 32 columns of its O row, divides by the row
//                      sum and stores 32 bf16 values (64 contiguous bytes).
// Keys beyond the sequence length are zero-filled by TMA and masked to -inf;
// query rows beyond it are computed and discarded.
// Every mbarrier wait is bounded (see mbar_wait): on expiry a code is recorded
// in the device status word, all roles drain, tensor memory is freed and the
// kernel returns.
#include "pd_common.cuh"
#include "sm100_ptx.cuh"

namespace pd {
namespace {

using namespace sm100;

constexpr int kD = 64;            // head dimension
constexpr int kBlockQ = 128;      // queries per block = TMEM lanes
constexpr int kBlockK = 128;      // keys per score block
constexpr int kMaxKeys = 512;     // TMEM columns
constexpr int kQBlocksPerUnit = 2;
constexpr int kThreads = 320;
constexpr int kSoftmaxThreads = 256;
constexpr int kHalfThreads = 128;
constexpr int kProducerWarp = 8, kMmaWarp = 9;

constexpr int kSmemK = kMaxKeys * kD * 2;        // 64 KiB
constexpr int kSmemV = kMaxKeys * kD * 2;        // 64 KiB
constexpr int kSmemQ = kBlockQ * kD * 2;         // 16 KiB
constexpr int kSmemP = kBlockQ * kBlockK * 2;    // 32 KiB per buffer, two buffers
constexpr int kSmemCtrl = 4096;
constexpr int kSmemBytes = kSmemK + kSmemV + kSmemQ + 2 * kSmemP + kSmemCtrl + 1024 /*alignment slack*/;

struct AttnParams {
  __nv_bfloat16* ctx;  // [batch*seq, hidden]
  int* status;
  int batch, seq, heads, hidden;
  int q_blocks;   // ceil(seq / 128)
  int k_blocks;   // ceil(seq / 128)
  int units_per_head, num_units;
};

enum : int { kTimeoutAttnProducer = 201, kTimeoutAttnMma = 202, kTimeoutAttnSoftmax = 203 };

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

__global__ void __launch_bounds__(kThreads, 1)
attention_fwd_tcgen05_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                             const __grid_constant__ CUtensorMap tmap_v, const AttnParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t sK = smem_base, sV = sK + kSmemK, sQ = sV + kSmemV, sP = sQ + kSmemQ;
  const uint32_t bar_base = sP + 2 * kSmemP;
  // barriers (8 bytes each)
  const uint32_t k_full = bar_base + 0, v_full = bar_base + 8, k_empty = bar_base + 16, v_empty = bar_base + 24;
  const uint32_t q_full = bar_base + 32, q_empty = bar_base + 40, s_full = bar_base + 48, s_empty = bar_base + 56;
  const uint32_t o_full = bar_base + 64, drain_bar = bar_base + 72;
  auto p_full = [&](int i) { return bar_base + 80u + 8u * i; };
  auto p_empty = [&](int i) { return bar_base + 96u + 8u * i; };
  const uint32_t max_bar = bar_base + 112, sum_bar = bar_base + 120;
  uint8_t* ctrl = smem_gen + (bar_base - smem_base) + 128;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(ctrl);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(ctrl + 4);
  float* xmax = reinterpret_cast<float*>(ctrl + 1024);  // [2][128] row maxima of the two halves
  float* xsum = reinterpret_cast<float*>(ctrl + 2048);  // [2][128] partial row sums

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    mbar_init(k_full, 1); mbar_init(v_full, 1); mbar_init(k_empty, 1); mbar_init(v_empty, 1);
    mbar_init(q_full, 1); mbar_init(q_empty, 1); mbar_init(s_full, 1); mbar_init(s_empty, kSoftmaxThreads);
    mbar_init(o_full, 1); mbar_init(drain_bar, 1);
    mbar_init(max_bar, kSoftmaxThreads); mbar_init(sum_bar, kSoftmaxThreads);
    for (int i = 0; i < 2; ++i) { mbar_init(p_full(i), kHalfThreads); mbar_init(p_empty(i), 1); }
    *abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async_smem();
  }
  if (warp == kMmaWarp) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), 512);
    tmem_relinquish_alloc_permit();
  }
  tcgen05_fence_before_sync();
  __syncthreads();
  tcgen05_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  // Work decomposition shared by all roles.
  auto unit_coords = [&](int unit, int& b, int& h, int& qb0, int& nqb) {
    const int per_bh = p.units_per_head;
    const int bh = unit / per_bh;
    b = bh / p.heads;
    h = bh % p.heads;
    qb0 = (unit % per_bh) * kQBlocksPerUnit;
    nqb = min(kQBlocksPerUnit, p.q_blocks - qb0);
  };

  if (warp == kProducerWarp) {
    // ------------------------------------------------------------- TMA producer
    if (lane == 0) {
      prefetch_tensormap(&tmap_q); prefetch_tensormap(&tmap_k); prefetch_tensormap(&tmap_v);
      uint32_t n_unit = 0, n_q = 0;
      bool ok = true;
      for (int unit = blockIdx.x; unit < p.num_units && ok; unit += gridDim.x, ++n_unit) {
        int b, h, qb0, nqb;
        unit_coords(unit, b, h, qb0, nqb);
        const uint32_t uph = n_unit & 1u;
        if (!mbar_wait(k_empty, uph ^ 1u, abort_flag, p.status, kTimeoutAttnProducer)) { ok = false; break; }
        mbar_arrive_expect_tx(k_full, kSmemK);
        tma_load_4d(sK, &tmap_k, k_full, 0, 0, h, b);
        tma_load_4d(sK + kSmemK / 2, &tmap_k, k_full, 0, 256, h, b);
        // the first Q of the unit goes out before V: the score product needs only Q and K
        for (int i = 0; i < nqb && ok; ++i, ++n_q) {
          if (!mbar_wait(q_empty, (n_q & 1u) ^ 1u, abort_flag, p.status, kTimeoutAttnProducer)) { ok = false; break; }
          mbar_arrive_expect_tx(q_full, kSmemQ);
          tma_load_4d(sQ, &tmap_q, q_full, 0, (qb0 + i) * kBlockQ, h, b);
          if (i == 0) {
            if (!mbar_wait(v_empty, uph ^ 1u, abort_flag, p.status, kTimeoutAttnProducer)) { ok = false; break; }
            mbar_arrive_expect_tx(v_full, kSmemV);
            tma_load_4d(sV, &tmap_v, v_full, 0, 0, h, b);
            tma_load_4d(sV + kSmemV / 2, &tmap_v, v_full, 0, 256, h, b);
          }
        }
      }
      if (!ok) {
        // leave no copy in flight: give the last armed barriers a short time to complete
        volatile int never = 0;
        if (n_unit > 0 || n_q > 0) {
          mbar_wait(k_full, (n_unit & 1u), &never, nullptr, 0, 20000000ull);
          mbar_wait(q_full, ((n_q - 1u) & 1u), &never, nullptr, 0, 20000000ull);
        }
      }
    }
  } else if (warp == kMmaWarp) {
    // --------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_s = make_idesc_bf16(kBlockQ, kBlockK, false, false);  // Q K^T: both K-major
      constexpr uint32_t idesc_o = make_idesc_bf16(kBlockQ, kD, false, true);        // P V: V is MN-major
      uint32_t n_unit = 0, n_q = 0, n_use0 = 0, n_use1 = 0;  // fills of each half's P tile consumed so far
      bool ok = true;
      for (int unit = blockIdx.x; unit < p.num_units && ok; unit += gridDim.x, ++n_unit) {
        int b, h, qb0, nqb;
        unit_coords(unit, b, h, qb0, nqb);
        const uint32_t uph = n_unit & 1u;
        if (!mbar_wait(k_full, uph, abort_flag, p.status, kTimeoutAttnMma)) { ok = false; break; }
        for (int i = 0; i < nqb && ok; ++i, ++n_q) {
          const uint32_t qph = n_q & 1u;
          if (!mbar_wait(q_full, qph, abort_flag, p.status, kTimeoutAttnMma)) { ok = false; break; }
          if (!mbar_wait(s_empty, qph ^ 1u, abort_flag, p.status, kTimeoutAttnMma)) { ok = false; break; }
          tcgen05_fence_after_sync();
          for (int j = 0; j < p.k_blocks; ++j) {
#pragma unroll
            for (int ks = 0; ks < kD / 16; ++ks) {
              const uint64_t a_desc = make_smem_desc(sQ + ks * 32, 0, 1024);
              const uint64_t b_desc = make_smem_desc(sK + j * (kBlockK * 128) + ks * 32, 0, 1024);
              mma_bf16_ss(tmem_base + j * kBlockK, a_desc, b_desc, idesc_s, ks != 0 ? 1u : 0u);
            }
          }
          mma_commit(s_full);
          mma_commit(q_empty);
          if (i == nqb - 1) mma_commit(k_empty);
          if (i == 0 && !mbar_wait(v_full, uph, abort_flag, p.status, kTimeoutAttnMma)) { ok = false; break; }
          for (int j = 0; j < p.k_blocks && ok; ++j) {
            const int buf = j & 1;  // key block j is produced by softmax half j % 2 into its own tile
            const uint32_t use = buf ? n_use1 : n_use0;
            if (!mbar_wait(p_full(buf), use & 1u, abort_flag, p.status, kTimeoutAttnMma)) { ok = false; break; }
            if (buf) ++n_use1; else ++n_use0;
            tcgen05_fence_after_sync();
#pragma unroll
            for (int ks = 0; ks < kBlockK / 16; ++ks) {
              const uint64_t a_desc = make_smem_desc(sP + buf * kSmemP + (ks >> 2) * (kBlockQ * 128) + (ks & 3) * 32, 0, 1024);
              const uint64_t b_desc = make_smem_desc(sV + (j * kBlockK + ks * 16) * 128, 0, 1024);
              mma_bf16_ss(tmem_base, a_desc, b_desc, idesc_o, (j | ks) != 0 ? 1u : 0u);
            }
            mma_commit(p_empty(buf));
          }
          if (!ok) break;
          mma_commit(o_full);
          if (i == nqb - 1) mma_commit(v_empty);
        }
      }
      if (!ok) {
        mma_commit(drain_bar);
        volatile int never = 0;
        mbar_wait(drain_bar, 0, &never, nullptr, 0, 20000000ull);
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax
    const int quarter = warp & 3, half = warp >> 2;
    const int row = quarter * 32 + lane;  // query row within the block = TMEM lane
    const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16);
    const uint32_t sw = (uint32_t)(lane & 7);
    const float kScale = 0.125f * 1.4426950408889634f;  // 1/sqrt(64) * log2(e)
    const uint32_t p_row = sP + half * kSmemP + (uint32_t)row * 128u;
    uint32_t n_q = 0, n_use = 0;  // n_use: how often this half has filled its P tile
    bool ok = true;
    for (int unit = blockIdx.x; unit < p.num_units && ok; unit += gridDim.x) {
      int b, h, qb0, nqb;
      unit_coords(unit, b, h, qb0, nqb);
      for (int i = 0; i < nqb && ok; ++i, ++n_q) {
        const uint32_t qph = n_q & 1u;
        if (!mbar_wait(s_full, qph, abort_flag, p.status, kTimeoutAttnSoftmax)) { ok = false; break; }
        tcgen05_fence_after_sync();
        // pass 1: maximum over this half's key blocks (j = half, half + 2), loads one chunk ahead
        float m = -INFINITY;
        {
          const int n_chunks = ((p.k_blocks - half + 1) >> 1) * (kBlockK / 32);  // 4 chunks per block
          auto col_of = [&](int c) { return ((c >> 2) * 2 + half) * kBlockK + (c & 3) * 32; };
          uint32_t r[2][32];
          if (n_chunks > 0) tmem_ld_32x32b_x32(t_row + col_of(0), r[0]);
#pragma unroll 1
          for (int c = 0; c < n_chunks; c += 2) {
#pragma unroll
            for (int u = 0; u < 2; ++u) {
              if (c + u >= n_chunks) break;
              tmem_ld_wait();
              if (c + u + 1 < n_chunks) tmem_ld_32x32b_x32(t_row + col_of(c + u + 1), r[u ^ 1]);
              const int c0 = col_of(c + u);
              if (c0 + 32 <= p.seq) {
#pragma unroll
                for (int t = 0; t < 32; ++t) m = fmaxf(m, __uint_as_float(r[u][t]));
              } else {
#pragma unroll
                for (int t = 0; t < 32; ++t)
                  if (c0 + t < p.seq) m = fmaxf(m, __uint_as_float(r[u][t]));
              }
            }
          }
        }
        xmax[half * kBlockQ + row] = m;
        mbar_arrive(max_bar);
        if (!mbar_wait(max_bar, qph, abort_flag, p.status, kTimeoutAttnSoftmax)) { ok = false; break; }
        m = fmaxf(xmax[row], xmax[kBlockQ + row]);
        const float mk = m * kScale;
        // pass 2: probabilities of this half's key blocks
        float sum = 0.f;
        for (int j = half; j < p.k_blocks && ok; j += 2, ++n_use) {
          if (!mbar_wait(p_empty(half), (n_use & 1u) ^ 1u, abort_flag, p.status, kTimeoutAttnSoftmax)) { ok = false; break; }
          uint32_t r[2][32];
          tmem_ld_32x32b_x32(t_row + j * kBlockK, r[0]);
#pragma unroll
          for (int cc = 0; cc < kBlockK / 32; ++cc) {
            const int c = cc * 32;
            const int c0 = j * kBlockK + c;
            tmem_ld_wait();
            if (cc + 1 < kBlockK / 32) tmem_ld_32x32b_x32(t_row + c0 + 32, r[(cc & 1) ^ 1]);
            const uint32_t(&rr)[32] = r[cc & 1];
            float e[32];
            if (c0 + 32 <= p.seq) {
#pragma unroll
              for (int t = 0; t < 32; ++t) e[t] = ex2_approx(fmaf(__uint_as_float(rr[t]), kScale, -mk));
            } else {
#pragma unroll
              for (int t = 0; t < 32; ++t)
                e[t] = (c0 + t < p.seq) ? ex2_approx(fmaf(__uint_as_float(rr[t]), kScale, -mk)) : 0.f;
            }
            float part = 0.f;
#pragma unroll
            for (int t = 0; t < 32; t += 4) part += (e[t] + e[t + 1]) + (e[t + 2] + e[t + 3]);
            sum += part;
            // keys c .. c+31 of the block: 16-byte units (c%64)/8 .. +3 of sub-tile c/64
            const uint32_t sub = p_row + (uint32_t)(c >> 6) * (kBlockQ * 128u);
            const uint32_t u0 = (uint32_t)((c & 63) >> 3);
#pragma unroll
            for (int u = 0; u < 4; ++u)
              st_shared_v4(sub + (((u0 + u) ^ sw) << 4),
                           make_uint4(pack_bf16x2(e[8 * u], e[8 * u + 1]), pack_bf16x2(e[8 * u + 2], e[8 * u + 3]),
                                      pack_bf16x2(e[8 * u + 4], e[8 * u + 5]), pack_bf16x2(e[8 * u + 6], e[8 * u + 7])));
          }
          fence_proxy_async_smem();
          mbar_arrive(p_full(half));
        }
        if (!ok) break;
        xsum[half * kBlockQ + row] = sum;
        mbar_arrive(sum_bar);
        if (!mbar_wait(sum_bar, qph, abort_flag, p.status, kTimeoutAttnSoftmax)) { ok = false; break; }
        const float inv = 1.0f / (xsum[row] + xsum[kBlockQ + row]);
        // output: this half's 32 columns of O / sum -> bf16 -> Ctx
        if (!mbar_wait(o_full, qph, abort_flag, p.status, kTimeoutAttnSoftmax)) { ok = false; break; }
        tcgen05_fence_after_sync();
        const int q = (qb0 + i) * kBlockQ + row;
        __nv_bfloat16* out = p.ctx + ((int64_t)b * p.seq + q) * p.hidden + h * kD + half * 32;
        {
          uint32_t r[32];
          tmem_ld_32x32b_x32(t_row + half * 32, r);
          tmem_ld_wait();
          if (q < p.seq) {
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              uint4 w;
              w.x = pack_bf16x2(__uint_as_float(r[8 * u]) * inv, __uint_as_float(r[8 * u + 1]) * inv);
              w.y = pack_bf16x2(__uint_as_float(r[8 * u + 2]) * inv, __uint_as_float(r[8 * u + 3]) * inv);
              w.z = pack_bf16x2(__uint_as_float(r[8 * u + 4]) * inv, __uint_as_float(r[8 * u + 5]) * inv);
              w.w = pack_bf16x2(__uint_as_float(r[8 * u + 6]) * inv, __uint_as_float(r[8 * u + 7]) * inv);
              *reinterpret_cast<uint4*>(out + 8 * u) = w;
            }
          }
        }
        tcgen05_fence_before_sync();
        mbar_arrive(s_empty);
      }
    }
  }

  // ------------------------------------------------------------------- teardown
  __syncwarp();
  tcgen05_fence_before_sync();
  __syncthreads();
  if (warp == kMmaWarp) {
    tcgen05_fence_after_sync();
    tmem_dealloc(tmem_base, 512);
  }
}

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

// One of Q, K, V inside qkv[batch*seq, 3*hidden]: dims {64, seq, heads, batch}.
bool make_head_map(CUtensorMap* map, const __nv_bfloat16* base, int64_t seq, int64_t heads, int64_t batch,
                   int64_t hidden, int box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  const cuuint64_t dims[4] = {(cuuint64_t)kD, (cuuint64_t)seq, (cuuint64_t)heads, (cuuint64_t)batch};
  const cuuint64_t strides[3] = {(cuuint64_t)(3 * hidden) * 2, (cuuint64_t)kD * 2, (cuuint64_t)(seq * 3 * hidden) * 2};
  const cuuint32_t box[4] = {(cuuint32_t)kD, (cuuint32_t)box_rows, 1, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<__nv_bfloat16*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool fused_attention_supported(int64_t seq, int64_t head_dim) { return head_dim == kD && seq >= 1 && seq <= kMaxKeys; }

pd_status launch_fused_attention(const __nv_bfloat16* qkv, __nv_bfloat16* ctx, int64_t batch, int64_t seq,
                                 int64_t heads, cudaStream_t s) {
  const int64_t hidden = heads * kD;
  CUtensorMap tq, tk, tv;
  if (!make_head_map(&tq, qkv, seq, heads, batch, hidden, kBlockQ) ||
      !make_head_map(&tk, qkv + hidden, seq, heads, batch, hidden, 256) ||
      !make_head_map(&tv, qkv + 2 * hidden, seq, heads, batch, hidden, 256))
    return PD_ERR_UNSUPPORTED;
  AttnParams p{};
  p.ctx = ctx;
  p.status = device_status_ptr();
  if (!p.status) return PD_ERR_CUDA;
  p.batch = (int)batch; p.seq = (int)seq; p.heads = (int)heads; p.hidden = (int)hidden;
  p.q_blocks = (int)((seq + kBlockQ - 1) / kBlockQ);
  p.k_blocks = (int)((seq + kBlockK - 1) / kBlockK);
  p.units_per_head = (p.q_blocks + kQBlocksPerUnit - 1) / kQBlocksPerUnit;
  const int64_t units = batch * heads * p.units_per_head;
  if (units > 0x7fffffff) return PD_ERR_BAD_SHAPE;
  p.num_units = (int)units;
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(attention_fwd_tcgen05_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         kSmemBytes);
    if (e != cudaSuccess) return record_cuda_error(e);
    attr_set = true;
  }
  const int grid = p.num_units < sm_count() ? p.num_units : sm_count();
  attention_fwd_tcgen05_kernel<<<grid, kThreads, kSmemBytes, s>>>(tq, tk, tv, p);
  return check_launch();
}

}  // namespace pd
