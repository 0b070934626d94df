// Fused multi-head attention for sequences of up to 512 keys, head dimension 64:
//
//   Ctx[b,h] = softmax(Q[b,h] K[b,h]^T / sqrt(64)) V[b,h]
//
// on the packed projection qkv[tokens, 3*hidden] = [Q | K | V].  Scores and
// probabilities never leave the SM.
//
// One persistent CTA of 544 threads per SM walks over work units of (batch,
// head, pair of 128-query blocks).  K and V of the head (up to 512 x 64 each)
// sit in shared memory in four chunks of 128 keys, each with its own full and
// empty barrier, so that the next unit's chunks stream in while the current
// unit is still working on the later ones; the query tiles are double
// buffered for the same reason.  The two query blocks ("slots") are in flight
// at the same time, and each slot works through the keys in blocks of 64 with
// two score buffers, two probability buffers and one output accumulator in
// tensor memory (all 512 columns), so that the tensor core, the exponential
// unit and the barrier round trips overlap, also across unit boundaries.
//
//   warp 16          : TMA producer (per unit: Q of each slot, then the K and V
//                      chunks in the order the previous unit releases them).
//                      Like the issuers below, the whole warp walks the loop
//                      and waits, so that its addresses and counters stay
//                      warp-uniform values, and one elected lane issues.
//   warps 8, 10      : score issuers, one warp per slot
//                      (see kScoreWarp0 below): for block g of
//                      64 keys S = Q K_g^T (128 x 64 x 64) into one of the slot's
//                      two score buffers, as soon as the softmax warps have
//                      read that buffer's previous contents.
//   warps 9, 11      : output issuers, one warp per slot: when the
//                      slot's softmax warps have published P_g,
//                      O += P_g V_g (128 x 64 x 64) into the slot's 64 output
//                      columns, P_g read from tensor memory as the A operand.
//                      (A single issuing thread for all four streams
//                      was the bottleneck: the per-product bookkeeping of one
//                      thread cost more than the products themselves.)
//   warps 0-3, 4-7   : softmax of slot 0 / slot 1, one thread per query row.
//                      The row keeps a reference exponent m (the maximum of its
//                      first 32 scores).  For each block it forms
//                      p = 2^(s * log2(e) / 8 - m) from the scores in tensor
//                      memory, adds them to the fp32 row sum l, releases the
//                      score buffer and writes P as bf16 into the probability
//                      buffer.  The block's sum shows whether any exponent
//                      exceeded 16 (p would
//                      still be far from overflow); only then is m raised, O and l rescaled
//                      by 2^(m_old - m_new) through a tensor-memory load / store
//                      round trip, and the block redone.  O / l is therefore the
//                      exact softmax for any finite input, and on ordinary
//                      inputs every score is read once.  At the end of the
//                      unit the row sums go to the epilogue warps through
//                      shared memory and the warp moves on to the next unit.
//   warps 12-15      : epilogue, one thread per query row and both slots in
//                      turn: when the unit's last product has landed, read the O
//                      row, divide by l, stage 64 bf16 values in shared memory,
//                      from where each warp's 32 rows go to Ctx with one TMA
//                      store; then release O to the next unit's products.
// Keys beyond the sequence length are zero-filled by TMA and masked out; query
// rows beyond it are computed and discarded.
// Every mbarrier wait is bounded (see mbar_wait): on expiry a code is recorded
// in the device status word, all roles drain, tensor memory is freed and the
// kernel returns.
#include "gemm_common.cuh"

namespace pd {
namespace {

using namespace sm100;

constexpr int kD = 64;            // head dimension
constexpr int kBlockQ = 128;      // queries per slot = TMEM lanes
constexpr int kBlockK = 64;       // keys per score block
constexpr int kMaxKeys = 512;
constexpr int kSlots = 2;         // query blocks in flight
constexpr int kThreads = 544;
constexpr int kSlotThreads = 128, kSlotWarps = kSlotThreads / 32;
// warps 0-7 softmax, 8-11 the four MMA-issuing warps, 12-15 epilogue, 16 the TMA producer (seventeen warps: 120 registers a thread).
// Every tcgen05.mma / tcgen05.commit issuing thread has a warp of its own: two lanes of one warp that reach the
// same tcgen05 instruction together, with different operands, do not get two independent operations (attention
// with peaked rows came out wrong that way whenever the two slots drifted apart).  The TMA producer issues no
// tcgen05 instruction and rides along as another lane of the first issuer's warp.
constexpr int kScoreWarp0 = 8, kOutputWarp0 = 9, kScoreWarp1 = 10, kOutputWarp1 = 11;
constexpr int kProducerWarp = 16;
constexpr int kEpilogueWarp0 = 12;  // warp w reads the tensor-memory lanes 32 * (w % 4) ... + 31
constexpr int kAllocWarp = kOutputWarp0;
static_assert(kEpilogueWarp0 % 4 == 0 && kProducerWarp == kEpilogueWarp0 + 4 && kThreads == 32 * (kProducerWarp + 1),
              "epilogue warps cover the four lane quarters; the producer warp comes last");

constexpr int kSmemK = kMaxKeys * kD * 2;        // 64 KiB
constexpr int kSmemV = kMaxKeys * kD * 2;        // 64 KiB
constexpr int kSmemQ = kBlockQ * kD * 2;         // 16 KiB per query tile, two per slot
constexpr int kSmemO = kBlockQ * kD * 2;         // 16 KiB of output staging per slot
constexpr int kChunkKeys = 128;                  // K and V arrive, and are released, in chunks of 128 keys
constexpr int kChunks = kMaxKeys / kChunkKeys;
constexpr int kSmemChunk = kChunkKeys * kD * 2;  // 16 KiB
constexpr int kSmemL = kSlots * kBlockQ * 4;     // row sums handed from the softmax warps to the epilogue warps
constexpr int kSmemCtrl = 1024;
constexpr int kSmemBytes = kSmemK + kSmemV + kSlots * (2 * kSmemQ + kSmemO) + kSmemL + kSmemCtrl + 1024 /*alignment slack*/;

// tensor-memory columns: score buffer b of slot s at 128*s + 64*b, output accumulator of slot s at 256 + 64*s,
// probability buffer b of slot s (64 bf16 per row in 32 columns) at 384 + 64*s + 32*b
constexpr uint32_t kTmemS = 0, kTmemO = 256, kTmemP = 384, kTmemCols = 512;

constexpr float kScale = 0.125f * 1.4426950408889634f;  // 1/sqrt(64) * log2(e)
constexpr float kRescaleThreshold = 16.0f;               // largest exponent of 2 tolerated before m is raised
// Five sixteenths of the exponentials are evaluated on the FMA pipe (2^a = 2^round(a) * P(a - round(a)), P the
// degree-3 fit printed by fit_exp2_poly.py, relative error 7.5e-5, far below the bf16 rounding of the stored
// probability), the rest by the special-function unit, which alone would bound the softmax warps; the fastest
// share measured (1/8: 65.4 us, 1/4: 64.2, 5/16: 62.7, 3/8: 64.7 for batch 32 x 16 heads x 512, standalone).
// Bit k of the mask = 1: pair k of each group of sixteen pairs takes the polynomial.
constexpr uint32_t kPolyPairMask = 0xA888u;
constexpr float kExp2C0 = 9.999280572e-01f, kExp2C1 = 6.932609677e-01f, kExp2C2 = 2.426111251e-01f,
                kExp2C3 = 5.517166853e-02f;
constexpr float kExp2Magic = 12582912.0f;  // 1.5 * 2^23: adding it leaves round(a) in the low mantissa bits
constexpr float kRescaleSum = 65536.0f;                  // 2^16: a block sum at most this large has no such exponent

struct AttnParams {
  __nv_bfloat16* ctx;  // [batch*seq, hidden]
  int* status;
  int batch, seq, heads, hidden;
  int q_blocks;   // ceil(seq / 128)
  int k_blocks;   // ceil(seq / 64)
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
                             const __grid_constant__ CUtensorMap tmap_v, const __grid_constant__ CUtensorMap tmap_o,
                             const AttnParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t sK = smem_base, sV = sK + kSmemK, sQ = sV + kSmemV, sO = sQ + kSlots * 2 * kSmemQ;
  const uint32_t sL = sO + kSlots * kSmemO;
  const uint32_t bar_base = sL + kSmemL;
  // barriers (8 bytes each); [c] = chunk of 128 keys, [s] = slot, [s][b] = slot and buffer
  auto k_full = [&](int c) { return bar_base + 8u * c; };
  auto k_empty = [&](int c) { return bar_base + 32u + 8u * c; };
  auto v_full = [&](int c) { return bar_base + 64u + 8u * c; };
  auto v_empty = [&](int c) { return bar_base + 96u + 8u * c; };
  auto q_full = [&](int s, int b) { return bar_base + 128u + 8u * (2 * s + b); };
  auto q_empty = [&](int s, int b) { return bar_base + 160u + 8u * (2 * s + b); };
  auto o_full = [&](int s) { return bar_base + 192u + 8u * s; };
  auto o_empty = [&](int s) { return bar_base + 208u + 8u * s; };
  auto s_full = [&](int s, int b) { return bar_base + 224u + 8u * (2 * s + b); };
  auto s_empty = [&](int s, int b) { return bar_base + 256u + 8u * (2 * s + b); };
  auto p_full = [&](int s, int b) { return bar_base + 288u + 8u * (2 * s + b); };
  auto p_empty = [&](int s, int b) { return bar_base + 320u + 8u * (2 * s + b); };
  auto l_full = [&](int s) { return bar_base + 352u + 8u * s; };
  const uint32_t drain_bar = bar_base + 368;  // four of them, one per MMA-issuing thread
  uint8_t* ctrl = smem_gen + (bar_base - smem_base) + 512;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(ctrl);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(ctrl + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int c = 0; c < kChunks; ++c) {
      mbar_init(k_full(c), 1); mbar_init(v_full(c), 1); mbar_init(k_empty(c), kSlots); mbar_init(v_empty(c), kSlots);
    }
    for (int i = 0; i < 4; ++i) mbar_init(drain_bar + 8u * i, 1);
    for (int s = 0; s < kSlots; ++s) {
      mbar_init(o_full(s), 1); mbar_init(o_empty(s), kSlotWarps); mbar_init(l_full(s), kSlotWarps);
      for (int b = 0; b < 2; ++b) {
        mbar_init(q_full(s, b), 1); mbar_init(q_empty(s, b), 1);
        mbar_init(s_full(s, b), 1); mbar_init(s_empty(s, b), kSlotWarps);
        mbar_init(p_full(s, b), kSlotWarps); mbar_init(p_empty(s, b), 1);
      }
    }
    *abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async_smem();
  }
  if (warp == kAllocWarp) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
    tmem_relinquish_alloc_permit();
  }
  tcgen05_fence_before_sync();
  __syncthreads();
  tcgen05_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  // everything above is independent of other kernels' data; from here on global memory is touched
  griddep_wait();
  griddep_launch_dependents();

  // Work decomposition shared by all roles: unit -> (batch, head, first query block, active slots).
  auto unit_coords = [&](int unit, int& b, int& h, int& qb0, int& nslots) {
    const int per_bh = p.units_per_head;
    const int bh = unit / per_bh;
    // last sequence first: inside the layer the projection before this kernel wrote qkv first row first, and what it
    // wrote last is what is still in L2
    b = p.batch - 1 - bh / p.heads;
    h = bh % p.heads;
    qb0 = (unit % per_bh) * kSlots;
    nslots = min(kSlots, p.q_blocks - qb0);
  };
  const int G = p.k_blocks;
  const int NC = (G + 1) >> 1;  // chunks of 128 keys in use; chunk c holds score blocks 2c and 2c + 1

  if (warp == kProducerWarp) {
    // ------------------------------------------------------------- TMA producer
    // Per unit: the two query tiles (into the slot's other buffer, normally free long before), then the chunks
    // of K and V in the order in which the previous unit releases them.
    // The whole warp walks the loop and waits; one elected lane issues the copies.
    {
      if (lane == 0) { prefetch_tensormap(&tmap_q); prefetch_tensormap(&tmap_k); prefetch_tensormap(&tmap_v); }
      uint32_t n_unit = 0, n_q[kSlots] = {0, 0};
      uint32_t armed_k = 0, armed_v = 0;  // bit c: chunk c of the current unit has been requested
      bool ok = true;
      auto load_k = [&](int c, int h, int b) {
        if (c >= NC || !ok) return;
        if (!mbar_wait_warp(k_empty(c), (n_unit & 1u) ^ 1u, abort_flag, p.status, kTimeoutAttnProducer)) { ok = false; return; }
        if (elect_one()) {
          mbar_arrive_expect_tx(k_full(c), kSmemChunk);
          tma_load_4d(sK + c * kSmemChunk, &tmap_k, k_full(c), 0, c * kChunkKeys, h, b);
        }
        __syncwarp();
        armed_k |= 1u << c;
      };
      auto load_v = [&](int c, int h, int b) {
        if (c >= NC || !ok) return;
        if (!mbar_wait_warp(v_empty(c), (n_unit & 1u) ^ 1u, abort_flag, p.status, kTimeoutAttnProducer)) { ok = false; return; }
        if (elect_one()) {
          mbar_arrive_expect_tx(v_full(c), kSmemChunk);
          tma_load_4d(sV + c * kSmemChunk, &tmap_v, v_full(c), 0, c * kChunkKeys, h, b);
        }
        __syncwarp();
        armed_v |= 1u << c;
      };
      for (int unit = blockIdx.x; unit < p.num_units && ok; unit += gridDim.x, ++n_unit) {
        int b, h, qb0, nslots;
        unit_coords(unit, b, h, qb0, nslots);
        armed_k = armed_v = 0;
        for (int s = 0; s < nslots && ok; ++s) {
          const uint32_t qb = n_q[s] & 1u; const uint32_t qpar = ((n_q[s] >> 1) & 1u) ^ 1u;
          if (!mbar_wait_warp(q_empty(s, qb), qpar, abort_flag, p.status, kTimeoutAttnProducer)) { ok = false; break; }
          ++n_q[s];
          if (elect_one()) {
            mbar_arrive_expect_tx(q_full(s, qb), kSmemQ);
            tma_load_4d(sQ + (2 * s + qb) * kSmemQ, &tmap_q, q_full(s, qb), 0, (qb0 + s) * kBlockQ, h, b);
          }
          __syncwarp();
        }
        load_k(0, h, b); load_k(1, h, b); load_v(0, h, b); load_k(2, h, b); load_v(1, h, b); load_k(3, h, b);
        load_v(2, h, b); load_v(3, h, b);
        if (!ok) break;  // n_unit stays the index of the unit that was cut short
      }
      if (!ok) {
        // leave no copy in flight: give the latest request on every barrier a short time to land
        volatile int never = 0;
        for (int c = 0; c < NC; ++c) {
          if ((armed_k >> c) & 1u) mbar_wait(k_full(c), n_unit & 1u, &never, nullptr, 0, 20000000ull);
          else if (n_unit > 0) mbar_wait(k_full(c), (n_unit - 1u) & 1u, &never, nullptr, 0, 20000000ull);
          if ((armed_v >> c) & 1u) mbar_wait(v_full(c), n_unit & 1u, &never, nullptr, 0, 20000000ull);
          else if (n_unit > 0) mbar_wait(v_full(c), (n_unit - 1u) & 1u, &never, nullptr, 0, 20000000ull);
        }
        for (int s = 0; s < kSlots; ++s)
          for (uint32_t back = 1; back <= 2 && back <= n_q[s]; ++back) {
            const uint32_t i = n_q[s] - back;
            mbar_wait(q_full(s, i & 1u), (i >> 1) & 1u, &never, nullptr, 0, 20000000ull);
          }
      }
    }
  } else if (warp == kScoreWarp0 || warp == kScoreWarp1) {
    // ---------------------- score-product issuers: one warp per slot walks the loop, one elected lane issues
    {
      const int s = warp == kScoreWarp0 ? 0 : 1;
      constexpr uint32_t idesc_s = make_idesc_bf16(kBlockQ, kBlockK, false, false);  // Q K^T: both K-major
      const uint64_t k_desc = make_smem_desc(sK, 0, 1024);
      const uint32_t d_tmem = tmem_base + kTmemS + s * 128;
      uint32_t t = 0, n_q = 0, n_unit = 0;
      bool ok = true;
      for (int unit = blockIdx.x; unit < p.num_units && ok; unit += gridDim.x, ++n_unit) {
        int b, h, qb0, nslots;
        unit_coords(unit, b, h, qb0, nslots);
        const bool active = s < nslots;
        const uint32_t qb = n_q & 1u; const uint32_t qpar = (n_q >> 1) & 1u;
        uint64_t q_desc = 0;
        if (active) {
          if (!mbar_wait_warp(q_full(s, qb), qpar, abort_flag, p.status, kTimeoutAttnMma)) { ok = false; break; }
          ++n_q;
          q_desc = make_smem_desc(sQ + (2 * s + qb) * kSmemQ, 0, 1024);
        }
        for (int c = 0; c < NC && ok; ++c) {
          if (!mbar_wait_warp(k_full(c), n_unit & 1u, abort_flag, p.status, kTimeoutAttnMma)) { ok = false; break; }
          if (active) {
            for (int g = 2 * c; g < min(2 * c + 2, G); ++g, ++t) {
              const uint32_t buf = t & 1u;
              if (!mbar_wait_warp(s_empty(s, buf), ((t >> 1) & 1u) ^ 1u, abort_flag, p.status, kTimeoutAttnMma)) { ok = false; break; }
              tcgen05_fence_after_sync();
              const uint64_t kg = k_desc + (uint64_t)(g * ((kBlockK * 128) >> 4));
              if (elect_one()) {
#pragma unroll
                for (int ks = 0; ks < kD / 16; ++ks)
                  mma_bf16_ss(d_tmem + buf * kBlockK, q_desc + 2 * ks, kg + 2 * ks, idesc_s, ks != 0 ? 1u : 0u);
                mma_commit(s_full(s, buf));
              }
              __syncwarp();
            }
            if (!ok) break;
          }
          if (elect_one()) mma_commit(k_empty(c));  // both score issuers arrive, whether or not their slot is in use
          __syncwarp();
        }
        if (!ok) break;
        if (active && elect_one()) mma_commit(q_empty(s, qb));
        __syncwarp();
      }
      if (!ok) {
        if (lane == 0) mma_commit(drain_bar + 16u + 8u * s);
        __syncwarp();
        volatile int never = 0;
        mbar_wait(drain_bar + 16u + 8u * s, 0, &never, nullptr, 0, 20000000ull);
      }
    }
  } else if (warp == kOutputWarp0 || warp == kOutputWarp1) {
    // ------------------------ P V product issuers: one warp per slot walks the loop, one elected lane issues
    {
      const int s = warp == kOutputWarp0 ? 0 : 1;
      constexpr uint32_t idesc_o = make_idesc_bf16(kBlockQ, kD, false, true);  // V is MN-major
      const uint64_t v_desc = make_smem_desc(sV, 0, 1024);
      const uint32_t d_tmem = tmem_base + kTmemO + s * kD;
      uint32_t t = 0, n_us = 0, n_unit = 0;
      bool ok = true;
      for (int unit = blockIdx.x; unit < p.num_units && ok; unit += gridDim.x, ++n_unit) {
        int b, h, qb0, nslots;
        unit_coords(unit, b, h, qb0, nslots);
        const bool active = s < nslots;
        if (active) {
          // the previous unit's output of this slot must have been read before it is overwritten
          if (!mbar_wait_warp(o_empty(s), (n_us & 1u) ^ 1u, abort_flag, p.status, kTimeoutAttnMma)) { ok = false; break; }
        }
        for (int c = 0; c < NC && ok; ++c) {
          if (!mbar_wait_warp(v_full(c), n_unit & 1u, abort_flag, p.status, kTimeoutAttnMma)) { ok = false; break; }
          if (active) {
            for (int g = 2 * c; g < min(2 * c + 2, G); ++g, ++t) {
              const uint32_t buf = t & 1u;
              if (!mbar_wait_warp(p_full(s, buf), (t >> 1) & 1u, abort_flag, p.status, kTimeoutAttnMma)) { ok = false; break; }
              tcgen05_fence_after_sync();
              // P_g is the A operand straight from tensor memory: keys 2j, 2j + 1 of the block in column j
              const uint32_t pg = tmem_base + kTmemP + s * 64 + buf * 32;
              const uint64_t vg = v_desc + (uint64_t)(g * ((kBlockK * 128) >> 4));
              if (elect_one()) {
#pragma unroll
                for (int ks = 0; ks < kBlockK / 16; ++ks)
                  mma_bf16_ts(d_tmem, pg + 8 * ks, vg + ks * ((16 * 128) >> 4), idesc_o, (g | ks) != 0 ? 1u : 0u);
                mma_commit(p_empty(s, buf));
              }
              __syncwarp();
            }
            if (!ok) break;
          }
          if (elect_one()) mma_commit(v_empty(c));  // both output issuers arrive
          __syncwarp();
        }
        if (!ok) break;
        if (active) {
          if (elect_one()) mma_commit(o_full(s));
          __syncwarp();
          ++n_us;
        }
      }
      if (!ok) {
        if (lane == 0) mma_commit(drain_bar + 8u * s);
        __syncwarp();
        volatile int never = 0;
        mbar_wait(drain_bar + 8u * s, 0, &never, nullptr, 0, 20000000ull);
      }
    }
  } else if (warp < 2 * kSlotWarps) {
    // ------------------------------------------------------------------ softmax
    const int slot = warp >> 2, quarter = warp & 3;
    const int row = quarter * 32 + lane;  // query row within the block = TMEM lane
    const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
    const uint32_t t_o = t_lane + kTmemO + slot * kD;
    uint32_t t = 0, n_us = 0;  // score blocks and units this slot has processed
    bool ok = true;
    for (int unit = blockIdx.x; unit < p.num_units && ok; unit += gridDim.x) {
      int b, h, qb0, nslots;
      unit_coords(unit, b, h, qb0, nslots);
      if (slot >= nslots) continue;
      float mk = 0.f, l = 0.f;  // reference exponent (already scaled by log2(e)/8) and row sum
      for (int g = 0; g < G && ok; ++g, ++t) {
        const int buf = t & 1u;
        const uint32_t use_ph = (t >> 1) & 1u;
        const uint32_t t_s = t_lane + kTmemS + slot * 128 + buf * kBlockK;
        const uint32_t t_p = t_lane + kTmemP + slot * 64 + buf * 32;
        const int key0 = g * kBlockK;
        if (!mbar_wait(s_full(slot, buf), use_ph, abort_flag, p.status, kTimeoutAttnSoftmax)) { ok = false; break; }
        tcgen05_fence_after_sync();
        // exponentials of the block against reference `ref`: fills pk and returns the row's partial sum
        // (two fp32 values per instruction where the operation exists in packed form)
        uint32_t pk[kBlockK / 2];  // the block's probabilities, two bf16 per register
        // `first`: the unit's first block, which also fixes the row's reference exponent: the maximum of the first
        // 32 scores, taken from the registers the exponentials are about to use (no second pass over the block).
        // Any reference that is attained by some key keeps l >= 1; the check below covers the rest.
        auto exp_block = [&](float ref, bool first) {
          uint64_t part2[2] = {0, 0};
          float part = 0.f;
          const uint64_t scale2 = pack_f32x2(kScale, kScale);
          uint64_t nref2 = pack_f32x2(-ref, -ref);
          uint32_t r[2][32];
          tmem_ld_32x32b_x32(t_s, r[0]);
#pragma unroll
          for (int cc = 0; cc < kBlockK / 32; ++cc) {
            tmem_ld_wait();
            if (cc + 1 < kBlockK / 32) tmem_ld_32x32b_x32(t_s + (cc + 1) * 32, r[(cc & 1) ^ 1]);
            const uint32_t(&rr)[32] = r[cc & 1];
            const int c0 = key0 + cc * 32;
            if (first && cc == 0) {
              float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
              for (int i = 0; i < 32; ++i)
                if (c0 + i < p.seq) m4[i & 3] = fmaxf(m4[i & 3], __uint_as_float(rr[i]));
              ref = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3])) * kScale;
              mk = ref;
              nref2 = pack_f32x2(-ref, -ref);
            }
            if (c0 + 32 <= p.seq) {
#pragma unroll
              for (int i = 0; i < 32; i += 2) {
                float a0, a1, e0, e1;
                unpack_f32x2(fma_f32x2(pack_b32x2(rr[i], rr[i + 1]), scale2, nref2), a0, a1);
                if ((kPolyPairMask >> (i / 2)) & 1u) {
                  // exponents outside [-125, 127] would wrap the exponent field; 2^127 still trips the sum check
                  const uint64_t ac = pack_f32x2(fminf(fmaxf(a0, -125.0f), 127.0f), fminf(fmaxf(a1, -125.0f), 127.0f));
                  const uint64_t t2 = add_f32x2(ac, pack_f32x2(kExp2Magic, kExp2Magic));
                  const uint64_t n2 = add_f32x2(t2, pack_f32x2(-kExp2Magic, -kExp2Magic));
                  const uint64_t f2 = fma_f32x2(n2, pack_f32x2(-1.0f, -1.0f), ac);
                  uint64_t p2 = fma_f32x2(pack_f32x2(kExp2C3, kExp2C3), f2, pack_f32x2(kExp2C2, kExp2C2));
                  p2 = fma_f32x2(p2, f2, pack_f32x2(kExp2C1, kExp2C1));
                  p2 = fma_f32x2(p2, f2, pack_f32x2(kExp2C0, kExp2C0));
                  uint32_t tb0, tb1, pb0, pb1;
                  unpack_b32x2(t2, tb0, tb1);
                  unpack_b32x2(p2, pb0, pb1);
                  e0 = __uint_as_float(pb0 + (tb0 << 23));
                  e1 = __uint_as_float(pb1 + (tb1 << 23));
                } else {
                  e0 = ex2_approx(a0);
                  e1 = ex2_approx(a1);
                }
                part2[(i >> 1) & 1] = add_f32x2(part2[(i >> 1) & 1], pack_f32x2(e0, e1));
                pk[cc * 16 + i / 2] = pack_bf16x2(e0, e1);
              }
            } else {
#pragma unroll
              for (int i = 0; i < 32; i += 2) {
                const float a0 = fmaf(__uint_as_float(rr[i]), kScale, -ref);
                const float a1 = fmaf(__uint_as_float(rr[i + 1]), kScale, -ref);
                const float e0 = c0 + i < p.seq ? ex2_approx(a0) : 0.f;
                const float e1 = c0 + i + 1 < p.seq ? ex2_approx(a1) : 0.f;
                part += e0 + e1;
                pk[cc * 16 + i / 2] = pack_bf16x2(e0, e1);
              }
            }
          }
          float s0, s1;
          unpack_f32x2(add_f32x2(part2[0], part2[1]), s0, s1);
          return part + (s0 + s1);
        };
        // largest exponent of the block against reference `ref` (only the rare path below needs it)
        auto block_amax = [&](float ref) {
          float amax = -INFINITY;
#pragma unroll 1
          for (int cc = 0; cc < kBlockK / 32; ++cc) {
            uint32_t rr[32];
            tmem_ld_32x32b_x32(t_s + cc * 32, rr);
            tmem_ld_wait();
            const int c0 = key0 + cc * 32;
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (c0 + i < p.seq) amax = fmaxf(amax, fmaf(__uint_as_float(rr[i]), kScale, -ref));
          }
          return amax;
        };
        float part = exp_block(mk, g == 0);
        // A term above 2^16 shows in the sum, so the sum alone clears the ordinary case; !(<=) also catches NaN.
        if (__any_sync(0xffffffffu, !(part <= kRescaleSum))) {
          // rare: this block towers over the reference.  Raise the reference of the rows concerned, rescale
          // what they have accumulated, and redo the block.  Every earlier P V product of the slot has to
          // be complete before O is touched: the latest one is the other tile's (there is one when g >= 1).
          const float amax = block_amax(mk);
          const bool raise = amax > kRescaleThreshold;
          if (g > 0) {
            if (!mbar_wait(p_empty(slot, buf ^ 1), ((t - 1u) >> 1) & 1u, abort_flag, p.status, kTimeoutAttnSoftmax)) { ok = false; break; }
            tcgen05_fence_after_sync();
            const float alpha = raise ? ex2_approx(-amax) : 1.0f;
            l *= alpha;
#pragma unroll
            for (int c0 = 0; c0 < kD; c0 += 32) {
              uint32_t o[32];
              tmem_ld_32x32b_x32(t_o + c0, o);
              tmem_ld_wait();
#pragma unroll
              for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
              tmem_st_32x32b_x32(t_o + c0, o);
            }
            tmem_st_wait();
          }
          if (raise) mk += amax;
          part = exp_block(mk, false);
        }
        l += part;
        // the scores have been read for good: the buffer may take the block after next
        tcgen05_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(s_empty(slot, buf));
        // P_g (keys 2j, 2j + 1 in column j: the A operand of P V) goes to its own tensor-memory buffer once the
        // product that read the buffer's previous contents has completed
        if (!mbar_wait(p_empty(slot, buf), use_ph ^ 1u, abort_flag, p.status, kTimeoutAttnSoftmax)) { ok = false; break; }
        tcgen05_fence_after_sync();
        tmem_st_32x32b_x32(t_p, pk);
        tmem_st_wait();
        tcgen05_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(p_full(slot, buf));
      }
      if (!ok) break;
      // ---- the row sums go to the epilogue warps, which finish the unit while this warp starts the next one.
      // The epilogue releases O after it has read the slot's previous sums; with eight blocks a unit that
      // happened long ago, with one or two this wait is what keeps the hand-over in step.
      if (!mbar_wait(o_empty(slot), (n_us & 1u) ^ 1u, abort_flag, p.status, kTimeoutAttnSoftmax)) { ok = false; break; }
      ++n_us;
      st_shared_f32(sL + (uint32_t)(slot * kBlockQ + row) * 4u, l);
      __syncwarp();
      if (lane == 0) mbar_arrive(l_full(slot));
    }
  } else {
    // ----------------------------------------------------------------- epilogue
    // O / l -> bf16 -> the slot's staging tile -> one TMA store of 32 rows x 128 bytes per warp; rows beyond the
    // sequence are clipped by the tensor map.
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
    const uint32_t sw = (uint32_t)(lane & 7);
    uint32_t n_us[kSlots] = {0, 0};
    bool ok = true;
    for (int unit = blockIdx.x; unit < p.num_units && ok; unit += gridDim.x) {
      int b, h, qb0, nslots;
      unit_coords(unit, b, h, qb0, nslots);
      for (int slot = 0; slot < nslots; ++slot) {
        const uint32_t ph = n_us[slot] & 1u;
        ++n_us[slot];
        if (!mbar_wait(l_full(slot), ph, abort_flag, p.status, kTimeoutAttnSoftmax)) { ok = false; break; }
        const float inv = 1.0f / ld_shared_f32(sL + (uint32_t)(slot * kBlockQ + row) * 4u);
        if (!mbar_wait(o_full(slot), ph, abort_flag, p.status, kTimeoutAttnSoftmax)) { ok = false; break; }
        tcgen05_fence_after_sync();
        // this warp's previous stores must have read their staging rows
        if (lane == 0) tma_store_wait_read<0>();
        __syncwarp();
        const uint32_t t_o = t_lane + kTmemO + slot * kD;
        const uint32_t o_row = sO + slot * kSmemO + (uint32_t)row * 128u;
#pragma unroll
        for (int c0 = 0; c0 < kD; c0 += 32) {
          uint32_t r[32];
          tmem_ld_32x32b_x32(t_o + c0, r);
          tmem_ld_wait();
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            uint4 w;
            w.x = pack_bf16x2(__uint_as_float(r[8 * u]) * inv, __uint_as_float(r[8 * u + 1]) * inv);
            w.y = pack_bf16x2(__uint_as_float(r[8 * u + 2]) * inv, __uint_as_float(r[8 * u + 3]) * inv);
            w.z = pack_bf16x2(__uint_as_float(r[8 * u + 4]) * inv, __uint_as_float(r[8 * u + 5]) * inv);
            w.w = pack_bf16x2(__uint_as_float(r[8 * u + 6]) * inv, __uint_as_float(r[8 * u + 7]) * inv);
            st_shared_v4(o_row + (((uint32_t)(c0 / 8 + u) ^ sw) << 4), w);
          }
        }
        // O (and the row sums) have been read: the next unit's products may overwrite them
        tcgen05_fence_before_sync();
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(o_empty(slot));
          tma_store_4d(&tmap_o, sO + slot * kSmemO + (uint32_t)(quarter * 32) * 128u, 0,
                       (qb0 + slot) * kBlockQ + quarter * 32, h, b);
          tma_store_commit();
        }
      }
    }
    // shared memory must outlive every store that still reads it
    if (lane == 0) tma_store_wait_read<0>();
    __syncwarp();
  }

  // ------------------------------------------------------------------- teardown
  __syncwarp();
  tcgen05_fence_before_sync();
  __syncthreads();
  if (warp == kAllocWarp) {
    tcgen05_fence_after_sync();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// One of Q, K, V inside qkv[batch*seq, 3*hidden]: dims {64, seq, heads, batch}.
bool make_head_map(CUtensorMap* map, const __nv_bfloat16* base, int64_t seq, int64_t heads, int64_t batch,
                   int64_t hidden, int box_rows) {
  gemm::EncodeTiledFn fn = gemm::encode_tiled_fn();
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
      !make_head_map(&tk, qkv + hidden, seq, heads, batch, hidden, kChunkKeys) ||
      !make_head_map(&tv, qkv + 2 * hidden, seq, heads, batch, hidden, kChunkKeys))
    return PD_ERR_UNSUPPORTED;
  // Ctx[batch*seq, hidden] seen as {64, seq, heads, batch}; written in boxes of 32 rows x 64 columns
  CUtensorMap to;
  if (!gemm::make_map(&to, false, ctx, kD, seq, hidden, heads, kD, batch, seq * hidden, kD, 32)) return PD_ERR_UNSUPPORTED;
  AttnParams p{};
  p.ctx = ctx;
  p.status = device_status_ptr();
  if (!p.status) return PD_ERR_CUDA;
  p.batch = (int)batch; p.seq = (int)seq; p.heads = (int)heads; p.hidden = (int)hidden;
  p.q_blocks = (int)((seq + kBlockQ - 1) / kBlockQ);
  p.k_blocks = (int)((seq + kBlockK - 1) / kBlockK);  // blocks of 64 keys
  p.units_per_head = (p.q_blocks + kSlots - 1) / kSlots;
  const int64_t units = batch * heads * p.units_per_head;
  if (units > 0x7fffffff) return PD_ERR_BAD_SHAPE;
  p.num_units = (int)units;
  static PerDeviceFlag smem_allowed;  // one per kernel (template instantiation)
  if (pd_status st = allow_dynamic_smem(attention_fwd_tcgen05_kernel, kSmemBytes, smem_allowed); st != PD_OK) return st;
  const int grid = p.num_units < sm_count() ? p.num_units : sm_count();
  logf("attention batch %lld seq %lld heads %lld: fused kernel, %d work units on %d CTAs", (long long)batch, (long long)seq,
       (long long)heads, p.num_units, grid);
  launch_pdl(attention_fwd_tcgen05_kernel, dim3(grid), dim3(kThreads), kSmemBytes, s, tq, tk, tv, to, p);
  return check_launch();
}

}  // namespace pd
