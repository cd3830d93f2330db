// Ragged-batch grouped-query extend-attention over the paged context cache, on the tcgen05 tensor cores.
//
// A CTA takes one AttnItem: the query rows of `ntok` consecutive new tokens of one step for the G query heads
// of one kv head (ntok = 128 / G, so at most 128 rows = the 128 lanes of the tensor memory; row = token * G +
// head-in-group), and a range of 64-key tiles. Context keys are all visible; the step's own keys are causal.
//
//   warp 0        TMA producer: Q tile once (one 3D box per 64-column half), then K/V tiles through a ring of
//                 stages (one 16-row box per page and half; the cache is bf16, the step's own K/V are fp16)
//   warp 1        issues tcgen05.mma: S_j = Q K_j^T into one of two TMEM buffers, O += P_j V_j
//   warps 2..5    softmax: one thread per query row reads its S row from TMEM, keeps the running reference
//                 maximum and the sum in registers, writes P_j (fp16) to shared memory as the next A operand
//   warps 6..9    re-encode cached bf16 K/V tiles to fp16 in place (exact), so that both MMA operands are fp16
//
// The exponent reference of a row only moves when the row maximum has grown by more than 2^8 since it was
// last set; O (in TMEM) is rescaled only then, so in steady state nobody touches O but the tensor core.
// When the key range is part of the sequence only, the unnormalised O, the reference and the sum go to a
// partial slot and attention_merge_kernel combines the slots.
#include "kernels.h"

#include "common.cuh"

namespace cs {

namespace {

constexpr int kKTile = 64;
constexpr int kPage = 16;
constexpr int kPagesPerTile = kKTile / kPage;
constexpr int kAttnThreads = 320;
constexpr int kStages = 3;
constexpr float kRescaleThreshold = 8.0f;   // log2 units

template <int HD>
struct AttnSmem {
  static constexpr int kHalves = HD / 64;
  static constexpr int kBoxBytes = kPage * 128;                            // 16 rows x 128 bytes
  static constexpr int kQBytes = kHalves * 128 * 128;                      // [half][128 rows][128 B]
  static constexpr int kKBytes = kHalves * kPagesPerTile * kBoxBytes;      // [half][page][16 rows][128 B]
  static constexpr int kStageBytes = 2 * kKBytes;                          // K then V
  static constexpr int kPBytes = 128 * 128;                                // [128 rows][64 keys] fp16
  static constexpr int kQOff = 0;
  static constexpr int kKVOff = kQBytes;
  static constexpr int kPOff = kKVOff + kStages * kStageBytes;
  static constexpr int kBarOff = kPOff + 2 * kPBytes;
  static constexpr int kTotal = kBarOff + 256 + 1024;
  static constexpr uint32_t kTmemCols = 256;                               // S0, S1 (64 each), O (HD)
  static constexpr uint32_t kOCol = 128;
};

// tcgen05.mma, both operands in shared memory; same instruction as the GEMM's.
__device__ __forceinline__ uint64_t desc_mn128(uint32_t smem_addr, uint32_t lbo_bytes) {
  // MN-major operand (the contiguous dimension is N): 64-element x 8-row swizzle atoms of 1024 bytes;
  // leading offset = distance between the 64-element column blocks, stride offset = between 8-row groups.
  uint64_t d = 0;
  d |= static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4);
  d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3FFF) << 16;
  d |= static_cast<uint64_t>(1024 >> 4) << 32;
  d |= static_cast<uint64_t>(1) << 46;
  d |= static_cast<uint64_t>(2) << 61;
  return d;
}
__host__ __device__ constexpr uint32_t idesc_f16(int m, int n, bool b_mn_major) {
  return (1u << 4) | (b_mn_major ? (1u << 16) : 0u) | (static_cast<uint32_t>(n >> 3) << 17) |
         (static_cast<uint32_t>(m >> 4) << 24);
}

__device__ __forceinline__ void tmem_st_32x32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
        "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
        "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ void tma_load_3d(void* smem_dst, const CUtensorMap* m, uint64_t* bar, int x, int y, int z) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z)
      : "memory");
}

struct Bars {
  uint64_t q_full;
  uint64_t kv_tma[kStages];    // TMA landed
  uint64_t kv_ready[kStages];  // converted (4 converter warps)
  uint64_t kv_empty[kStages];  // P V of the tile complete
  uint64_t s_full[2];          // Q K^T complete
  uint64_t s_empty[2];         // S read out by the 4 softmax warps
  uint64_t p_full[2];          // P written by the 4 softmax warps
  uint64_t p_empty[2];         // P V complete
  uint32_t tmem_slot;
  uint32_t abort_flag;
};

template <int HD>
__global__ void __launch_bounds__(kAttnThreads, 1)
attention_kernel(const AttnParams p, const __grid_constant__ CUtensorMap tm_pool,
                 const __grid_constant__ CUtensorMap tm_qkv, const __grid_constant__ CUtensorMap tm_q3d,
                 const AttnItem* __restrict__ items) {
  using L = AttnSmem<HD>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  Bars* bars = reinterpret_cast<Bars*>(smem + L::kBarOff);
  volatile uint32_t* abort_flag = &bars->abort_flag;

  const AttnItem it = items[blockIdx.x];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tok0 = p.cu_new[it.step];
  const int n_new = p.cu_new[it.step + 1] - tok0;
  const int ctx = p.ctx_len[it.step];
  const int G = p.n_q_heads / p.n_kv_heads;
  const int ctx_tiles = (ctx + kKTile - 1) / kKTile;
  const int n_tiles = it.tile_end - it.tile_begin;

  if (threadIdx.x == 0) {
    mbar_init(&bars->q_full, 1);
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&bars->kv_tma[s], 1);
      mbar_init(&bars->kv_ready[s], 4);
      mbar_init(&bars->kv_empty[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&bars->s_full[b], 1);
      mbar_init(&bars->s_empty[b], 4);
      mbar_init(&bars->p_full[b], 4);
      mbar_init(&bars->p_empty[b], 1);
    }
    bars->abort_flag = 0;
    fence_barrier_init();
    tma_prefetch_desc(&tm_pool);
    tma_prefetch_desc(&tm_qkv);
    tma_prefetch_desc(&tm_q3d);
  }
  if (warp == 1) {
    tmem_alloc(&bars->tmem_slot, L::kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      mbar_arrive_expect_tx(&bars->q_full, L::kHalves * (128 / G) * G * 128);
#pragma unroll
      for (int h = 0; h < L::kHalves; ++h)
        tma_load_3d(smem + L::kQOff + h * 128 * 128, &tm_q3d, &bars->q_full, h * 64, it.kv_head * G, tok0 + it.q_tok0);
      const int32_t* pages = p.page_table + static_cast<size_t>(p.seq_id[it.step]) * p.max_pages_per_seq;
      const int n_pages = (ctx + kPage - 1) / kPage;
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int t = it.tile_begin; t < it.tile_end; ++t) {
        if (!mbar_wait(&bars->kv_empty[stage], phase ^ 1u, abort_flag, p.status)) { ok = false; break; }
        uint8_t* sk = smem + L::kKVOff + stage * L::kStageBytes;
        uint8_t* sv = sk + L::kKBytes;
        mbar_arrive_expect_tx(&bars->kv_tma[stage], L::kStageBytes);
        if (t < ctx_tiles) {
#pragma unroll
          for (int pg = 0; pg < kPagesPerTile; ++pg) {
            // Pages past the end of the context are replaced by the last real page; their keys are masked.
            const int pi = min(t * kPagesPerTile + pg, n_pages - 1);
            const int row = (pages[pi] * p.n_kv_heads + it.kv_head) * kPage;
#pragma unroll
            for (int h = 0; h < L::kHalves; ++h) {
              tma_load_2d(sk + (h * kPagesPerTile + pg) * L::kBoxBytes, &tm_pool, &bars->kv_tma[stage], h * 64, p.k_row_base + row);
              tma_load_2d(sv + (h * kPagesPerTile + pg) * L::kBoxBytes, &tm_pool, &bars->kv_tma[stage], h * 64, p.v_row_base + row);
            }
          }
        } else {
          const int row0 = tok0 + (t - ctx_tiles) * kKTile;
          const int kcol = (p.n_q_heads + it.kv_head) * HD;
          const int vcol = (p.n_q_heads + p.n_kv_heads + it.kv_head) * HD;
#pragma unroll
          for (int pg = 0; pg < kPagesPerTile; ++pg) {
#pragma unroll
            for (int h = 0; h < L::kHalves; ++h) {
              // Rows past the end of the batch are zero-filled by TMA; rows of the next step are masked.
              tma_load_2d(sk + (h * kPagesPerTile + pg) * L::kBoxBytes, &tm_qkv, &bars->kv_tma[stage], kcol + h * 64, row0 + pg * kPage);
              tma_load_2d(sv + (h * kPagesPerTile + pg) * L::kBoxBytes, &tm_qkv, &bars->kv_tma[stage], vcol + h * 64, row0 + pg * kPage);
            }
          }
        }
        if (++stage == kStages) { stage = 0; phase ^= 1u; }
      }
      if (!ok)
        for (int i = 0; i < 64; ++i) __nanosleep(10000);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t kIdescQK = idesc_f16(128, kKTile, false);
      constexpr uint32_t kIdescPV = idesc_f16(128, HD, true);
      const uint32_t q_addr = smem_u32(smem + L::kQOff);
      const uint32_t p_addr = smem_u32(smem + L::kPOff);
      bool ok = mbar_wait(&bars->q_full, 0, abort_flag, p.status);
      int stage = 0;                 // stage of tile j (for Q K^T)
      uint32_t kv_phase = 0;
      int pv_stage = 0;              // stage of tile j-1 (for P V)
      for (int j = 0; j <= n_tiles && ok; ++j) {
        if (j < n_tiles) {
          const int b = j & 1;
          const uint32_t use = static_cast<uint32_t>(j >> 1) & 1u;   // phase of this use of buffer b
          if (!mbar_wait(&bars->kv_tma[stage], kv_phase, abort_flag, p.status) ||
              !mbar_wait(&bars->kv_ready[stage], kv_phase, abort_flag, p.status) ||
              !mbar_wait(&bars->s_empty[b], use ^ 1u, abort_flag, p.status)) { ok = false; break; }
          tc_fence_after();
          const uint32_t k_addr = smem_u32(smem + L::kKVOff + stage * L::kStageBytes);
#pragma unroll
          for (int k = 0; k < HD / 16; ++k) {
            const uint64_t adesc = umma_desc_k128(q_addr + (k >> 2) * (128 * 128) + (k & 3) * 32);
            const uint64_t bdesc = umma_desc_k128(k_addr + (k >> 2) * (kPagesPerTile * L::kBoxBytes) + (k & 3) * 32);
            umma_f16(tmem_base + b * kKTile, adesc, bdesc, kIdescQK, k != 0);
          }
          umma_commit(&bars->s_full[b]);
          if (++stage == kStages) { stage = 0; kv_phase ^= 1u; }
        }
        if (j > 0) {
          const int i = j - 1, b = i & 1;
          const uint32_t use = static_cast<uint32_t>(i >> 1) & 1u;
          if (!mbar_wait(&bars->p_full[b], use, abort_flag, p.status)) { ok = false; break; }
          tc_fence_after();
          const uint32_t v_addr = smem_u32(smem + L::kKVOff + pv_stage * L::kStageBytes + L::kKBytes);
#pragma unroll
          for (int ks = 0; ks < kKTile / 16; ++ks) {
            const uint64_t adesc = umma_desc_k128(p_addr + b * L::kPBytes + ks * 32);
            const uint64_t bdesc = desc_mn128(v_addr + ks * L::kBoxBytes, kPagesPerTile * L::kBoxBytes);
            umma_f16(tmem_base + L::kOCol, adesc, bdesc, kIdescPV, (i | ks) != 0);
          }
          umma_commit(&bars->kv_empty[pv_stage]);
          umma_commit(&bars->p_empty[b]);
          if (++pv_stage == kStages) pv_stage = 0;
        }
      }
    }
  } else if (warp < 6) {
    // ------------------------------------------------------------ softmax: one thread per query row
    const int quad = warp & 3;
    const int row = quad * 32 + lane;
    const int ntok = 128 / G;
    const int p_local = row / G;
    const int pos = it.q_tok0 + p_local;            // new-token index of this row within the step
    const bool row_ok = (p_local < ntok) && (pos < n_new);
    const float sc = p.scale_log2e;
    const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(quad * 32) << 16);
    float m_ref = -INFINITY;   // raw score units
    float l = 0.f;
    bool ok = true;
    uint8_t* p_row_base = smem + L::kPOff + row * 128;

    for (int j = 0; j < n_tiles; ++j) {
      const int t = it.tile_begin + j;
      const int b = j & 1;
      const uint32_t use = static_cast<uint32_t>(j >> 1) & 1u;
      if (!mbar_wait(&bars->s_full[b], use, abort_flag, p.status)) { ok = false; break; }
      tc_fence_after();
      uint32_t s0[32], s1[32];
      tmem_ld_32x32(t_lane + b * kKTile, s0);
      tmem_ld_32x32(t_lane + b * kKTile + 32, s1);
      tmem_ld_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->s_empty[b]);

      // number of visible keys of this tile for this row
      int lim;
      if (t < ctx_tiles) lim = ctx - t * kKTile;
      else lim = pos + 1 - (t - ctx_tiles) * kKTile;
      float mx = -INFINITY;
#pragma unroll
      for (int c = 0; c < 32; ++c) {
        if (c >= lim) s0[c] = 0xff800000u;
        if (c + 32 >= lim) s1[c] = 0xff800000u;
        mx = fmaxf(mx, fmaxf(__uint_as_float(s0[c]), __uint_as_float(s1[c])));
      }
      // Move the reference only when the maximum has outgrown it by the threshold (or on first sight).
      const bool grow = (mx > -INFINITY) && (m_ref == -INFINITY || (mx - m_ref) * sc > kRescaleThreshold);
      if (__any_sync(0xffffffffu, grow && j > 0)) {
        // O holds tiles < j scaled to the old reference: wait for P V of tile j-1, then rescale in place.
        const int ib = (j - 1) & 1;
        const uint32_t iuse = static_cast<uint32_t>((j - 1) >> 1) & 1u;
        if (!mbar_wait(&bars->p_empty[ib], iuse, abort_flag, p.status)) { ok = false; break; }
        tc_fence_after();
        const float alpha = (grow && m_ref != -INFINITY) ? fast_exp2((m_ref - mx) * sc) : 1.0f;
#pragma unroll 1
        for (int c = 0; c < HD / 32; ++c) {
          uint32_t o[32];
          tmem_ld_32x32(t_lane + L::kOCol + c * 32, o);
          tmem_ld_wait();
#pragma unroll
          for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
          tmem_st_32x32(t_lane + L::kOCol + c * 32, o);
        }
        tmem_st_wait();
        tc_fence_before();
        l *= alpha;
      }
      if (grow) m_ref = mx;
      const float ref = (m_ref == -INFINITY) ? 0.f : m_ref * sc;
      uint32_t pk[32];
      float sum = 0.f;
#pragma unroll
      for (int c = 0; c < 16; ++c) {
        const float a0 = fast_exp2(fmaf(__uint_as_float(s0[2 * c]), sc, -ref));
        const float a1 = fast_exp2(fmaf(__uint_as_float(s0[2 * c + 1]), sc, -ref));
        const float b0 = fast_exp2(fmaf(__uint_as_float(s1[2 * c]), sc, -ref));
        const float b1 = fast_exp2(fmaf(__uint_as_float(s1[2 * c + 1]), sc, -ref));
        sum += (a0 + a1) + (b0 + b1);
        pk[c] = pack_f16x2(a0, a1);
        pk[16 + c] = pack_f16x2(b0, b1);
      }
      l += sum;
      // P buffer b is free once P V of tile j-2 has completed.
      if (!mbar_wait(&bars->p_empty[b], use ^ 1u, abort_flag, p.status)) { ok = false; break; }
      uint8_t* prow = p_row_base + b * L::kPBytes;
#pragma unroll
      for (int c = 0; c < 8; ++c)
        *reinterpret_cast<uint4*>(prow + ((c ^ (row & 7)) << 4)) = make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
      fence_proxy_async();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->p_full[b]);
    }

    // ---- epilogue: O is final once P V of the last tile has completed
    if (ok) {
      const int ib = (n_tiles - 1) & 1;
      const uint32_t iuse = static_cast<uint32_t>((n_tiles - 1) >> 1) & 1u;
      ok = mbar_wait(&bars->p_empty[ib], iuse, abort_flag, p.status);
    }
    if (ok) {
      tc_fence_after();
      const int g = row - p_local * G;
      if (it.slot < 0) {
        const float inv = 1.f / l;
        uint16_t* dst = p.out + static_cast<size_t>(tok0 + pos) * (p.n_q_heads * HD) + (it.kv_head * G + g) * HD;
#pragma unroll 1
        for (int c = 0; c < HD / 32; ++c) {
          uint32_t o[32];
          tmem_ld_32x32(t_lane + L::kOCol + c * 32, o);
          tmem_ld_wait();
          if (row_ok) {
#pragma unroll
            for (int e = 0; e < 4; ++e)
              *reinterpret_cast<uint4*>(dst + c * 32 + e * 8) = make_uint4(
                  pack_f16x2(__uint_as_float(o[8 * e]) * inv, __uint_as_float(o[8 * e + 1]) * inv),
                  pack_f16x2(__uint_as_float(o[8 * e + 2]) * inv, __uint_as_float(o[8 * e + 3]) * inv),
                  pack_f16x2(__uint_as_float(o[8 * e + 4]) * inv, __uint_as_float(o[8 * e + 5]) * inv),
                  pack_f16x2(__uint_as_float(o[8 * e + 6]) * inv, __uint_as_float(o[8 * e + 7]) * inv));
          }
        }
      } else {
        float* po = p.part_o + (static_cast<size_t>(it.slot) * 128 + row) * HD;
#pragma unroll 1
        for (int c = 0; c < HD / 32; ++c) {
          uint32_t o[32];
          tmem_ld_32x32(t_lane + L::kOCol + c * 32, o);
          tmem_ld_wait();
#pragma unroll
          for (int e = 0; e < 8; ++e)
            *reinterpret_cast<uint4*>(po + c * 32 + e * 4) = make_uint4(o[4 * e], o[4 * e + 1], o[4 * e + 2], o[4 * e + 3]);
        }
        *reinterpret_cast<float2*>(p.part_ml + (static_cast<size_t>(it.slot) * 128 + row) * 2) = make_float2(m_ref, l);
      }
    }
  } else {
    // ------------------------------------------------------------ bf16 -> fp16 re-encoding of cached tiles
    const int ct = threadIdx.x - 6 * 32;   // 0..127
    int stage = 0;
    uint32_t phase = 0;
    for (int t = it.tile_begin; t < it.tile_end; ++t) {
      if (!mbar_wait(&bars->kv_tma[stage], phase, abort_flag, p.status)) break;
      if (t < ctx_tiles) {
        uint4* tile = reinterpret_cast<uint4*>(smem + L::kKVOff + stage * L::kStageBytes);
#pragma unroll 4
        for (int i = ct; i < L::kStageBytes / 16; i += 128) {
          uint4 v = tile[i];
          v.x = bf16x2_to_f16x2(v.x); v.y = bf16x2_to_f16x2(v.y); v.z = bf16x2_to_f16x2(v.z); v.w = bf16x2_to_f16x2(v.w);
          tile[i] = v;
        }
        fence_proxy_async();
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->kv_ready[stage]);
      if (++stage == kStages) { stage = 0; phase ^= 1u; }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, L::kTmemCols);
  }
}

// One CTA per query tile that was split: thread per (row, 4 columns).
template <int HD>
__global__ void attention_merge_kernel(const AttnParams p, const AttnMerge* __restrict__ merges) {
  const AttnMerge mg = merges[blockIdx.x];
  const int tok0 = p.cu_new[mg.step];
  const int n_new = p.cu_new[mg.step + 1] - tok0;
  const int G = p.n_q_heads / p.n_kv_heads;
  const int ntok = 128 / G;
  const int q_dim = p.n_q_heads * HD;
  for (int i = threadIdx.x; i < 128 * (HD / 4); i += blockDim.x) {
    const int row = i / (HD / 4), c = (i - row * (HD / 4)) * 4;
    const int p_local = row / G;
    const int pos = mg.q_tok0 + p_local;
    if (p_local >= ntok || pos >= n_new) continue;
    float mmax = -INFINITY;
    for (int s = 0; s < mg.n_splits; ++s)
      mmax = fmaxf(mmax, p.part_ml[(static_cast<size_t>(mg.slot0 + s) * 128 + row) * 2]);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float l = 0.f;
    for (int s = 0; s < mg.n_splits; ++s) {
      const float2 ml = *reinterpret_cast<const float2*>(p.part_ml + (static_cast<size_t>(mg.slot0 + s) * 128 + row) * 2);
      const float w = (ml.x == -INFINITY) ? 0.f : fast_exp2((ml.x - mmax) * p.scale_log2e);
      const float4 v = *reinterpret_cast<const float4*>(p.part_o + (static_cast<size_t>(mg.slot0 + s) * 128 + row) * HD + c);
      if (w != 0.f) { acc.x += w * v.x; acc.y += w * v.y; acc.z += w * v.z; acc.w += w * v.w; }
      l += w * ml.y;
    }
    const float inv = 1.f / l;
    uint16_t* dst = p.out + static_cast<size_t>(tok0 + pos) * q_dim + (mg.kv_head * G + (row - p_local * G)) * HD + c;
    *reinterpret_cast<uint2*>(dst) = make_uint2(pack_f16x2(acc.x * inv, acc.y * inv), pack_f16x2(acc.z * inv, acc.w * inv));
  }
}

template <int HD>
cudaError_t launch_hd(const AttnParams& p, const CUtensorMap& tm_pool, const CUtensorMap& tm_qkv,
                      const CUtensorMap& tm_q3d, const AttnItem* items, int n_items, const AttnMerge* merges,
                      int n_merges, cudaStream_t s) {
  using L = AttnSmem<HD>;
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(attention_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kTotal);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  attention_kernel<HD><<<n_items, kAttnThreads, L::kTotal, s>>>(p, tm_pool, tm_qkv, tm_q3d, items);
  count_launch();
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  if (n_merges > 0) {
    attention_merge_kernel<HD><<<n_merges, 256, 0, s>>>(p, merges);
    count_launch();
    e = cudaGetLastError();
  }
  return e;
}

}  // namespace

cudaError_t launch_attention(const AttnParams& p, const CUtensorMap& tm_pool, const CUtensorMap& tm_qkv,
                             const CUtensorMap& tm_q3d, const AttnItem* items, int n_items, const AttnMerge* merges,
                             int n_merges, cudaStream_t s) {
  if (n_items <= 0) return cudaSuccess;
  if (p.head_dim == 128) return launch_hd<128>(p, tm_pool, tm_qkv, tm_q3d, items, n_items, merges, n_merges, s);
  if (p.head_dim == 64) return launch_hd<64>(p, tm_pool, tm_qkv, tm_q3d, items, n_items, merges, n_merges, s);
  return cudaErrorInvalidValue;
}

}  // namespace cs
