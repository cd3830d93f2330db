// Ragged-batch grouped-query extend-attention over the paged context cache.
//
// A CTA takes one AttnItem: 64 query rows (pairs (new position, head in group) of one step and kv head) and a
// range of 64-key tiles. A producer warp stages K and V tiles in shared memory with TMA (one 16-row x 64-column
// box per page and half head, 128-byte swizzle) through a ring of stages; four consumer warps (16 query rows
// each) run S = Q K^T and O += P V on the tensor cores with the running softmax kept in registers and the row
// maximum / sum exchanged by warp shuffles. Context keys are all visible; a step's own new keys are causal.
// When the key range is only part of the sequence the unnormalised result goes to a partial slot and a second
// kernel merges the slots.
#include "kernels.h"

#include "common.cuh"

namespace cs {

namespace {

constexpr int kQTile = 64;
constexpr int kKTile = 64;
constexpr int kPage = 16;
constexpr int kConsumerWarps = 4;
constexpr int kAttnThreads = (kConsumerWarps + 1) * 32;
constexpr int kAttnStages = 3;

template <int HD>
struct AttnSmem {
  static constexpr int kHalves = HD / 64;
  static constexpr int kBoxBytes = kPage * 128;                        // 16 rows x 128 bytes
  static constexpr int kTileBytes = (kKTile / kPage) * kHalves * kBoxBytes;  // K or V tile
  static constexpr int kStageBytes = 2 * kTileBytes;
  static constexpr int kTotal = kAttnStages * kStageBytes + 128 + 1024;
};

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void mma_f16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                        uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Byte offset, inside a K or V tile, of the 16-byte chunk holding elements [e, e+8) of key row `key`.
template <int HD>
__device__ __forceinline__ uint32_t tile_offset(int key, int e) {
  constexpr int kHalves = HD / 64;
  const int page = key >> 4, r = key & 15;
  const int half = e >> 6, chunk = (e & 63) >> 3;
  return static_cast<uint32_t>(((page * kHalves + half) * kPage + r) * 128 + ((chunk ^ (r & 7)) << 4));
}

template <int HD>
__global__ void __launch_bounds__(kAttnThreads)
attention_kernel(const AttnParams p, const __grid_constant__ CUtensorMap tm_pool,
                 const __grid_constant__ CUtensorMap tm_qkv, const AttnItem* __restrict__ items) {
  using L = AttnSmem<HD>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + kAttnStages * L::kStageBytes);
  uint64_t* empty_bar = full_bar + kAttnStages;
  volatile uint32_t* abort_flag = reinterpret_cast<uint32_t*>(empty_bar + kAttnStages);

  const AttnItem it = items[blockIdx.x];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tok0 = p.cu_new[it.step];
  const int n_new = p.cu_new[it.step + 1] - tok0;
  const int ctx = p.ctx_len[it.step];
  const int G = p.n_q_heads / p.n_kv_heads;
  const int ctx_tiles = (ctx + kKTile - 1) / kKTile;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kAttnStages; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], kConsumerWarps);
    }
    *abort_flag = 0;
    fence_barrier_init();
    tma_prefetch_desc(&tm_pool);
    tma_prefetch_desc(&tm_qkv);
  }
  __syncthreads();

  if (warp == kConsumerWarps) {
    // ------------------------------------------------------------ producer
    if (lane == 0) {
      const int32_t* pages = p.page_table + static_cast<size_t>(p.seq_id[it.step]) * p.max_pages_per_seq;
      const int n_pages = (ctx + kPage - 1) / kPage;
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int t = it.tile_begin; t < it.tile_end; ++t) {
        if (!mbar_wait(&empty_bar[stage], phase ^ 1u, abort_flag, p.status)) { ok = false; break; }
        uint8_t* sk = smem + stage * L::kStageBytes;
        uint8_t* sv = sk + L::kTileBytes;
        mbar_arrive_expect_tx(&full_bar[stage], L::kStageBytes);
        if (t < ctx_tiles) {
#pragma unroll
          for (int pg = 0; pg < kKTile / kPage; ++pg) {
            // Pages past the end of the context are replaced by the last real page; their keys are masked.
            const int pi = min(t * (kKTile / kPage) + pg, n_pages - 1);
            const int row = (pages[pi] * p.n_kv_heads + it.kv_head) * kPage;
#pragma unroll
            for (int h = 0; h < L::kHalves; ++h) {
              tma_load_2d(sk + (pg * L::kHalves + h) * L::kBoxBytes, &tm_pool, &full_bar[stage], h * 64, p.k_row_base + row);
              tma_load_2d(sv + (pg * L::kHalves + h) * L::kBoxBytes, &tm_pool, &full_bar[stage], h * 64, p.v_row_base + row);
            }
          }
        } else {
          const int row0 = tok0 + (t - ctx_tiles) * kKTile;
          const int kcol = (p.n_q_heads + it.kv_head) * HD;
          const int vcol = (p.n_q_heads + p.n_kv_heads + it.kv_head) * HD;
#pragma unroll
          for (int pg = 0; pg < kKTile / kPage; ++pg) {
#pragma unroll
            for (int h = 0; h < L::kHalves; ++h) {
              // Rows past the end of the batch are zero-filled by TMA; rows of the next step are masked.
              tma_load_2d(sk + (pg * L::kHalves + h) * L::kBoxBytes, &tm_qkv, &full_bar[stage], kcol + h * 64, row0 + pg * kPage);
              tma_load_2d(sv + (pg * L::kHalves + h) * L::kBoxBytes, &tm_qkv, &full_bar[stage], vcol + h * 64, row0 + pg * kPage);
            }
          }
        }
        if (++stage == kAttnStages) { stage = 0; phase ^= 1u; }
      }
      if (!ok)
        for (int i = 0; i < 64; ++i) __nanosleep(10000);
    }
    return;
  }

  // -------------------------------------------------------------- consumers
  const int g = lane >> 2, tq = lane & 3;
  const int rows_total = n_new * G;
  const int r_lo = it.q_row0 + warp * 16 + g;  // flattened query rows of this thread: r_lo and r_lo + 8
  const int r_hi = r_lo + 8;
  const int p_lo = r_lo / G, p_hi = r_hi / G;  // their new-token positions (causal bound on new keys)

  // Q fragments straight from global memory (A operand layout of m16n8k16).
  uint32_t qf[HD / 16][4];
  {
    const uint16_t* q_lo = p.qkv + static_cast<size_t>(tok0 + p_lo) * p.n_qkv + (it.kv_head * G + (r_lo - p_lo * G)) * HD;
    const uint16_t* q_hi = p.qkv + static_cast<size_t>(tok0 + p_hi) * p.n_qkv + (it.kv_head * G + (r_hi - p_hi * G)) * HD;
    const bool v_lo = r_lo < rows_total, v_hi = r_hi < rows_total;
#pragma unroll
    for (int ks = 0; ks < HD / 16; ++ks) {
      const int c = ks * 16 + 2 * tq;
      qf[ks][0] = v_lo ? *reinterpret_cast<const uint32_t*>(q_lo + c) : 0u;
      qf[ks][1] = v_hi ? *reinterpret_cast<const uint32_t*>(q_hi + c) : 0u;
      qf[ks][2] = v_lo ? *reinterpret_cast<const uint32_t*>(q_lo + c + 8) : 0u;
      qf[ks][3] = v_hi ? *reinterpret_cast<const uint32_t*>(q_hi + c + 8) : 0u;
    }
  }

  float o[HD / 8][4];
#pragma unroll
  for (int i = 0; i < HD / 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
  float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;
  const float sc = p.scale_log2e;

  int stage = 0;
  uint32_t phase = 0;
  bool ok = true;
  for (int t = it.tile_begin; t < it.tile_end; ++t) {
    if (!mbar_wait(&full_bar[stage], phase, abort_flag, p.status)) { ok = false; break; }
    const uint32_t sk = smem_u32(smem + stage * L::kStageBytes);
    const uint32_t sv = sk + L::kTileBytes;
    const bool cached = t < ctx_tiles;

    // S = Q K^T for 64 keys: 8 key groups of 8.
    float s[kKTile / 8][4];
#pragma unroll
    for (int nt = 0; nt < kKTile / 8; ++nt) {
      s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
      const int key = nt * 8 + (lane & 7);
#pragma unroll
      for (int j = 0; j < HD / 32; ++j) {
        uint32_t b0, b1, b2, b3;
        ldsm_x4(sk + tile_offset<HD>(key, j * 32 + (lane >> 3) * 8), b0, b1, b2, b3);
        if (cached) {  // cache pages hold bf16; the query and the step's own keys are fp16
          b0 = bf16x2_to_f16x2(b0); b1 = bf16x2_to_f16x2(b1); b2 = bf16x2_to_f16x2(b2); b3 = bf16x2_to_f16x2(b3);
        }
        mma_f16(s[nt], qf[2 * j][0], qf[2 * j][1], qf[2 * j][2], qf[2 * j][3], b0, b1);
        mma_f16(s[nt], qf[2 * j + 1][0], qf[2 * j + 1][1], qf[2 * j + 1][2], qf[2 * j + 1][3], b2, b3);
      }
    }

    // Visibility: context keys below ctx; new key j visible to new position p when j <= p.
    int lim_lo, lim_hi;  // number of visible keys of this tile for the two rows
    if (t < ctx_tiles) {
      lim_lo = lim_hi = ctx - t * kKTile;
    } else {
      const int j0 = (t - ctx_tiles) * kKTile;
      lim_lo = p_lo + 1 - j0;
      lim_hi = p_hi + 1 - j0;
    }
    float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
    for (int nt = 0; nt < kKTile / 8; ++nt) {
      const int c0 = nt * 8 + 2 * tq;
      if (c0 >= lim_lo) s[nt][0] = -INFINITY;
      if (c0 + 1 >= lim_lo) s[nt][1] = -INFINITY;
      if (c0 >= lim_hi) s[nt][2] = -INFINITY;
      if (c0 + 1 >= lim_hi) s[nt][3] = -INFINITY;
      mx_lo = fmaxf(mx_lo, fmaxf(s[nt][0], s[nt][1]));
      mx_hi = fmaxf(mx_hi, fmaxf(s[nt][2], s[nt][3]));
    }
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
    const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);
    // A row that has seen no key yet keeps max = -inf; use 0 as the reference so that exp2 gives 0, not NaN.
    const float ref_lo = (mn_lo == -INFINITY) ? 0.f : mn_lo * sc;
    const float ref_hi = (mn_hi == -INFINITY) ? 0.f : mn_hi * sc;
    const float al_lo = fast_exp2(m_lo * sc - ref_lo), al_hi = fast_exp2(m_hi * sc - ref_hi);
    m_lo = mn_lo;
    m_hi = mn_hi;
    l_lo *= al_lo;
    l_hi *= al_hi;
#pragma unroll
    for (int i = 0; i < HD / 8; ++i) {
      o[i][0] *= al_lo; o[i][1] *= al_lo; o[i][2] *= al_hi; o[i][3] *= al_hi;
    }
    uint32_t pf[kKTile / 16][4];  // P as A-operand fragments
#pragma unroll
    for (int nt = 0; nt < kKTile / 8; ++nt) {
      const float p0 = fast_exp2(fmaf(s[nt][0], sc, -ref_lo)), p1 = fast_exp2(fmaf(s[nt][1], sc, -ref_lo));
      const float p2 = fast_exp2(fmaf(s[nt][2], sc, -ref_hi)), p3 = fast_exp2(fmaf(s[nt][3], sc, -ref_hi));
      l_lo += p0 + p1;
      l_hi += p2 + p3;
      pf[nt >> 1][(nt & 1) * 2] = pack_f16x2(p0, p1);
      pf[nt >> 1][(nt & 1) * 2 + 1] = pack_f16x2(p2, p3);
    }

    // O += P V
#pragma unroll
    for (int ks = 0; ks < kKTile / 16; ++ks) {
      const int key = ks * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
      for (int np = 0; np < HD / 16; ++np) {
        uint32_t b0, b1, b2, b3;
        ldsm_x4_t(sv + tile_offset<HD>(key, np * 16 + (lane >> 4) * 8), b0, b1, b2, b3);
        if (cached) {
          b0 = bf16x2_to_f16x2(b0); b1 = bf16x2_to_f16x2(b1); b2 = bf16x2_to_f16x2(b2); b3 = bf16x2_to_f16x2(b3);
        }
        mma_f16(o[2 * np], pf[ks][0], pf[ks][1], pf[ks][2], pf[ks][3], b0, b1);
        mma_f16(o[2 * np + 1], pf[ks][0], pf[ks][1], pf[ks][2], pf[ks][3], b2, b3);
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&empty_bar[stage]);
    if (++stage == kAttnStages) { stage = 0; phase ^= 1u; }
  }
  if (!ok) return;

  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
  l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
  l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);

  if (it.slot < 0) {
    const float inv_lo = 1.f / l_lo, inv_hi = 1.f / l_hi;
    const int q_dim = p.n_q_heads * HD;
    if (r_lo < rows_total) {
      uint16_t* dst = p.out + static_cast<size_t>(tok0 + p_lo) * q_dim + (it.kv_head * G + (r_lo - p_lo * G)) * HD;
#pragma unroll
      for (int i = 0; i < HD / 8; ++i)
        *reinterpret_cast<uint32_t*>(dst + i * 8 + 2 * tq) = pack_f16x2(o[i][0] * inv_lo, o[i][1] * inv_lo);
    }
    if (r_hi < rows_total) {
      uint16_t* dst = p.out + static_cast<size_t>(tok0 + p_hi) * q_dim + (it.kv_head * G + (r_hi - p_hi * G)) * HD;
#pragma unroll
      for (int i = 0; i < HD / 8; ++i)
        *reinterpret_cast<uint32_t*>(dst + i * 8 + 2 * tq) = pack_f16x2(o[i][2] * inv_hi, o[i][3] * inv_hi);
    }
  } else {
    const int row_lo = warp * 16 + g, row_hi = row_lo + 8;
    float* po = p.part_o + static_cast<size_t>(it.slot) * kQTile * HD;
    float* pml = p.part_ml + static_cast<size_t>(it.slot) * kQTile * 2;
#pragma unroll
    for (int i = 0; i < HD / 8; ++i) {
      *reinterpret_cast<float2*>(po + row_lo * HD + i * 8 + 2 * tq) = make_float2(o[i][0], o[i][1]);
      *reinterpret_cast<float2*>(po + row_hi * HD + i * 8 + 2 * tq) = make_float2(o[i][2], o[i][3]);
    }
    if (tq == 0) {
      *reinterpret_cast<float2*>(pml + row_lo * 2) = make_float2(m_lo, l_lo);
      *reinterpret_cast<float2*>(pml + row_hi * 2) = make_float2(m_hi, l_hi);
    }
  }
}

// One CTA per query tile that was split: thread per (row, 4 columns).
template <int HD>
__global__ void attention_merge_kernel(const AttnParams p, const AttnMerge* __restrict__ merges) {
  const AttnMerge mg = merges[blockIdx.x];
  const int tok0 = p.cu_new[mg.step];
  const int n_new = p.cu_new[mg.step + 1] - tok0;
  const int G = p.n_q_heads / p.n_kv_heads;
  const int rows_total = n_new * G;
  const int q_dim = p.n_q_heads * HD;
  for (int i = threadIdx.x; i < kQTile * (HD / 4); i += blockDim.x) {
    const int row = i / (HD / 4), c = (i - row * (HD / 4)) * 4;
    const int r = mg.q_row0 + row;
    if (r >= rows_total) continue;
    float mmax = -INFINITY;
    for (int s = 0; s < mg.n_splits; ++s)
      mmax = fmaxf(mmax, p.part_ml[(static_cast<size_t>(mg.slot0 + s) * kQTile + row) * 2]);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float l = 0.f;
    for (int s = 0; s < mg.n_splits; ++s) {
      const float2 ml = *reinterpret_cast<const float2*>(p.part_ml + (static_cast<size_t>(mg.slot0 + s) * kQTile + row) * 2);
      const float w = (ml.x == -INFINITY) ? 0.f : fast_exp2((ml.x - mmax) * p.scale_log2e);
      const float4 v = *reinterpret_cast<const float4*>(p.part_o + (static_cast<size_t>(mg.slot0 + s) * kQTile + row) * HD + c);
      acc.x += w * v.x; acc.y += w * v.y; acc.z += w * v.z; acc.w += w * v.w;
      l += w * ml.y;
    }
    const float inv = 1.f / l;
    const int pos = r / G;
    uint16_t* dst = p.out + static_cast<size_t>(tok0 + pos) * q_dim + (mg.kv_head * G + (r - pos * G)) * HD + c;
    *reinterpret_cast<uint2*>(dst) = make_uint2(pack_f16x2(acc.x * inv, acc.y * inv), pack_f16x2(acc.z * inv, acc.w * inv));
  }
}

template <int HD>
cudaError_t launch_hd(const AttnParams& p, const CUtensorMap& tm_pool, const CUtensorMap& tm_qkv,
                      const AttnItem* items, int n_items, const AttnMerge* merges, int n_merges, cudaStream_t s) {
  using L = AttnSmem<HD>;
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(attention_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kTotal);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  attention_kernel<HD><<<n_items, kAttnThreads, L::kTotal, s>>>(p, tm_pool, tm_qkv, items);
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
                             const AttnItem* items, int n_items, const AttnMerge* merges, int n_merges,
                             cudaStream_t s) {
  if (n_items <= 0) return cudaSuccess;
  if (p.head_dim == 128) return launch_hd<128>(p, tm_pool, tm_qkv, items, n_items, merges, n_merges, s);
  if (p.head_dim == 64) return launch_hd<64>(p, tm_pool, tm_qkv, items, n_items, merges, n_merges, s);
  return cudaErrorInvalidValue;
}

}  // namespace cs
