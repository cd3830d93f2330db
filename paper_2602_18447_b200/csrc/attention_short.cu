// Extend-attention for short steps (at most 32 query rows per kv head: new tokens x heads in the group) over a cache
// kept in one of the two 8-bit formats. With so few rows the pass is bound by reading the cache, not by arithmetic, so the
// kernel is organised around bytes: every warp streams whole 16-key pages of one (step, kv head) from global memory
// with asynchronous copies, two or three pages in flight, widens the codes to fp16 in registers (exact: every 8-bit value is
// an fp16 value) and runs the two small products of the page on warp-level tensor-core instructions. There is no wait on
// another CTA and no spin: pieces of a long context leave partial results that a second kernel combines.
#include <cuda_fp16.h>

#include <type_traits>

#include "common.cuh"
#include "kernels.h"

namespace cs {

namespace {

constexpr int kShortThreads = 128;
constexpr int kShortWarps = 4;
constexpr int kPage = 16;
constexpr float kNegBig = -1.0e30f;

__device__ __forceinline__ void cp_async_16(void* smem_dst, const void* gmem_src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(smem_dst)), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
// D (16 x 8, fp32) += A (16 x 16, fp16, row) * B (16 x 8, fp16, col)
__device__ __forceinline__ void mma_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// Two 8-bit floats (4 exponent, 3 mantissa bits) -> two fp16, exactly.
__device__ __forceinline__ uint32_t e4m3x2_to_f16x2(uint16_t v) {
  uint32_t r;
  asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(r) : "h"(v));
  return r;
}
// Two codes of the 5-exponent-bit format -> two fp16: each code is the upper byte of its fp16. lo = true takes
// bytes 0, 1 of w, lo = false bytes 2, 3.
__device__ __forceinline__ uint32_t e5m2x2_to_f16x2(uint32_t w, bool lo) {
  uint32_t r;
  if (lo) asm("prmt.b32 %0, %1, %2, 0x1404;" : "=r"(r) : "r"(w), "r"(0u));
  else    asm("prmt.b32 %0, %1, %2, 0x3424;" : "=r"(r) : "r"(w), "r"(0u));
  return r;
}
// Codes -> fp16 pairs for either 8-bit format (E5M2 = false: 4 exponent / 3 mantissa bits).
template <bool E5M2>
__device__ __forceinline__ uint32_t widen2(uint32_t w, bool lo) {
  if (E5M2) return e5m2x2_to_f16x2(w, lo);
  return e4m3x2_to_f16x2(static_cast<uint16_t>(lo ? (w & 0xffffu) : (w >> 16)));
}
// 2^x for x <= 0 by the special-function unit alone; results below the normal range flush to zero, which is what a
// probability that small contributes anyway.
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_half2(float a, float b) {
  __half2 h = __floats2half2_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&h);
}

// Fragments are built straight from the codes, without a pass through shared memory in fp16:
//  - K page [16 keys][HD codes]. The score product sums over the head dimension, in any order, so the dimension
//    index is permuted to make every lane's operands contiguous: in each block of 32 dimensions lane q = lane % 4 owns
//    dimensions 8q .. 8q+7 (one 8-byte load = the B operands of two k-steps), and the query fragments use the same
//    permutation. The 16 keys are likewise assigned to the columns of the two 8-column score tiles so that lane q ends
//    up holding the probabilities of keys 4q .. 4q+3: tile 0 column c is key 4 (c / 2) + c % 2, tile 1 that plus 2.
//  - V page TRANSPOSED, [HD][16 keys codes] (the layout of the 8-bit pool's V planes): the B operand of
//    O += P V for output column d and keys 4q .. 4q+3 is one 4-byte load.
// Shared memory of one warp: kStages pages in flight (K codes, 16-byte chunks XOR-swizzled per key row; V^T codes).
// One 16-row tile of queries: 3 stages and 4 CTAs per SM; two tiles: 4 stages (the partial results need the room)
// and 2 CTAs per SM.
template <int HD, int MT>
struct ShortSmem {
  static constexpr int kStages = MT == 1 ? 3 : 4;
  static constexpr int kRawPage = kPage * HD;                  // bytes of one K or V page of one head
  static constexpr int kStage = 2 * kRawPage;
  static constexpr int kWarp = kStages * kStage;
  static constexpr int kQBytes = 16 * MT * HD * 2;
  static constexpr int kTotal = kQBytes + kShortWarps * kWarp;
  // reused after the loop: the step's own keys in fp16 (K [16][HD], V^T [HD][16]) in warp 0's stages, and the
  // warps' partial results [warp][16 MT rows][HD] fp32 (+ [warp][32][2] over the queries)
  static_assert(kWarp >= 2 * kPage * HD * 2, "own keys must fit in one warp's stages");
  static_assert(kShortWarps * kWarp >= kShortWarps * 16 * MT * HD * 4, "partial results must fit");
  static_assert(kQBytes >= kShortWarps * 32 * 2 * 4, "row statistics must fit over the queries");
};

// swizzle of the 16-byte chunks of a K row: distinct for the 8 keys one score tile reads at once
template <int HD>
__device__ __forceinline__ int k_swz(int key) { return (((key >> 2) << 1) | (key & 1)) & (HD / 16 - 1); }

// MT = number of 16-row tiles of query rows (1 or 2).
template <int HD, int MT, bool E5M2>
__global__ void __launch_bounds__(kShortThreads, MT == 1 ? 4 : 2)
attention_short_kernel(const AttnParams p, const uint8_t* __restrict__ pool_k, const uint8_t* __restrict__ pool_v,
                       const AttnItem* __restrict__ items) {
  constexpr int KS = HD / 16;        // k-steps of the score product
  constexpr int NT = HD / 8;         // 8-column tiles of the output
  constexpr int RAW = ShortSmem<HD, MT>::kRawPage;
  constexpr int STAGE = ShortSmem<HD, MT>::kStage;
  constexpr int kStages = ShortSmem<HD, MT>::kStages;
  extern __shared__ __align__(128) uint8_t smem[];
  pdl_launch_dependents();
  const AttnItem it = items[blockIdx.x];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, q = lane & 3;
  const int G = p.n_q_heads / p.n_kv_heads;
  const int R = it.n_new * G;                       // query rows in use (<= 16 MT)
  uint8_t* q_s = smem;
  uint8_t* my = smem + ShortSmem<HD, MT>::kQBytes + warp * ShortSmem<HD, MT>::kWarp;
  const int32_t* table = p.page_table + static_cast<size_t>(it.seq) * p.max_pages_per_seq;
  const size_t head_off = static_cast<size_t>(it.kv_head) * kPage * HD;
  const size_t page_stride = static_cast<size_t>(p.n_kv_heads) * kPage * HD;

  // cached pages of this warp: page_begin + warp, + 4, ...; the copies touch only the cache and the page table, which
  // no kernel of the pass writes, so the first ones go out before the wait on the previous kernel
  auto fetch = [&](int32_t id, int stage) {
    if (!debug_in_range(id >= 0 && id < p.num_pages, p.status)) id = 0;
    const uint8_t* gk = pool_k + static_cast<size_t>(id) * page_stride + head_off;
    const uint8_t* gv = pool_v + static_cast<size_t>(id) * page_stride + head_off;
    uint8_t* dst = my + stage * STAGE;
    for (int c = lane; c < RAW / 16; c += 32) {
      const int key = c / (HD / 16), ch = c % (HD / 16);
      cp_async_16(dst + key * HD + ((ch ^ k_swz<HD>(key)) << 4), gk + c * 16);
      cp_async_16(dst + RAW + c * 16, gv + c * 16);
    }
  };
  const int pg0 = it.tile_begin + warp;
  // page ids are read one round before the copies that need them, so that the look-up never stalls the stream
  int32_t ids[kStages];
#pragma unroll
  for (int st = 0; st < kStages; ++st)
    ids[st] = pg0 + st * kShortWarps < it.tile_end ? __ldg(table + pg0 + st * kShortWarps) : 0;
#pragma unroll
  for (int st = 0; st < kStages - 1; ++st) {
    if (pg0 + st * kShortWarps < it.tile_end) fetch(ids[st], st);
    cp_async_commit();
  }
  int32_t id_ahead = ids[kStages - 1];

  pdl_wait();

  // query rows (token t, head hq of the group) -> row t * G + hq, fp16 from the projection workspace
  for (int c = threadIdx.x; c < 16 * MT * (HD / 8); c += kShortThreads) {
    const int row = c / (HD / 8), ch = c % (HD / 8);
    uint4 v = make_uint4(0, 0, 0, 0);
    if (row < R) {
      const int t = row / G, hq = row % G;
      const uint16_t* src = p.qkv + static_cast<size_t>(it.tok0 + t) * p.n_qkv + (it.kv_head * G + hq) * HD + ch * 8;
      v = *reinterpret_cast<const uint4*>(src);
    }
    *reinterpret_cast<uint4*>(q_s + (row * HD + ch * 8) * 2) = v;
  }
  __syncthreads();

  // A fragments of the query rows, with the permuted dimension index, stay in registers:
  // k-step ks = 2 blk + j covers dimensions 32 blk + 8 q + 4 j + {0, 1} (a0, a1) and + {2, 3} (a2, a3)
  uint32_t qa[MT][KS][4];
#pragma unroll
  for (int mt = 0; mt < MT; ++mt)
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      const int dim = 32 * (ks >> 1) + 8 * q + 4 * (ks & 1);
      const uint8_t* r0 = q_s + ((mt * 16 + g) * HD + dim) * 2;
      const uint8_t* r1 = r0 + 8 * HD * 2;
      qa[mt][ks][0] = *reinterpret_cast<const uint32_t*>(r0);
      qa[mt][ks][1] = *reinterpret_cast<const uint32_t*>(r1);
      qa[mt][ks][2] = *reinterpret_cast<const uint32_t*>(r0 + 4);
      qa[mt][ks][3] = *reinterpret_cast<const uint32_t*>(r1 + 4);
    }

  float o[MT][NT][4];
  float m_run[MT][2], l_run[MT][2];
#pragma unroll
  for (int mt = 0; mt < MT; ++mt) {
    m_run[mt][0] = m_run[mt][1] = kNegBig;
    l_run[mt][0] = l_run[mt][1] = 0.f;
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) o[mt][nt][0] = o[mt][nt][1] = o[mt][nt][2] = o[mt][nt][3] = 0.f;
  }

  // One page of 16 keys. WIDE = false: kb = K codes (swizzled rows), vb = V^T codes. WIDE = true: the step's own keys
  // in fp16, kb = K [16][HD], vb = V^T [HD][16], both plain. key_limit: keys at or beyond it are masked; causal: the
  // page holds the step's keys key0 .. key0 + 15, and key j is visible to the rows of token t only when j <= t.
  auto process = [&](auto wide_tag, const uint8_t* kb, const uint8_t* vb, int key_limit, bool causal, int key0) {
    constexpr bool WIDE = decltype(wide_tag)::value;
    float s[MT][2][4];               // [row tile][score tile]
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) s[mt][nt][0] = s[mt][nt][1] = s[mt][nt][2] = s[mt][nt][3] = 0.f;
#pragma unroll
    for (int blk = 0; blk < KS / 2; ++blk)
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
        const int key = 4 * (g >> 1) + (g & 1) + 2 * nt;
        uint32_t b[2][2];
        if (WIDE) {
          const uint4 w = *reinterpret_cast<const uint4*>(kb + (key * HD + 32 * blk + 8 * q) * 2);
          b[0][0] = w.x; b[0][1] = w.y; b[1][0] = w.z; b[1][1] = w.w;
        } else {
          const int chunk = 2 * blk + (q >> 1);
          const uint2 w = *reinterpret_cast<const uint2*>(kb + key * HD + ((chunk ^ k_swz<HD>(key)) << 4) + (q & 1) * 8);
          b[0][0] = widen2<E5M2>(w.x, true);
          b[0][1] = widen2<E5M2>(w.x, false);
          b[1][0] = widen2<E5M2>(w.y, true);
          b[1][1] = widen2<E5M2>(w.y, false);
        }
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
          mma_16816(s[mt][nt], qa[mt][2 * blk], b[0][0], b[0][1]);
          mma_16816(s[mt][nt], qa[mt][2 * blk + 1], b[1][0], b[1][1]);
        }
      }
    uint32_t pa[MT][4];
    bool rescale = false;
    float corr[MT][2];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      float sc[2][4];
      const int r0 = mt * 16 + g;
#pragma unroll
      for (int nt = 0; nt < 2; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) sc[nt][e] = s[mt][nt][e] * p.scale_log2e;
      // Only the last page of the context and the step's own keys have anything to mask (a warp-uniform branch).
      // A masked score becomes kNegBig and its probability exp2(kNegBig - reference) = 0: the reference is finite,
      // because every page has a key that all rows see (a context page's first key; the step's first own key).
      if (causal || key_limit < kPage) {
#pragma unroll
        for (int nt = 0; nt < 2; ++nt)
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int key = 4 * q + (e & 1) + 2 * nt;
            const int row = r0 + (e >> 1) * 8;
            bool vis = key < key_limit;
            if (causal) vis = vis && key0 + key <= row / G;
            if (!vis) sc[nt][e] = kNegBig;
          }
      }
      float mx[2] = {fmaxf(fmaxf(sc[0][0], sc[0][1]), fmaxf(sc[1][0], sc[1][1])),
                     fmaxf(fmaxf(sc[0][2], sc[0][3]), fmaxf(sc[1][2], sc[1][3]))};
      float sum[2] = {0.f, 0.f};
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 1));
        mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 2));
        const float m_new = fmaxf(m_run[mt][h], mx[h]);
        corr[mt][h] = fast_exp2(m_run[mt][h] - m_new);
        rescale = rescale || (m_new != m_run[mt][h]);
        m_run[mt][h] = m_new;
      }
#pragma unroll
      for (int nt = 0; nt < 2; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float pe = fast_exp2(sc[nt][e] - m_run[mt][e >> 1]);
          sc[nt][e] = pe;
          sum[e >> 1] += pe;
        }
      // the sums stay per lane (a quarter of each row's keys) until the pages are done
#pragma unroll
      for (int h = 0; h < 2; ++h) l_run[mt][h] = l_run[mt][h] * corr[mt][h] + sum[h];
      pa[mt][0] = pack_half2(sc[0][0], sc[0][1]);
      pa[mt][1] = pack_half2(sc[0][2], sc[0][3]);
      pa[mt][2] = pack_half2(sc[1][0], sc[1][1]);
      pa[mt][3] = pack_half2(sc[1][2], sc[1][3]);
    }
    // the running maxima settle after a few pages: the accumulators are rescaled only when one of them moved
    if (__any_sync(0xffffffffu, rescale)) {
#pragma unroll
      for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
          for (int e = 0; e < 4; ++e) o[mt][nt][e] *= corr[mt][e >> 1];
    }
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      uint32_t b0, b1;
      if (WIDE) {
        const uint2 w = *reinterpret_cast<const uint2*>(vb + ((nt * 8 + g) * kPage + 4 * q) * 2);
        b0 = w.x; b1 = w.y;
      } else {
        const uint32_t w = *reinterpret_cast<const uint32_t*>(vb + (nt * 8 + g) * kPage + 4 * q);
        b0 = widen2<E5M2>(w, true);
        b1 = widen2<E5M2>(w, false);
      }
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) mma_16816(o[mt][nt], pa[mt], b0, b1);
    }
  };

  // ------------------------------------------------------------------ cached pages
  int i = 0;
  for (int pg = pg0; pg < it.tile_end; pg += kShortWarps, ++i) {
    cp_async_wait<kStages - 2>();
    __syncwarp();
    // the stage read in the previous round is free: request the page kStages - 1 rounds ahead
    const int ahead = pg + (kStages - 1) * kShortWarps;
    if (ahead < it.tile_end) fetch(id_ahead, (i + kStages - 1) % kStages);
    cp_async_commit();
    if (ahead + kShortWarps < it.tile_end) id_ahead = __ldg(table + ahead + kShortWarps);
    const uint8_t* st = my + (i % kStages) * STAGE;
    process(std::false_type{}, st, st + RAW, it.ctx - pg * kPage, false, 0);
  }
  cp_async_wait<0>();

  // ------------------------------------------------------------------ the step's own keys (last piece, warp 0)
  const bool last_piece = it.slot == it.slot0 + it.n_splits - 1;
  if (last_piece && warp == 0) {
    uint8_t* k_n = my;                       // [16 keys][HD] fp16
    uint8_t* v_n = my + kPage * HD * 2;      // [HD][16 keys] fp16
    for (int key0 = 0; key0 < it.n_new; key0 += kPage) {       // up to two pages of them (32 rows, one head per group)
      __syncwarp();
      for (int c = lane; c < kPage * (HD / 8); c += 32) {
        const int key = c / (HD / 8), ch = c % (HD / 8);
        uint4 kv4 = make_uint4(0, 0, 0, 0), vv4 = make_uint4(0, 0, 0, 0);
        if (key0 + key < it.n_new) {
          const uint16_t* row = p.qkv + static_cast<size_t>(it.tok0 + key0 + key) * p.n_qkv;
          kv4 = *reinterpret_cast<const uint4*>(row + (p.n_q_heads + it.kv_head) * HD + ch * 8);
          vv4 = *reinterpret_cast<const uint4*>(row + (p.n_q_heads + p.n_kv_heads + it.kv_head) * HD + ch * 8);
        }
        *reinterpret_cast<uint4*>(k_n + (key * HD + ch * 8) * 2) = kv4;
        const uint32_t vw[4] = {vv4.x, vv4.y, vv4.z, vv4.w};
#pragma unroll
        for (int j = 0; j < 8; ++j)
          *reinterpret_cast<uint16_t*>(v_n + ((ch * 8 + j) * kPage + key) * 2) =
              static_cast<uint16_t>(j & 1 ? vw[j >> 1] >> 16 : vw[j >> 1] & 0xffffu);
      }
      __syncwarp();
      process(std::true_type{}, k_n, v_n, it.n_new - key0, true, key0);
    }
  }
  __syncthreads();

#pragma unroll
  for (int mt = 0; mt < MT; ++mt)
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      l_run[mt][h] += __shfl_xor_sync(0xffffffffu, l_run[mt][h], 1);
      l_run[mt][h] += __shfl_xor_sync(0xffffffffu, l_run[mt][h], 2);
    }

  // ------------------------------------------------------------------ combine the four warps
  float* po = reinterpret_cast<float*>(smem + ShortSmem<HD, MT>::kQBytes);           // [warp][16 MT rows][HD]
  float* pml = reinterpret_cast<float*>(q_s);                                    // [warp][32 rows][2], over the queries
#pragma unroll
  for (int mt = 0; mt < MT; ++mt) {
    const int r0 = mt * 16 + g;
    if (q == 0) {
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        pml[(warp * 32 + r0 + h * 8) * 2] = m_run[mt][h];
        pml[(warp * 32 + r0 + h * 8) * 2 + 1] = l_run[mt][h];
      }
    }
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int e = 0; e < 4; ++e)
        po[(static_cast<size_t>(warp) * 16 * MT + r0 + (e >> 1) * 8) * HD + nt * 8 + 2 * q + (e & 1)] = o[mt][nt][e];
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < R * HD; idx += kShortThreads) {
    const int row = idx / HD, d = idx % HD;
    float M = kNegBig;
#pragma unroll
    for (int w = 0; w < kShortWarps; ++w) M = fmaxf(M, pml[(w * 32 + row) * 2]);
    float acc = 0.f, L = 0.f;
#pragma unroll
    for (int w = 0; w < kShortWarps; ++w) {
      const float f = exp2f(pml[(w * 32 + row) * 2] - M);
      acc += f * po[(static_cast<size_t>(w) * 16 * MT + row) * HD + d];
      L += f * pml[(w * 32 + row) * 2 + 1];
    }
    if (it.n_splits == 1) {
      const int t = row / G, hq = row % G;
      reinterpret_cast<__half*>(p.out)[static_cast<size_t>(it.tok0 + t) * (p.n_q_heads * HD) + (it.kv_head * G + hq) * HD + d] =
          __float2half_rn(acc / L);
    } else {
      p.part_o[(static_cast<size_t>(it.slot) * 32 + row) * HD + d] = acc;
      if (d == 0) {
        p.part_ml[(static_cast<size_t>(it.slot) * 32 + row) * 2] = M;
        p.part_ml[(static_cast<size_t>(it.slot) * 32 + row) * 2 + 1] = L;
      }
    }
  }
}

// Pieces of one (step, kv head) -> output. One CTA per work item; only the first piece of a cut range does anything.
template <int HD>
__global__ void attention_short_merge_kernel(const AttnParams p, const AttnItem* __restrict__ items) {
  pdl_launch_dependents();
  pdl_wait();
  const AttnItem it = items[blockIdx.x];
  if (it.n_splits <= 1 || it.slot != it.slot0) return;
  const int G = p.n_q_heads / p.n_kv_heads;
  const int R = it.n_new * G;
  for (int idx = threadIdx.x; idx < R * HD; idx += blockDim.x) {
    const int row = idx / HD, d = idx % HD;
    float M = kNegBig;
    for (int s = 0; s < it.n_splits; ++s) M = fmaxf(M, p.part_ml[(static_cast<size_t>(it.slot0 + s) * 32 + row) * 2]);
    float acc = 0.f, L = 0.f;
    for (int s = 0; s < it.n_splits; ++s) {
      const size_t base = static_cast<size_t>(it.slot0 + s) * 32 + row;
      const float f = exp2f(p.part_ml[base * 2] - M);
      acc += f * p.part_o[base * HD + d];
      L += f * p.part_ml[base * 2 + 1];
    }
    const int t = row / G, g = row % G;
    reinterpret_cast<__half*>(p.out)[static_cast<size_t>(it.tok0 + t) * (p.n_q_heads * HD) + (it.kv_head * G + g) * HD + d] =
        __float2half_rn(acc / L);
  }
}

template <int HD, int MT, bool E5M2>
cudaError_t launch_short(const AttnParams& p, const uint8_t* pool_k, const uint8_t* pool_v, const AttnItem* items,
                         int n_items, cudaStream_t s) {
  static std::atomic<uint64_t> smem_opted{0};
  if (cudaError_t e = opt_in_dynamic_smem(attention_short_kernel<HD, MT, E5M2>, ShortSmem<HD, MT>::kTotal, smem_opted);
      e != cudaSuccess)
    return e;
  cudaError_t le = launch_pdl(attention_short_kernel<HD, MT, E5M2>, dim3(n_items), dim3(kShortThreads), ShortSmem<HD, MT>::kTotal, s,
                              p, pool_k, pool_v, items);
  count_launch();
  return le != cudaSuccess ? le : cudaGetLastError();
}

}  // namespace

cudaError_t launch_attention_short(const AttnParams& p, const uint8_t* pool_k, const uint8_t* pool_v,
                                   const AttnItem* items, int n_items, int max_rows, bool any_split, bool e5m2,
                                   cudaStream_t s) {
  if (n_items <= 0) return cudaSuccess;
  if (max_rows < 1 || max_rows > 32 || (p.head_dim != 64 && p.head_dim != 128)) return cudaErrorInvalidValue;
  cudaError_t e;
#define CS_SHORT(HD_, MT_)                                                               \
  (e5m2 ? launch_short<HD_, MT_, true>(p, pool_k, pool_v, items, n_items, s)            \
        : launch_short<HD_, MT_, false>(p, pool_k, pool_v, items, n_items, s))
  if (p.head_dim == 128) e = max_rows <= 16 ? CS_SHORT(128, 1) : CS_SHORT(128, 2);
  else e = max_rows <= 16 ? CS_SHORT(64, 1) : CS_SHORT(64, 2);
#undef CS_SHORT
  if (e != cudaSuccess || !any_split) return e;
  if (p.head_dim == 128)
    e = launch_pdl(attention_short_merge_kernel<128>, dim3(n_items), dim3(128), 0, s, p, items);
  else
    e = launch_pdl(attention_short_merge_kernel<64>, dim3(n_items), dim3(128), 0, s, p, items);
  count_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace cs
