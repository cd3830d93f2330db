// Extend-attention for short steps (at most 32 query rows per kv head: new tokens x heads in the group) over a cache
// kept in the 8-bit format. With so few rows the pass is bound by reading the cache, not by arithmetic, so the
// kernel is organised around bytes: every warp streams whole 16-key pages of one (step, kv head) from global memory
// with asynchronous copies, two pages in flight, widens them to fp16 in shared memory (exact: every 8-bit value is an
// fp16 value) and runs the two small products of the page on warp-level tensor-core instructions. There is no wait on
// another CTA and no spin: pieces of a long context leave partial results that a second kernel combines.
#include <cuda_fp16.h>

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
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
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
__device__ __forceinline__ uint32_t pack_half2(float a, float b) {
  __half2 h = __floats2half2_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&h);
}

// Shared memory of one warp: two raw pages in flight (K and V codes), and the current page widened to fp16 in
// rows of HD halves whose 16-byte chunks are XOR-swizzled with the row, which keeps ldmatrix free of bank conflicts.
template <int HD>
struct WarpSmem {
  static constexpr int kRawPage = kPage * HD;          // bytes of one K or V page of one head, 8-bit
  static constexpr int kWidePage = kPage * HD * 2;     // the same as fp16
  static constexpr int kBytes = 2 * 2 * kRawPage + 2 * kWidePage;
};
template <int HD>
struct ShortSmem {
  static constexpr int kQBytes = 32 * HD * 2;
  static constexpr int kWarp = WarpSmem<HD>::kBytes;
  static constexpr int kTotal = kQBytes + kShortWarps * kWarp;
  // the combining step reuses the warps' buffers: [warp][32 rows][HD] fp32 + [warp][32][2]
  static_assert(kShortWarps * kWarp >= kShortWarps * 16 * HD * 4, "partial results of one row tile must fit");
};

__device__ __forceinline__ uint32_t swz(int row, int chunk) { return (static_cast<uint32_t>(chunk) ^ (row & 7)) << 4; }

// MT = number of 16-row tiles of query rows (1 or 2).
template <int HD, int MT>
__global__ void __launch_bounds__(kShortThreads, MT == 1 ? 3 : 2)
attention_short_kernel(const AttnParams p, const uint8_t* __restrict__ pool_k, const uint8_t* __restrict__ pool_v,
                       const AttnItem* __restrict__ items) {
  constexpr int KS = HD / 16;        // k-steps of the score product
  constexpr int NT = HD / 8;         // 8-column tiles of the output
  constexpr int RAW = WarpSmem<HD>::kRawPage;
  constexpr int WIDE = WarpSmem<HD>::kWidePage;
  constexpr int ROWB = HD * 2;       // bytes of one fp16 row
  extern __shared__ __align__(128) uint8_t smem[];
  pdl_launch_dependents();
  const AttnItem it = items[blockIdx.x];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = p.n_q_heads / p.n_kv_heads;
  const int R = it.n_new * G;                       // query rows in use (<= 16 MT)
  uint8_t* q_s = smem;
  uint8_t* my = smem + ShortSmem<HD>::kQBytes + warp * ShortSmem<HD>::kWarp;
  auto raw_of = [&](int stage) { return my + stage * 2 * RAW; };   // each stage: K codes then V codes
  uint8_t* k_w = my + 4 * RAW;
  uint8_t* v_w = k_w + WIDE;
  const int32_t* table = p.page_table + static_cast<size_t>(it.seq) * p.max_pages_per_seq;
  const size_t head_off = static_cast<size_t>(it.kv_head) * kPage * HD;
  const size_t page_stride = static_cast<size_t>(p.n_kv_heads) * kPage * HD;

  // cached pages of this warp: page_begin + warp, + 4, ...; the copies touch only the cache and the page table, which
  // no kernel of the pass writes, so the first two go out before the wait on the previous kernel
  auto fetch = [&](int pg, int stage) {
    const int32_t id = __ldg(table + pg);
    const uint8_t* gk = pool_k + static_cast<size_t>(id) * page_stride + head_off;
    const uint8_t* gv = pool_v + static_cast<size_t>(id) * page_stride + head_off;
    for (int c = lane; c < RAW / 16; c += 32) {
      cp_async_16(raw_of(stage) + c * 16, gk + c * 16);
      cp_async_16(raw_of(stage) + RAW + c * 16, gv + c * 16);
    }
  };
  int pg = it.tile_begin + warp;
  if (pg < it.tile_end) fetch(pg, 0);
  cp_async_commit();
  if (pg + kShortWarps < it.tile_end) fetch(pg + kShortWarps, 1);
  cp_async_commit();

  pdl_wait();

  // query rows (token t, head g of the group) -> row t * G + g, fp16 from the projection workspace
  for (int c = threadIdx.x; c < 32 * (HD / 8); c += kShortThreads) {
    const int row = c / (HD / 8), ch = c % (HD / 8);
    uint4 v = make_uint4(0, 0, 0, 0);
    if (row < R) {
      const int t = row / G, g = row % G;
      const uint16_t* src = p.qkv + static_cast<size_t>(it.tok0 + t) * p.n_qkv + (it.kv_head * G + g) * HD + ch * 8;
      v = *reinterpret_cast<const uint4*>(src);
    }
    *reinterpret_cast<uint4*>(q_s + row * ROWB + swz(row, ch)) = v;
  }
  __syncthreads();

  // A fragments of the query rows stay in registers
  uint32_t qa[MT][KS][4];
#pragma unroll
  for (int mt = 0; mt < MT; ++mt)
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      const int mat = lane >> 3;
      const int row = mt * 16 + (mat & 1) * 8 + (lane & 7);
      ldsm_x4(smem_u32(q_s + row * ROWB + swz(row, 2 * ks + (mat >> 1))), qa[mt][ks]);
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

  // One page of 16 keys, already widened into k_w / v_w. key_limit: keys at or beyond it are masked; causal: the
  // page holds the step's own keys key0 .. key0 + 15, and key j is visible to the rows of token t only when j <= t.
  auto process = [&](int key_limit, bool causal, int key0) {
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      float s[2][4];
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        uint32_t kb[4];
        const int mat = lane >> 3;
        const int key = (mat >> 1) * 8 + (lane & 7);
        ldsm_x4(smem_u32(k_w + key * ROWB + swz(key, 2 * ks + (mat & 1))), kb);
        mma_16816(s[0], qa[mt][ks], kb[0], kb[1]);
        mma_16816(s[1], qa[mt][ks], kb[2], kb[3]);
      }
      // mask, running maximum per row (rows lane/4 and lane/4 + 8 of the tile)
      const int r0 = mt * 16 + (lane >> 2);
#pragma unroll
      for (int nt = 0; nt < 2; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int key = nt * 8 + 2 * (lane & 3) + (e & 1);
          const int row = r0 + (e >> 1) * 8;
          bool vis = key < key_limit;
          if (causal) vis = vis && key0 + key <= row / G;
          s[nt][e] = vis ? s[nt][e] * p.scale_log2e : kNegBig;
        }
      float mx[2] = {fmaxf(fmaxf(s[0][0], s[0][1]), fmaxf(s[1][0], s[1][1])),
                     fmaxf(fmaxf(s[0][2], s[0][3]), fmaxf(s[1][2], s[1][3]))};
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 1));
        mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 2));
      }
      float corr[2], sum[2] = {0.f, 0.f};
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const float m_new = fmaxf(m_run[mt][h], mx[h]);
        corr[h] = exp2f(m_run[mt][h] - m_new);
        m_run[mt][h] = m_new;
      }
#pragma unroll
      for (int nt = 0; nt < 2; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          // a masked score stays at kNegBig; against a row that has seen nothing yet (m_new == kNegBig) it must
          // still contribute nothing
          const float pe = s[nt][e] <= 0.5f * kNegBig ? 0.f : exp2f(s[nt][e] - m_run[mt][e >> 1]);
          s[nt][e] = pe;
          sum[e >> 1] += pe;
        }
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        sum[h] += __shfl_xor_sync(0xffffffffu, sum[h], 1);
        sum[h] += __shfl_xor_sync(0xffffffffu, sum[h], 2);
        l_run[mt][h] = l_run[mt][h] * corr[h] + sum[h];
      }
      uint32_t pa[4] = {pack_half2(s[0][0], s[0][1]), pack_half2(s[0][2], s[0][3]), pack_half2(s[1][0], s[1][1]),
                        pack_half2(s[1][2], s[1][3])};
#pragma unroll
      for (int nt = 0; nt < NT; nt += 2) {
        uint32_t vb[4];
        const int mat = lane >> 3;
        const int key = (mat & 1) * 8 + (lane & 7);
        ldsm_x4_trans(smem_u32(v_w + key * ROWB + swz(key, nt + (mat >> 1))), vb);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          o[mt][nt][e] *= corr[e >> 1];
          o[mt][nt + 1][e] *= corr[e >> 1];
        }
        mma_16816(o[mt][nt], pa, vb[0], vb[1]);
        mma_16816(o[mt][nt + 1], pa, vb[2], vb[3]);
      }
    }
  };

  // ------------------------------------------------------------------ cached pages
  int stage = 0;
  for (; pg < it.tile_end; pg += kShortWarps) {
    cp_async_wait<1>();
    __syncwarp();
    // widen the page: a lane takes 16-byte pieces (16 codes) of K and of V and writes two swizzled chunks of halves
    const uint8_t* rk = raw_of(stage);
    for (int c = lane; c < 2 * RAW / 16; c += 32) {
      const bool is_v = c >= RAW / 16;
      const int cc = is_v ? c - RAW / 16 : c;
      const uint4 codes = *reinterpret_cast<const uint4*>(rk + (is_v ? RAW : 0) + cc * 16);
      const int key = cc / (HD / 16), ch = cc % (HD / 16);
      const uint32_t w[4] = {codes.x, codes.y, codes.z, codes.w};
      uint32_t h[8];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        h[2 * j] = e4m3x2_to_f16x2(static_cast<uint16_t>(w[j] & 0xffffu));
        h[2 * j + 1] = e4m3x2_to_f16x2(static_cast<uint16_t>(w[j] >> 16));
      }
      uint8_t* dst = (is_v ? v_w : k_w) + key * ROWB;
      *reinterpret_cast<uint4*>(dst + swz(key, 2 * ch)) = make_uint4(h[0], h[1], h[2], h[3]);
      *reinterpret_cast<uint4*>(dst + swz(key, 2 * ch + 1)) = make_uint4(h[4], h[5], h[6], h[7]);
    }
    __syncwarp();
    // the raw stage is free again: request the page after next
    if (pg + 2 * kShortWarps < it.tile_end) fetch(pg + 2 * kShortWarps, stage);
    cp_async_commit();
    process(it.ctx - pg * kPage, false, 0);
    __syncwarp();
    stage ^= 1;
  }
  cp_async_wait<0>();

  // ------------------------------------------------------------------ the step's own keys (last piece, warp 0)
  const bool last_piece = it.slot == it.slot0 + it.n_splits - 1;
  if (last_piece && warp == 0) {
    for (int key0 = 0; key0 < it.n_new; key0 += kPage) {       // up to two pages of them (32 rows, one head per group)
      __syncwarp();
      for (int c = lane; c < 2 * kPage * (HD / 8); c += 32) {
        const bool is_v = c >= kPage * (HD / 8);
        const int cc = is_v ? c - kPage * (HD / 8) : c;
        const int key = cc / (HD / 8), ch = cc % (HD / 8);
        uint4 v = make_uint4(0, 0, 0, 0);
        if (key0 + key < it.n_new) {
          const int col = (p.n_q_heads + (is_v ? p.n_kv_heads : 0) + it.kv_head) * HD + ch * 8;
          v = *reinterpret_cast<const uint4*>(p.qkv + static_cast<size_t>(it.tok0 + key0 + key) * p.n_qkv + col);
        }
        *reinterpret_cast<uint4*>((is_v ? v_w : k_w) + key * ROWB + swz(key, ch)) = v;
      }
      __syncwarp();
      process(it.n_new - key0, true, key0);
    }
  }
  __syncthreads();

  // ------------------------------------------------------------------ combine the four warps
  float* po = reinterpret_cast<float*>(smem + ShortSmem<HD>::kQBytes);           // [warp][16 MT rows][HD]
  float* pml = reinterpret_cast<float*>(q_s);                                    // [warp][32 rows][2], over the queries
#pragma unroll
  for (int mt = 0; mt < MT; ++mt) {
    const int r0 = mt * 16 + (lane >> 2);
    if ((lane & 3) == 0) {
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
        po[(static_cast<size_t>(warp) * 16 * MT + r0 + (e >> 1) * 8) * HD + nt * 8 + 2 * (lane & 3) + (e & 1)] = o[mt][nt][e];
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
      const int t = row / G, g = row % G;
      reinterpret_cast<__half*>(p.out)[static_cast<size_t>(it.tok0 + t) * (p.n_q_heads * HD) + (it.kv_head * G + g) * HD + d] =
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

template <int HD, int MT>
cudaError_t launch_short(const AttnParams& p, const uint8_t* pool_k, const uint8_t* pool_v, const AttnItem* items,
                         int n_items, cudaStream_t s) {
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(attention_short_kernel<HD, MT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         ShortSmem<HD>::kTotal);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  cudaError_t le = launch_pdl(attention_short_kernel<HD, MT>, dim3(n_items), dim3(kShortThreads), ShortSmem<HD>::kTotal, s,
                              p, pool_k, pool_v, items);
  count_launch();
  return le != cudaSuccess ? le : cudaGetLastError();
}

}  // namespace

cudaError_t launch_attention_short(const AttnParams& p, const uint8_t* pool_k, const uint8_t* pool_v,
                                   const AttnItem* items, int n_items, int max_rows, bool any_split, cudaStream_t s) {
  if (n_items <= 0) return cudaSuccess;
  if (max_rows < 1 || max_rows > 32 || (p.head_dim != 64 && p.head_dim != 128)) return cudaErrorInvalidValue;
  cudaError_t e;
  if (p.head_dim == 128)
    e = max_rows <= 16 ? launch_short<128, 1>(p, pool_k, pool_v, items, n_items, s)
                       : launch_short<128, 2>(p, pool_k, pool_v, items, n_items, s);
  else
    e = max_rows <= 16 ? launch_short<64, 1>(p, pool_k, pool_v, items, n_items, s)
                       : launch_short<64, 2>(p, pool_k, pool_v, items, n_items, s);
  if (e != cudaSuccess || !any_split) return e;
  if (p.head_dim == 128)
    e = launch_pdl(attention_short_merge_kernel<128>, dim3(n_items), dim3(128), 0, s, p, items);
  else
    e = launch_pdl(attention_short_merge_kernel<64>, dim3(n_items), dim3(128), 0, s, p, items);
  count_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace cs
