// Ragged-batch grouped-query extend-attention over the paged context cache, on the tcgen05 tensor cores.
//
// A CTA takes one AttnItem: the query rows of `ntok` consecutive new tokens of one step for the G query heads
// of one kv head (ntok = 128 / G, so at most 128 rows = the 128 lanes of the tensor memory; row = token * G +
// head-in-group), and a range of 128-key tiles. Context keys are all visible; the step's own keys are causal.
//
//   warp 0        TMA producer of Q (once) and of the K tiles, into a ring of K stages
//   warp 6        TMA producer of the V tiles, into a ring of V stages
//                 A cached tile is 8 pages, one 4D box per page, issued by 8 lanes at once (one thread issuing
//                 them in turn takes about three times as long); a tile of the step's own keys is one box from
//                 the qkv workspace. Every box lands as [8-key group][64-column half][8 keys][128 B] with the
//                 128-byte swizzle, which serves K as a K-major operand and V as an MN-major operand with
//                 uniform strides.
//   warp 1        one thread issues tcgen05.mma: S_j = Q K_j^T into one of three TMEM buffers (both operands from
//                 shared memory), O += P_j V_j with P_j read from TMEM. S_{j+2} is issued before P_j V_j, so the
//                 softmax never waits for the tensor core.
//   warps 2..5    softmax: one thread per query row reads its S row from TMEM, keeps the running reference
//                 maximum and the sum in registers and writes P_j (fp16) back into the columns S_j came from.
//
// The exponent reference of a row only moves when the row maximum has grown by more than 2^8 since it was
// last set; O (in TMEM) is rescaled only then, so in steady state nobody touches O but the tensor core.
// When the key range is only part of the sequence, the unnormalised O, the reference and the sum go to a
// partial slot; the CTA that finishes last among the pieces of one query tile (a counter per query tile,
// which that CTA sets back to zero) combines the slots and writes the output.
#include "kernels.h"

#include "common.cuh"

namespace cs {

namespace {

constexpr int kKTile = 128;
constexpr int kPage = 16;
constexpr int kPagesPerTile = kKTile / kPage;
constexpr int kAttnThreads = 224;
constexpr int kStages = 3;                  // K stages and, separately, V stages
constexpr float kRescaleThreshold = 8.0f;   // log2 units
constexpr int kMaxSplits = 32;
constexpr int kSBufs = 3;                   // S/P buffers in tensor memory

template <int HD>
struct AttnSmem {
  static constexpr int kHalves = HD / 64;
  static constexpr int kGroupBytes = kHalves * 1024;                   // 8 keys: [half][8 keys][128 B]
  static constexpr int kPageBytes = 2 * kGroupBytes;
  static constexpr int kTileBytes = kPagesPerTile * kPageBytes;        // 128 keys of K (or of V)
  static constexpr int kQBytes = kHalves * 128 * 128;                  // [half][128 rows][128 B]
  static constexpr int kQOff = 0;
  static constexpr int kKOff = kQBytes;
  static constexpr int kVOff = kKOff + kStages * kTileBytes;
  static constexpr int kBarOff = kVOff + kStages * kTileBytes;
  static constexpr int kUsed = kBarOff + 256 + 1024;                   // + slack for 1024-byte alignment
  // At least 116 KB so that two CTAs never share an SM: each allocates all 512 TMEM columns.
  static constexpr int kTotal = kUsed > 118784 ? kUsed : 118784;
  static constexpr uint32_t kTmemCols = 512;                           // S0, S1, S2 at 0, 128, 256; O [384,384+HD)
  static constexpr uint32_t kOCol = 384;
};

// Shared-memory descriptor, 128-byte swizzle: `lbo` = distance between 64-element blocks along the contiguous
// dimension (MN-major operands only), `sbo` = distance between 8-row groups.
__device__ __forceinline__ uint64_t smem_desc(uint32_t smem_addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4);
  d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3FFF) << 16;
  d |= static_cast<uint64_t>((sbo_bytes >> 4) & 0x3FFF) << 32;
  d |= static_cast<uint64_t>(1) << 46;
  d |= static_cast<uint64_t>(2) << 61;
  return d;
}
__host__ __device__ constexpr uint32_t idesc_f16(int m, int n, bool b_mn_major) {
  return (1u << 4) | (b_mn_major ? (1u << 16) : 0u) | (static_cast<uint32_t>(n >> 3) << 17) |
         (static_cast<uint32_t>(m >> 4) << 24);
}
// The thread that feeds the tensor core must not stall: even a wait on a barrier that is already complete costs a
// round trip of a few hundred cycles, in which the short queue of issued products runs dry. Both groups below
// therefore start with a non-blocking test of the barrier the NEXT group will need, issue their products and
// their two completion arrivals, and only then read the test's answer (true = that phase is complete).

// S = Q K^T for one 128-key tile: HD / 16 products with both operands in shared memory. The Q tile is
// [half][128 rows][128 B]; the K tile [8-key group][half][8 keys][128 B].
template <int HD>
__device__ __forceinline__ bool umma_qk_group(uint32_t tmem_s, uint64_t q_desc, uint64_t k_desc, uint32_t idesc,
                                              uint64_t* commit1, uint64_t* commit2, uint64_t* peek_bar,
                                              uint32_t peek_parity);
template <>
__device__ __forceinline__ bool umma_qk_group<128>(uint32_t tmem_s, uint64_t q_desc, uint64_t k_desc, uint32_t idesc,
                                                   uint64_t* commit1, uint64_t* commit2, uint64_t* peek_bar,
                                                   uint32_t peek_parity) {
  uint32_t ready;
  asm volatile(
      "{\n\t.reg .pred P;\n\t.reg .b64 da, db;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 P, [%1], %2;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%3], %4, %5, %6, 0;\n\t"
      "add.u64 da, %4, 2;\n\tadd.u64 db, %5, 2;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%3], da, db, %6, 1;\n\t"
      "add.u64 da, %4, 4;\n\tadd.u64 db, %5, 4;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%3], da, db, %6, 1;\n\t"
      "add.u64 da, %4, 6;\n\tadd.u64 db, %5, 6;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%3], da, db, %6, 1;\n\t"
      "add.u64 da, %4, 1024;\n\tadd.u64 db, %5, 64;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%3], da, db, %6, 1;\n\t"
      "add.u64 da, %4, 1026;\n\tadd.u64 db, %5, 66;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%3], da, db, %6, 1;\n\t"
      "add.u64 da, %4, 1028;\n\tadd.u64 db, %5, 68;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%3], da, db, %6, 1;\n\t"
      "add.u64 da, %4, 1030;\n\tadd.u64 db, %5, 70;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%3], da, db, %6, 1;\n\t"
      "tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%7];\n\t"
      "tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%8];\n\t"
      "selp.u32 %0, 1, 0, P;\n\t}"
      : "=r"(ready)
      : "r"(smem_u32(peek_bar)), "r"(peek_parity), "r"(tmem_s), "l"(q_desc), "l"(k_desc), "r"(idesc),
        "r"(smem_u32(commit1)), "r"(smem_u32(commit2))
      : "memory");
  return ready != 0;
}
template <>
__device__ __forceinline__ bool umma_qk_group<64>(uint32_t tmem_s, uint64_t q_desc, uint64_t k_desc, uint32_t idesc,
                                                  uint64_t* commit1, uint64_t* commit2, uint64_t* peek_bar,
                                                  uint32_t peek_parity) {
  uint32_t ready;
  asm volatile(
      "{\n\t.reg .pred P;\n\t.reg .b64 da, db;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 P, [%1], %2;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%3], %4, %5, %6, 0;\n\t"
      "add.u64 da, %4, 2;\n\tadd.u64 db, %5, 2;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%3], da, db, %6, 1;\n\t"
      "add.u64 da, %4, 4;\n\tadd.u64 db, %5, 4;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%3], da, db, %6, 1;\n\t"
      "add.u64 da, %4, 6;\n\tadd.u64 db, %5, 6;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%3], da, db, %6, 1;\n\t"
      "tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%7];\n\t"
      "tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%8];\n\t"
      "selp.u32 %0, 1, 0, P;\n\t}"
      : "=r"(ready)
      : "r"(smem_u32(peek_bar)), "r"(peek_parity), "r"(tmem_s), "l"(q_desc), "l"(k_desc), "r"(idesc),
        "r"(smem_u32(commit1)), "r"(smem_u32(commit2))
      : "memory");
  return ready != 0;
}

// O (+)= P V for one 128-key tile: eight products of 16 keys each. P comes from tensor memory (128 lanes x 16 fp16
// values per product, two per 32-bit column, so 8 columns per product); V from shared memory, one 16-key page per
// product.
template <int HD>
__device__ __forceinline__ bool umma_pv_group(uint32_t tmem_o, uint32_t tmem_p, uint64_t v_desc, uint32_t idesc,
                                              uint32_t accumulate_first, uint64_t* commit1, uint64_t* commit2,
                                              uint64_t* peek_bar, uint32_t peek_parity);
template <>
__device__ __forceinline__ bool umma_pv_group<128>(uint32_t tmem_o, uint32_t tmem_p, uint64_t v_desc, uint32_t idesc,
                                                   uint32_t accumulate_first, uint64_t* commit1, uint64_t* commit2,
                                                   uint64_t* peek_bar, uint32_t peek_parity) {
  uint32_t ready;
  asm volatile(
      "{\n\t.reg .pred P, Q;\n\t.reg .b64 db;\n\t.reg .b32 ta;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 P, [%1], %2;\n\t"
      "setp.ne.b32 Q, %7, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%3], [%4], %5, %6, Q;\n\t"
      "add.u32 ta, %4, 8;\n\tadd.u64 db, %5, 256;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%3], [ta], db, %6, 1;\n\t"
      "add.u32 ta, %4, 16;\n\tadd.u64 db, %5, 512;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%3], [ta], db, %6, 1;\n\t"
      "add.u32 ta, %4, 24;\n\tadd.u64 db, %5, 768;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%3], [ta], db, %6, 1;\n\t"
      "add.u32 ta, %4, 32;\n\tadd.u64 db, %5, 1024;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%3], [ta], db, %6, 1;\n\t"
      "add.u32 ta, %4, 40;\n\tadd.u64 db, %5, 1280;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%3], [ta], db, %6, 1;\n\t"
      "add.u32 ta, %4, 48;\n\tadd.u64 db, %5, 1536;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%3], [ta], db, %6, 1;\n\t"
      "add.u32 ta, %4, 56;\n\tadd.u64 db, %5, 1792;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%3], [ta], db, %6, 1;\n\t"
      "tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%8];\n\t"
      "tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%9];\n\t"
      "selp.u32 %0, 1, 0, P;\n\t}"
      : "=r"(ready)
      : "r"(smem_u32(peek_bar)), "r"(peek_parity), "r"(tmem_o), "r"(tmem_p), "l"(v_desc), "r"(idesc),
        "r"(accumulate_first), "r"(smem_u32(commit1)), "r"(smem_u32(commit2))
      : "memory");
  return ready != 0;
}
template <>
__device__ __forceinline__ bool umma_pv_group<64>(uint32_t tmem_o, uint32_t tmem_p, uint64_t v_desc, uint32_t idesc,
                                                  uint32_t accumulate_first, uint64_t* commit1, uint64_t* commit2,
                                                  uint64_t* peek_bar, uint32_t peek_parity) {
  uint32_t ready;
  asm volatile(
      "{\n\t.reg .pred P, Q;\n\t.reg .b64 db;\n\t.reg .b32 ta;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 P, [%1], %2;\n\t"
      "setp.ne.b32 Q, %7, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%3], [%4], %5, %6, Q;\n\t"
      "add.u32 ta, %4, 8;\n\tadd.u64 db, %5, 128;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%3], [ta], db, %6, 1;\n\t"
      "add.u32 ta, %4, 16;\n\tadd.u64 db, %5, 256;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%3], [ta], db, %6, 1;\n\t"
      "add.u32 ta, %4, 24;\n\tadd.u64 db, %5, 384;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%3], [ta], db, %6, 1;\n\t"
      "add.u32 ta, %4, 32;\n\tadd.u64 db, %5, 512;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%3], [ta], db, %6, 1;\n\t"
      "add.u32 ta, %4, 40;\n\tadd.u64 db, %5, 640;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%3], [ta], db, %6, 1;\n\t"
      "add.u32 ta, %4, 48;\n\tadd.u64 db, %5, 768;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%3], [ta], db, %6, 1;\n\t"
      "add.u32 ta, %4, 56;\n\tadd.u64 db, %5, 896;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%3], [ta], db, %6, 1;\n\t"
      "tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%8];\n\t"
      "tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%9];\n\t"
      "selp.u32 %0, 1, 0, P;\n\t}"
      : "=r"(ready)
      : "r"(smem_u32(peek_bar)), "r"(peek_parity), "r"(tmem_o), "r"(tmem_p), "l"(v_desc), "r"(idesc),
        "r"(accumulate_first), "r"(smem_u32(commit1)), "r"(smem_u32(commit2))
      : "memory");
  return ready != 0;
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
__device__ __forceinline__ void tmem_st_32x16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ void tma_load_3d(void* smem_dst, const CUtensorMap* m, uint64_t* bar, int x, int y, int z) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z)
      : "memory");
}
__device__ __forceinline__ void tma_load_4d(void* smem_dst, const CUtensorMap* m, uint64_t* bar, int x, int y, int z,
                                            int w) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z), "r"(w)
      : "memory");
}

struct Bars {
  uint64_t q_full;
  uint64_t k_full[kStages], k_empty[kStages];   // TMA landed / Q K^T of the tile complete
  uint64_t v_full[kStages], v_empty[kStages];   // TMA landed / P V of the tile complete
  uint64_t s_full[kSBufs];                      // Q K^T complete
  uint64_t p_full[kSBufs];                      // P written by the 4 softmax warps
  uint64_t pv_done[kSBufs];                     // P V complete
  uint32_t tmem_slot;
  uint32_t abort_flag;
  uint64_t merge_bar;                           // partial blocks of a round have landed (combining piece only)
  uint32_t is_last;
};

template <int HD>
__global__ void __launch_bounds__(kAttnThreads, 1)
attention_kernel(const AttnParams p, const __grid_constant__ CUtensorMap tm_pool,
                 const __grid_constant__ CUtensorMap tm_kv_new, const __grid_constant__ CUtensorMap tm_q3d,
                 const AttnItem* __restrict__ items) {
  using L = AttnSmem<HD>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  Bars* bars = reinterpret_cast<Bars*>(smem + L::kBarOff);
  volatile uint32_t* abort_flag = &bars->abort_flag;

  const AttnItem it = items[blockIdx.x];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tok0 = it.tok0, n_new = it.n_new, ctx = it.ctx;
  const int G = p.n_q_heads / p.n_kv_heads;
  const int ctx_tiles = (ctx + kKTile - 1) / kKTile;
  const int n_tiles = it.tile_end - it.tile_begin;

  if (threadIdx.x == 0) {
    mbar_init(&bars->q_full, 1);
    mbar_init(&bars->merge_bar, 1);
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&bars->k_full[s], 1);
      mbar_init(&bars->k_empty[s], 1);
      mbar_init(&bars->v_full[s], 1);
      mbar_init(&bars->v_empty[s], 1);
    }
    for (int b = 0; b < kSBufs; ++b) {
      mbar_init(&bars->s_full[b], 1);
      mbar_init(&bars->p_full[b], 4);
      mbar_init(&bars->pv_done[b], 1);
    }
    bars->abort_flag = 0;
    bars->is_last = 0;
    fence_barrier_init();
    tma_prefetch_desc(&tm_pool);
    tma_prefetch_desc(&tm_kv_new);
    tma_prefetch_desc(&tm_q3d);
  }
  if (warp == 1) {
    tmem_alloc(&bars->tmem_slot, L::kTmemCols);
    tmem_relinquish();
  }
  {
    // The Q box covers (128 / G) * G rows; the rest of the 128-row operand is zeroed so that its scores are finite.
    // A row keeps to its own 128 bytes under the swizzle.
    const int used_rows = (128 / G) * G;
    const int n16 = (128 - used_rows) * 8;
    for (int i = threadIdx.x; i < n16 * L::kHalves; i += kAttnThreads) {
      const int h = i / n16, r = i - h * n16;
      reinterpret_cast<uint4*>(smem + L::kQOff + h * 128 * 128 + used_rows * 128)[r] = make_uint4(0u, 0u, 0u, 0u);
    }
    fence_proxy_async();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem_slot;
  // Set-up overlapped the previous kernel's tail; q, k, v of the new tokens are needed from here on. The producer
  // warps wait a little later: the cached pages do not depend on the previous kernel, so they first send for the
  // cached tiles that fit their rings.
  pdl_launch_dependents();
  if (warp != 0 && warp != 6) pdl_wait();

  if (warp == 0 || warp == 6) {
    // ------------------------------------------------------------ TMA producers (whole warps): warp 0 K, warp 6 V
    const bool is_k = warp == 0;
    bool waited = false;
    auto dependency_wait = [&]() {
      if (waited) return;
      pdl_wait();
      waited = true;
      if (is_k && lane == 0) {
        mbar_arrive_expect_tx(&bars->q_full, L::kHalves * (128 / G) * G * 128);
#pragma unroll
        for (int h = 0; h < L::kHalves; ++h)
          tma_load_3d(smem + L::kQOff + h * 128 * 128, &tm_q3d, &bars->q_full, h * 64, it.kv_head * G, tok0 + it.q_tok0);
      }
    };
    const int32_t* pages = p.page_table + static_cast<size_t>(it.seq) * p.max_pages_per_seq;
    const int n_pages = (ctx + kPage - 1) / kPage;
    // Lane l < 8 fetches page l of a cached tile. Pages past the end of the context are replaced by the last
    // real page; their keys are masked.
    auto page_of = [&](int t) -> int {
      if (!(t < ctx_tiles && lane < kPagesPerTile)) return 0;
      const int id = __ldg(pages + min(t * kPagesPerTile + lane, n_pages - 1));
      return debug_in_range(id >= 0 && id < p.num_pages, p.status) ? id : 0;
    };
    // token rows of this item lie inside the batch, its key tiles inside its sequence, its tensor-memory buffers
    // inside the allocation
    if (lane == 0) {
      debug_in_range(tok0 >= 0 && n_new > 0 && tok0 + n_new <= p.n_rows && it.q_tok0 >= 0 && it.q_tok0 < n_new, p.status);
      debug_in_range(it.tile_begin >= 0 && it.tile_begin < it.tile_end &&
                     it.tile_end <= ctx_tiles + (n_new + kKTile - 1) / kKTile && n_pages <= p.max_pages_per_seq, p.status);
      debug_in_range(L::kOCol + HD <= L::kTmemCols && kSBufs * kKTile <= static_cast<int>(L::kOCol), p.status);
    }
    int page = page_of(it.tile_begin);
    // column of this kv head's K (or V) in the qkv workspace, in 64-column units
    const int col = (p.n_q_heads + (is_k ? 0 : p.n_kv_heads) + it.kv_head) * L::kHalves;
    const int group_base = is_k ? p.k_group_base : p.v_group_base;
    uint64_t* full = is_k ? bars->k_full : bars->v_full;
    uint64_t* empty = is_k ? bars->k_empty : bars->v_empty;
    uint8_t* ring = smem + (is_k ? L::kKOff : L::kVOff);
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;
    for (int t = it.tile_begin; t < it.tile_end; ++t) {
      // the first cached tiles, as many as the ring holds, go out before the previous kernel is known to be complete
      if (t >= ctx_tiles || t - it.tile_begin >= kStages) dependency_wait();
      const int next_page = page_of(t + 1 < it.tile_end ? t + 1 : t);
      const int group = ((page * p.n_kv_heads + it.kv_head) * kPage) >> 3;     // 8-row group within a K or V plane
      uint8_t* dst = ring + stage * L::kTileBytes;
      if (lane == 0) ok = mbar_wait(&empty[stage], phase ^ 1u, abort_flag, p.status);
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      if (lane == 0) mbar_arrive_expect_tx(&full[stage], L::kTileBytes);
      __syncwarp();
      if (t < ctx_tiles) {
        if (lane < kPagesPerTile) tma_load_4d(dst + lane * L::kPageBytes, &tm_pool, &full[stage], 0, 0, 0, group_base + group);
      } else if (lane == 0) {
        // Rows past the step's own tokens belong to the next step or to the zeroed tail of the workspace;
        // their keys are masked.
        tma_load_4d(dst, &tm_kv_new, &full[stage], 0, tok0 + (t - ctx_tiles) * kKTile, col, 0);
      }
      page = next_page;
      if (++stage == kStages) { stage = 0; phase ^= 1u; }
    }
    dependency_wait();
    // In a healthy run the MMA warp has waited for every copy before the CTA exits. After an abort, give
    // the copies still in flight time to land in shared memory before the CTA may go away.
    if (!ok)
      for (int i = 0; i < 64; ++i) __nanosleep(10000);
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t kIdescQK = idesc_f16(128, kKTile, false);
      constexpr uint32_t kIdescPV = idesc_f16(128, HD, true);
      const uint64_t q_desc = smem_desc(smem_u32(smem + L::kQOff), 16, 1024);
      const uint64_t k_desc0 = smem_desc(smem_u32(smem + L::kKOff), 16, L::kGroupBytes);
      const uint64_t v_desc0 = smem_desc(smem_u32(smem + L::kVOff), 1024, L::kGroupBytes);
      bool ok = mbar_wait(&bars->q_full, 0, abort_flag, p.status);
      int k_stage = 0, v_stage = 0;
      uint32_t k_phase = 0, v_phase = 0;
      bool k_ready = false, v_ready = false;
      // Issue order: S_0, S_1, then for every tile j: S_{j+2}, O += P_j V_j. With three S/P buffers S_{j+2} lands in the
      // buffer that P_{j-1} V_{j-1} (issued earlier, and executed in issue order) has read P from, while the softmax
      // works on S_j and S_{j+1} waits in the third: the softmax never waits for the tensor core.
      for (int j = -2; j < n_tiles && ok; ++j) {
        if (j + 2 < n_tiles) {
          const int b = (j + 2) % kSBufs;
          if (!k_ready && !mbar_wait(&bars->k_full[k_stage], k_phase, abort_flag, p.status)) { ok = false; break; }
          // next needed: V of tile j (or of tile 0)
          v_ready = umma_qk_group<HD>(tmem_base + b * kKTile, q_desc,
                                      k_desc0 + static_cast<uint64_t>(k_stage * (L::kTileBytes >> 4)), kIdescQK,
                                      &bars->s_full[b], &bars->k_empty[k_stage], &bars->v_full[v_stage], v_phase);
          if (++k_stage == kStages) { k_stage = 0; k_phase ^= 1u; }
          k_ready = false;
        }
        if (j >= 0) {
          const int b = j % kSBufs;
          const uint32_t use = static_cast<uint32_t>(j / kSBufs) & 1u;
          if ((!v_ready && !mbar_wait(&bars->v_full[v_stage], v_phase, abort_flag, p.status)) ||
              !mbar_wait(&bars->p_full[b], use, abort_flag, p.status)) { ok = false; break; }
          tc_fence_after();
          // next needed: K of tile j+3
          k_ready = umma_pv_group<HD>(tmem_base + L::kOCol, tmem_base + b * kKTile,
                                      v_desc0 + static_cast<uint64_t>(v_stage * (L::kTileBytes >> 4)), kIdescPV, j != 0,
                                      &bars->v_empty[v_stage], &bars->pv_done[b], &bars->k_full[k_stage], k_phase);
          if (++v_stage == kStages) { v_stage = 0; v_phase ^= 1u; }
          v_ready = false;
        }
      }
    }
  } else {
    // ------------------------------------------------------------ softmax: one thread per query row
    const int quad = warp & 3;
    const int row = quad * 32 + lane;
    const int ntok = 128 / G;
    const int p_local = row / G;
    const int g = row - p_local * G;
    const int pos = it.q_tok0 + p_local;            // new-token index of this row within the step
    const bool row_ok = (p_local < ntok) && (pos < n_new);
    const float sc = p.scale_log2e;
    const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(quad * 32) << 16);
    // Reference of the exponents, raw score units; -inf until the row meets a visible key. Unused rows of the tile
    // start at 0 so that they never ask for the first-sight maximum.
    float m_ref = row_ok ? -INFINITY : 0.f;
    float l = 0.f;
    bool ok = true;

    for (int j = 0; j < n_tiles; ++j) {
      const int t = it.tile_begin + j;
      const int b = j % kSBufs;
      const uint32_t use = static_cast<uint32_t>(j / kSBufs) & 1u;
      if (!mbar_wait(&bars->s_full[b], use, abort_flag, p.status)) { ok = false; break; }
      tc_fence_after();
      uint32_t s[4][32];
#pragma unroll
      for (int c = 0; c < 4; ++c) tmem_ld_32x32(t_lane + b * kKTile + c * 32, s[c]);
      tmem_ld_wait();

      // Number of visible keys of this tile for this row. The branch is taken by whole warps: the code after it
      // contains warp-wide tensor-memory stores.
      const int lim = (t < ctx_tiles) ? ctx - t * kKTile : pos + 1 - (t - ctx_tiles) * kKTile;
      if (__any_sync(0xffffffffu, lim < kKTile)) {
#pragma unroll
        for (int c = 0; c < 4; ++c)
#pragma unroll
          for (int e = 0; e < 32; ++e)
            if (c * 32 + e >= lim) s[c][e] = 0xff800000u;
      }
      // A row that has not seen a visible key yet takes the maximum of this tile as its reference.
      if (__any_sync(0xffffffffu, m_ref == -INFINITY)) {
        float mx4[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          float a = fmaxf(__uint_as_float(s[c][0]), __uint_as_float(s[c][1]));
#pragma unroll
          for (int e = 2; e < 32; e += 2)
            a = fmaxf(a, fmaxf(__uint_as_float(s[c][e]), __uint_as_float(s[c][e + 1])));
          mx4[c] = a;
        }
        const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
        if (m_ref == -INFINITY && row_ok) m_ref = mx;      // may stay -inf (no visible key in this tile either)
      }
      // One pass: exponentials against the standing reference, their sum, and the largest exponent met. P_j replaces
      // S_j in tensor memory: keys 2e, 2e+1 of this row share one 32-bit column.
      float ref = (m_ref == -INFINITY) ? 0.f : m_ref * sc;
      float xmax, tile_sum;
      auto exp_pass = [&]() {
        float xm4[4], sum4[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint32_t pk[16];
          float sa = 0.f, sb = 0.f, xa = -INFINITY, xb = -INFINITY;
#pragma unroll
          for (int e = 0; e < 16; ++e) {
            const float x0 = fmaf(__uint_as_float(s[c][2 * e]), sc, -ref);
            const float x1 = fmaf(__uint_as_float(s[c][2 * e + 1]), sc, -ref);
            xa = fmaxf(xa, x0);
            xb = fmaxf(xb, x1);
            const float a0 = fast_exp2(x0), a1 = fast_exp2(x1);
            sa += a0;
            sb += a1;
            pk[e] = pack_f16x2(a0, a1);
          }
          sum4[c] = sa + sb;
          xm4[c] = fmaxf(xa, xb);
          tmem_st_32x16(t_lane + b * kKTile + c * 16, pk);
        }
        xmax = fmaxf(fmaxf(xm4[0], xm4[1]), fmaxf(xm4[2], xm4[3]));
        tile_sum = (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
      };
      exp_pass();
      // The reference only moves when some exponent outgrew it by more than the threshold: then O (which holds the
      // tiles before this one, scaled to the old reference) and the running sum are rescaled, and P_j is redone.
      const bool grow = row_ok && xmax > kRescaleThreshold;
      if (__any_sync(0xffffffffu, grow)) {
        if (j > 0) {
          const int ib = (j - 1) % kSBufs;
          const uint32_t iuse = static_cast<uint32_t>((j - 1) / kSBufs) & 1u;
          if (!mbar_wait(&bars->pv_done[ib], iuse, abort_flag, p.status)) { ok = false; break; }
          tc_fence_after();
          const float alpha = grow ? fast_exp2(-xmax) : 1.0f;
#pragma unroll 1
          for (int c = 0; c < HD / 32; ++c) {
            uint32_t o[32];
            tmem_ld_32x32(t_lane + L::kOCol + c * 32, o);
            tmem_ld_wait();
#pragma unroll
            for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
            tmem_st_32x32(t_lane + L::kOCol + c * 32, o);
          }
          l *= alpha;
        }
        if (grow) {
          ref += xmax;
          m_ref = ref / sc;
        }
        exp_pass();
      }
      l += tile_sum;
      tmem_st_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->p_full[b]);
    }

    // ---- epilogue: O is final once P V of the last tile has completed
    if (ok) {
      const int ib = (n_tiles - 1) % kSBufs;
      const uint32_t iuse = static_cast<uint32_t>((n_tiles - 1) / kSBufs) & 1u;
      ok = mbar_wait(&bars->pv_done[ib], iuse, abort_flag, p.status);
    }
    const int q_dim = p.n_q_heads * HD;
    if (ok && it.n_splits <= 1) {
      tc_fence_after();
      const float inv = 1.f / l;
      uint16_t* dst = p.out + static_cast<size_t>(tok0 + pos) * q_dim + (it.kv_head * G + g) * HD;
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
    } else if (it.n_splits > 1) {
      // ---- piece of a split key range: store the partial result, then the last piece to arrive combines them
      // The partial O goes out as one bulk copy: every thread puts its row into the (now idle) K ring, 16-byte
      // chunk c of row r at chunk position c ^ (r & 7) so that the writes do not collide on the banks, and one
      // thread hands the [128][HD] block to the copy engine. The slot keeps that chunk order; the combining
      // step undoes it.
      uint8_t* stage = smem + L::kKOff;
      if (ok) {
        tc_fence_after();
#pragma unroll 1
        for (int c = 0; c < HD / 32; ++c) {
          uint32_t o[32];
          tmem_ld_32x32(t_lane + L::kOCol + c * 32, o);
          tmem_ld_wait();
#pragma unroll
          for (int e = 0; e < 8; ++e)
            *reinterpret_cast<uint4*>(stage + row * (HD * 4) + (((c * 8 + e) ^ (row & 7)) << 4)) =
                make_uint4(o[4 * e], o[4 * e + 1], o[4 * e + 2], o[4 * e + 3]);
        }
        __stcg(reinterpret_cast<float2*>(p.part_ml + (static_cast<size_t>(it.slot) * 128 + row) * 2), make_float2(m_ref, l));
        fence_proxy_async();
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (ok && warp == 2 && lane == 0) {
        asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                     ::"l"(p.part_o + static_cast<size_t>(it.slot) * 128 * HD), "r"(smem_u32(stage)), "r"(128 * HD * 4)
                     : "memory");
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
      }
      __threadfence();
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (warp == 2 && lane == 0) {
        // A piece that gave up still counts, so that the counter returns to zero; its slot is then stale and the
        // timeout is reported through the status word.
        const int seen = atomicAdd(p.counters + it.slot0, 1);
        if (seen == it.n_splits - 1) {
          p.counters[it.slot0] = 0;
          bars->is_last = 1;
        }
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (bars->is_last) {
        __threadfence();
        // Combine the pieces. Their partial O blocks are fetched into the idle K/V rings by bulk copies, as many
        // per round as fit, so that the whole round costs one trip to L2; then every thread combines its own row
        // from shared memory. (Reading the blocks from global memory a few rows at a time took ~15 k cycles.)
        constexpr int kBlockBytes = 128 * HD * 4;
        constexpr int kPerRound = (2 * kStages * L::kTileBytes) / kBlockBytes;
        float mmax = -INFINITY;
        for (int sp = 0; sp < it.n_splits; ++sp)
          mmax = fmaxf(mmax, __ldcg(p.part_ml + (static_cast<size_t>(it.slot0 + sp) * 128 + row) * 2));
        float acc[HD];
#pragma unroll
        for (int e = 0; e < HD; ++e) acc[e] = 0.f;
        float lsum = 0.f;
        uint32_t round = 0;
        for (int s0 = 0; s0 < it.n_splits && ok; s0 += kPerRound, ++round) {
          const int cnt = min(kPerRound, it.n_splits - s0);
          if (warp == 2 && lane == 0) {
            mbar_arrive_expect_tx(&bars->merge_bar, static_cast<uint32_t>(cnt) * kBlockBytes);
            for (int i = 0; i < cnt; ++i)
              asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                           ::"r"(smem_u32(stage + i * kBlockBytes)),
                             "l"(p.part_o + static_cast<size_t>(it.slot0 + s0 + i) * 128 * HD), "r"(kBlockBytes),
                             "r"(smem_u32(&bars->merge_bar))
                           : "memory");
          }
          if (!mbar_wait(&bars->merge_bar, round & 1u, abort_flag, p.status)) { ok = false; break; }
          for (int i = 0; i < cnt; ++i) {
            const float2 ml = __ldcg(reinterpret_cast<const float2*>(p.part_ml + (static_cast<size_t>(it.slot0 + s0 + i) * 128 + row) * 2));
            if (ml.x == -INFINITY) continue;
            const float w = fast_exp2((ml.x - mmax) * sc);
            lsum += w * ml.y;
            const uint8_t* src = stage + i * kBlockBytes + row * (HD * 4);
#pragma unroll
            for (int c = 0; c < HD / 4; ++c) {
              const float4 v = *reinterpret_cast<const float4*>(src + ((c ^ (row & 7)) << 4));
              acc[4 * c] += w * v.x; acc[4 * c + 1] += w * v.y; acc[4 * c + 2] += w * v.z; acc[4 * c + 3] += w * v.w;
            }
          }
          asm volatile("bar.sync 1, 128;" ::: "memory");     // the next round overwrites the blocks
        }
        if (ok && row_ok) {
          const float inv = 1.f / lsum;
          uint16_t* dst = p.out + static_cast<size_t>(tok0 + pos) * q_dim + (it.kv_head * G + g) * HD;
#pragma unroll
          for (int c = 0; c < HD / 8; ++c)
            *reinterpret_cast<uint4*>(dst + c * 8) = make_uint4(
                pack_f16x2(acc[8 * c] * inv, acc[8 * c + 1] * inv), pack_f16x2(acc[8 * c + 2] * inv, acc[8 * c + 3] * inv),
                pack_f16x2(acc[8 * c + 4] * inv, acc[8 * c + 5] * inv), pack_f16x2(acc[8 * c + 6] * inv, acc[8 * c + 7] * inv));
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, L::kTmemCols);
  }
}

template <int HD>
cudaError_t launch_hd(const AttnParams& p, const CUtensorMap& tm_pool, const CUtensorMap& tm_kv_new,
                      const CUtensorMap& tm_q3d, const AttnItem* items, int n_items, cudaStream_t s) {
  using L = AttnSmem<HD>;
  static std::atomic<uint64_t> smem_opted{0};
  if (cudaError_t e = opt_in_dynamic_smem(attention_kernel<HD>, L::kTotal, smem_opted); e != cudaSuccess) return e;
  cudaError_t le = launch_pdl(attention_kernel<HD>, dim3(n_items), dim3(kAttnThreads), L::kTotal, s, p, tm_pool, tm_kv_new, tm_q3d,
                              items);
  count_launch();
  return le != cudaSuccess ? le : cudaGetLastError();
}

}  // namespace

int attention_max_splits() { return kMaxSplits; }

cudaError_t launch_attention(const AttnParams& p, const CUtensorMap& tm_pool, const CUtensorMap& tm_kv_new,
                             const CUtensorMap& tm_q3d, const AttnItem* items, int n_items, cudaStream_t s) {
  if (n_items <= 0) return cudaSuccess;
  if (p.head_dim == 128) return launch_hd<128>(p, tm_pool, tm_kv_new, tm_q3d, items, n_items, s);
  if (p.head_dim == 64) return launch_hd<64>(p, tm_pool, tm_kv_new, tm_q3d, items, n_items, s);
  return cudaErrorInvalidValue;
}

}  // namespace cs
