// Projection GEMMs of the decoder layers: out = a[M,K] * w[N,K]^T, fp16 in, fp32 accumulate in TMEM.
//
// One persistent CTA per SM. Warp 0 feeds a ring of shared-memory stages with TMA (128-byte swizzle), warp 1
// issues tcgen05.mma into one of two TMEM accumulators, warps 2-5 drain the other accumulator (tcgen05.ld)
// and apply the epilogue, so the epilogue of one tile overlaps the main loop of the next.
//
// Work is measured in k-blocks (128 x BN x 64 products). Each CTA owns a contiguous range of k-blocks in the
// order (n tile, m tile, k); a range may start or end inside a tile. For the two epilogues that need the whole
// sum (fp16 store, SwiGLU) the ranges are whole tiles. For the residual epilogue (x += a * w^T, fp32) the
// range is cut evenly over the SMs whatever the tile boundaries are, and every piece is added into x by the copy
// engine (TMA reduce-add from a shared-memory box), which is what lets the narrow O and down projections fill all SMs.
// The pieces of one tile belong to consecutive CTAs. In the ordered mode they add in a fixed order - the piece with the
// highest k range first, which is also the one that finishes first - so that every element of x receives its pieces
// in the same order in every run and the result is bit-identical from run to run: a piece waits (bounded) for a word
// that the CTA holding the next k range of its tile sets once its own additions have been performed.
#include "gemm.h"

#include <algorithm>

#include "kernels.h"

#include "common.cuh"

namespace cs {

namespace {

constexpr int BM = 128;
constexpr int BK = 64;
constexpr int kGemmThreads = 192;
constexpr int kABytes = BM * BK * 2;
constexpr int kMaxOrderedPieces = 4;    // ordered residual epilogue: a tile's k range is cut into about this many pieces at most
constexpr int kShortK = 2048;           // residual projections with K up to this run on whole 128-wide tiles

template <int BN>
struct GemmSmem {
  static constexpr int kBBytes = BN * BK * 2;
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kStages = (BN == 256) ? 4 : 6;
  static constexpr int kBarBytes = 256;
  // Residual epilogue only: per epilogue warp two 32-row x 32-column fp32 boxes (4 KB each) from which the copy
  // engine adds into the output.
  static constexpr int kStagingBytes = 4 * 2 * 4096;
  static constexpr int kStagingOff = kStages * kStageBytes;
  static constexpr int kTotal = kStages * kStageBytes + kStagingBytes + kBarBytes + 1024;  // + slack for alignment
};

struct Segment {
  int tile, kb0, len;
};

// A CTA's range of k-blocks [start, end) as a sequence of segments. A range may begin inside a tile (a "head" piece
// up to that tile's end, or a "middle" piece if the whole range lies inside the tile) and may stop short of a tile's
// end (a "tail" piece, which begins at its tile's start). The pieces come first, the whole tiles after them: what other
// CTAs wait for (ordered residual epilogue) is finished early, and a CTA ends on a tile that it shares with nobody.
struct SegPlan {
  int start, kblocks, head_len, tail_len, whole0, n_whole, count;
};
__device__ __forceinline__ SegPlan make_plan(int start, int end, int kblocks) {
  SegPlan p;
  p.start = start;
  p.kblocks = kblocks;
  p.head_len = p.tail_len = p.n_whole = p.count = 0;
  p.whole0 = start;
  if (start >= end) return p;
  const int r = start % kblocks;
  if (r != 0) p.head_len = min(kblocks - r, end - start);
  p.whole0 = start + p.head_len;
  const int rem = end - p.whole0;
  p.n_whole = rem / kblocks;
  p.tail_len = rem - p.n_whole * kblocks;
  p.count = (p.head_len > 0) + (p.tail_len > 0) + p.n_whole;
  return p;
}
__device__ __forceinline__ Segment plan_segment(const SegPlan& p, int i) {
  Segment s;
  if (p.head_len > 0) {
    if (i == 0) {
      s.tile = p.start / p.kblocks;
      s.kb0 = p.start - s.tile * p.kblocks;
      s.len = p.head_len;
      return s;
    }
    --i;
  }
  if (p.tail_len > 0) {
    if (i == 0) {
      s.tile = p.whole0 / p.kblocks + p.n_whole;
      s.kb0 = 0;
      s.len = p.tail_len;
      return s;
    }
    --i;
  }
  s.tile = p.whole0 / p.kblocks + i;
  s.kb0 = 0;
  s.len = p.kblocks;
  return s;
}

// Order of the tiles. A CTA of the whole-tile epilogues (fp16 store, SwiGLU) takes consecutive tiles: with the column
// tile running fastest it keeps its rows of A and walks through the weights, and the CTAs that hold other rows walk
// through the same weights at the same time, so the weights stream from DRAM evenly over the whole launch (with the
// row tile fastest, every CTA wanted its share of the weights in its first tile and waited for DRAM there).
__device__ __forceinline__ int tile_m(int tile, int m_tiles, int n_tiles, int epi) {
  return epi == kEpiResidAdd ? tile % m_tiles : tile / n_tiles;
}
__device__ __forceinline__ int tile_n(int tile, int m_tiles, int n_tiles, int epi) {
  return epi == kEpiResidAdd ? tile / m_tiles : tile % n_tiles;
}

// out[tile] += shared-memory box, by the copy engine (element-wise fp32 atomics at L2, whole sectors at a time). The
// box is [32 rows][32 floats] with the 128-byte swizzle; rows and columns past the tensor's extent are dropped.
__device__ __forceinline__ void tma_reduce_add_2d(const CUtensorMap* m, const void* smem_src, int x, int y) {
  asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%2, %3}], [%1];"
               ::"l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(smem_src)), "r"(x), "r"(y)
               : "memory");
}
__device__ __forceinline__ void bulk_commit_group() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// Until at most `N` of this thread's groups still have to read their shared-memory source.
template <int N>
__device__ __forceinline__ void bulk_wait_group_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void bulk_wait_group_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
// Ordered mode of the residual epilogue. The pieces of a tile belong to consecutive CTAs and add in descending order
// of their k range: head, middle pieces, tail. Every CTA owns one word, which it sets to the launch's number once the
// additions of the piece at the start of its range (head or middle) have been performed; a middle or tail piece waits
// (bounded) for the word of the CTA above it. A head piece is the first thing its CTA computes, so in launches whose
// CTAs each hold more than a tile nobody ever waits long.
constexpr uint32_t kTurnSpinLimit = 1u << 22;     // polls of ~0.1-0.3 us each: about a second
__device__ __forceinline__ bool wait_turn(const uint32_t* flag, uint32_t epoch, volatile uint32_t* abort_flag,
                                          uint32_t* status) {
  for (uint32_t i = 0; i < kTurnSpinLimit; ++i) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(flag) : "memory");
    if (v == epoch) return true;
    if ((i & 255u) == 255u && *abort_flag) return false;
    __nanosleep(i < 64 ? 32 : 256);
  }
  *abort_flag = 1;
  atomicOr(status, kStatusTimeout);
  return false;
}
__device__ __forceinline__ void publish_turn(uint32_t* flag, uint32_t epoch) {
  asm volatile("fence.proxy.async;" ::: "memory");     // the additions went through the copy engine
  __threadfence();
  asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(flag), "r"(epoch) : "memory");
}
__device__ __forceinline__ void st_shared_v4(void* p, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(smem_u32(p)), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ void tmem_ld_32x16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void st_v4(void* p, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.global.v4.b32 [%0], {%1, %2, %3, %4};" ::"l"(p), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
// z * sigmoid(z) with the fast exponential and the fast reciprocal: an IEEE division here made the epilogue of a
// SwiGLU tile as long as its main loop.
__device__ __forceinline__ float silu_f(float z) { return __fdividef(z, 1.0f + __expf(-z)); }

// One 64-deep block of products D (+)= A B^T (four K = 16 steps; the descriptors advance by 32 bytes per step),
// then an arrival on `commit_bar` once they have completed. Before them a non-blocking test of `peek_bar` is
// issued; its answer (1 = that phase is complete) is only read after everything else has been issued.
__device__ __forceinline__ bool umma_kblock_peek(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                                 uint32_t accumulate_first, uint64_t* commit_bar, uint64_t* peek_bar,
                                                 uint32_t peek_parity) {
  uint32_t ready;
  asm volatile(
      "{\n\t.reg .pred P, Q;\n\t.reg .b64 a1, a2, a3, b1, b2, b3;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 P, [%1], %2;\n\t"
      "setp.ne.b32 Q, %7, 0;\n\t"
      "add.u64 a1, %4, 2;\n\tadd.u64 b1, %5, 2;\n\t"
      "add.u64 a2, %4, 4;\n\tadd.u64 b2, %5, 4;\n\t"
      "add.u64 a3, %4, 6;\n\tadd.u64 b3, %5, 6;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%3], %4, %5, %6, Q;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%3], a1, b1, %6, 1;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%3], a2, b2, %6, 1;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%3], a3, b3, %6, 1;\n\t"
      "tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%8];\n\t"
      "selp.u32 %0, 1, 0, P;\n\t}"
      : "=r"(ready)
      : "r"(smem_u32(peek_bar)), "r"(peek_parity), "r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc),
        "r"(accumulate_first), "r"(smem_u32(commit_bar))
      : "memory");
  return ready != 0;
}

template <int BN, int EPI>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_f16_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                 const __grid_constant__ CUtensorMap tm_b2, const __grid_constant__ CUtensorMap tm_out,
                 void* __restrict__ out, int M, int N, int m_tiles, int n_tiles, int kblocks, int total_units,
                 int units_per_cta, const RopeEpilogue rope, uint32_t* status, uint32_t* turn_flags, uint32_t epoch) {
  using L = GemmSmem<BN>;
  constexpr int OUT_BN = (EPI == kEpiSwiGLU) ? BN / 2 : BN;
  constexpr uint32_t kTmemCols = 2 * BN;
  constexpr uint32_t kIdesc = umma_idesc_f16(BM, BN);

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::kStagingOff + L::kStagingBytes);
  uint64_t* full_bar = bars;                       // [kStages] TMA -> MMA
  uint64_t* empty_bar = bars + L::kStages;         // [kStages] MMA -> TMA
  uint64_t* acc_full = bars + 2 * L::kStages;      // [2] MMA -> epilogue
  uint64_t* acc_empty = bars + 2 * L::kStages + 2; // [2] epilogue -> MMA
  uint64_t* turn_bar = bars + 2 * L::kStages + 4;  // the epilogue warps' additions of the first piece are done
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * L::kStages + 5);
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  const int start = blockIdx.x * units_per_cta;
  const int end = min(total_units, start + units_per_cta);
  const SegPlan plan = make_plan(start, end, kblocks);

  if (threadIdx.x == 0) {
    for (int s = 0; s < L::kStages; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(&acc_full[a], 1);
      mbar_init(&acc_empty[a], 4);
    }
    mbar_init(turn_bar, 4);
    *abort_flag = 0;
    fence_barrier_init();
    tma_prefetch_desc(&tm_a);
    tma_prefetch_desc(&tm_b);
    if (EPI == kEpiSwiGLU) tma_prefetch_desc(&tm_b2);
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // Everything above overlapped the previous kernel's tail; its results (the A operand, x) are needed from here on.
  pdl_launch_dependents();
  // The producer thread waits a little later: the weights do not depend on the previous kernel, so it first sends
  // for the B boxes of its first stages (all stages are empty at this point).
  int pre = 0;
  if (threadIdx.x == 0) {
    for (int si = 0; si < plan.count && pre < L::kStages; ++si) {
      const Segment sg = plan_segment(plan, si);
      const int n0 = tile_n(sg.tile, m_tiles, n_tiles, EPI) * OUT_BN;
      for (int kb = sg.kb0; kb < sg.kb0 + sg.len && pre < L::kStages; ++kb, ++pre) {
        uint8_t* sb = smem + pre * L::kStageBytes + kABytes;
        mbar_arrive_expect_tx(&full_bar[pre], L::kStageBytes);
        tma_load_2d(sb, &tm_b, &full_bar[pre], kb * BK, n0);
        if (EPI == kEpiSwiGLU) tma_load_2d(sb + 128 * BK * 2, &tm_b2, &full_bar[pre], kb * BK, n0);
        else if (BN == 256) tma_load_2d(sb + 128 * BK * 2, &tm_b, &full_bar[pre], kb * BK, n0 + 128);
      }
    }
  }
  pdl_wait();

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    // One thread issues the two or three 16 KB boxes of a stage in turn. (Spreading them over lanes of the warp,
    // which pays for 4 KB boxes, was measured slower here.)
    if (lane == 0) {
      int stage = 0, issued = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int si = 0; si < plan.count && ok; ++si) {
        const Segment sg = plan_segment(plan, si);
        const int m0 = tile_m(sg.tile, m_tiles, n_tiles, EPI) * BM;
        const int n0 = tile_n(sg.tile, m_tiles, n_tiles, EPI) * OUT_BN;
        for (int kb = sg.kb0; kb < sg.kb0 + sg.len; ++kb, ++issued) {
          uint8_t* sa = smem + stage * L::kStageBytes;
          uint8_t* sb = sa + kABytes;
          if (issued < pre) {
            // first use of the stage: its bytes are announced and its weight boxes already on their way
            tma_load_2d(sa, &tm_a, &full_bar[stage], kb * BK, m0);
          } else {
            if (!mbar_wait(&empty_bar[stage], phase ^ 1u, abort_flag, status)) { ok = false; break; }
            mbar_arrive_expect_tx(&full_bar[stage], L::kStageBytes);
            tma_load_2d(sa, &tm_a, &full_bar[stage], kb * BK, m0);
            tma_load_2d(sb, &tm_b, &full_bar[stage], kb * BK, n0);
            if (EPI == kEpiSwiGLU) tma_load_2d(sb + 128 * BK * 2, &tm_b2, &full_bar[stage], kb * BK, n0);
            else if (BN == 256) tma_load_2d(sb + 128 * BK * 2, &tm_b, &full_bar[stage], kb * BK, n0 + 128);
          }
          if (++stage == L::kStages) { stage = 0; phase ^= 1u; }
        }
      }
      // In a healthy run the MMA warp has waited for every copy before the CTA exits. After an abort, give
      // the copies still in flight time to land in shared memory before the CTA may go away.
      if (!ok)
        for (int i = 0; i < 64; ++i) __nanosleep(10000);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    // The thread that feeds the tensor core must not stall: a wait on a barrier that is already complete still
    // costs a round trip of a few hundred cycles, in which the short queue of issued products runs dry. So the
    // test of the NEXT stage's barrier is issued before this stage's products and its answer is read after them.
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      const uint32_t smem_base = smem_u32(smem);
      const uint64_t adesc0 = umma_desc_k128(smem_base);
      const uint64_t bdesc0 = umma_desc_k128(smem_base + kABytes);
      bool ready = false;
      for (int si = 0; si < plan.count && ok; ++si) {
        const Segment sg = plan_segment(plan, si);
        if (!mbar_wait(&acc_empty[acc], acc_phase ^ 1u, abort_flag, status)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * BN;
        for (int i = 0; i < sg.len; ++i) {
          if (!ready && !mbar_wait(&full_bar[stage], phase, abort_flag, status)) { ok = false; break; }
          const int ns = (stage + 1 == L::kStages) ? 0 : stage + 1;
          const uint32_t np = (ns == 0) ? phase ^ 1u : phase;
          const uint64_t off = static_cast<uint64_t>(stage * (L::kStageBytes >> 4));
          ready = umma_kblock_peek(d_tmem, adesc0 + off, bdesc0 + off, kIdesc, i != 0, &empty_bar[stage], &full_bar[ns], np);
          stage = ns;
          phase = np;
        }
        if (!ok) break;
        umma_commit(&acc_full[acc]);
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1u;
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..5)
    const int quad = warp & 3;  // the TMEM lane quadrant this warp may read
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    const bool ordered = EPI == kEpiResidAdd && turn_flags != nullptr;
    bool owes_turn = ordered && plan.head_len > 0;
    for (int si = 0; si < plan.count && ok; ++si) {
      const Segment sg = plan_segment(plan, si);
      const int m0 = tile_m(sg.tile, m_tiles, n_tiles, EPI) * BM;
      const int n0 = tile_n(sg.tile, m_tiles, n_tiles, EPI) * OUT_BN;
      const int row = m0 + quad * 32 + lane;
      const bool row_ok = row < M;
      // Rotary epilogue: this row's (cos, sin) pairs are fetched while the tile is still being accumulated.
      float4 rot[32];
      if ((EPI == kEpiStoreRope || EPI == kEpiStoreNormRope) && row_ok && n0 < rope.n_rot_cols) {
        const float4* tb = reinterpret_cast<const float4*>(rope.table + static_cast<size_t>(row) * rope.half);
#pragma unroll
        for (int j = 0; j < 32; ++j)
          if (2 * j < rope.half) rot[j] = __ldg(tb + j);
      }
      if (!mbar_wait(&acc_full[acc], acc_phase, abort_flag, status)) { ok = false; break; }
      tc_fence_after();
      const uint32_t t_row = tmem_base + acc * BN + (static_cast<uint32_t>(quad * 32) << 16);
      // the tile lies inside the output and its accumulator inside the tensor-memory allocation
      if (lane == 0) debug_in_range(m0 >= 0 && m0 < M && n0 >= 0 && n0 < N && acc * BN + BN <= static_cast<int>(kTmemCols), status);
      uint32_t r[32];
      if (EPI == kEpiSwiGLU) {
        uint32_t r2[32];
        __half* o = reinterpret_cast<__half*>(out) + static_cast<size_t>(row) * N;
#pragma unroll 1
        for (int c = 0; c < OUT_BN / 32; ++c) {
          tmem_ld_32x32(t_row + c * 32, r);
          tmem_ld_32x32(t_row + OUT_BN + c * 32, r2);
          tmem_ld_wait();
          uint32_t p[16];
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const float g0 = __uint_as_float(r[2 * j]), g1 = __uint_as_float(r[2 * j + 1]);
            const float u0 = __uint_as_float(r2[2 * j]), u1 = __uint_as_float(r2[2 * j + 1]);
            p[j] = pack_f16x2(silu_f(g0) * u0, silu_f(g1) * u1);
          }
          const int col = n0 + c * 32;
          if (row_ok) {
#pragma unroll
            for (int j = 0; j < 4; ++j)
              if (col + j * 8 < N) st_v4(o + col + j * 8, p[4 * j], p[4 * j + 1], p[4 * j + 2], p[4 * j + 3]);
          }
        }
      } else if (EPI == kEpiStoreRope || EPI == kEpiStoreNormRope) {
        __half* o = reinterpret_cast<__half*>(out) + static_cast<size_t>(row) * N;
        const int hd = 2 * rope.half;
#pragma unroll 1
        for (int h0 = 0; h0 < BN && n0 + h0 < N; h0 += hd) {
          if (n0 + h0 < rope.n_rot_cols) {
            // Query/key normalisation: a first sweep over the head's columns for this row's mean square.
            float inv_rms = 1.f;
            const float* gain = nullptr;
            if (EPI == kEpiStoreNormRope) {
              float ss = 0.f;
#pragma unroll 1
              for (int c = 0; c < hd / 32; ++c) {
                tmem_ld_32x32(t_row + h0 + c * 32, r);
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 32; ++j) ss = fmaf(__uint_as_float(r[j]), __uint_as_float(r[j]), ss);
              }
              inv_rms = rsqrtf(ss / static_cast<float>(hd) + rope.eps);
              gain = rope.qk_gain + (n0 + h0 < rope.q_cols ? 0 : hd);
            }
            // pairs (j, j + half) of one head, 16 pairs at a time
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              if (c * 16 < rope.half) {
                uint32_t lo[16], hi[16];
                tmem_ld_32x16(t_row + h0 + c * 16, lo);
                tmem_ld_32x16(t_row + h0 + rope.half + c * 16, hi);
                tmem_ld_wait();
                uint32_t plo[8], phi[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                  const float4 cs = rot[c * 8 + e];      // (cos, sin) of pairs 2e and 2e + 1 of this chunk
                  float a0 = __uint_as_float(lo[2 * e]), a1 = __uint_as_float(lo[2 * e + 1]);
                  float b0 = __uint_as_float(hi[2 * e]), b1 = __uint_as_float(hi[2 * e + 1]);
                  if (EPI == kEpiStoreNormRope) {
                    const float2 ga = __ldg(reinterpret_cast<const float2*>(gain + c * 16 + 2 * e));
                    const float2 gb = __ldg(reinterpret_cast<const float2*>(gain + rope.half + c * 16 + 2 * e));
                    a0 *= inv_rms * ga.x;
                    a1 *= inv_rms * ga.y;
                    b0 *= inv_rms * gb.x;
                    b1 *= inv_rms * gb.y;
                  }
                  plo[e] = pack_f16x2(a0 * cs.x - b0 * cs.y, a1 * cs.z - b1 * cs.w);
                  phi[e] = pack_f16x2(b0 * cs.x + a0 * cs.y, b1 * cs.z + a1 * cs.w);
                }
                if (row_ok) {
                  __half* ol = o + n0 + h0 + c * 16;
                  st_v4(ol, plo[0], plo[1], plo[2], plo[3]);
                  st_v4(ol + 8, plo[4], plo[5], plo[6], plo[7]);
                  st_v4(ol + rope.half, phi[0], phi[1], phi[2], phi[3]);
                  st_v4(ol + rope.half + 8, phi[4], phi[5], phi[6], phi[7]);
                }
              }
            }
          } else {
#pragma unroll 1
            for (int c = 0; c < hd / 32; ++c) {
              tmem_ld_32x32(t_row + h0 + c * 32, r);
              tmem_ld_wait();
              if (row_ok) {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                  st_v4(o + n0 + h0 + c * 32 + j * 8, pack_f16x2(__uint_as_float(r[8 * j]), __uint_as_float(r[8 * j + 1])),
                        pack_f16x2(__uint_as_float(r[8 * j + 2]), __uint_as_float(r[8 * j + 3])),
                        pack_f16x2(__uint_as_float(r[8 * j + 4]), __uint_as_float(r[8 * j + 5])),
                        pack_f16x2(__uint_as_float(r[8 * j + 6]), __uint_as_float(r[8 * j + 7])));
              }
            }
          }
        }
      } else if (EPI == kEpiStoreF16) {
        __half* o = reinterpret_cast<__half*>(out) + static_cast<size_t>(row) * N;
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c) {
          tmem_ld_32x32(t_row + c * 32, r);
          tmem_ld_wait();
          const int col = n0 + c * 32;
          if (row_ok) {
#pragma unroll
            for (int j = 0; j < 4; ++j)
              if (col + j * 8 < N)
                st_v4(o + col + j * 8, pack_f16x2(__uint_as_float(r[8 * j]), __uint_as_float(r[8 * j + 1])),
                      pack_f16x2(__uint_as_float(r[8 * j + 2]), __uint_as_float(r[8 * j + 3])),
                      pack_f16x2(__uint_as_float(r[8 * j + 4]), __uint_as_float(r[8 * j + 5])),
                      pack_f16x2(__uint_as_float(r[8 * j + 6]), __uint_as_float(r[8 * j + 7])));
          }
        }
      } else {
        // x += acc. Each warp stages its 32 rows, 32 columns at a time, in shared memory and lets the copy engine add
        // the box into x: per-lane atomics on 16-byte pieces of 32 different rows took as long as a third of the
        // main loop. Two boxes per warp alternate; lane 0 owns the warp's copy groups.
        uint8_t* stage0 = smem + L::kStagingOff + quad * 2 * 4096;
        const int y = m0 + quad * 32;
        // Ordered mode: a piece that stops short of its tile's end adds after the piece above it (next CTA); a piece
        // that starts inside its tile tells the piece below it (previous CTA) when its own additions are done.
        const bool partial = ordered && sg.len < kblocks;
        const bool publishes = partial && sg.kb0 > 0;
        const int me = blockIdx.x;
        if (partial && sg.kb0 + sg.len < kblocks) {
          if (!wait_turn(turn_flags + me + 1, epoch, abort_flag, status)) { ok = false; break; }
          asm volatile("fence.proxy.async;" ::: "memory");
        }
#pragma unroll 1
        for (int c = 0; c < BN / 32 && n0 + c * 32 < N; ++c) {
          tmem_ld_32x32(t_row + c * 32, r);
          if (c >= 2) {
            if (lane == 0) bulk_wait_group_read<1>();      // the box written two rounds ago has been read
            __syncwarp();
          }
          tmem_ld_wait();
          uint8_t* box = stage0 + (c & 1) * 4096;
#pragma unroll
          for (int j = 0; j < 8; ++j)
            st_shared_v4(box + lane * 128 + ((j ^ (lane & 7)) << 4), r[4 * j], r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]);
          fence_proxy_async();
          __syncwarp();
          if (lane == 0) {     // one group per round, empty or not: the wait above counts groups
            if (y < M) tma_reduce_add_2d(&tm_out, box, n0 + c * 32, y);
            bulk_commit_group();
          }
        }
        if (lane == 0) bulk_wait_group_read<0>();
        __syncwarp();
        if (publishes) {
          // additions performed by all four warps -> the piece below may add
          if (lane == 0) {
            bulk_wait_group_all();
            mbar_arrive(turn_bar);
          }
          if (warp == 2 && lane == 0 && mbar_wait(turn_bar, 0, abort_flag, status)) {
            publish_turn(turn_flags + me, epoch);
            owes_turn = false;
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&acc_empty[acc]);
      acc ^= 1;
      if (acc == 0) acc_phase ^= 1u;
    }
    if (EPI == kEpiResidAdd && lane == 0) bulk_wait_group_all();   // the additions have been performed
    // A CTA that gave up still lets the pieces that wait for it go on (the time-out is reported through the status word).
    if (owes_turn && warp == 2 && lane == 0) publish_turn(turn_flags + blockIdx.x, epoch);
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = []() -> EncodeTiledFn {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &p, 12000, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      return nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

// fp32 [rows, cols] row-major, boxes of 32 rows x 32 columns (128 bytes per row), 128-byte swizzle.
bool make_out_f32_map(CUtensorMap* tm, void* base, int rows, int cols) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
  cuuint64_t strides[1] = {static_cast<cuuint64_t>(cols) * 4};
  cuuint32_t box[2] = {32, 32};
  cuuint32_t estr[2] = {1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int BN, int EPI>
cudaError_t launch(const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap& tb2, void* out, int M, int N,
                   int K, uint32_t* status, cudaStream_t stream, const RopeEpilogue& rope = RopeEpilogue{nullptr, 0, 0},
                   const TurnOrder* turn = nullptr, bool whole_tiles = false) {
  using L = GemmSmem<BN>;
  constexpr int OUT_BN = (EPI == kEpiSwiGLU) ? BN / 2 : BN;
  static std::atomic<uint64_t> smem_opted{0};
  if (cudaError_t e = opt_in_dynamic_smem(gemm_f16_kernel<BN, EPI>, L::kTotal, smem_opted); e != cudaSuccess) return e;
  const int m_tiles = (M + BM - 1) / BM;
  const int n_tiles = (N + OUT_BN - 1) / OUT_BN;
  const int kblocks = (K + BK - 1) / BK;
  const int tiles = m_tiles * n_tiles;
  const int total = tiles * kblocks;
  int grid, upc;
  uint32_t* turn_flags = nullptr;
  uint32_t epoch = 0;
  if (EPI == kEpiResidAdd && !whole_tiles) {
    grid = total < kNumSMs ? total : kNumSMs;
    upc = (total + grid - 1) / grid;
    if (turn) {
      // The pieces of a tile add one after the other: keep them few when the even cut would make them many (few rows).
      upc = std::max(upc, (kblocks + kMaxOrderedPieces - 1) / kMaxOrderedPieces);
      turn_flags = turn->flags;
      epoch = ++*turn->epoch;
      if (epoch == 0) epoch = ++*turn->epoch;       // 0 is what a fresh flag array holds
    }
    grid = (total + upc - 1) / upc;
  } else {
    const int tpc = (tiles + kNumSMs - 1) / kNumSMs;
    grid = (tiles + tpc - 1) / tpc;
    upc = tpc * kblocks;
  }
  CUtensorMap tout = ta;   // only the residual epilogue reads it
  if (EPI == kEpiResidAdd) {
    // The output of the residual projections is the same buffer and shape for every layer of a pass (x, and the last
    // rows' copy of it): its tensor map is encoded when either changes, not per launch.
    struct OutMap { void* base = nullptr; int rows = 0, cols = 0; CUtensorMap tm; };
    thread_local OutMap cache[2];
    thread_local int next = 0;
    const OutMap* hit = nullptr;
    for (const OutMap& c : cache)
      if (c.base == out && c.rows == M && c.cols == N) hit = &c;
    if (!hit) {
      OutMap& c = cache[next];
      next ^= 1;
      if (!make_out_f32_map(&c.tm, out, M, N)) { c.base = nullptr; return cudaErrorInvalidValue; }
      c.base = out; c.rows = M; c.cols = N;
      hit = &c;
    }
    tout = hit->tm;
  }
  cudaError_t le = launch_pdl(gemm_f16_kernel<BN, EPI>, dim3(grid), dim3(kGemmThreads), L::kTotal, stream, ta, tb, tb2, tout, out, M,
                              N, m_tiles, n_tiles, kblocks, total, upc, rope, status, turn_flags, epoch);
  count_launch();
  return le != cudaSuccess ? le : cudaGetLastError();
}

}  // namespace

bool make_tensor_map_16b(CUtensorMap* tm, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows,
                         uint32_t box_cols, bool swizzle128, bool is_bf16) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {cols * 2};
  cuuint32_t box[2] = {box_cols, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(tm, is_bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

bool make_tensor_map_heads3d(CUtensorMap* tm, const void* base, uint64_t tokens, uint64_t heads, uint32_t head_dim,
                             uint64_t row_elems, uint32_t box_tokens, uint32_t box_heads) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[3] = {head_dim, heads, tokens};
  cuuint64_t strides[2] = {static_cast<cuuint64_t>(head_dim) * 2, row_elems * 2};
  cuuint32_t box[3] = {64, box_heads, box_tokens};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

bool make_kv_group_map(CUtensorMap* tm, const void* base, uint64_t rows, uint32_t hd, uint32_t groups_per_box) {
  EncodeTiledFn fn = encode_fn();
  if (!fn || hd % 64 || rows % 8) return false;
  cuuint64_t dims[4] = {64, 8, hd / 64, rows / 8};
  cuuint64_t strides[3] = {static_cast<cuuint64_t>(hd) * 2, 128, static_cast<cuuint64_t>(hd) * 2 * 8};
  cuuint32_t box[4] = {64, 8, hd / 64, groups_per_box};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

bool make_kv_rows_map(CUtensorMap* tm, const void* base, uint64_t rows, uint64_t row_elems, uint32_t hd) {
  EncodeTiledFn fn = encode_fn();
  if (!fn || hd % 64 || row_elems % 64) return false;
  // The row coordinate (dimension 1) and the group coordinate (dimension 3) address the same rows: row + 8 * group.
  cuuint64_t dims[4] = {64, rows + 8, row_elems / 64, 16};
  cuuint64_t strides[3] = {row_elems * 2, 128, row_elems * 2 * 8};
  cuuint32_t box[4] = {64, 8, hd / 64, 16};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

bool make_gemm_operand_map(CUtensorMap* tm, const void* base, int rows, int k) {
  return make_tensor_map_16b(tm, base, static_cast<uint64_t>(rows), static_cast<uint64_t>(k), 128, 64, true, false);
}

cudaError_t gemm_f16_rope(const CUtensorMap& ta, const CUtensorMap& tb, void* out, int M, int N, int K,
                          const RopeEpilogue& rope, uint32_t* status, cudaStream_t stream) {
  if (M <= 0) return cudaSuccess;
  if (!rope.table || (rope.half != 32 && rope.half != 64) || N % (2 * rope.half) || rope.n_rot_cols % (2 * rope.half))
    return cudaErrorInvalidValue;
  if (rope.qk_gain) {
    if (rope.q_cols % (2 * rope.half) || rope.q_cols > rope.n_rot_cols) return cudaErrorInvalidValue;
    return launch<256, kEpiStoreNormRope>(ta, tb, tb, out, M, N, K, status, stream, rope);
  }
  return launch<256, kEpiStoreRope>(ta, tb, tb, out, M, N, K, status, stream, rope);
}

cudaError_t gemm_f16(const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap* tb2, void* out, int M, int N,
                      int K, int epilogue, uint32_t* status, cudaStream_t stream, const TurnOrder* turn) {
  if (M <= 0) return cudaSuccess;
  switch (epilogue) {
    case kEpiStoreF16:
      // Issuing a product costs the issuing thread about 70 cycles whatever its size, so 128-wide tiles (64-cycle
      // products) leave the tensor core waiting for the issuer: 256-wide tiles even when they fill fewer SMs.
      if (N <= 128) return launch<128, kEpiStoreF16>(ta, tb, tb, out, M, N, K, status, stream);
      return launch<256, kEpiStoreF16>(ta, tb, tb, out, M, N, K, status, stream);
    case kEpiResidAdd:
      // Short k ranges (the O projection): whole 128-wide tiles. The narrow tiles are issue-bound, but there are twice
      // as many of them, no tile is shared between CTAs and every element of the output receives one addition.
      if (K <= kShortK && N >= 128)
        return launch<128, kEpiResidAdd>(ta, tb, tb, out, M, N, K, status, stream, RopeEpilogue{nullptr, 0, 0}, nullptr, true);
      return launch<256, kEpiResidAdd>(ta, tb, tb, out, M, N, K, status, stream, RopeEpilogue{nullptr, 0, 0}, turn);
    case kEpiSwiGLU:
      return launch<256, kEpiSwiGLU>(ta, tb, *tb2, out, M, N, K, status, stream);
    default:
      return cudaErrorInvalidValue;
  }
}

}  // namespace cs
