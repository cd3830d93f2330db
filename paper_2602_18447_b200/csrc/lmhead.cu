// Last-position LM head with the logsumexp over the vocabulary fused in, and the confidence gate.
//
// logits^T[V, B] = W_lm[V, d] * h[B, d]^T is a weight-streaming product (B is 8..64): each CTA walks over
// 128-row tiles of W_lm, brought in by TMA, multiplies them on the tensor cores (tcgen05, M = 128 vocabulary
// rows, N = padded batch) and never writes the logits: every epilogue thread owns one TMEM lane (one
// vocabulary row of each tile) and keeps, per step, a running maximum and a running sum of exp(z - max) over
// the rows it has seen. At the end the 128 threads merge their pairs and the CTA emits one (max, sum) pair per
// step; the gate kernel merges the CTAs' pairs, forms p = exp(z_verdict - lse) and applies the threshold.
#include "kernels.h"

#include "common.cuh"

namespace cs {

namespace {

constexpr int kLmBM = 128;
constexpr int kLmBK = 64;
constexpr int kLmThreads = 192;
constexpr int kLmWBytes = kLmBM * kLmBK * 2;
constexpr int kLmMaxVerdict = 8;

template <int NB>
struct LmSmem {
  static constexpr int kHBytes = NB * kLmBK * 2;
  // a stage: two 128-row tiles of W (a 256-row "double tile") and the one tile of hidden states they share
  static constexpr int kStageBytes = 2 * kLmWBytes + ((kHBytes + 1023) / 1024) * 1024;
  static constexpr int kStages = 5;
  static constexpr int kBarOff = kStages * kStageBytes;
  static constexpr int kRedOff = kBarOff + 256;                 // [4 warps][NB][2] floats
  static constexpr int kTotal = kRedOff + 4 * NB * 2 * 4 + 1024;
};

__device__ __forceinline__ void tmem_ld_32x16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}

// One 64-deep block of products (four K = 16 steps; the descriptors advance by 32 bytes per step), then an arrival on
// `commit_bar` once they have completed. Before them a non-blocking test of `peek_bar` is issued; its answer (1 = that
// phase is complete) is read after everything else has been issued: with at most 64 steps per pass the products are
// short, and a blocking wait between them would leave the tensor core idle for longer than they run.
__device__ __forceinline__ bool lm_kblock_peek(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
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

// The same for a double tile: the second 128 rows of W lie 16 KB behind the first in the stage and accumulate NB
// columns further on in tensor memory; both read the same hidden-state tile.
__device__ __forceinline__ bool lm_kblock2_peek(uint32_t tmem_d, uint32_t tmem_d2, uint64_t adesc, uint64_t bdesc,
                                                uint32_t idesc, uint32_t accumulate_first, uint64_t* commit_bar,
                                                uint64_t* peek_bar, uint32_t peek_parity) {
  uint32_t ready;
  asm volatile(
      "{\n\t.reg .pred P, Q;\n\t.reg .b64 a1, a2, a3, b1, b2, b3, c0, c1, c2, c3;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 P, [%1], %2;\n\t"
      "setp.ne.b32 Q, %7, 0;\n\t"
      "add.u64 a1, %4, 2;\n\tadd.u64 b1, %5, 2;\n\t"
      "add.u64 a2, %4, 4;\n\tadd.u64 b2, %5, 4;\n\t"
      "add.u64 a3, %4, 6;\n\tadd.u64 b3, %5, 6;\n\t"
      "add.u64 c0, %4, 1024;\n\tadd.u64 c1, %4, 1026;\n\tadd.u64 c2, %4, 1028;\n\tadd.u64 c3, %4, 1030;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%3], %4, %5, %6, Q;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%9], c0, %5, %6, Q;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%3], a1, b1, %6, 1;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%9], c1, b1, %6, 1;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%3], a2, b2, %6, 1;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%9], c2, b2, %6, 1;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%3], a3, b3, %6, 1;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%9], c3, b3, %6, 1;\n\t"
      "tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%8];\n\t"
      "selp.u32 %0, 1, 0, P;\n\t}"
      : "=r"(ready)
      : "r"(smem_u32(peek_bar)), "r"(peek_parity), "r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc),
        "r"(accumulate_first), "r"(smem_u32(commit_bar)), "r"(tmem_d2)
      : "memory");
  return ready != 0;
}

// Rows of the vocabulary [blockIdx.x * rows_per_cta, + rows_per_cta) belong to a CTA, cut evenly so that every SM
// streams the same number of bytes. A range is walked in 256-row double tiles (two products per tile of hidden states:
// with 32-64 steps per pass the hidden states re-read from L2 for every tile of W are half as many bytes again as W
// itself, more than an SM takes in at the clock the power cap leaves); when the range is not a multiple of 256 its
// last, partial double tile (one 128-row tile if that covers it) comes FIRST: the rows that tile fetches beyond the range are the first tile of the next CTA, which
// fetches them at the same moment, so they cross the DRAM interface once.
struct LmArgs {
  int B, vocab, kblocks, rows_per_cta, n_verdict, h_row0;
  int verdict[kLmMaxVerdict];
  float* part_max;        // [grid, NB]
  float* part_sum;        // [grid, NB]
  float* verdict_logits;  // [B, n_verdict]
  float* logits;          // [B, vocab] or nullptr
  uint32_t* status;
};

template <int NB>
__global__ void __launch_bounds__(kLmThreads, 1)
lm_head_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_h, const LmArgs a) {
  using L = LmSmem<NB>;
  constexpr uint32_t kTmemCols = (4 * NB < 32) ? 32 : 4 * NB;     // two accumulators of two tiles of NB columns
  constexpr uint32_t kIdesc = umma_idesc_f16(kLmBM, NB);

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::kBarOff);
  uint64_t* full_bar = bars;
  uint64_t* empty_bar = bars + L::kStages;
  uint64_t* acc_full = bars + 2 * L::kStages;
  uint64_t* acc_empty = bars + 2 * L::kStages + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * L::kStages + 4);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  float* red = reinterpret_cast<float*>(smem + L::kRedOff);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row_begin = blockIdx.x * a.rows_per_cta;
  const int row_end = min(a.vocab, row_begin + a.rows_per_cta);
  constexpr int kDouble = 2 * kLmBM;
  const int n_my_tiles = (row_end - row_begin + kDouble - 1) / kDouble;
  const bool tail_first = ((row_end - row_begin) % kDouble) != 0 && n_my_tiles > 1;
  // first row of the i-th double tile this CTA works on, and whether its second 128 rows hold any row of the range
  auto tile_row0 = [&](int i) {
    const int t = tail_first ? (i == 0 ? n_my_tiles - 1 : i - 1) : i;
    return row_begin + t * kDouble;
  };
  auto tile_is_double = [&](int i) { return tile_row0(i) + kLmBM < row_end; };

  if (threadIdx.x == 0) {
    for (int s = 0; s < L::kStages; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&acc_full[i], 1);
      mbar_init(&acc_empty[i], 4);
    }
    *abort_flag = 0;
    fence_barrier_init();
    tma_prefetch_desc(&tm_w);
    tma_prefetch_desc(&tm_h);
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_launch_dependents();
  pdl_wait();

  if (warp == 0) {
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int i = 0; i < n_my_tiles && ok; ++i) {
        const int r0 = tile_row0(i);
        const bool two = tile_is_double(i);
        for (int kb = 0; kb < a.kblocks; ++kb) {
          if (!mbar_wait(&empty_bar[stage], phase ^ 1u, abort_flag, a.status)) { ok = false; break; }
          uint8_t* sw = smem + stage * L::kStageBytes;
          mbar_arrive_expect_tx(&full_bar[stage], (two ? 2 : 1) * kLmWBytes + L::kHBytes);
          tma_load_2d(sw, &tm_w, &full_bar[stage], kb * kLmBK, r0);
          if (two) tma_load_2d(sw + kLmWBytes, &tm_w, &full_bar[stage], kb * kLmBK, r0 + kLmBM);
          tma_load_2d(sw + 2 * kLmWBytes, &tm_h, &full_bar[stage], kb * kLmBK, a.h_row0);
          if (++stage == L::kStages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok)
        for (int i = 0; i < 64; ++i) __nanosleep(10000);
    }
  } else if (warp == 1) {
    if (lane == 0) {
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true, ready = false;
      const uint32_t smem_base = smem_u32(smem);
      const uint64_t adesc0 = umma_desc_k128(smem_base);
      const uint64_t bdesc0 = umma_desc_k128(smem_base + 2 * kLmWBytes);
      for (int i = 0; i < n_my_tiles && ok; ++i) {
        if (!mbar_wait(&acc_empty[acc], acc_phase ^ 1u, abort_flag, a.status)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * 2 * NB;
        const bool two = tile_is_double(i);
        for (int kb = 0; kb < a.kblocks; ++kb) {
          if (!ready && !mbar_wait(&full_bar[stage], phase, abort_flag, a.status)) { ok = false; break; }
          const int ns = (stage + 1 == L::kStages) ? 0 : stage + 1;
          const uint32_t np = (ns == 0) ? phase ^ 1u : phase;
          const uint64_t off = static_cast<uint64_t>(stage * (L::kStageBytes >> 4));
          ready = two ? lm_kblock2_peek(d_tmem, d_tmem + NB, adesc0 + off, bdesc0 + off, kIdesc, kb != 0, &empty_bar[stage],
                                        &full_bar[ns], np)
                      : lm_kblock_peek(d_tmem, adesc0 + off, bdesc0 + off, kIdesc, kb != 0, &empty_bar[stage], &full_bar[ns], np);
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
    const int quad = warp & 3;
    float run_m[NB], run_l[NB];
#pragma unroll
    for (int b = 0; b < NB; ++b) { run_m[b] = -INFINITY; run_l[b] = 0.f; }
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    for (int i = 0; i < n_my_tiles; ++i) {
      if (!mbar_wait(&acc_full[acc], acc_phase, abort_flag, a.status)) { ok = false; break; }
      tc_fence_after();
      const int n_sub = tile_is_double(i) ? 2 : 1;
#pragma unroll 1
      for (int sub = 0; sub < n_sub; ++sub) {
      const uint32_t t_row = tmem_base + acc * 2 * NB + sub * NB + (static_cast<uint32_t>(quad * 32) << 16);
      const int row = tile_row0(i) + sub * kLmBM + quad * 32 + lane;   // vocabulary id of this thread's lane
      const bool row_ok = row < row_end;                 // rows past the range belong to the next CTA (or to nobody)
      uint32_t vmask = 0;   // which entries of verdict_ids name this row (an id may be listed twice)
      for (int j = 0; j < a.n_verdict; ++j)
        if (a.verdict[j] == row) vmask |= 1u << j;
#pragma unroll
      for (int c = 0; c < NB / 16; ++c) {
        uint32_t r[16];
        tmem_ld_32x16(t_row + c * 16, r);
        tmem_ld_wait();
        if (row_ok) {
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int b = c * 16 + j;
            const float z = __uint_as_float(r[j]);
            const float mn = fmaxf(run_m[b], z);
            run_l[b] = run_l[b] * __expf(run_m[b] - mn) + __expf(z - mn);
            run_m[b] = mn;
            if (b < a.B) {
              for (uint32_t vm = vmask; vm; vm &= vm - 1) a.verdict_logits[b * a.n_verdict + (__ffs(vm) - 1)] = z;
              if (a.logits) a.logits[static_cast<size_t>(b) * a.vocab + row] = z;
            }
          }
        }
      }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&acc_empty[acc]);
      acc ^= 1;
      if (acc == 0) acc_phase ^= 1u;
    }
    // Merge the per-thread pairs: across the warp by shuffles, across the four warps through shared memory.
    if (ok) {
#pragma unroll
      for (int b = 0; b < NB; ++b) {
        const float m = warp_max(run_m[b]);
        const float l = warp_sum(run_m[b] == -INFINITY ? 0.f : run_l[b] * __expf(run_m[b] - m));
        if (lane == 0) {
          red[(quad * NB + b) * 2] = m;
          red[(quad * NB + b) * 2 + 1] = l;
        }
      }
    }
    asm volatile("bar.sync 1, 128;" ::: "memory");
    if (ok && quad == 0) {
      for (int b = lane; b < NB; b += 32) {
        float m = -INFINITY;
        for (int q = 0; q < 4; ++q) m = fmaxf(m, red[(q * NB + b) * 2]);
        float l = 0.f;
        for (int q = 0; q < 4; ++q) {
          const float mq = red[(q * NB + b) * 2];
          l += (mq == -INFINITY) ? 0.f : red[(q * NB + b) * 2 + 1] * __expf(mq - m);
        }
        a.part_max[blockIdx.x * NB + b] = m;
        a.part_sum[blockIdx.x * NB + b] = l;
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// One warp per step.
// x_last[b] = x[last row of step b]: one warp per step.
__global__ void gather_last_rows_kernel(const float* __restrict__ x, const int32_t* __restrict__ cu_new,
                                        float* __restrict__ x_last, int B, int d) {
  pdl_launch_dependents();
  pdl_wait();
  const int b = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (b >= B) return;
  const float4* src = reinterpret_cast<const float4*>(x + static_cast<size_t>(cu_new[b + 1] - 1) * d);
  float4* dst = reinterpret_cast<float4*>(x_last + static_cast<size_t>(b) * d);
  for (int i = lane; i < d / 4; i += 32) dst[i] = src[i];
}

__global__ void last_rows_norm_kernel(const float* __restrict__ x, const int32_t* __restrict__ cu_new,
                                      const float* __restrict__ gain, uint16_t* __restrict__ h, int B, int B_pad,
                                      int d, float eps) {
  pdl_launch_dependents();
  pdl_wait();
  const int b = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (b >= B_pad) return;
  uint2* o = reinterpret_cast<uint2*>(h + static_cast<size_t>(b) * d);
  if (b >= B) {
    for (int i = lane; i < d / 4; i += 32) o[i] = make_uint2(0u, 0u);
    return;
  }
  const float4* xr = reinterpret_cast<const float4*>(x + static_cast<size_t>(cu_new ? cu_new[b + 1] - 1 : b) * d);
  float ss = 0.f;
  for (int i = lane; i < d / 4; i += 32) {
    const float4 v = xr[i];
    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
  }
  ss = warp_sum(ss);
  const float r = rsqrtf(ss / static_cast<float>(d) + eps);
  const float4* g4 = reinterpret_cast<const float4*>(gain);
  for (int i = lane; i < d / 4; i += 32) {
    const float4 v = xr[i];
    const float4 g = g4[i];
    o[i] = make_uint2(pack_f16x2(v.x * r * g.x, v.y * r * g.y), pack_f16x2(v.z * r * g.z, v.w * r * g.w));
  }
}

// One warp per step: merge the vocabulary slices, then confidence, decision and threshold (Eq. 4).
__global__ void gate_kernel(const float* __restrict__ part_max, const float* __restrict__ part_sum, int n_slices,
                            int nb_stride, const float* __restrict__ verdict_logits, int n_verdict, int B, float tau,
                            float* __restrict__ out_conf, uint8_t* __restrict__ out_accept,
                            int32_t* __restrict__ out_verdict, float* __restrict__ out_lse) {
  pdl_launch_dependents();
  pdl_wait();
  const int b = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (b >= B) return;
  float m = -INFINITY;
  for (int s = lane; s < n_slices; s += 32) m = fmaxf(m, part_max[s * nb_stride + b]);
  m = warp_max(m);
  float l = 0.f;
  for (int s = lane; s < n_slices; s += 32) {
    const float ms = part_max[s * nb_stride + b];
    if (ms != -INFINITY) l += part_sum[s * nb_stride + b] * expf(ms - m);
  }
  l = warp_sum(l);
  if (lane == 0) {
    const float lse = m + logf(l);
    float best = -1.f;
    int arg = 0;
    bool nan = false;
    for (int j = 0; j < n_verdict; ++j) {
      const float pj = expf(verdict_logits[b * n_verdict + j] - lse);
      if (pj != pj) nan = true;
      if (pj > best) { best = pj; arg = j; }
    }
    const float conf = nan ? __int_as_float(0x7fc00000) : best;
    out_conf[b] = conf;
    out_accept[b] = (conf >= tau) ? 1 : 0;   // false for NaN: such a step is escalated
    if (out_verdict) out_verdict[b] = arg;
    if (out_lse) out_lse[b] = lse;
  }
}

// Single CTA: flags, then an ordered compaction of the escalated indices by a block-wide scan.
// With req_start (linear drafting; req_start[i] = first step of step i's request) a step is listed only while its
// request is still open: Algorithm 1's loop over a request's steps breaks at the first rejection, so a step behind a
// trusted draft rejection (conf >= tau and verdict != accept_index at an earlier step of the request) is left out.
__global__ void escalate_kernel(const float* __restrict__ conf, int B, float tau, uint8_t* __restrict__ out_accept,
                                int32_t* __restrict__ out_idx, int32_t* __restrict__ out_count,
                                const int32_t* __restrict__ verdict_d, const int32_t* __restrict__ req_start,
                                int accept_index) {
  __shared__ int warp_tot[32];
  __shared__ int base;
  if (threadIdx.x == 0) base = 0;
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  for (int i0 = 0; i0 < B; i0 += blockDim.x) {
    const int i = i0 + threadIdx.x;
    int esc = 0;
    if (i < B) {
      const int acc = (conf[i] >= tau) ? 1 : 0;
      if (out_accept) out_accept[i] = static_cast<uint8_t>(acc);
      esc = 1 - acc;
      if (esc && req_start) {
        for (int j = req_start[i]; j < i; ++j)
          if (conf[j] >= tau && verdict_d[j] != accept_index) { esc = 0; break; }
      }
    }
    const unsigned ball = __ballot_sync(0xffffffffu, esc);
    const int before = __popc(ball & ((1u << lane) - 1u));
    if (lane == 0) warp_tot[warp] = __popc(ball);
    __syncthreads();
    int off = base;
    for (int w = 0; w < warp; ++w) off += warp_tot[w];
    if (esc) out_idx[off + before] = i;
    __syncthreads();
    if (threadIdx.x == 0) {
      int tot = 0;
      for (int w = 0; w < nw; ++w) tot += warp_tot[w];
      base += tot;
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) *out_count = base;
}

// Eq. 4 per step, after the target pass over the escalated steps only: idx[0 .. *count) lists those steps in
// ascending order and verdict_c / conf_c hold the target's results in that order. A trusted step keeps the draft's
// decision and gets (-1, 0) as its target result; an escalated one takes the target's.
__global__ void cascade_scatter_kernel(int B, const uint8_t* __restrict__ trusted, const int32_t* __restrict__ verdict_d,
                                       const float* __restrict__ conf_d, const int32_t* __restrict__ idx,
                                       const int32_t* __restrict__ count, const int32_t* __restrict__ verdict_c,
                                       const float* __restrict__ conf_c, int32_t* __restrict__ out_verdict_t,
                                       float* __restrict__ out_conf_t, int32_t* __restrict__ out_verdict,
                                       float* __restrict__ out_conf) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= B) return;
  int v = verdict_d[i], vt = -1;
  float c = conf_d[i], ct = 0.f;
  if (!trusted[i]) {
    const int n = *count;
    int lo = 0, hi = n;                 // position of i in the ascending list
    while (lo < hi) {
      const int mid = (lo + hi) >> 1;
      if (idx[mid] < i) lo = mid + 1; else hi = mid;
    }
    if (lo < n && idx[lo] == i) {
      vt = verdict_c[lo];
      ct = conf_c[lo];
    }
    v = vt;
    c = ct;
  }
  if (out_verdict_t) out_verdict_t[i] = vt;
  if (out_conf_t) out_conf_t[i] = ct;
  out_verdict[i] = v;
  out_conf[i] = c;
}

// One warp per request: final decision and confidence of each of its steps (Eq. 4), the length of the leading run
// of accepted steps (Algorithm 1's loop with break) and the accepted step with the highest confidence (Eq. 5).
__global__ void cascade_select_kernel(const uint8_t* __restrict__ trusted, const int32_t* __restrict__ verdict_d,
                                      const float* __restrict__ conf_d, const int32_t* __restrict__ verdict_t,
                                      const float* __restrict__ conf_t, const int32_t* __restrict__ req_offsets, int R,
                                      int accept_index, int32_t* __restrict__ out_prefix_len,
                                      int32_t* __restrict__ out_best, uint8_t* __restrict__ out_pass,
                                      float* __restrict__ out_conf) {
  pdl_launch_dependents();
  pdl_wait();
  const int r = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (r >= R) return;
  const int lo = req_offsets[r], hi = req_offsets[r + 1];
  int prefix = -1;                       // first rejected position, once found
  float best_c = -INFINITY;
  int best_i = -1;
  for (int i0 = lo; i0 < hi; i0 += 32) {
    const int i = i0 + lane;
    bool pass = false;
    float c = 0.f;
    if (i < hi) {
      if (trusted[i]) {
        pass = verdict_d[i] == accept_index;
        c = conf_d[i];
      } else if (verdict_t) {
        pass = verdict_t[i] == accept_index;
        c = conf_t[i];
      } else {
        c = conf_d[i];
      }
      if (out_pass) out_pass[i] = pass ? 1 : 0;
      if (out_conf) out_conf[i] = c;
    }
    const unsigned rejected = __ballot_sync(0xffffffffu, i < hi && !pass);
    if (prefix < 0 && rejected) prefix = i0 - lo + (__ffs(rejected) - 1);
    // highest confidence among the accepted steps, the earliest on ties (NaN never wins)
    float cand = (i < hi && pass && c == c) ? c : -INFINITY;
    int idx = (cand > -INFINITY) ? i : 0x7fffffff;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float oc = __shfl_xor_sync(0xffffffffu, cand, o);
      const int oi = __shfl_xor_sync(0xffffffffu, idx, o);
      if (oc > cand || (oc == cand && oi < idx)) { cand = oc; idx = oi; }
    }
    if (idx != 0x7fffffff && (best_i < 0 || cand > best_c)) { best_c = cand; best_i = idx; }
  }
  if (lane == 0) {
    out_prefix_len[r] = prefix < 0 ? hi - lo : prefix;
    out_best[r] = best_i;
  }
}

template <int NB>
cudaError_t launch_lm_nb(const CUtensorMap& tm_w, const CUtensorMap& tm_h, const LmArgs& a, int grid, cudaStream_t s) {
  using L = LmSmem<NB>;
  static std::atomic<uint64_t> smem_opted{0};
  if (cudaError_t e = opt_in_dynamic_smem(lm_head_kernel<NB>, L::kTotal, smem_opted); e != cudaSuccess) return e;
  cudaError_t le = launch_pdl(lm_head_kernel<NB>, dim3(grid), dim3(kLmThreads), L::kTotal, s, tm_w, tm_h, a);
  count_launch();
  return le != cudaSuccess ? le : cudaGetLastError();
}

}  // namespace

int lm_head_grid(int vocab, int* rows_per_cta) {
  const int n_tiles = (vocab + kLmBM - 1) / kLmBM;
  const int ctas = n_tiles < kNumSMs ? n_tiles : kNumSMs;
  const int rows = (vocab + ctas - 1) / ctas;
  *rows_per_cta = rows;
  return (vocab + rows - 1) / rows;
}

int lm_head_batch_pad(int B) { return B <= 16 ? 16 : (B <= 32 ? 32 : 64); }

cudaError_t launch_lm_head(const CUtensorMap& tm_w, const CUtensorMap& tm_h, int h_row0, int B, int B_pad, int d,
                           int vocab, const int32_t* verdict_ids_host, int n_verdict, float* part_max,
                           float* part_sum, float* verdict_logits, float* logits_or_null, uint32_t* status,
                           cudaStream_t s) {
  LmArgs a;
  a.B = B;
  a.h_row0 = h_row0;
  a.vocab = vocab;
  a.kblocks = (d + kLmBK - 1) / kLmBK;
  const int grid = lm_head_grid(vocab, &a.rows_per_cta);
  a.n_verdict = n_verdict;
  for (int j = 0; j < kLmMaxVerdict; ++j) a.verdict[j] = j < n_verdict ? verdict_ids_host[j] : -1;
  a.part_max = part_max;
  a.part_sum = part_sum;
  a.verdict_logits = verdict_logits;
  a.logits = logits_or_null;
  a.status = status;
  switch (B_pad) {
    case 16: return launch_lm_nb<16>(tm_w, tm_h, a, grid, s);
    case 32: return launch_lm_nb<32>(tm_w, tm_h, a, grid, s);
    case 64: return launch_lm_nb<64>(tm_w, tm_h, a, grid, s);
    default: return cudaErrorInvalidValue;
  }
}

cudaError_t launch_last_rows_norm(const float* x, const int32_t* cu_new, const float* gain, uint16_t* h, int B,
                                  int B_pad, int d, float eps, cudaStream_t s) {
  const int warps = 4;
  last_rows_norm_kernel<<<(B_pad + warps - 1) / warps, warps * 32, 0, s>>>(x, cu_new, gain, h, B, B_pad, d, eps);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_gather_last_rows(const float* x, const int32_t* cu_new, float* x_last, int B, int d, cudaStream_t s) {
  if (B <= 0) return cudaSuccess;
  const int warps = 4;
  cudaError_t le = launch_pdl(gather_last_rows_kernel, dim3((B + warps - 1) / warps), dim3(warps * 32), 0, s, x, cu_new,
                              x_last, B, d);
  count_launch();
  return le != cudaSuccess ? le : cudaGetLastError();
}

cudaError_t launch_gate(const float* part_max, const float* part_sum, int n_slices, int nb_stride,
                        const float* verdict_logits, int n_verdict, int B, float tau, float* out_conf,
                        uint8_t* out_accept, int32_t* out_verdict, float* out_lse, cudaStream_t s) {
  const int warps = 4;
  gate_kernel<<<(B + warps - 1) / warps, warps * 32, 0, s>>>(part_max, part_sum, n_slices, nb_stride, verdict_logits,
                                                           n_verdict, B, tau, out_conf, out_accept, out_verdict,
                                                           out_lse);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_cascade_select(const uint8_t* trusted, const int32_t* verdict_d, const float* conf_d,
                                  const int32_t* verdict_t, const float* conf_t, const int32_t* req_offsets, int R,
                                  int accept_index, int32_t* out_prefix_len, int32_t* out_best, uint8_t* out_pass,
                                  float* out_conf, cudaStream_t s) {
  if (R <= 0) return cudaSuccess;
  const int warps = 4;
  cascade_select_kernel<<<(R + warps - 1) / warps, warps * 32, 0, s>>>(trusted, verdict_d, conf_d, verdict_t, conf_t,
                                                                     req_offsets, R, accept_index, out_prefix_len,
                                                                     out_best, out_pass, out_conf);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_cascade_scatter(int B, const uint8_t* trusted, const int32_t* verdict_d, const float* conf_d,
                                   const int32_t* idx, const int32_t* count, const int32_t* verdict_c,
                                   const float* conf_c, int32_t* out_verdict_t, float* out_conf_t,
                                   int32_t* out_verdict, float* out_conf, cudaStream_t s) {
  if (B <= 0) return cudaSuccess;
  cascade_scatter_kernel<<<(B + 127) / 128, 128, 0, s>>>(B, trusted, verdict_d, conf_d, idx, count, verdict_c, conf_c,
                                                         out_verdict_t, out_conf_t, out_verdict, out_conf);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_escalate(const float* conf, int B, float tau, uint8_t* out_accept, int32_t* out_idx,
                            int32_t* out_count, cudaStream_t s, const int32_t* verdict_d, const int32_t* req_start,
                            int accept_index) {
  escalate_kernel<<<1, 1024, 0, s>>>(conf, B, tau, out_accept, out_idx, out_count, verdict_d, req_start, accept_index);
  count_launch();
  return cudaGetLastError();
}

}  // namespace cs

// ------------------------------------------------------------------------------------------------------------------
// cs_lm_head_gate_static: the LM-head + gate stage for callers that must not allocate device memory.
// ------------------------------------------------------------------------------------------------------------------
#include "../../include/confspec.h"

#include "gemm.h"

namespace {

constexpr int kStaticMaxSteps = CS_LM_HEAD_STATIC_MAX_STEPS;
constexpr int kStaticPartFloats = 2 * cs::kNumSMs * kStaticMaxSteps;      // per-CTA (max, sum exp) pairs
constexpr int kStaticVerdictFloats = kStaticMaxSteps * 8;                 // logits of the verdict ids
constexpr int kStaticStatusFloats = 64;                                   // status word, padded to 256 bytes
constexpr int kStaticFloats = kStaticPartFloats + kStaticVerdictFloats + kStaticStatusFloats;

// The scratch of the no-allocation entry point: about 78 KB that every GPU which loads the library holds until the
// process exits. In host code this name is only a handle; the device address comes from cudaGetSymbolAddress.
static __device__ __align__(256) float g_lm_static_scratch[kStaticFloats];

constexpr int kMaxDevices = 64;
float* g_lm_static_ptr[kMaxDevices] = {};

// A pass that gave up on a bounded wait leaves no usable numbers: make that visible in the outputs themselves.
__global__ void poison_on_timeout_kernel(const uint32_t* status, float* out_conf, uint8_t* out_accept,
                                         int32_t* out_verdict, float* out_lse, int B) {
  if (*status == 0) return;
  for (int i = threadIdx.x; i < B; i += blockDim.x) {
    out_conf[i] = __int_as_float(0x7fc00000);
    out_accept[i] = 0;
    if (out_verdict) out_verdict[i] = -1;
    if (out_lse) out_lse[i] = __int_as_float(0x7fc00000);
  }
}

}  // namespace

extern "C" int cs_lm_head_gate_static(const uint16_t* w_lm, const uint16_t* h, int B, int d_model, int vocab,
                                      const int32_t* verdict_ids, int n_verdict, float tau, float* out_conf,
                                      uint8_t* out_accept, int32_t* out_verdict, float* out_lse, void* stream) {
  using namespace cs;
  if (!w_lm || !h || B < 0 || d_model < 8 || (d_model % 8) || vocab < 1 || tau != tau) return CS_EINVAL;
  if (n_verdict < 1 || n_verdict > 8 || !verdict_ids) return CS_EINVAL;
  for (int j = 0; j < n_verdict; ++j)
    if (verdict_ids[j] < 0 || verdict_ids[j] >= vocab) return CS_EINVAL;
  if (B > kStaticMaxSteps) return CS_ELIMIT;
  if (B == 0) return CS_OK;
  if (!out_conf || !out_accept) return CS_EINVAL;

  // Set-up, once per device, with that device current: the device address of the scratch array.
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return CS_ECUDA;
  if (!g_lm_static_ptr[dev]) {
    float* ptr = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_lm_static_scratch) != cudaSuccess || !ptr) {
      cudaGetLastError();
      return CS_ECUDA;
    }
    g_lm_static_ptr[dev] = ptr;
  }
  float* scratch = g_lm_static_ptr[dev];
  float* part_max = scratch;
  float* part_sum = scratch + kNumSMs * kStaticMaxSteps;
  float* vlog = scratch + kStaticPartFloats;
  uint32_t* status = reinterpret_cast<uint32_t*>(scratch + kStaticPartFloats + kStaticVerdictFloats);

  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // The array keeps what the previous call left. The partial pairs and the verdict logits are overwritten in full
  // by this call; the status word is the one thing that must start at zero.
  if (cudaMemsetAsync(status, 0, sizeof(uint32_t), s) != cudaSuccess) { cudaGetLastError(); return CS_ECUDA; }
  CUtensorMap tm_w, tm_h;
  const int bp = lm_head_batch_pad(B);
  if (!make_gemm_operand_map(&tm_w, w_lm, vocab, d_model) ||
      !make_tensor_map_16b(&tm_h, h, B, d_model, bp, 64, true, false))      // rows past B read as zeros
    return CS_ECUDA;
  int rows_per_cta;
  const int grid = lm_head_grid(vocab, &rows_per_cta);
  if (launch_lm_head(tm_w, tm_h, 0, B, bp, d_model, vocab, verdict_ids, n_verdict, part_max, part_sum, vlog, nullptr,
                     status, s) != cudaSuccess ||
      launch_gate(part_max, part_sum, grid, bp, vlog, n_verdict, B, tau, out_conf, out_accept, out_verdict, out_lse,
                  s) != cudaSuccess) {
    cudaGetLastError();
    return CS_ECUDA;
  }
  poison_on_timeout_kernel<<<1, 64, 0, s>>>(status, out_conf, out_accept, out_verdict, out_lse, B);
  count_launch();
  if (cudaGetLastError() != cudaSuccess) return CS_ECUDA;
  return CS_OK;
}
