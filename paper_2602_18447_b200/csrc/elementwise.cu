// Memory-bound pieces of the decoder layers: embedding gather, RMSNorm, rotary tables (the rotation itself is the
// epilogue of the QKV projection), and the scatter of K/V rows into cache pages.
#include "kernels.h"

#include "common.cuh"

namespace cs {

namespace {

thread_local int64_t g_launches = 0;

__global__ void embed_kernel(const int32_t* __restrict__ tokens, const uint16_t* __restrict__ embed,
                             float* __restrict__ x, int T, int d, int vocab, uint32_t* status) {
  pdl_launch_dependents();
  pdl_wait();
  const int t = blockIdx.x;
  int tok = tokens[t];
  if (threadIdx.x == 0) debug_in_range(tok >= 0 && tok < vocab, status);
  tok = tok < 0 ? 0 : (tok >= vocab ? vocab - 1 : tok);
  const uint4* src = reinterpret_cast<const uint4*>(embed + static_cast<size_t>(tok) * d);
  float4* dst = reinterpret_cast<float4*>(x + static_cast<size_t>(t) * d);
  for (int i = threadIdx.x; i < d / 8; i += blockDim.x) {
    const uint4 v = src[i];
    dst[2 * i] = make_float4(bf16_lo(v.x), bf16_hi(v.x), bf16_lo(v.y), bf16_hi(v.y));
    dst[2 * i + 1] = make_float4(bf16_lo(v.z), bf16_hi(v.z), bf16_lo(v.w), bf16_hi(v.w));
  }
}

// One warp per row. A row of up to 128 NV values is held in registers between the sum of squares and the scaling, so x
// is read once and all of a row's loads are in flight together; longer rows are read twice. The gains are requested
// together with the row (while they fit the register file): the kernel moves a few MB and lasts as long as its
// longest chain of dependent memory accesses.
template <int NV>
__global__ void rmsnorm_kernel(const float* __restrict__ x, const float* __restrict__ gain,
                               uint16_t* __restrict__ out, int rows, int d, float eps) {
  pdl_launch_dependents();
  pdl_wait();
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= rows) return;
  const float4* xr = reinterpret_cast<const float4*>(x + static_cast<size_t>(row) * d);
  const float4* g4 = reinterpret_cast<const float4*>(gain);
  uint2* o = reinterpret_cast<uint2*>(out + static_cast<size_t>(row) * d);
  const int n = d >> 2;
  if (n <= 32 * NV) {
    constexpr bool kGainsAhead = NV <= 16;
    float4 v[NV], gv[kGainsAhead ? NV : 1];
    float ss = 0.f;
#pragma unroll
    for (int i = 0; i < NV; ++i) {
      const int idx = lane + 32 * i;
      if (idx < n) v[i] = xr[idx];
    }
    if (kGainsAhead) {
#pragma unroll
      for (int i = 0; i < NV; ++i) {
        const int idx = lane + 32 * i;
        if (idx < n) gv[kGainsAhead ? i : 0] = __ldg(g4 + idx);
      }
    }
#pragma unroll
    for (int i = 0; i < NV; ++i)
      if (lane + 32 * i < n) ss += v[i].x * v[i].x + v[i].y * v[i].y + v[i].z * v[i].z + v[i].w * v[i].w;
    ss = warp_sum(ss);
    const float r = rsqrtf(ss / static_cast<float>(d) + eps);
#pragma unroll
    for (int i = 0; i < NV; ++i) {
      const int idx = lane + 32 * i;
      if (idx < n) {
        const float4 g = kGainsAhead ? gv[kGainsAhead ? i : 0] : __ldg(g4 + idx);
        o[idx] = make_uint2(pack_f16x2(v[i].x * r * g.x, v[i].y * r * g.y), pack_f16x2(v[i].z * r * g.z, v[i].w * r * g.w));
      }
    }
    return;
  }
  float ss = 0.f;
  for (int i = lane; i < n; i += 32) {
    const float4 v = xr[i];
    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
  }
  ss = warp_sum(ss);
  const float r = rsqrtf(ss / static_cast<float>(d) + eps);
  for (int i = lane; i < n; i += 32) {
    const float4 v = xr[i];
    const float4 g = g4[i];
    o[i] = make_uint2(pack_f16x2(v.x * r * g.x, v.y * r * g.y), pack_f16x2(v.z * r * g.z, v.w * r * g.w));
  }
}

__global__ void rope_table_kernel(const int32_t* __restrict__ pos, const double* __restrict__ inv_freq,
                                  float2* __restrict__ table, int T, int half) {
  pdl_launch_dependents();
  pdl_wait();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= T * half) return;
  const int t = i / half, j = i - t * half;
  double s, c;
  sincos(static_cast<double>(pos[t]) * inv_freq[j], &s, &c);
  table[i] = make_float2(static_cast<float>(c), static_cast<float>(s));
}

// Thread per 16 bytes of a K row and of a V row.
__global__ void kv_scatter_kernel(const uint16_t* __restrict__ src_k, const uint16_t* __restrict__ src_v,
                                  int row_stride, const int32_t* __restrict__ tok_seq,
                                  const int32_t* __restrict__ tok_pos, int const_seq, int pos0,
                                  const int32_t* __restrict__ page_table,
                                  int max_pages_per_seq, uint16_t* __restrict__ pool_k, uint16_t* __restrict__ pool_v,
                                  int n_kv_heads, int hd, int page_size, int T, int src_is_f16, int num_pages,
                                  uint32_t* status) {
  pdl_launch_dependents();
  pdl_wait();
  const int chunks = n_kv_heads * hd / 8;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= T * chunks) return;
  const int t = i / chunks;
  const int c = i - t * chunks;
  const int head = (c * 8) / hd;
  const int e = c * 8 - head * hd;
  const int pos = tok_seq ? tok_pos[t] : pos0 + t;
  const int seq = tok_seq ? tok_seq[t] : const_seq;
  if (!debug_in_range(pos >= 0 && pos / page_size < max_pages_per_seq, status)) return;
  const int page = page_table[static_cast<size_t>(seq) * max_pages_per_seq + pos / page_size];
  if (!debug_in_range(page >= 0 && page < num_pages, status)) return;
  const int slot = pos % page_size;
  const size_t dst = ((static_cast<size_t>(page) * n_kv_heads + head) * page_size + slot) * hd + e;
  const size_t src = static_cast<size_t>(t) * row_stride + c * 8;
  uint4 k = *reinterpret_cast<const uint4*>(src_k + src);
  uint4 v = *reinterpret_cast<const uint4*>(src_v + src);
  if (src_is_f16) {  // the cache keeps bf16 precision: round the fp16 activations to the nearest bf16 value
    k = make_uint4(f16x2_to_bf16x2(k.x), f16x2_to_bf16x2(k.y), f16x2_to_bf16x2(k.z), f16x2_to_bf16x2(k.w));
    v = make_uint4(f16x2_to_bf16x2(v.x), f16x2_to_bf16x2(v.y), f16x2_to_bf16x2(v.z), f16x2_to_bf16x2(v.w));
  }
  // ... and stores those bf16 values in the fp16 encoding, the operand format of the attention products
  k = make_uint4(bf16x2_to_f16x2(k.x), bf16x2_to_f16x2(k.y), bf16x2_to_f16x2(k.z), bf16x2_to_f16x2(k.w));
  v = make_uint4(bf16x2_to_f16x2(v.x), bf16x2_to_f16x2(v.y), bf16x2_to_f16x2(v.z), bf16x2_to_f16x2(v.w));
  *reinterpret_cast<uint4*>(pool_k + dst) = k;
  *reinterpret_cast<uint4*>(pool_v + dst) = v;
}

__global__ void kv_scatter_u8_kernel(const uint8_t* __restrict__ src_k, const uint8_t* __restrict__ src_v, int seq,
                                     const int32_t* __restrict__ page_table, int max_pages_per_seq,
                                     uint8_t* __restrict__ pool_k, uint8_t* __restrict__ pool_v, int n_kv_heads, int hd,
                                     int page_size, int T) {
  const int chunks = n_kv_heads * hd / 16;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= T * chunks) return;
  const int t = i / chunks;
  const int c = i - t * chunks;
  const int head = (c * 16) / hd;
  const int e = c * 16 - head * hd;
  const int page = page_table[static_cast<size_t>(seq) * max_pages_per_seq + t / page_size];
  const int slot = t % page_size;
  const size_t dst = ((static_cast<size_t>(page) * n_kv_heads + head) * page_size + slot) * hd + e;
  const size_t src = static_cast<size_t>(t) * n_kv_heads * hd + c * 16;
  *reinterpret_cast<uint4*>(pool_k + dst) = *reinterpret_cast<const uint4*>(src_k + src);
  // V pages are kept transposed, [hd][page_size]: the short-step attention reads four consecutive keys of one column
  const uint4 vv = *reinterpret_cast<const uint4*>(src_v + src);
  const uint32_t w[4] = {vv.x, vv.y, vv.z, vv.w};
  uint8_t* vt = pool_v + (static_cast<size_t>(page) * n_kv_heads + head) * page_size * hd;
#pragma unroll
  for (int j = 0; j < 16; ++j) vt[static_cast<size_t>(e + j) * page_size + slot] = static_cast<uint8_t>(w[j >> 2] >> (8 * (j & 3)));
}

// In-place re-encoding of bf16 bit patterns as fp16 (same size). Exact for magnitudes in [2^-14, 65504];
// smaller values round to the fp16 subnormal grid (absolute error <= 2^-25).
__global__ void bf16_to_f16_kernel(uint32_t* __restrict__ p, size_t n_pairs) {
  for (size_t i = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x; i < n_pairs;
       i += static_cast<size_t>(gridDim.x) * blockDim.x)
    p[i] = bf16x2_to_f16x2(p[i]);
}

// One thread waits, with the library's bounded wait, on a barrier of its own that nothing ever arrives at: the wait
// runs out after `limit` polls, raises the time-out bit of the status word and the kernel returns normally.
__global__ void wait_timeout_selftest_kernel(uint32_t* status, uint32_t limit, int32_t* gave_up) {
  __shared__ uint64_t bar;
  __shared__ uint32_t abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    abort_flag = 0;
    fence_barrier_init();
    const bool ok = mbar_wait_limited(&bar, 0, &abort_flag, status, limit);
    *gave_up = ok ? 0 : 1;
  }
}

__global__ void range_check_selftest_kernel(uint32_t* status) {
  const int index = 7, extent = 4;                  // out of range by construction; nothing is accessed
  debug_in_range(index < extent, status);
}

}  // namespace

cudaError_t launch_range_check_selftest(uint32_t* status, cudaStream_t s) {
  range_check_selftest_kernel<<<1, 1, 0, s>>>(status);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_wait_timeout_selftest(uint32_t* status, uint32_t limit, int32_t* gave_up, cudaStream_t s) {
  wait_timeout_selftest_kernel<<<1, 32, 0, s>>>(status, limit, gave_up);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_bf16_to_f16(uint16_t* p, size_t n, cudaStream_t s) {
  if (n == 0) return cudaSuccess;
  bf16_to_f16_kernel<<<1184, 256, 0, s>>>(reinterpret_cast<uint32_t*>(p), n / 2);
  return cudaGetLastError();
}

void count_launch(int n) { g_launches += n; }
int64_t take_launch_count() {
  const int64_t v = g_launches;
  g_launches = 0;
  return v;
}

cudaError_t launch_embed(const int32_t* tokens, const uint16_t* embed, float* x, int T, int d, int vocab,
                         uint32_t* status, cudaStream_t s) {
  if (T <= 0) return cudaSuccess;
  cudaError_t le = launch_pdl(embed_kernel, dim3(T), dim3(128), 0, s, tokens, embed, x, T, d, vocab, status);
  count_launch();
  return le != cudaSuccess ? le : cudaGetLastError();
}

cudaError_t launch_rmsnorm(const float* x, const float* gain, uint16_t* out, int rows, int d, float eps,
                           cudaStream_t s) {
  if (rows <= 0) return cudaSuccess;
  const int warps = 4;
  const dim3 grid((rows + warps - 1) / warps), block(warps * 32);
  cudaError_t le;
  if (d <= 1024) le = launch_pdl(rmsnorm_kernel<8>, grid, block, 0, s, x, gain, out, rows, d, eps);
  else if (d <= 2048) le = launch_pdl(rmsnorm_kernel<16>, grid, block, 0, s, x, gain, out, rows, d, eps);
  else le = launch_pdl(rmsnorm_kernel<32>, grid, block, 0, s, x, gain, out, rows, d, eps);
  count_launch();
  return le != cudaSuccess ? le : cudaGetLastError();
}

cudaError_t launch_rope_table(const int32_t* pos, const double* inv_freq, float2* table, int T, int half,
                              cudaStream_t s) {
  if (T <= 0) return cudaSuccess;
  const int n = T * half;
  cudaError_t le = launch_pdl(rope_table_kernel, dim3((n + 255) / 256), dim3(256), 0, s, pos, inv_freq, table, T, half);
  count_launch();
  return le != cudaSuccess ? le : cudaGetLastError();
}

cudaError_t launch_kv_scatter(const uint16_t* src_k, const uint16_t* src_v, int row_stride, const int32_t* tok_seq,
                              const int32_t* tok_pos, int const_seq, int pos0, const int32_t* page_table,
                              int max_pages_per_seq,
                              uint16_t* pool_k_plane, uint16_t* pool_v_plane, int n_kv_heads, int hd, int page_size,
                              int T, int src_is_f16, int num_pages, uint32_t* status, cudaStream_t s) {
  if (T <= 0) return cudaSuccess;
  const int n = T * n_kv_heads * hd / 8;
  kv_scatter_kernel<<<(n + 255) / 256, 256, 0, s>>>(src_k, src_v, row_stride, tok_seq, tok_pos, const_seq, pos0, page_table,
                                                    max_pages_per_seq, pool_k_plane, pool_v_plane, n_kv_heads, hd,
                                                    page_size, T, src_is_f16, num_pages, status);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_kv_scatter_u8(const uint8_t* src_k, const uint8_t* src_v, int seq, const int32_t* page_table,
                                 int max_pages_per_seq, uint8_t* pool_k_plane, uint8_t* pool_v_plane, int n_kv_heads,
                                 int hd, int page_size, int T, cudaStream_t s) {
  if (T <= 0) return cudaSuccess;
  const int n = T * n_kv_heads * hd / 16;
  kv_scatter_u8_kernel<<<(n + 255) / 256, 256, 0, s>>>(src_k, src_v, seq, page_table, max_pages_per_seq, pool_k_plane,
                                                       pool_v_plane, n_kv_heads, hd, page_size, T);
  count_launch();
  return cudaGetLastError();
}

}  // namespace cs
