// Launchers of the non-GEMM kernels of the verification pass. All are asynchronous on `stream`.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

namespace cs {

constexpr int kNumSMs = 148;

// Opt-in to more than 48 KB of dynamic shared memory. cudaFuncSetAttribute applies to the CURRENT device only, so
// the "already done" flag is kept per device (one bit each; devices beyond 63 simply set the attribute every time).
// Setting it twice is harmless, so two host threads racing on the first call need no lock.
template <typename Kernel>
cudaError_t opt_in_dynamic_smem(Kernel kernel, int bytes, std::atomic<uint64_t>& done) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const bool tracked = dev >= 0 && dev < 64;
  if (tracked && (done.load(std::memory_order_relaxed) >> dev & 1ull)) return cudaSuccess;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess && tracked) done.fetch_or(1ull << dev, std::memory_order_relaxed);
  return e;
}

// One unit of attention work: the query rows of 128 / G consecutive new tokens of one step for the G query
// heads of one kv head (row = token * G + head-in-group, at most 128 rows), over a range of 128-key tiles.
// Key tiles 0 .. ctx_tiles-1 cover the cached context (8 pages each), the following ones the step's own
// new keys. A query tile whose key range is cut into n_splits > 1 pieces owns the partial-result slots
// [slot0, slot0 + n_splits) and the counter counters[slot0].
struct AttnItem {
  int32_t step;       // index into the batch
  int32_t kv_head;
  int32_t q_tok0;     // first new token of the query tile, relative to the step (multiple of 128 / G)
  int32_t tile_begin; // key tile range [tile_begin, tile_end)
  int32_t tile_end;
  int32_t slot;       // this piece's partial-result slot (unused when n_splits == 1)
  int32_t slot0;      // first slot of the query tile
  int32_t n_splits;   // pieces the query tile's key range is cut into (1 = whole range, at most 32)
  int32_t tok0;       // first row of the step in the batch's token order
  int32_t n_new;      // new tokens of the step
  int32_t ctx;        // cached context length of the step's sequence
  int32_t seq;        // row of the page table
  int32_t pad[4];
};

struct AttnParams {
  const uint16_t* qkv;      // [T, n_qkv] fp16: q heads, k heads, v heads (q, k already rotated)
  uint16_t* out;            // [T, Hq*hd] fp16
  const int32_t* page_table;// [max_seqs, max_pages_per_seq]
  int32_t max_pages_per_seq;
  int32_t n_q_heads, n_kv_heads, head_dim, n_qkv;
  int32_t k_group_base, v_group_base;  // first 8-row group of this layer's K and V planes in the pool
  float scale_log2e;        // log2(e) / sqrt(head_dim)
  float* part_o;            // [slots, 128, hd] unnormalised partial outputs
  float* part_ml;           // [slots, 128, 2]  exponent reference (raw score units) and sum
  int32_t* counters;        // [slots] zero between launches
  uint32_t* status;
  int32_t num_pages;        // pages of the pool and rows of the qkv workspace in use: range checks of debug builds
  int32_t n_rows;
};

cudaError_t launch_embed(const int32_t* tokens, const uint16_t* embed, float* x, int T, int d, int vocab,
                         uint32_t* status, cudaStream_t s);
cudaError_t launch_rmsnorm(const float* x, const float* gain, uint16_t* out, int rows, int d, float eps,
                           cudaStream_t s);
// cos/sin of pos[t] * inv_freq[j] in double, stored as float2 [T, half].
cudaError_t launch_rope_table(const int32_t* pos, const double* inv_freq, float2* table, int T, int half,
                              cudaStream_t s);
// Copy K and V rows into cache pages. src rows are [n_kv_heads*hd] wide at src_k/src_v + t*row_stride.
// Row t goes to sequence tok_seq[t], position tok_pos[t]; when tok_seq is NULL, to sequence const_seq,
// position pos0 + t. The cache holds bf16 values in the fp16 encoding: bf16 sources are re-encoded (exact in
// the fp16 normal range), fp16 sources are first rounded to the nearest bf16 value.
cudaError_t launch_kv_scatter(const uint16_t* src_k, const uint16_t* src_v, int row_stride, const int32_t* tok_seq,
                              const int32_t* tok_pos, int const_seq, int pos0, const int32_t* page_table,
                              int max_pages_per_seq,
                              uint16_t* pool_k_plane, uint16_t* pool_v_plane, int n_kv_heads, int hd, int page_size,
                              int T, int src_is_f16, int num_pages, uint32_t* status, cudaStream_t s);
// Re-encode n bf16 values (n even) as fp16 in place.
cudaError_t launch_bf16_to_f16(uint16_t* p, size_t n, cudaStream_t s);

// tm_pool: 4D map of the cache (make_kv_group_map over all pool rows, one 16-row page per box); tm_kv_new: the
// same kind of map over the qkv workspace (128 rows per box; see make_kv_rows_map); tm_q3d: 3D map (head_dim,
// head, token) of the workspace with box (64, G, 128 / G).
cudaError_t launch_attention(const AttnParams& p, const CUtensorMap& tm_pool, const CUtensorMap& tm_kv_new,
                             const CUtensorMap& tm_q3d, const AttnItem* items, int n_items, cudaStream_t s);
int attention_max_splits();
// Short steps over an 8-bit cache (attention_short.cu). Items reuse AttnItem with [tile_begin, tile_end) counted in
// 16-key PAGES of the cached context; the piece with slot == slot0 + n_splits - 1 also covers the step's own keys.
// pool_k / pool_v: this layer's planes, K [pages][kv heads][16][head_dim] codes, V [pages][kv heads][head_dim][16]. max_rows = the largest n_new * G of
// the batch (<= 32); e5m2 selects the 5-exponent-bit format (else 4 exponent / 3 mantissa bits). Partial results: part_o [slots][32][head_dim], part_ml [slots][32][2].
cudaError_t launch_attention_short(const AttnParams& p, const uint8_t* pool_k, const uint8_t* pool_v,
                                   const AttnItem* items, int n_items, int max_rows, bool any_split, bool e5m2,
                                   cudaStream_t s);
// Codes of an 8-bit cache into their pages (V transposed within the page): thread per 16 bytes; rows of src are
// [n_kv_heads * hd] codes.
cudaError_t launch_kv_scatter_u8(const uint8_t* src_k, const uint8_t* src_v, int seq, const int32_t* page_table,
                                 int max_pages_per_seq, uint8_t* pool_k_plane, uint8_t* pool_v_plane, int n_kv_heads,
                                 int hd, int page_size, int T, cudaStream_t s);

// x_last[b] = x[cu_new[b + 1] - 1], fp32 [B, d].
cudaError_t launch_gather_last_rows(const float* x, const int32_t* cu_new, float* x_last, int B, int d, cudaStream_t s);
// h[b] = RMSNorm(x[last_row[b]]) as bf16 [B_pad, d]; rows B..B_pad-1 are zeroed. cu_new == nullptr: row b itself.
cudaError_t launch_last_rows_norm(const float* x, const int32_t* cu_new, const float* gain, uint16_t* h, int B,
                                  int B_pad, int d, float eps, cudaStream_t s);
// LM head over 128-row vocabulary tiles (tcgen05): per CTA and step the maximum and the sum of exp(z - max)
// of the CTA's rows, the logits of the verdict ids, and optionally all logits. h rows [h_row0, h_row0 + B_pad)
// of the tensor map tm_h are the batch; B_pad is 16, 32 or 64. part_max / part_sum are [grid, B_pad].
cudaError_t launch_lm_head(const CUtensorMap& tm_w, const CUtensorMap& tm_h, int h_row0, int B, int B_pad, int d,
                           int vocab, const int32_t* verdict_ids_host, int n_verdict, float* part_max,
                           float* part_sum, float* verdict_logits, float* logits_or_null, uint32_t* status,
                           cudaStream_t s);
// Grid of the LM-head launch: the vocabulary is cut evenly into one range of rows per CTA.
int lm_head_grid(int vocab, int* rows_per_cta);
int lm_head_batch_pad(int B);
// Merge the CTAs' pairs, form the confidence and apply the threshold.
cudaError_t launch_gate(const float* part_max, const float* part_sum, int n_slices, int nb_stride,
                        const float* verdict_logits, int n_verdict, int B, float tau, float* out_conf,
                        uint8_t* out_accept, int32_t* out_verdict, float* out_lse, cudaStream_t s);
cudaError_t launch_cascade_select(const uint8_t* trusted, const int32_t* verdict_d, const float* conf_d,
                                  const int32_t* verdict_t, const float* conf_t, const int32_t* req_offsets, int R,
                                  int accept_index, int32_t* out_prefix_len, int32_t* out_best, uint8_t* out_pass,
                                  float* out_conf, cudaStream_t s);
// verdict_d / req_start non-null: steps behind a trusted rejection of their request are not listed (see the kernel).
cudaError_t launch_escalate(const float* conf, int B, float tau, uint8_t* out_accept, int32_t* out_idx,
                            int32_t* out_count, cudaStream_t s, const int32_t* verdict_d = nullptr,
                            const int32_t* req_start = nullptr, int accept_index = 0);
// Results of the target pass (compact, over the escalated steps idx[0 .. *count)) back to batch order, and the
// final decision of Eq. 4 for every step.
cudaError_t launch_cascade_scatter(int B, const uint8_t* trusted, const int32_t* verdict_d, const float* conf_d,
                                   const int32_t* idx, const int32_t* count, const int32_t* verdict_c,
                                   const float* conf_c, int32_t* out_verdict_t, float* out_conf_t,
                                   int32_t* out_verdict, float* out_conf, cudaStream_t s);

// Evaluates one range check that fails by construction (no memory is touched): in a debug build the status word gets
// its range bit, in a release build nothing happens.
cudaError_t launch_range_check_selftest(uint32_t* status, cudaStream_t s);

// Failure-detection self-test: a bounded wait that is made to run out (see cs_selftest_wait_timeout).
cudaError_t launch_wait_timeout_selftest(uint32_t* status, uint32_t limit, int32_t* gave_up, cudaStream_t s);

// Launch with programmatic stream serialisation (see pdl_wait in common.cuh).
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

void count_launch(int n = 1);
int64_t take_launch_count();

}  // namespace cs
