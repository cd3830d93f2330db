// C ABI of the library: handles, argument checks, host-side batch metadata and the launch sequence.
#include "../../include/confspec.h"

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "gemm.h"
#include "kernels.h"

using namespace cs;

namespace {

thread_local std::string g_cuda_error;

int cuda_fail(cudaError_t e, const char* what) {
  g_cuda_error = std::string(what) + ": " + cudaGetErrorString(e);
  cudaGetLastError();
  return e == cudaErrorMemoryAllocation ? CS_ENOMEM : CS_ECUDA;
}
#define CS_CUDA(call)                                     \
  do {                                                    \
    cudaError_t e__ = (call);                             \
    if (e__ != cudaSuccess) return cuda_fail(e__, #call); \
  } while (0)

constexpr int kPageSize = 16;
constexpr int kStagingRing = 4;

struct LayerDev {
  uint16_t *wqkv, *wo, *wg, *wu, *wd;
  float *norm1, *norm2;
  float* qk_gain = nullptr;   // [2 * head_dim]: query gains then key gains; null when the family has no such norm
  CUtensorMap tm_wqkv, tm_wo, tm_wg, tm_wu, tm_wd;
};

// A workspace buffer. Behind its `cap` usable bytes lie kCanaryBytes of a fixed pattern that nothing may write: a
// kernel that runs past the end of a workspace disturbs them, which cs_check_workspace finds.
constexpr size_t kCanaryBytes = 256;
constexpr int kCanaryByte = 0xC5;

struct DevBuf {
  void* p = nullptr;
  size_t cap = 0;
  int ensure(size_t bytes, bool zero = false) {
    if (bytes <= cap) return CS_OK;
    if (p) {
      cudaDeviceSynchronize();
      cudaFree(p);
      p = nullptr;
      cap = 0;
    }
    const size_t want = ((bytes + bytes / 4 + 256) + 255) & ~static_cast<size_t>(255);
    cudaError_t e = cudaMalloc(&p, want + kCanaryBytes);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMalloc(workspace)");
    if (zero && (e = cudaMemset(p, 0, want)) != cudaSuccess) return cuda_fail(e, "cudaMemset(workspace)");
    if ((e = cudaMemset(static_cast<uint8_t*>(p) + want, kCanaryByte, kCanaryBytes)) != cudaSuccess)
      return cuda_fail(e, "cudaMemset(workspace canary)");
    cap = want;
    return CS_OK;
  }
  // 0 = intact, 1 = disturbed, -1 = the read-back failed
  int canary_state(cudaStream_t s) const {
    if (!p) return 0;
    uint8_t h[kCanaryBytes];
    if (cudaMemcpyAsync(h, static_cast<const uint8_t*>(p) + cap, kCanaryBytes, cudaMemcpyDeviceToHost, s) != cudaSuccess ||
        cudaStreamSynchronize(s) != cudaSuccess)
      return -1;
    for (size_t i = 0; i < kCanaryBytes; ++i)
      if (h[i] != kCanaryByte) return 1;
    return 0;
  }
  void release() {
    if (p) cudaFree(p);
    p = nullptr;
    cap = 0;
  }
};

// Optional per-kernel-class timing: a pair of events around every launch of the pass.
enum ProfClass { kProfEmbed = 0, kProfNorm, kProfQkv, kProfRope, kProfAttn, kProfO, kProfGateUp, kProfDown,
                 kProfLmHead, kProfGate, kProfOther, kProfClasses };
struct Prof {
  bool on = false;
  std::vector<cudaEvent_t> pool;   // events, used in pairs
  std::vector<int> cls;            // class of pair i
  size_t used = 0;                 // pairs in use
};

struct Staging {
  int32_t* host[kStagingRing] = {nullptr, nullptr, nullptr, nullptr};
  size_t host_cap[kStagingRing] = {0, 0, 0, 0};
  cudaEvent_t ev[kStagingRing] = {nullptr, nullptr, nullptr, nullptr};
  bool pending[kStagingRing] = {false, false, false, false};
  int next = 0;
  DevBuf dev;
};

}  // namespace

struct cs_model {
  cs_model_desc d;
  int q_dim, kv_dim, n_qkv;
  uint16_t *embed = nullptr, *lm_head = nullptr;
  float* final_norm = nullptr;
  double* inv_freq = nullptr;
  std::vector<LayerDev> layers;
  std::vector<void*> owned;
  CUtensorMap tm_lm;
  // workspace
  DevBuf x, x_last, a, qkv, attn_o, hmlp, rope, h_last, lm_part, vlogits, logits, lse, attn_part_o, attn_part_ml, attn_counters;
  uint32_t* status = nullptr;
  // fixed order of the residual projections' additions (bit-identical passes); see TurnOrder
  uint32_t* turn_flags = nullptr;
  uint32_t turn_epoch = 0;
  bool deterministic = true;
  Staging stg;
  bool keep_logits = false;
  bool last_rows_compact = false;   // the last run_layers left the steps' final hidden rows in x_last, in step order
  int last_B = 0;
  int64_t last_h2d_bytes = 0;   // bytes the last cs_verify_steps / cs_prefill call copied to the device
  // two-tier pass: list of escalated steps (+ its length) on the draft model, compact results on the target model
  DevBuf casc_idx, casc_conf, casc_verdict, casc_accept;
  int32_t* casc_host = nullptr;   // pinned copy of the list
  size_t casc_host_cap = 0;
  Prof prof;
};

struct cs_kv {
  const cs_model* model;
  int num_pages, page_size, max_seqs, max_pages_per_seq;
  uint16_t* pool = nullptr;   // 16-bit cells (bf16 values in the fp16 encoding), or 8-bit codes when format == 1
  bool own_pool = false;
  int format = 0;             // 0: 16-bit cells; CS_KV_E4M3 / CS_KV_E5M2: 8-bit codes (read-only for the pass)
  size_t plane_elems;  // elements of one (layer, K or V) plane
  CUtensorMap tm_pool;
  int32_t* table_host = nullptr;  // pinned [max_seqs, max_pages_per_seq]
  int32_t* table_dev = nullptr;
  std::vector<int32_t> ctx_len, n_pages;  // per sequence; ctx_len < 0 = not set
  bool dirty = true;
  cudaEvent_t upload_ev = nullptr;
  bool upload_pending = false;
  DevBuf fill_tmp;
};

namespace {

int upload_table(cs_kv* kv, cudaStream_t s) {
  if (!kv->dirty) return CS_OK;
  CS_CUDA(cudaMemcpyAsync(kv->table_dev, kv->table_host,
                          sizeof(int32_t) * static_cast<size_t>(kv->max_seqs) * kv->max_pages_per_seq,
                          cudaMemcpyHostToDevice, s));
  CS_CUDA(cudaEventRecord(kv->upload_ev, s));
  kv->upload_pending = true;
  kv->dirty = false;
  return CS_OK;
}

// Host staging slot of at least `ints` int32, safe to overwrite.
int staging_slot(Staging& st, size_t ints, int* slot_out) {
  const int slot = st.next;
  st.next = (st.next + 1) % kStagingRing;
  if (st.pending[slot]) {
    CS_CUDA(cudaEventSynchronize(st.ev[slot]));
    st.pending[slot] = false;
  }
  if (!st.ev[slot]) CS_CUDA(cudaEventCreateWithFlags(&st.ev[slot], cudaEventDisableTiming));
  if (st.host_cap[slot] < ints) {
    if (st.host[slot]) cudaFreeHost(st.host[slot]);
    st.host[slot] = nullptr;
    const size_t want = ints + ints / 2 + 1024;
    CS_CUDA(cudaMallocHost(reinterpret_cast<void**>(&st.host[slot]), want * sizeof(int32_t)));
    st.host_cap[slot] = want;
  }
  *slot_out = slot;
  return CS_OK;
}

// Pinned host buffer of at least `ints` int32 for small device-to-host read-backs.
int ensure_readback(cs_model* m, size_t ints) {
  if (m->casc_host_cap >= ints) return CS_OK;
  if (m->casc_host) cudaFreeHost(m->casc_host);
  m->casc_host = nullptr;
  m->casc_host_cap = 0;
  const size_t want = 2 * ints + 64;
  CS_CUDA(cudaMallocHost(reinterpret_cast<void**>(&m->casc_host), want * sizeof(int32_t)));
  m->casc_host_cap = want;
  return CS_OK;
}

struct BatchLayout {
  int B = 0, T = 0;
  size_t off_cu, off_pos, off_tseq, off_tok, off_items, total;
  int n_items = 0, n_slots = 0;
  int max_rows = 0;        // 8-bit cache: the largest number of query rows (new tokens x heads per kv head) of a step
  bool any_split = false;  // 8-bit cache: some context is cut into pieces
};

// Cost of an attention work item in key tiles: the tiles themselves plus the fixed part of a CTA (set-up, Q load,
// pipeline fill, epilogue), what being a piece of a split query tile adds (the partial result goes through global
// memory), and what the last piece adds by combining the partial results.
// Measured on B200: a tile takes ~2 k cycles; set-up to first S ~5.5 k; the epilogue of a piece (partial block out
// by bulk copy, fence, counter) ~5 k against ~1.5 k for a whole range; the combining piece fetches all blocks in one
// round of bulk copies.
constexpr double kAttnItemFixed = 3.5;
constexpr double kAttnPieceExtra = 2.0;
constexpr double kAttnMergeFixed = 1.0;
constexpr double kAttnMergePerSplit = 0.5;

// Time at which the last SM finishes when the items, sorted by decreasing cost, are handed to whichever of
// `machines` SMs is free first (what the hardware does with one CTA per SM and the grid in that order).
double list_schedule_makespan(std::vector<double>& cost, int machines) {
  std::sort(cost.begin(), cost.end(), std::greater<double>());
  if (static_cast<int>(cost.size()) <= machines) return cost.empty() ? 0.0 : cost[0];
  std::vector<double> heap(cost.begin(), cost.begin() + machines);   // min-heap of finish times
  std::make_heap(heap.begin(), heap.end(), std::greater<double>());
  for (size_t i = machines; i < cost.size(); ++i) {
    std::pop_heap(heap.begin(), heap.end(), std::greater<double>());
    heap.back() += cost[i];
    std::push_heap(heap.begin(), heap.end(), std::greater<double>());
  }
  return *std::max_element(heap.begin(), heap.end());
}

// Work items of one attention launch: every (step, kv head, query tile of 128 / G tokens) over its key tiles,
// long key ranges cut into pieces of at most `max_tiles` tiles. `max_tiles` is the candidate with the smallest
// estimated finish time on the SMs; cutting is only worth it when it shortens the longest item by more than the
// extra fixed cost and the combining step add.
void build_attention_work(const cs_model* m, int B, const int32_t* lens, const int32_t* ctx, std::vector<AttnItem>& items,
                          int* n_slots) {
  const int G = m->d.n_q_heads / m->d.n_kv_heads;
  const int ntok = 128 / G;
  const int max_splits = attention_max_splits();
  struct Unit { int step, q0, nt; };
  std::vector<Unit> units;
  int longest = 1;
  for (int i = 0; i < B; ++i) {
    const int ctx_tiles = (ctx[i] + 127) / 128;
    for (int q0 = 0; q0 < lens[i]; q0 += ntok) {
      const int p_max = std::min(lens[i] - 1, q0 + ntok - 1);
      const int nt = ctx_tiles + p_max / 128 + 1;
      units.push_back(Unit{i, q0, nt});
      longest = std::max(longest, nt);
    }
  }
  const int heads = m->d.n_kv_heads;
  auto pieces = [&](int nt, int cap) { return std::min(max_splits, (nt + cap - 1) / cap); };
  // No schedule finishes before its longest item or before the work divided by the SMs: a candidate whose bound
  // cannot beat `to_beat` is dropped without being scheduled (the call runs on the host before the first launch).
  std::vector<double> cost;
  cost.reserve(units.size() * heads * 2);
  auto estimate = [&](int cap, double to_beat) {
    cost.clear();
    double longest_item = 0.0, total = 0.0;
    for (const Unit& u : units) {
      const int n = pieces(u.nt, cap);
      for (int s = 0; s < n; ++s) {
        const int len = static_cast<int>(static_cast<long>(u.nt) * (s + 1) / n - static_cast<long>(u.nt) * s / n);
        double c = kAttnItemFixed + len;
        if (n > 1) c += kAttnPieceExtra;
        if (n > 1 && s == n - 1) c += kAttnMergeFixed + kAttnMergePerSplit * n;
        for (int h = 0; h < heads; ++h) cost.push_back(c);
        longest_item = std::max(longest_item, c);
        total += c * heads;
      }
    }
    if (static_cast<int>(cost.size()) <= kNumSMs) return longest_item;
    if (std::max(longest_item, total / kNumSMs) >= to_beat) return to_beat;
    return list_schedule_makespan(cost, kNumSMs);
  };
  int best_cap = longest;
  double best = estimate(longest, 1e300);
  int last_cap = longest;
  auto consider = [&](int cap) {
    if (cap < 2 || cap >= last_cap) return;
    last_cap = cap;
    const double e = estimate(cap, 0.97 * best);
    if (e < 0.97 * best) { best = e; best_cap = cap; }
  };
  // caps just below the longest range cut only the few longest query tiles (in two) ...
  for (int pct = 92; pct >= 52; pct -= 8) consider((longest * pct + 99) / 100);
  // ... smaller ones cut most of them, into more pieces
  for (int k = 2; k <= 16; ++k) consider((longest + k - 1) / k);
  items.clear();
  int slots = 0;
  for (const Unit& u : units)
    for (int h = 0; h < heads; ++h) {
      const int n = pieces(u.nt, best_cap);
      for (int s = 0; s < n; ++s) {
        const int b = static_cast<int>(static_cast<long>(u.nt) * s / n);
        const int e = static_cast<int>(static_cast<long>(u.nt) * (s + 1) / n);
        items.push_back(AttnItem{u.step, h, u.q0, b, e, n > 1 ? slots + s : 0, n > 1 ? slots : 0, n, 0, lens[u.step],
                                 ctx[u.step], 0, {0, 0, 0, 0}});
      }
      if (n > 1) slots += n;
    }
  std::stable_sort(items.begin(), items.end(), [](const AttnItem& a, const AttnItem& b) {
    return (a.tile_end - a.tile_begin) > (b.tile_end - b.tile_begin);
  });
  *n_slots = slots;
}

// Work items of the short-step attention over an 8-bit cache: one per (step, kv head, piece of the context's pages).
// The pieces are sized so that the launch has a few CTAs per SM; the last piece of a step also covers its own keys.
void build_short_work(const cs_model* m, int B, const int32_t* lens, const int32_t* ctx, std::vector<AttnItem>& items,
                      int* n_slots, bool* any_split) {
  const int heads = m->d.n_kv_heads;
  long units = 0;
  for (int i = 0; i < B; ++i) units += static_cast<long>((ctx[i] + kPageSize - 1) / kPageSize) * heads;
  // measured: an item costs ~9 us of its own (query load, first pages' latency, combining), so few long items win
  const long chunk = std::max<long>(32, units / (kNumSMs * 6L) + 1);
  items.clear();
  int slots = 0;
  *any_split = false;
  for (int i = 0; i < B; ++i) {
    const int pages = (ctx[i] + kPageSize - 1) / kPageSize;
    const int n = static_cast<int>(std::min<long>(32, std::max<long>(1, (pages + chunk - 1) / chunk)));
    for (int h = 0; h < heads; ++h) {
      for (int s = 0; s < n; ++s) {
        const int b = static_cast<int>(static_cast<long>(pages) * s / n);
        const int e = static_cast<int>(static_cast<long>(pages) * (s + 1) / n);
        items.push_back(AttnItem{i, h, 0, b, e, n > 1 ? slots + s : 0, n > 1 ? slots : 0, n, 0, lens[i], ctx[i], 0,
                                 {0, 0, 0, 0}});
      }
      if (n > 1) { slots += n; *any_split = true; }
    }
  }
  std::stable_sort(items.begin(), items.end(), [](const AttnItem& a, const AttnItem& b) {
    return (a.tile_end - a.tile_begin) > (b.tile_end - b.tile_begin);
  });
  *n_slots = slots;
}

int check_model_desc(const cs_model_desc* d) {
  if (!d) return CS_EINVAL;
  if (d->n_layers < 1 || d->d_model < 8 || d->n_q_heads < 1 || d->n_kv_heads < 1 || d->d_ffn < 8 || d->vocab < 1)
    return CS_EINVAL;
  if (d->head_dim != 64 && d->head_dim != 128) return CS_EINVAL;
  if (d->n_q_heads % d->n_kv_heads) return CS_EINVAL;
  // a query tile holds the rows of 128 / G tokens for the G query heads of one kv head: G beyond 128 leaves no token
  if (d->n_q_heads / d->n_kv_heads > 128) return CS_EINVAL;
  if (d->d_model % 8 || d->d_ffn % 8) return CS_EINVAL;
  if (!(d->rope_theta > 0.f) || !(d->rms_eps >= 0.f)) return CS_EINVAL;
  return CS_OK;
}

template <typename T>
int dev_copy(cs_model* m, T** dst, const T* src, size_t n, bool src_dev) {
  void* p = nullptr;
  cudaError_t e = cudaMalloc(&p, n * sizeof(T));
  if (e != cudaSuccess) return cuda_fail(e, "cudaMalloc(weights)");
  m->owned.push_back(p);
  CS_CUDA(cudaMemcpy(p, src, n * sizeof(T), src_dev ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice));
  *dst = static_cast<T*>(p);
  return CS_OK;
}

void prof_begin(cs_model* m, int cls, cudaStream_t s) {
  Prof& p = m->prof;
  if (!p.on) return;
  if (p.pool.size() < 2 * (p.used + 1)) {
    cudaEvent_t a = nullptr, b = nullptr;
    if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) { p.on = false; return; }
    p.pool.push_back(a);
    p.pool.push_back(b);
    p.cls.push_back(cls);
  }
  p.cls[p.used] = cls;
  cudaEventRecord(p.pool[2 * p.used], s);
}
void prof_end(cs_model* m, cudaStream_t s) {
  Prof& p = m->prof;
  if (!p.on) return;
  cudaEventRecord(p.pool[2 * p.used + 1], s);
  ++p.used;
}
#define CS_STEP(cls, call)                                \
  do {                                                    \
    prof_begin(m, cls, s);                                \
    cudaError_t e__ = (call);                             \
    prof_end(m, s);                                       \
    if (e__ != cudaSuccess) return cuda_fail(e__, #call); \
  } while (0)

// The forward over all layers for a staged batch. When `append_kv` is given the new K/V of every layer are
// also written to that cache's pages.
int run_layers(cs_model* m, const cs_kv* kv, cs_kv* append_kv, const BatchLayout& L, const int32_t* dev_meta,
               const int32_t* d_tok, cudaStream_t s) {
  const cs_model_desc& d = m->d;
  const int T = L.T;
  m->last_rows_compact = false;
  const int32_t* d_pos = dev_meta + L.off_pos;
  const int32_t* d_tseq = dev_meta + L.off_tseq;
  const AttnItem* d_items = reinterpret_cast<const AttnItem*>(dev_meta + L.off_items);

  float* x = static_cast<float*>(m->x.p);
  uint16_t* a = static_cast<uint16_t*>(m->a.p);
  uint16_t* qkv = static_cast<uint16_t*>(m->qkv.p);
  uint16_t* attn_o = static_cast<uint16_t*>(m->attn_o.p);
  uint16_t* hmlp = static_cast<uint16_t*>(m->hmlp.p);
  float2* rope = static_cast<float2*>(m->rope.p);

  CUtensorMap tm_a, tm_o, tm_h, tm_qkv_attn, tm_q3d;
  const int group = d.n_q_heads / d.n_kv_heads;
  if (!make_gemm_operand_map(&tm_a, a, T, d.d_model) || !make_gemm_operand_map(&tm_o, attn_o, T, m->q_dim) ||
      !make_gemm_operand_map(&tm_h, hmlp, T, d.d_ffn) ||
      !make_kv_rows_map(&tm_qkv_attn, qkv, T, m->n_qkv, d.head_dim) ||
      !make_tensor_map_heads3d(&tm_q3d, qkv, T, d.n_q_heads + 2 * d.n_kv_heads, d.head_dim, m->n_qkv, 128 / group,
                               group)) {
    g_cuda_error = "cuTensorMapEncodeTiled failed for an activation buffer";
    return CS_ECUDA;
  }

  CS_STEP(kProfEmbed, launch_embed(d_tok, m->embed, x, T, d.d_model, d.vocab, m->status, s));
  CS_STEP(kProfOther, launch_rope_table(d_pos, m->inv_freq, rope, T, d.head_dim / 2, s));

  AttnParams ap;
  ap.qkv = qkv;
  ap.out = attn_o;
  ap.page_table = kv->table_dev;
  ap.max_pages_per_seq = kv->max_pages_per_seq;
  ap.n_q_heads = d.n_q_heads;
  ap.n_kv_heads = d.n_kv_heads;
  ap.head_dim = d.head_dim;
  ap.n_qkv = m->n_qkv;
  ap.scale_log2e = static_cast<float>(1.4426950408889634 / std::sqrt(static_cast<double>(d.head_dim)));
  ap.part_o = static_cast<float*>(m->attn_part_o.p);
  ap.part_ml = static_cast<float*>(m->attn_part_ml.p);
  ap.counters = static_cast<int32_t*>(m->attn_counters.p);
  ap.status = m->status;
  ap.num_pages = kv->num_pages;
  ap.n_rows = T;
  const int plane_groups = kv->num_pages * d.n_kv_heads * kPageSize / 8;

  TurnOrder turn_order{m->turn_flags, &m->turn_epoch};
  const TurnOrder* turn = m->deterministic ? &turn_order : nullptr;
  RopeEpilogue rope_epi{rope, d.head_dim / 2, (d.n_q_heads + d.n_kv_heads) * d.head_dim};
  rope_epi.q_cols = m->q_dim;
  rope_epi.eps = d.rms_eps;
  for (int l = 0; l < d.n_layers; ++l) {
    const LayerDev& lw = m->layers[l];
    rope_epi.qk_gain = lw.qk_gain;
    CS_STEP(kProfNorm, launch_rmsnorm(x, lw.norm1, a, T, d.d_model, d.rms_eps, s));
    // q and k heads leave the projection already rotated (the turn is applied to the fp32 accumulators)
    CS_STEP(kProfQkv, gemm_f16_rope(tm_a, lw.tm_wqkv, qkv, T, m->n_qkv, d.d_model, rope_epi, m->status, s));
    ap.k_group_base = (2 * l) * plane_groups;
    ap.v_group_base = (2 * l + 1) * plane_groups;
    if (l == d.n_layers - 1 && append_kv) {
      // A pass that only appends to the cache has no use for what follows the last layer's K/V projection.
      CS_STEP(kProfOther, launch_kv_scatter(qkv + m->q_dim, qkv + m->q_dim + m->kv_dim, m->n_qkv, d_tseq, d_pos, 0, 0,
                                append_kv->table_dev, append_kv->max_pages_per_seq,
                                append_kv->pool + static_cast<size_t>(2 * l) * append_kv->plane_elems,
                                append_kv->pool + static_cast<size_t>(2 * l + 1) * append_kv->plane_elems,
                                d.n_kv_heads, d.head_dim, kPageSize, T, 1, append_kv->num_pages, m->status, s));
      break;
    }
    if (kv->format != 0) {
      const uint8_t* pool8 = reinterpret_cast<const uint8_t*>(kv->pool);
      CS_STEP(kProfAttn, launch_attention_short(ap, pool8 + static_cast<size_t>(2 * l) * kv->plane_elems,
                                                pool8 + static_cast<size_t>(2 * l + 1) * kv->plane_elems, d_items,
                                                L.n_items, L.max_rows, L.any_split, kv->format == 2, s));
    } else {
      CS_STEP(kProfAttn, launch_attention(ap, kv->tm_pool, tm_qkv_attn, tm_q3d, d_items, L.n_items, s));
    }
    if (append_kv) {
      CS_STEP(kProfOther, launch_kv_scatter(qkv + m->q_dim, qkv + m->q_dim + m->kv_dim, m->n_qkv, d_tseq, d_pos, 0, 0,
                                append_kv->table_dev, append_kv->max_pages_per_seq,
                                append_kv->pool + static_cast<size_t>(2 * l) * append_kv->plane_elems,
                                append_kv->pool + static_cast<size_t>(2 * l + 1) * append_kv->plane_elems,
                                d.n_kv_heads, d.head_dim, kPageSize, T, 1, append_kv->num_pages, m->status, s));
    }
    CS_STEP(kProfO, gemm_f16(tm_o, lw.tm_wo, nullptr, x, T, d.d_model, m->q_dim, kEpiResidAdd, m->status, s, turn));
    if (l == d.n_layers - 1 && !append_kv) {
      // Only each step's last position feeds the LM head, and after the last attention no row depends on another:
      // the last MLP runs on those B rows alone. Same arithmetic per row; the launches are small and bound by
      // reading the weights, and are timed under "other" so that the per-launch figures of the projection classes
      // stay those of full launches.
      float* xl = static_cast<float*>(m->x_last.p);
      CUtensorMap tm_a_last, tm_h_last;
      if (!make_gemm_operand_map(&tm_a_last, a, L.B, d.d_model) || !make_gemm_operand_map(&tm_h_last, hmlp, L.B, d.d_ffn)) {
        g_cuda_error = "cuTensorMapEncodeTiled failed for the last-row buffers";
        return CS_ECUDA;
      }
      CS_STEP(kProfOther, launch_gather_last_rows(x, dev_meta + L.off_cu, xl, L.B, d.d_model, s));
      CS_STEP(kProfOther, launch_rmsnorm(xl, lw.norm2, a, L.B, d.d_model, d.rms_eps, s));
      CS_STEP(kProfOther, gemm_f16(tm_a_last, lw.tm_wg, &lw.tm_wu, hmlp, L.B, d.d_ffn, d.d_model, kEpiSwiGLU, m->status, s));
      CS_STEP(kProfOther, gemm_f16(tm_h_last, lw.tm_wd, nullptr, xl, L.B, d.d_model, d.d_ffn, kEpiResidAdd, m->status, s, turn));
      m->last_rows_compact = true;
      break;
    }
    CS_STEP(kProfNorm, launch_rmsnorm(x, lw.norm2, a, T, d.d_model, d.rms_eps, s));
    CS_STEP(kProfGateUp, gemm_f16(tm_a, lw.tm_wg, &lw.tm_wu, hmlp, T, d.d_ffn, d.d_model, kEpiSwiGLU, m->status, s));
    CS_STEP(kProfDown, gemm_f16(tm_h, lw.tm_wd, nullptr, x, T, d.d_model, d.d_ffn, kEpiResidAdd, m->status, s, turn));
  }
  return CS_OK;
}

int ensure_workspace(cs_model* m, int B, int T) {
  const cs_model_desc& d = m->d;
  int rc;
  const size_t t = static_cast<size_t>(T);
  if ((rc = m->x.ensure(t * d.d_model * 4))) return rc;
  if ((rc = m->a.ensure(t * d.d_model * 2))) return rc;
  if ((rc = m->x_last.ensure(static_cast<size_t>(B) * d.d_model * 4))) return rc;
  // A 128-row K/V box of the attention kernel may start at any of the T rows: the rows it reaches past the end
  // must exist and be finite (they are masked, but they are multiplied), so the buffer is zeroed when it is made.
  if ((rc = m->qkv.ensure((t + 128) * m->n_qkv * 2, true))) return rc;
  if ((rc = m->attn_o.ensure(t * m->q_dim * 2))) return rc;
  if ((rc = m->hmlp.ensure(t * d.d_ffn * 2))) return rc;
  if ((rc = m->rope.ensure(t * (d.head_dim / 2) * sizeof(float2)))) return rc;
  const size_t bp = static_cast<size_t>((B + 63) / 64) * 64;
  if ((rc = m->h_last.ensure(bp * d.d_model * 2))) return rc;
  if ((rc = m->lm_part.ensure(static_cast<size_t>((B + 63) / 64) * 2 * kNumSMs * 64 * 4))) return rc;
  if ((rc = m->vlogits.ensure(bp * 8 * 4))) return rc;
  if ((rc = m->lse.ensure(bp * 4))) return rc;
  if (m->keep_logits && (rc = m->logits.ensure(static_cast<size_t>(B) * d.vocab * 4))) return rc;
  return CS_OK;
}

// Checks a batch, writes its metadata into a staging slot and enqueues the upload.
int stage_batch(cs_model* m, const cs_kv* kv, const int32_t* seq_ids, int B, const int32_t* tokens,
                int tokens_on_device, const int32_t* lens, BatchLayout* out, const int32_t** dev_meta,
                const int32_t** dev_tokens, cudaStream_t s) {
  long T = 0;
  for (int i = 0; i < B; ++i) {
    if (lens[i] < 1) return CS_EINVAL;
    if (seq_ids[i] < 0 || seq_ids[i] >= kv->max_seqs) return CS_EINVAL;
    if (kv->ctx_len[seq_ids[i]] < 0) return CS_ESTATE;
    T += lens[i];
    if (T > (1 << 24)) return CS_EINVAL;
  }
  if (!tokens_on_device)
    for (long t = 0; t < T; ++t)
      if (tokens[t] < 0 || tokens[t] >= m->d.vocab) return CS_EINVAL;

  std::vector<int32_t> ctx(B);
  for (int i = 0; i < B; ++i) ctx[i] = kv->ctx_len[seq_ids[i]];
  std::vector<AttnItem> items;
  int n_slots = 0, max_rows = 0;
  bool any_split = false;
  if (kv->format != 0) {
    const int G = m->d.n_q_heads / m->d.n_kv_heads;
    for (int i = 0; i < B; ++i) max_rows = std::max(max_rows, lens[i] * G);
    if (max_rows > 32) return CS_EINVAL;     // the 8-bit cache serves short steps only
    build_short_work(m, B, lens, ctx.data(), items, &n_slots, &any_split);
  } else {
    build_attention_work(m, B, lens, ctx.data(), items, &n_slots);
  }

  BatchLayout L;
  L.B = B;
  L.T = static_cast<int>(T);
  size_t o = 0;
  auto take = [&o](size_t n) { size_t r = o; o += (n + 3) & ~size_t(3); return r; };  // keep 16-byte alignment
  L.off_cu = take(B + 1);
  L.off_pos = take(T);
  L.off_tseq = take(T);
  L.off_tok = take(tokens_on_device ? 0 : T);
  L.off_items = take(items.size() * (sizeof(AttnItem) / 4));
  L.total = o;
  L.n_items = static_cast<int>(items.size());
  L.n_slots = n_slots;
  L.max_rows = max_rows;
  L.any_split = any_split;

  int rc;
  if ((rc = ensure_workspace(m, B, L.T))) return rc;
  const int hd = m->d.head_dim;
  if ((rc = m->attn_part_o.ensure(static_cast<size_t>(std::max(1, n_slots)) * 128 * hd * 4))) return rc;
  if ((rc = m->attn_part_ml.ensure(static_cast<size_t>(std::max(1, n_slots)) * 128 * 2 * 4))) return rc;
  // One counter per split query tile; every launch leaves them at zero again.
  if ((rc = m->attn_counters.ensure(static_cast<size_t>(std::max(1, n_slots)) * 4, true))) return rc;
  if ((rc = m->stg.dev.ensure(L.total * 4))) return rc;
  int slot;
  if ((rc = staging_slot(m->stg, L.total, &slot))) return rc;
  int32_t* h = m->stg.host[slot];
  int32_t* cu = h + L.off_cu;
  cu[0] = 0;
  for (int i = 0; i < B; ++i) {
    cu[i + 1] = cu[i] + lens[i];
    for (int p = 0; p < lens[i]; ++p) {
      h[L.off_pos + cu[i] + p] = ctx[i] + p;
      h[L.off_tseq + cu[i] + p] = seq_ids[i];
    }
  }
  if (!tokens_on_device) std::memcpy(h + L.off_tok, tokens, sizeof(int32_t) * T);
  for (AttnItem& it : items) {
    it.tok0 = cu[it.step];
    it.seq = seq_ids[it.step];
  }
  if (!items.empty()) std::memcpy(h + L.off_items, items.data(), items.size() * sizeof(AttnItem));
  CS_CUDA(cudaMemcpyAsync(m->stg.dev.p, h, L.total * 4, cudaMemcpyHostToDevice, s));
  m->last_h2d_bytes = static_cast<int64_t>(L.total) * 4;
  CS_CUDA(cudaEventRecord(m->stg.ev[slot], s));
  m->stg.pending[slot] = true;
  *out = L;
  *dev_meta = static_cast<const int32_t*>(m->stg.dev.p);
  *dev_tokens = tokens_on_device ? tokens : *dev_meta + L.off_tok;
  return CS_OK;
}

uint32_t* g_test_status = nullptr;
uint32_t* g_test_turn_flags = nullptr;
uint32_t g_test_turn_epoch = 0;

}  // namespace

extern "C" {

int cs_version(void) { return 100; }

const char* cs_strerror(int status) {
  switch (status) {
    case CS_OK: return "ok";
    case CS_EINVAL: return "invalid argument";
    case CS_ENOMEM: return "out of memory";
    case CS_ECUDA: return "CUDA error";
    case CS_ETIMEOUT: return "a kernel gave up on a bounded wait";
    case CS_ESTATE: return "call does not fit the handle's state";
    case CS_ELIMIT: return "size exceeds the fixed capacity of an entry point that never allocates";
    case CS_ERANGE: return "a range check failed: an index left its array (debug build) or a workspace's guard bytes were written";
    default: return "unknown status";
  }
}

const char* cs_last_cuda_error(void) { return g_cuda_error.c_str(); }

int64_t cs_take_launch_count(void) { return take_launch_count(); }

int cs_model_load(const cs_model_desc* desc, const cs_model_tensors* t, int on_dev, cs_model** out) {
  if (!out) return CS_EINVAL;
  *out = nullptr;
  int rc = check_model_desc(desc);
  if (rc) return rc;
  if (!t || !t->embed || !t->lm_head || !t->final_norm || !t->wq || !t->wk || !t->wv || !t->wo || !t->wg || !t->wu ||
      !t->wd || !t->norm1 || !t->norm2)
    return CS_EINVAL;
  for (int l = 0; l < desc->n_layers; ++l)
    if (!t->wq[l] || !t->wk[l] || !t->wv[l] || !t->wo[l] || !t->wg[l] || !t->wu[l] || !t->wd[l] || !t->norm1[l] ||
        !t->norm2[l])
      return CS_EINVAL;
  if ((t->q_norm == nullptr) != (t->k_norm == nullptr)) return CS_EINVAL;
  if (t->q_norm)
    for (int l = 0; l < desc->n_layers; ++l)
      if (!t->q_norm[l] || !t->k_norm[l]) return CS_EINVAL;
  int dev = 0;
  cudaDeviceProp prop;
  CS_CUDA(cudaGetDevice(&dev));
  CS_CUDA(cudaGetDeviceProperties(&prop, dev));
  if (prop.major != 10) {
    g_cuda_error = "this library contains sm_100a code only; the current device is not compute capability 10.x";
    return CS_ECUDA;
  }
  cs_model* m = new (std::nothrow) cs_model();
  if (!m) return CS_ENOMEM;
  m->d = *desc;
  m->q_dim = desc->n_q_heads * desc->head_dim;
  m->kv_dim = desc->n_kv_heads * desc->head_dim;
  m->n_qkv = m->q_dim + 2 * m->kv_dim;
  const bool sd = on_dev != 0;
  const size_t dm = desc->d_model, V = desc->vocab, F = desc->d_ffn;
#define CS_TRY(expr)     \
  do {                   \
    rc = (expr);         \
    if (rc) {            \
      cs_model_free(m);  \
      return rc;         \
    }                    \
  } while (0)
  CS_TRY(dev_copy(m, &m->embed, t->embed, V * dm, sd));
  CS_TRY(dev_copy(m, &m->lm_head, t->lm_head, V * dm, sd));
  CS_TRY(dev_copy(m, &m->final_norm, t->final_norm, dm, sd));
  m->layers.resize(desc->n_layers);
  for (int l = 0; l < desc->n_layers; ++l) {
    LayerDev& lw = m->layers[l];
    void* p = nullptr;
    cudaError_t e = cudaMalloc(&p, static_cast<size_t>(m->n_qkv) * dm * 2);
    if (e != cudaSuccess) { rc = cuda_fail(e, "cudaMalloc(wqkv)"); cs_model_free(m); return rc; }
    m->owned.push_back(p);
    lw.wqkv = static_cast<uint16_t*>(p);
    const cudaMemcpyKind kind = sd ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice;
    e = cudaMemcpy(lw.wqkv, t->wq[l], static_cast<size_t>(m->q_dim) * dm * 2, kind);
    if (e == cudaSuccess) e = cudaMemcpy(lw.wqkv + static_cast<size_t>(m->q_dim) * dm, t->wk[l], static_cast<size_t>(m->kv_dim) * dm * 2, kind);
    if (e == cudaSuccess) e = cudaMemcpy(lw.wqkv + static_cast<size_t>(m->q_dim + m->kv_dim) * dm, t->wv[l], static_cast<size_t>(m->kv_dim) * dm * 2, kind);
    if (e != cudaSuccess) { rc = cuda_fail(e, "cudaMemcpy(wqkv)"); cs_model_free(m); return rc; }
    CS_TRY(dev_copy(m, &lw.wo, t->wo[l], dm * m->q_dim, sd));
    CS_TRY(dev_copy(m, &lw.wg, t->wg[l], F * dm, sd));
    CS_TRY(dev_copy(m, &lw.wu, t->wu[l], F * dm, sd));
    CS_TRY(dev_copy(m, &lw.wd, t->wd[l], dm * F, sd));
    CS_TRY(dev_copy(m, &lw.norm1, t->norm1[l], dm, sd));
    CS_TRY(dev_copy(m, &lw.norm2, t->norm2[l], dm, sd));
    if (t->q_norm) {
      void* g = nullptr;
      e = cudaMalloc(&g, 2 * sizeof(float) * desc->head_dim);
      if (e != cudaSuccess) { rc = cuda_fail(e, "cudaMalloc(qk gains)"); cs_model_free(m); return rc; }
      m->owned.push_back(g);
      lw.qk_gain = static_cast<float*>(g);
      e = cudaMemcpy(lw.qk_gain, t->q_norm[l], sizeof(float) * desc->head_dim, kind);
      if (e == cudaSuccess) e = cudaMemcpy(lw.qk_gain + desc->head_dim, t->k_norm[l], sizeof(float) * desc->head_dim, kind);
      if (e != cudaSuccess) { rc = cuda_fail(e, "cudaMemcpy(qk gains)"); cs_model_free(m); return rc; }
    }
    // The matrices arrive as bf16 and are kept as fp16 (same size; see launch_bf16_to_f16): the tensor cores
    // take both operands in one 16-bit format and fp16 activations carry three more mantissa bits.
    e = launch_bf16_to_f16(lw.wqkv, static_cast<size_t>(m->n_qkv) * dm, nullptr);
    if (e == cudaSuccess) e = launch_bf16_to_f16(lw.wo, dm * m->q_dim, nullptr);
    if (e == cudaSuccess) e = launch_bf16_to_f16(lw.wg, F * dm, nullptr);
    if (e == cudaSuccess) e = launch_bf16_to_f16(lw.wu, F * dm, nullptr);
    if (e == cudaSuccess) e = launch_bf16_to_f16(lw.wd, dm * F, nullptr);
    if (e != cudaSuccess) { rc = cuda_fail(e, "bf16->fp16 weight conversion"); cs_model_free(m); return rc; }
    if (!make_gemm_operand_map(&lw.tm_wqkv, lw.wqkv, m->n_qkv, desc->d_model) ||
        !make_gemm_operand_map(&lw.tm_wo, lw.wo, desc->d_model, m->q_dim) ||
        !make_gemm_operand_map(&lw.tm_wg, lw.wg, desc->d_ffn, desc->d_model) ||
        !make_gemm_operand_map(&lw.tm_wu, lw.wu, desc->d_ffn, desc->d_model) ||
        !make_gemm_operand_map(&lw.tm_wd, lw.wd, desc->d_model, desc->d_ffn)) {
      g_cuda_error = "cuTensorMapEncodeTiled failed for a weight matrix";
      cs_model_free(m);
      return CS_ECUDA;
    }
  }
  {
    cudaError_t e = launch_bf16_to_f16(m->lm_head, V * dm, nullptr);
    if (e != cudaSuccess) { rc = cuda_fail(e, "bf16->fp16 weight conversion"); cs_model_free(m); return rc; }
  }
  if (!make_gemm_operand_map(&m->tm_lm, m->lm_head, desc->vocab, desc->d_model)) {
    g_cuda_error = "cuTensorMapEncodeTiled failed for the LM head";
    cs_model_free(m);
    return CS_ECUDA;
  }
  {
    const int half = desc->head_dim / 2;
    std::vector<double> f(half);
    for (int j = 0; j < half; ++j)
      f[j] = std::pow(static_cast<double>(desc->rope_theta), -2.0 * j / static_cast<double>(desc->head_dim));
    CS_TRY(dev_copy(m, &m->inv_freq, f.data(), static_cast<size_t>(half), false));
  }
  {
    void* p = nullptr;
    cudaError_t e = cudaMalloc(&p, 256);
    if (e != cudaSuccess) { rc = cuda_fail(e, "cudaMalloc(status)"); cs_model_free(m); return rc; }
    m->owned.push_back(p);
    m->status = static_cast<uint32_t*>(p);
    cudaMemset(p, 0, 256);
    p = nullptr;
    e = cudaMalloc(&p, sizeof(uint32_t) * kTurnWords);
    if (e != cudaSuccess) { rc = cuda_fail(e, "cudaMalloc(turn flags)"); cs_model_free(m); return rc; }
    m->owned.push_back(p);
    m->turn_flags = static_cast<uint32_t*>(p);
    cudaMemset(p, 0, sizeof(uint32_t) * kTurnWords);
  }
#undef CS_TRY
  CS_CUDA(cudaDeviceSynchronize());
  *out = m;
  return CS_OK;
}

int cs_model_free(cs_model* m) {
  if (!m) return CS_OK;
  cudaDeviceSynchronize();
  for (void* p : m->owned) cudaFree(p);
  DevBuf* bufs[] = {&m->x, &m->x_last, &m->a, &m->qkv, &m->attn_o, &m->hmlp, &m->rope, &m->h_last, &m->lm_part, &m->vlogits,
                    &m->logits, &m->lse, &m->attn_part_o, &m->attn_part_ml, &m->attn_counters, &m->stg.dev,
                    &m->casc_idx, &m->casc_conf, &m->casc_verdict, &m->casc_accept};
  for (DevBuf* b : bufs) b->release();
  if (m->casc_host) cudaFreeHost(m->casc_host);
  for (cudaEvent_t e : m->prof.pool) cudaEventDestroy(e);
  for (int i = 0; i < kStagingRing; ++i) {
    if (m->stg.host[i]) cudaFreeHost(m->stg.host[i]);
    if (m->stg.ev[i]) cudaEventDestroy(m->stg.ev[i]);
  }
  delete m;
  return CS_OK;
}

int cs_model_set_lm_head_rows(cs_model* m, const int32_t* row_ids, int n_rows, const uint16_t* rows_bf16, void* stream) {
  if (!m || n_rows < 0) return CS_EINVAL;
  if (n_rows == 0) return CS_OK;
  if (!row_ids || !rows_bf16) return CS_EINVAL;
  for (int i = 0; i < n_rows; ++i)
    if (row_ids[i] < 0 || row_ids[i] >= m->d.vocab) return CS_EINVAL;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t dm = static_cast<size_t>(m->d.d_model);
  for (int i = 0; i < n_rows; ++i) {
    uint16_t* dst = m->lm_head + static_cast<size_t>(row_ids[i]) * dm;
    CS_CUDA(cudaMemcpyAsync(dst, rows_bf16 + static_cast<size_t>(i) * dm, dm * 2, cudaMemcpyHostToDevice, s));
    CS_CUDA(launch_bf16_to_f16(dst, dm, s));   // same re-encoding as at load
  }
  CS_CUDA(cudaStreamSynchronize(s));            // the host rows may be released on return
  return CS_OK;
}

int cs_reserve(cs_model* m, int max_steps, int max_tokens) {
  if (!m || max_steps < 1 || max_tokens < max_steps) return CS_EINVAL;
  return ensure_workspace(m, max_steps, max_tokens);
}

uint64_t cs_kv_pool_bytes(const cs_model* m, int num_pages, int page_size) {
  if (!m || num_pages < 1 || page_size != kPageSize) return 0;
  return static_cast<uint64_t>(m->d.n_layers) * 2 * num_pages * m->d.n_kv_heads * page_size * m->d.head_dim * 2;
}

static int kv_alloc_impl(const cs_model* m, int num_pages, int page_size, int max_seqs, int max_pages_per_seq,
                         void* dev_pool, int format, cs_kv** out);

int cs_kv_alloc(const cs_model* m, int num_pages, int page_size, int max_seqs, int max_pages_per_seq, void* dev_pool,
                cs_kv** out) {
  return kv_alloc_impl(m, num_pages, page_size, max_seqs, max_pages_per_seq, dev_pool, 0, out);
}

int cs_kv_alloc_8bit(const cs_model* m, int num_pages, int page_size, int max_seqs, int max_pages_per_seq, int format,
                     cs_kv** out) {
  if (format != CS_KV_E4M3 && format != CS_KV_E5M2) {
    if (out) *out = nullptr;
    return CS_EINVAL;
  }
  return kv_alloc_impl(m, num_pages, page_size, max_seqs, max_pages_per_seq, nullptr, format, out);
}

static int kv_alloc_impl(const cs_model* m, int num_pages, int page_size, int max_seqs, int max_pages_per_seq,
                         void* dev_pool, int format, cs_kv** out) {
  if (!out) return CS_EINVAL;
  *out = nullptr;
  if (!m || num_pages < 1 || page_size != kPageSize || max_seqs < 1 || max_pages_per_seq < 1) return CS_EINVAL;
  const uint64_t rows = static_cast<uint64_t>(m->d.n_layers) * 2 * num_pages * m->d.n_kv_heads * page_size;
  if (rows >= (1ull << 31)) return CS_EINVAL;
  if (dev_pool && (reinterpret_cast<uintptr_t>(dev_pool) & 255)) return CS_EINVAL;
  cs_kv* kv = new (std::nothrow) cs_kv();
  if (!kv) return CS_ENOMEM;
  kv->model = m;
  kv->format = format;
  kv->num_pages = num_pages;
  kv->page_size = page_size;
  kv->max_seqs = max_seqs;
  kv->max_pages_per_seq = max_pages_per_seq;
  kv->plane_elems = static_cast<size_t>(num_pages) * m->d.n_kv_heads * page_size * m->d.head_dim;
  kv->ctx_len.assign(max_seqs, -1);
  kv->n_pages.assign(max_seqs, 0);
  const uint64_t bytes = cs_kv_pool_bytes(m, num_pages, page_size) / (format != 0 ? 2 : 1);
  int rc = CS_OK;
  cudaError_t e;
  if (dev_pool) {
    kv->pool = static_cast<uint16_t*>(dev_pool);
  } else {
    void* p = nullptr;
    e = cudaMalloc(&p, bytes);
    if (e != cudaSuccess) { rc = cuda_fail(e, "cudaMalloc(kv pool)"); cs_kv_free(kv); return rc; }
    kv->pool = static_cast<uint16_t*>(p);
    kv->own_pool = true;
    e = cudaMemset(p, 0, bytes);
    if (e != cudaSuccess) { rc = cuda_fail(e, "cudaMemset(kv pool)"); cs_kv_free(kv); return rc; }
  }
  const size_t tbytes = sizeof(int32_t) * static_cast<size_t>(max_seqs) * max_pages_per_seq;
  e = cudaMallocHost(reinterpret_cast<void**>(&kv->table_host), tbytes);
  if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void**>(&kv->table_dev), tbytes);
  if (e == cudaSuccess) e = cudaMemset(kv->table_dev, 0, tbytes);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&kv->upload_ev, cudaEventDisableTiming);
  if (e != cudaSuccess) { rc = cuda_fail(e, "kv page table"); cs_kv_free(kv); return rc; }
  std::memset(kv->table_host, 0, tbytes);
  if (format == 0 && !make_kv_group_map(&kv->tm_pool, kv->pool, rows, m->d.head_dim, kPageSize / 8)) {
    g_cuda_error = "cuTensorMapEncodeTiled failed for the kv pool";
    cs_kv_free(kv);
    return CS_ECUDA;
  }
  *out = kv;
  return CS_OK;
}

int cs_kv_free(cs_kv* kv) {
  if (!kv) return CS_OK;
  cudaDeviceSynchronize();
  if (kv->own_pool && kv->pool) cudaFree(kv->pool);
  if (kv->table_host) cudaFreeHost(kv->table_host);
  if (kv->table_dev) cudaFree(kv->table_dev);
  if (kv->upload_ev) cudaEventDestroy(kv->upload_ev);
  kv->fill_tmp.release();
  delete kv;
  return CS_OK;
}

int cs_kv_set_seq(cs_kv* kv, int seq, const int32_t* page_ids, int n_pages, int ctx_len) {
  if (!kv || seq < 0 || seq >= kv->max_seqs || n_pages < 0 || n_pages > kv->max_pages_per_seq || ctx_len < 0 ||
      ctx_len > n_pages * kv->page_size || (n_pages > 0 && !page_ids))
    return CS_EINVAL;
  for (int i = 0; i < n_pages; ++i)
    if (page_ids[i] < 0 || page_ids[i] >= kv->num_pages) return CS_EINVAL;
  if (kv->upload_pending) {
    CS_CUDA(cudaEventSynchronize(kv->upload_ev));
    kv->upload_pending = false;
  }
  int32_t* row = kv->table_host + static_cast<size_t>(seq) * kv->max_pages_per_seq;
  for (int i = 0; i < n_pages; ++i) row[i] = page_ids[i];
  kv->ctx_len[seq] = ctx_len;
  kv->n_pages[seq] = n_pages;
  kv->dirty = true;
  return CS_OK;
}

int cs_kv_fill(cs_kv* kv, int seq, int layer, const uint16_t* host_k, const uint16_t* host_v, void* stream) {
  if (!kv || seq < 0 || seq >= kv->max_seqs || layer < 0 || layer >= kv->model->d.n_layers) return CS_EINVAL;
  if (kv->ctx_len[seq] < 0) return CS_ESTATE;
  const int c = kv->ctx_len[seq];
  if (c == 0) return CS_OK;
  if (!host_k || !host_v) return CS_EINVAL;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const cs_model_desc& d = kv->model->d;
  const size_t row = static_cast<size_t>(d.n_kv_heads) * d.head_dim;
  const size_t elems = static_cast<size_t>(c) * row;
  int rc;
  if ((rc = kv->fill_tmp.ensure(2 * elems * 2))) return rc;
  if ((rc = upload_table(kv, s))) return rc;
  if (kv->format != 0) {   // 8-bit cache: host_k / host_v hold one code per element
    uint8_t* tk8 = static_cast<uint8_t*>(kv->fill_tmp.p);
    uint8_t* tv8 = tk8 + elems;
    uint8_t* pool8 = reinterpret_cast<uint8_t*>(kv->pool);
    CS_CUDA(cudaMemcpyAsync(tk8, host_k, elems, cudaMemcpyHostToDevice, s));
    CS_CUDA(cudaMemcpyAsync(tv8, host_v, elems, cudaMemcpyHostToDevice, s));
    CS_CUDA(launch_kv_scatter_u8(tk8, tv8, seq, kv->table_dev, kv->max_pages_per_seq,
                                 pool8 + static_cast<size_t>(2 * layer) * kv->plane_elems,
                                 pool8 + static_cast<size_t>(2 * layer + 1) * kv->plane_elems, d.n_kv_heads, d.head_dim,
                                 kPageSize, c, s));
    CS_CUDA(cudaStreamSynchronize(s));
    return CS_OK;
  }
  uint16_t* tk = static_cast<uint16_t*>(kv->fill_tmp.p);
  uint16_t* tv = tk + elems;
  CS_CUDA(cudaMemcpyAsync(tk, host_k, elems * 2, cudaMemcpyHostToDevice, s));
  CS_CUDA(cudaMemcpyAsync(tv, host_v, elems * 2, cudaMemcpyHostToDevice, s));
  CS_CUDA(launch_kv_scatter(tk, tv, static_cast<int>(row), nullptr, nullptr, seq, 0, kv->table_dev,
                            kv->max_pages_per_seq, kv->pool + static_cast<size_t>(2 * layer) * kv->plane_elems,
                            kv->pool + static_cast<size_t>(2 * layer + 1) * kv->plane_elems, d.n_kv_heads, d.head_dim,
                            kPageSize, c, 0, kv->num_pages, nullptr, s));
  CS_CUDA(cudaStreamSynchronize(s));
  return CS_OK;
}

int cs_prefill(cs_model* m, cs_kv* kv, const int32_t* seq_ids, const int32_t* tokens, const int32_t* lens, int B,
               void* stream) {
  if (!m || !kv || kv->model != m || B < 0) return CS_EINVAL;
  if (kv->format != 0) return CS_EINVAL;   // the 8-bit cache is filled with given codes, not appended to
  if (B == 0) return CS_OK;
  if (!seq_ids || !tokens || !lens) return CS_EINVAL;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  for (int i = 0; i < B; ++i) {
    if (seq_ids[i] < 0 || seq_ids[i] >= kv->max_seqs || lens[i] < 1) return CS_EINVAL;
    if (kv->ctx_len[seq_ids[i]] < 0) return CS_ESTATE;
    if (kv->ctx_len[seq_ids[i]] + lens[i] > kv->n_pages[seq_ids[i]] * kv->page_size) return CS_EINVAL;
    for (int j = 0; j < i; ++j)
      if (seq_ids[j] == seq_ids[i]) return CS_EINVAL;
  }
  int rc;
  BatchLayout L;
  const int32_t *dev_meta, *dev_tok;
  if ((rc = stage_batch(m, kv, seq_ids, B, tokens, 0, lens, &L, &dev_meta, &dev_tok, s))) return rc;
  if ((rc = upload_table(kv, s))) return rc;
  if ((rc = run_layers(m, kv, kv, L, dev_meta, dev_tok, s))) return rc;
  for (int i = 0; i < B; ++i) kv->ctx_len[seq_ids[i]] += lens[i];
  return CS_OK;
}

int cs_append_accepted(cs_model* m, cs_kv* kv, int R, const int32_t* req_seq_ids, const int32_t* req_offsets,
                       const int32_t* dev_prefix_len, const int32_t* step_tokens, const int32_t* step_lens,
                       const int32_t* draft_lens, int32_t* host_prefix_len, void* stream) {
  if (!m || !kv || kv->model != m || R < 0 || kv->format != 0) return CS_EINVAL;
  if (R == 0) return CS_OK;
  if (!req_seq_ids || !req_offsets || !dev_prefix_len || !step_tokens || !step_lens || !draft_lens) return CS_EINVAL;
  if (req_offsets[0] != 0) return CS_EINVAL;
  for (int r = 0; r < R; ++r) {
    if (req_offsets[r + 1] < req_offsets[r]) return CS_EINVAL;
    if (req_seq_ids[r] < 0 || req_seq_ids[r] >= kv->max_seqs) return CS_EINVAL;
    if (kv->ctx_len[req_seq_ids[r]] < 0) return CS_ESTATE;
    for (int q = 0; q < r; ++q)
      if (req_seq_ids[q] == req_seq_ids[r]) return CS_EINVAL;
  }
  const int B = req_offsets[R];
  std::vector<int64_t> cu(static_cast<size_t>(B) + 1, 0);
  for (int i = 0; i < B; ++i) {
    if (step_lens[i] < 1 || draft_lens[i] < 0 || draft_lens[i] > step_lens[i]) return CS_EINVAL;
    cu[i + 1] = cu[i] + step_lens[i];
  }
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int rc;
  if ((rc = ensure_readback(m, static_cast<size_t>(R)))) return rc;
  CS_CUDA(cudaMemcpyAsync(m->casc_host, dev_prefix_len, sizeof(int32_t) * R, cudaMemcpyDeviceToHost, s));
  CS_CUDA(cudaStreamSynchronize(s));
  std::vector<int32_t> seqs, lens, toks;
  for (int r = 0; r < R; ++r) {
    const int mr = m->casc_host[r];
    if (mr < 0 || mr > req_offsets[r + 1] - req_offsets[r]) return CS_EINVAL;
    if (host_prefix_len) host_prefix_len[r] = mr;
    int n = 0;
    for (int j = 0; j < mr; ++j) {
      const int i = req_offsets[r] + j;
      toks.insert(toks.end(), step_tokens + cu[i], step_tokens + cu[i] + draft_lens[i]);
      n += draft_lens[i];
    }
    if (n > 0) {
      seqs.push_back(req_seq_ids[r]);
      lens.push_back(n);
    }
  }
  if (seqs.empty()) return CS_OK;
  return cs_prefill(m, kv, seqs.data(), toks.data(), lens.data(), static_cast<int>(seqs.size()), stream);
}

int cs_verify_steps(cs_model* m, const cs_kv* ckv, const int32_t* seq_ids, int B, const int32_t* step_tokens,
                    int tokens_on_device, const int32_t* step_lens, const int32_t* verdict_ids, int n_verdict,
                    float tau, float* out_conf, uint8_t* out_accept, int32_t* out_verdict, void* stream) {
  if (!m || !ckv || ckv->model != m || B < 0) return CS_EINVAL;
  if (tau != tau) return CS_EINVAL;
  if (n_verdict < 1 || n_verdict > 8 || !verdict_ids) return CS_EINVAL;
  for (int j = 0; j < n_verdict; ++j)
    if (verdict_ids[j] < 0 || verdict_ids[j] >= m->d.vocab) return CS_EINVAL;
  if (B == 0) return CS_OK;
  if (!seq_ids || !step_tokens || !step_lens || !out_conf || !out_accept) return CS_EINVAL;
  cs_kv* kv = const_cast<cs_kv*>(ckv);  // only the upload bookkeeping of the page table changes
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int rc;
  BatchLayout L;
  const int32_t *dev_meta, *dev_tok;
  if ((rc = stage_batch(m, kv, seq_ids, B, step_tokens, tokens_on_device, step_lens, &L, &dev_meta, &dev_tok, s)))
    return rc;
  if ((rc = upload_table(kv, s))) return rc;
  if ((rc = run_layers(m, kv, nullptr, L, dev_meta, dev_tok, s))) return rc;

  const cs_model_desc& d = m->d;
  float* x = static_cast<float*>(m->x.p);
  uint16_t* h_last = static_cast<uint16_t*>(m->h_last.p);
  const int B_all = ((B + 63) / 64) * 64;
  if (m->last_rows_compact)
    CS_STEP(kProfNorm, launch_last_rows_norm(static_cast<float*>(m->x_last.p), nullptr, m->final_norm, h_last, B, B_all,
                                             d.d_model, d.rms_eps, s));
  else
    CS_STEP(kProfNorm, launch_last_rows_norm(x, dev_meta + L.off_cu, m->final_norm, h_last, B, B_all, d.d_model, d.rms_eps, s));
  CUtensorMap tm_h;
  int rows_per_cta;
  const int grid = lm_head_grid(d.vocab, &rows_per_cta);
  for (int b0 = 0; b0 < B; b0 += 64) {
    const int bc = std::min(64, B - b0);
    const int bp = lm_head_batch_pad(bc);
    if (!make_tensor_map_16b(&tm_h, h_last, B_all, d.d_model, bp, 64, true, false)) {
      g_cuda_error = "cuTensorMapEncodeTiled failed for the last-position hidden states";
      return CS_ECUDA;
    }
    float* part_max = static_cast<float*>(m->lm_part.p) + static_cast<size_t>(b0 / 64) * 2 * kNumSMs * 64;
    float* part_sum = part_max + kNumSMs * 64;
    float* vlog = static_cast<float*>(m->vlogits.p) + static_cast<size_t>(b0) * 8;
    float* logits = m->keep_logits ? static_cast<float*>(m->logits.p) + static_cast<size_t>(b0) * d.vocab : nullptr;
    CS_STEP(kProfLmHead, launch_lm_head(m->tm_lm, tm_h, b0, bc, bp, d.d_model, d.vocab, verdict_ids, n_verdict, part_max, part_sum,
                           vlog, logits, m->status, s));
    CS_STEP(kProfGate, launch_gate(part_max, part_sum, grid, bp, vlog, n_verdict, bc, tau, out_conf + b0, out_accept + b0,
                        out_verdict ? out_verdict + b0 : nullptr, static_cast<float*>(m->lse.p) + b0, s));
  }
  m->last_B = B;
  return CS_OK;
}

int cs_escalate_mask(const float* conf, int B, float tau, uint8_t* out_accept, int32_t* out_idx, int32_t* out_count,
                     void* stream) {
  if (B < 0 || B > 65536 || tau != tau || !out_count) return CS_EINVAL;
  if (B > 0 && (!conf || !out_idx)) return CS_EINVAL;
  CS_CUDA(launch_escalate(conf, B, tau, out_accept, out_idx, out_count, static_cast<cudaStream_t>(stream)));
  return CS_OK;
}

int cs_verify_cascade(cs_model* draft, const cs_kv* kv_d, cs_model* target, const cs_kv* kv_t, const int32_t* seq_ids,
                      int B, const int32_t* step_tokens, const int32_t* step_lens, const int32_t* verdict_ids,
                      int n_verdict, float tau, float* out_conf_d, uint8_t* out_trusted, int32_t* out_verdict_d,
                      float* out_conf_t, int32_t* out_verdict_t, int32_t* out_verdict, float* out_conf,
                      const int32_t* req_offsets, int R, int accept_index, int32_t* host_n_escalated, void* stream) {
  if (!draft || !target || draft == target || !kv_d || !kv_t || kv_d->model != draft || kv_t->model != target || B < 0)
    return CS_EINVAL;
  if (tau != tau || n_verdict < 1 || n_verdict > 8 || !verdict_ids) return CS_EINVAL;
  for (int j = 0; j < n_verdict; ++j)
    if (verdict_ids[j] < 0 || verdict_ids[j] >= draft->d.vocab || verdict_ids[j] >= target->d.vocab) return CS_EINVAL;
  if (host_n_escalated) *host_n_escalated = 0;
  if (req_offsets) {
    if (R < 0 || accept_index < 0 || accept_index >= n_verdict || req_offsets[0] != 0 || req_offsets[R] != B)
      return CS_EINVAL;
    for (int r = 0; r < R; ++r)
      if (req_offsets[r + 1] < req_offsets[r]) return CS_EINVAL;
  }
  if (B == 0) return CS_OK;
  if (B > 65536) return CS_EINVAL;
  if (!seq_ids || !step_tokens || !step_lens || !out_conf_d || !out_trusted || !out_verdict_d || !out_verdict ||
      !out_conf)
    return CS_EINVAL;
  // everything the target pass would reject is rejected before the draft pass is launched
  {
    int64_t t = 0;
    for (int i = 0; i < B; ++i) {
      if (step_lens[i] < 1 || seq_ids[i] < 0 || seq_ids[i] >= kv_t->max_seqs || seq_ids[i] >= kv_d->max_seqs)
        return CS_EINVAL;
      if (kv_t->ctx_len[seq_ids[i]] < 0 || kv_d->ctx_len[seq_ids[i]] < 0) return CS_ESTATE;
      t += step_lens[i];
    }
    for (int64_t k = 0; k < t; ++k)
      if (step_tokens[k] < 0 || step_tokens[k] >= target->d.vocab) return CS_EINVAL;
  }
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int rc;
  if ((rc = draft->casc_idx.ensure(sizeof(int32_t) * (2 * static_cast<size_t>(B) + 1)))) return rc;
  if ((rc = ensure_readback(draft, 2 * static_cast<size_t>(B) + 1))) return rc;
  int32_t* idx = static_cast<int32_t*>(draft->casc_idx.p);
  int32_t* count = idx + B;
  int32_t* req_start = nullptr;
  if (req_offsets) {
    // first step of each step's request, for the rule that closes a request at a trusted rejection
    req_start = count + 1;
    int32_t* h = draft->casc_host + B + 1;
    for (int r = 0; r < R; ++r)
      for (int i = req_offsets[r]; i < req_offsets[r + 1]; ++i) h[i] = req_offsets[r];
    CS_CUDA(cudaMemcpyAsync(req_start, h, sizeof(int32_t) * B, cudaMemcpyHostToDevice, s));
  }
  // tier 1: every step through the draft model
  if ((rc = cs_verify_steps(draft, kv_d, seq_ids, B, step_tokens, 0, step_lens, verdict_ids, n_verdict, tau, out_conf_d,
                            out_trusted, out_verdict_d, stream)))
    return rc;
  // the steps it is not confident about, listed on the device; the host needs the list to lay out the second batch
  CS_CUDA(launch_escalate(out_conf_d, B, tau, nullptr, idx, count, s, out_verdict_d, req_start, accept_index));
  CS_CUDA(cudaMemcpyAsync(draft->casc_host + B, count, sizeof(int32_t), cudaMemcpyDeviceToHost, s));
  CS_CUDA(cudaMemcpyAsync(draft->casc_host, idx, sizeof(int32_t) * B, cudaMemcpyDeviceToHost, s));
  CS_CUDA(cudaStreamSynchronize(s));
  const int n_esc = draft->casc_host[B];
  if (n_esc < 0 || n_esc > B) return CS_ECUDA;
  if (host_n_escalated) *host_n_escalated = n_esc;
  // tier 2: the escalated steps, as one smaller batch, through the target model
  const int32_t* verdict_c = nullptr;
  const float* conf_c = nullptr;
  if (n_esc > 0) {
    if ((rc = target->casc_conf.ensure(sizeof(float) * n_esc))) return rc;
    if ((rc = target->casc_verdict.ensure(sizeof(int32_t) * n_esc))) return rc;
    if ((rc = target->casc_accept.ensure(n_esc))) return rc;
    std::vector<int64_t> cu(static_cast<size_t>(B) + 1, 0);
    for (int i = 0; i < B; ++i) cu[i + 1] = cu[i] + step_lens[i];
    std::vector<int32_t> sub_seq(n_esc), sub_len(n_esc), sub_tok;
    for (int j = 0; j < n_esc; ++j) {
      const int i = draft->casc_host[j];
      if (i < 0 || i >= B) return CS_ECUDA;
      sub_seq[j] = seq_ids[i];
      sub_len[j] = step_lens[i];
      sub_tok.insert(sub_tok.end(), step_tokens + cu[i], step_tokens + cu[i + 1]);
    }
    if ((rc = cs_verify_steps(target, kv_t, sub_seq.data(), n_esc, sub_tok.data(), 0, sub_len.data(), verdict_ids,
                              n_verdict, tau, static_cast<float*>(target->casc_conf.p),
                              static_cast<uint8_t*>(target->casc_accept.p),
                              static_cast<int32_t*>(target->casc_verdict.p), stream)))
      return rc;
    verdict_c = static_cast<const int32_t*>(target->casc_verdict.p);
    conf_c = static_cast<const float*>(target->casc_conf.p);
  }
  CS_CUDA(launch_cascade_scatter(B, out_trusted, out_verdict_d, out_conf_d, idx, count, verdict_c, conf_c, out_verdict_t,
                                 out_conf_t, out_verdict, out_conf, s));
  return CS_OK;
}

int cs_cascade_select(const uint8_t* trusted, const int32_t* verdict_d, const float* conf_d, const int32_t* verdict_t,
                      const float* conf_t, const int32_t* req_offsets, int R, int accept_index, int32_t* out_prefix_len,
                      int32_t* out_best, uint8_t* out_pass, float* out_conf, void* stream) {
  if (R < 0 || accept_index < 0 || accept_index > 7) return CS_EINVAL;
  if (R == 0) return CS_OK;
  if (!trusted || !verdict_d || !conf_d || !req_offsets || !out_prefix_len || !out_best) return CS_EINVAL;
  if ((verdict_t == nullptr) != (conf_t == nullptr)) return CS_EINVAL;
  CS_CUDA(launch_cascade_select(trusted, verdict_d, conf_d, verdict_t, conf_t, req_offsets, R, accept_index,
                                out_prefix_len, out_best, out_pass, out_conf, static_cast<cudaStream_t>(stream)));
  return CS_OK;
}

int64_t cs_last_h2d_bytes(const cs_model* m) { return m ? m->last_h2d_bytes : 0; }

int cs_set_deterministic(cs_model* m, int on) {
  if (!m) return CS_EINVAL;
  m->deterministic = on != 0;
  return CS_OK;
}

int cs_set_keep_logits(cs_model* m, int keep) {
  if (!m) return CS_EINVAL;
  m->keep_logits = keep != 0;
  return CS_OK;
}

int cs_get_last_logits(cs_model* m, float* dev_out, int B, void* stream) {
  if (!m || !dev_out || B < 1) return CS_EINVAL;
  if (!m->keep_logits || B > m->last_B || !m->logits.p) return CS_ESTATE;
  CS_CUDA(cudaMemcpyAsync(dev_out, m->logits.p, static_cast<size_t>(B) * m->d.vocab * 4, cudaMemcpyDeviceToDevice,
                          static_cast<cudaStream_t>(stream)));
  return CS_OK;
}

int cs_get_last_lse(cs_model* m, float* dev_out, int B, void* stream) {
  if (!m || !dev_out || B < 1) return CS_EINVAL;
  if (B > m->last_B || !m->lse.p) return CS_ESTATE;
  CS_CUDA(cudaMemcpyAsync(dev_out, m->lse.p, static_cast<size_t>(B) * 4, cudaMemcpyDeviceToDevice,
                          static_cast<cudaStream_t>(stream)));
  return CS_OK;
}

int cs_last_status(cs_model* m, void* stream) {
  if (!m) return CS_EINVAL;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  uint32_t v = 0;
  CS_CUDA(cudaMemcpyAsync(&v, m->status, 4, cudaMemcpyDeviceToHost, s));
  CS_CUDA(cudaStreamSynchronize(s));
  if (v) CS_CUDA(cudaMemsetAsync(m->status, 0, 4, s));
  return (v & 1u) ? CS_ETIMEOUT : (v & 2u) ? CS_ERANGE : CS_OK;
}

int cs_check_workspace(cs_model* m, void* stream) {
  if (!m) return CS_EINVAL;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const DevBuf* bufs[] = {&m->x, &m->x_last, &m->a, &m->qkv, &m->attn_o, &m->hmlp, &m->rope, &m->h_last, &m->lm_part,
                          &m->vlogits, &m->logits, &m->lse, &m->attn_part_o, &m->attn_part_ml, &m->attn_counters,
                          &m->stg.dev, &m->casc_idx, &m->casc_conf, &m->casc_verdict, &m->casc_accept};
  for (const DevBuf* b : bufs) {
    const int st = b->canary_state(s);
    if (st < 0) return cuda_fail(cudaGetLastError(), "workspace canary read-back");
    if (st > 0) return CS_ERANGE;
  }
  return CS_OK;
}

int cs_selftest_range_check(cs_model* m, void* stream) {
  if (!m) return CS_EINVAL;
  CS_CUDA(launch_range_check_selftest(m->status, static_cast<cudaStream_t>(stream)));
  return CS_OK;
}

int cs_debug_build(void) {
#ifdef CS_DEBUG
  return 1;
#else
  return 0;
#endif
}

int cs_selftest_wait_timeout(cs_model* m, int polls, void* stream) {
  if (!m || polls < 1 || polls > (1 << 20)) return CS_EINVAL;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int rc;
  if ((rc = m->casc_idx.ensure(sizeof(int32_t) * 4))) return rc;
  int32_t* gave_up = static_cast<int32_t*>(m->casc_idx.p);
  CS_CUDA(cudaMemsetAsync(gave_up, 0, sizeof(int32_t), s));
  CS_CUDA(launch_wait_timeout_selftest(m->status, static_cast<uint32_t>(polls), gave_up, s));
  int32_t h = 0;
  CS_CUDA(cudaMemcpyAsync(&h, gave_up, sizeof(int32_t), cudaMemcpyDeviceToHost, s));
  CS_CUDA(cudaStreamSynchronize(s));
  return h == 1 ? CS_OK : CS_ESTATE;
}

int cs_profile(cs_model* m, int enable) {
  if (!m) return CS_EINVAL;
  m->prof.on = enable != 0;
  m->prof.used = 0;
  return CS_OK;
}

int cs_profile_read(cs_model* m, float* ms_out, int32_t* launches_out, int n_classes) {
  if (!m || !ms_out || !launches_out || n_classes < kProfClasses) return CS_EINVAL;
  for (int c = 0; c < n_classes; ++c) { ms_out[c] = 0.f; launches_out[c] = 0; }
  Prof& p = m->prof;
  for (size_t i = 0; i < p.used; ++i) {
    CS_CUDA(cudaEventSynchronize(p.pool[2 * i + 1]));
    float ms = 0.f;
    CS_CUDA(cudaEventElapsedTime(&ms, p.pool[2 * i], p.pool[2 * i + 1]));
    ms_out[p.cls[i]] += ms;
    launches_out[p.cls[i]] += 1;
  }
  p.used = 0;
  return CS_OK;
}

int cs_gemm_f16(const uint16_t* a, const uint16_t* w, const uint16_t* w2, void* out, int M, int N, int K,
                 int epilogue, void* stream) {
  if (!a || !w || !out || M < 0 || N < 8 || K < 8 || (N % 8) || (K % 8) || epilogue < 0 || epilogue > 3)
    return CS_EINVAL;
  if (epilogue == kEpiSwiGLU && !w2) return CS_EINVAL;
  if (M == 0) return CS_OK;
  if (!g_test_status) {
    CS_CUDA(cudaMalloc(reinterpret_cast<void**>(&g_test_status), 256));
    CS_CUDA(cudaMemset(g_test_status, 0, 256));
  }
  CUtensorMap ta, tb, tb2;
  if (!make_gemm_operand_map(&ta, a, M, K) || !make_gemm_operand_map(&tb, w, N, K) ||
      (w2 && !make_gemm_operand_map(&tb2, w2, N, K))) {
    g_cuda_error = "cuTensorMapEncodeTiled failed";
    return CS_ECUDA;
  }
  if (!g_test_turn_flags) {
    CS_CUDA(cudaMalloc(reinterpret_cast<void**>(&g_test_turn_flags), sizeof(uint32_t) * kTurnWords));
    CS_CUDA(cudaMemset(g_test_turn_flags, 0, sizeof(uint32_t) * kTurnWords));
  }
  TurnOrder turn{g_test_turn_flags, &g_test_turn_epoch};
  CS_CUDA(gemm_f16(ta, tb, w2 ? &tb2 : nullptr, out, M, N, K, epilogue == 3 ? kEpiResidAdd : epilogue, g_test_status,
                    static_cast<cudaStream_t>(stream), epilogue == 1 ? &turn : nullptr));
  return CS_OK;
}

int cs_lm_head_gate(const uint16_t* w_lm, const uint16_t* h, int B, int d_model, int vocab, const int32_t* verdict_ids,
                    int n_verdict, float tau, float* out_conf, uint8_t* out_accept, int32_t* out_verdict, float* out_lse,
                    void* stream) {
  if (!w_lm || !h || B < 0 || d_model < 8 || (d_model % 8) || vocab < 1 || tau != tau) return CS_EINVAL;
  if (n_verdict < 1 || n_verdict > 8 || !verdict_ids) return CS_EINVAL;
  for (int j = 0; j < n_verdict; ++j)
    if (verdict_ids[j] < 0 || verdict_ids[j] >= vocab) return CS_EINVAL;
  if (B == 0) return CS_OK;
  if (!out_conf || !out_accept) return CS_EINVAL;
  if (!g_test_status) {
    CS_CUDA(cudaMalloc(reinterpret_cast<void**>(&g_test_status), 256));
    CS_CUDA(cudaMemset(g_test_status, 0, 256));
  }
  // scratch: per-CTA (max, sum exp) pairs and the verdict logits of one chunk of up to 64 steps
  static DevBuf scratch;
  const size_t part_floats = static_cast<size_t>(2) * kNumSMs * 64;
  int rc;
  if ((rc = scratch.ensure((part_floats + 64 * 8) * sizeof(float)))) return rc;
  float* part_max = static_cast<float*>(scratch.p);
  float* part_sum = part_max + kNumSMs * 64;
  float* vlog = part_max + part_floats;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  CUtensorMap tm_w, tm_h;
  if (!make_gemm_operand_map(&tm_w, w_lm, vocab, d_model)) {
    g_cuda_error = "cuTensorMapEncodeTiled failed for the LM head";
    return CS_ECUDA;
  }
  int rows_per_cta;
  const int grid = lm_head_grid(vocab, &rows_per_cta);
  for (int b0 = 0; b0 < B; b0 += 64) {
    const int bc = std::min(64, B - b0);
    const int bp = lm_head_batch_pad(bc);
    // rows past B are filled with zeros by the copy engine
    if (!make_tensor_map_16b(&tm_h, h, B, d_model, bp, 64, true, false)) {
      g_cuda_error = "cuTensorMapEncodeTiled failed for the hidden states";
      return CS_ECUDA;
    }
    CS_CUDA(launch_lm_head(tm_w, tm_h, b0, bc, bp, d_model, vocab, verdict_ids, n_verdict, part_max, part_sum, vlog,
                           nullptr, g_test_status, s));
    CS_CUDA(launch_gate(part_max, part_sum, grid, bp, vlog, n_verdict, bc, tau, out_conf + b0, out_accept + b0,
                        out_verdict ? out_verdict + b0 : nullptr, out_lse ? out_lse + b0 : nullptr, s));
  }
  return CS_OK;
}

int cs_rmsnorm(const float* x, const float* gain, uint16_t* out, int rows, int d, float eps, void* stream) {
  if (!x || !gain || !out || rows < 0 || d < 4 || (d % 4)) return CS_EINVAL;
  CS_CUDA(launch_rmsnorm(x, gain, out, rows, d, eps, static_cast<cudaStream_t>(stream)));
  return CS_OK;
}

}  // extern "C"
