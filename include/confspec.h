/*
 * confspec.h — C ABI of the batched draft-verification pass of confidence-gated cascaded verification.
 *
 * What the library computes (paper Section 4.2; Algorithm 1, Stage 2): a batch of candidate reasoning
 * steps, each appended to its cached reasoning context, is run through one extend-prefill of a
 * decoder-only transformer; the hidden state of each step's last new position goes through the LM head;
 * the probability of the decision ("verdict") token under the softmax over the whole vocabulary is the
 * confidence p_D (Eqs. 2-3); the draft verifier's decision is trusted when p_D >= gamma and the step is
 * escalated to the target model otherwise (Eq. 4). Every step of that path runs in CUDA kernels written
 * for sm_100a; there is no CPU fallback.
 *
 * Conventions
 *  - Every function returns an int status (CS_OK = 0). Nothing throws, exits or prints.
 *  - "host" / "device" in a parameter comment says where the pointer must point. Device pointers are
 *    plain CUDA device addresses on the current device (for instance torch.Tensor.data_ptr()).
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream). Calls that take a
 *    stream only enqueue work; results are valid once the stream has been synchronised.
 *  - Handles are not thread-safe: use one handle from one host thread at a time.
 *  - bf16 values are passed as uint16_t bit patterns.
 */
#ifndef CONFSPEC_H
#define CONFSPEC_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  CS_OK = 0,
  CS_EINVAL = 1,   /* an argument is out of range or NULL; nothing was launched */
  CS_ENOMEM = 2,   /* a device or host allocation failed */
  CS_ECUDA = 3,    /* a CUDA runtime / driver call failed; see cs_last_cuda_error */
  CS_ETIMEOUT = 4, /* a kernel gave up on a bounded wait (reported by cs_last_status) */
  CS_ESTATE = 5,   /* the call does not fit the handle's state (e.g. sequence not set) */
  CS_ELIMIT = 6,   /* a size exceeds the fixed capacity of an entry point that never allocates */
  CS_ERANGE = 7    /* a device-side range check of a debug build failed, or a workspace's guard bytes were written */
};

typedef struct cs_model cs_model;
typedef struct cs_kv cs_kv;

/* Geometry of the decoder. n_q_heads must be a multiple of n_kv_heads; head_dim is 64 or 128;
 * d_model, n_q_heads*head_dim and d_ffn must be multiples of 8 (16-byte rows for TMA). */
typedef struct cs_model_desc {
  int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ffn, vocab;
  float rope_theta; /* rotary base; pair (j, j + head_dim/2) turns by pos * theta^(-2j/head_dim) */
  float rms_eps;    /* added to the mean square inside every RMSNorm */
} cs_model_desc;

/* Weights handed to cs_model_load. Matrices are bf16, row-major [out_features, in_features].
 * The per-layer members are arrays of n_layers pointers. No biases; embedding and LM head are separate. */
typedef struct cs_model_tensors {
  const uint16_t* embed;        /* [vocab, d_model] */
  const uint16_t* lm_head;      /* [vocab, d_model] */
  const float* final_norm;      /* [d_model] RMSNorm gain before the LM head */
  const uint16_t* const* wq;    /* [n_q_heads*head_dim, d_model] */
  const uint16_t* const* wk;    /* [n_kv_heads*head_dim, d_model] */
  const uint16_t* const* wv;    /* [n_kv_heads*head_dim, d_model] */
  const uint16_t* const* wo;    /* [d_model, n_q_heads*head_dim] */
  const uint16_t* const* wg;    /* [d_ffn, d_model]  SwiGLU gate */
  const uint16_t* const* wu;    /* [d_ffn, d_model]  SwiGLU up */
  const uint16_t* const* wd;    /* [d_model, d_ffn]  SwiGLU down */
  const float* const* norm1;    /* [d_model] gain of the pre-attention RMSNorm */
  const float* const* norm2;    /* [d_model] gain of the pre-MLP RMSNorm */
  /* Second model family of the paper's experiments (Section 5.1): every head's query and key vector is
   * RMS-normalised over its head_dim entries (eps = rms_eps) before the rotary turn, with one gain vector per layer
   * shared by all query heads and one shared by all key heads. Both NULL: no such normalisation. */
  const float* const* q_norm;   /* [head_dim] or NULL */
  const float* const* k_norm;   /* [head_dim] or NULL */
} cs_model_tensors;

/* Library version as major*10000 + minor*100 + patch. */
int cs_version(void);
/* Static English text for a status code. */
const char* cs_strerror(int status);
/* Text of the last CUDA error seen by a call on this host thread ("" if none). */
const char* cs_last_cuda_error(void);

/*
 * cs_model_load — copy a verifier model (the M_D, or M_T for escalated steps, of Algorithm 1) into
 * library-owned device memory and prepare everything that does not depend on a batch (fused QKV matrix,
 * TMA descriptors, rotary frequencies). The projection and LM-head matrices are re-encoded from bf16 to fp16
 * on the device (exact for magnitudes in [2^-14, 65504], absolute error <= 2^-25 below): the tensor cores take
 * both operands in one 16-bit format, and the activations are kept in fp16, whose rounding error is 8x smaller
 * than bf16's. Activations beyond the fp16 range (|v| > 65504) are not supported.
 *   desc               host. Geometry.
 *   tensors            host struct; the tensor pointers inside are host pointers when
 *                      tensors_on_device == 0, device pointers otherwise. The caller keeps ownership and
 *                      may free them once the call returns (the copy is synchronous).
 *   out                receives the handle; release with cs_model_free.
 * Errors: CS_EINVAL (NULL, bad geometry), CS_ENOMEM, CS_ECUDA (e.g. not an sm_100 device).
 */
int cs_model_load(const cs_model_desc* desc, const cs_model_tensors* tensors, int tensors_on_device,
                  cs_model** out);
int cs_model_free(cs_model* model);

/*
 * cs_model_set_lm_head_rows - replace rows of a loaded model's LM head, e.g. the rows of the verdict tokens whose
 * probability is the confidence of Eqs. 2-3 (a verifier whose decision tokens were tuned after the base model was
 * loaded; the tests use it to give the verdict rows a weight that spreads the confidences over (0, 1)).
 *   row_ids            host int32[n_rows], each in [0, vocab).
 *   rows_bf16          host bf16 [n_rows, d_model]; re-encoded like the matrices at load.
 * Enqueued on `stream` behind earlier passes and synchronised before returning. Errors: CS_EINVAL, CS_ECUDA.
 */
int cs_model_set_lm_head_rows(cs_model* model, const int32_t* row_ids, int n_rows, const uint16_t* rows_bf16,
                              void* stream);

/*
 * cs_reserve — size the per-model activation workspace for batches of up to max_steps steps and
 * max_tokens new tokens in total. Optional: cs_verify_steps / cs_prefill grow the workspace on demand, but
 * growing synchronises the device, so latency-sensitive callers reserve once up front.
 */
int cs_reserve(cs_model* model, int max_steps, int max_tokens);

/*
 * cs_kv_alloc — the paged bf16 cache of reasoning contexts ("context" of Algorithm 1, which grows by the
 * accepted steps and is re-read by every verification).
 * Pool layout (bf16): [n_layers][2 (K, V)][num_pages][n_kv_heads][page_size][head_dim]; K is stored
 * already rotated. page_size must be 16. The pool is zero-filled at allocation; slots past a sequence's
 * length inside its last page must hold finite values (they are masked, not skipped).
 *   dev_pool           device or NULL. When given, caller-owned memory of cs_kv_pool_bytes() bytes,
 *                      256-byte aligned, already zeroed; otherwise the library allocates and owns the pool.
 *   max_seqs, max_pages_per_seq   capacity of the page table.
 */
int cs_kv_alloc(const cs_model* model, int num_pages, int page_size, int max_seqs, int max_pages_per_seq,
                void* dev_pool, cs_kv** out);
/*
 * cs_kv_alloc_8bit - the same cache in an optional 8-bit format (no counterpart in the paper, which leaves the
 * cache to its serving engine): one byte per element, unscaled, in one of two floating-point formats,
 *   CS_KV_E4M3  4 exponent bits (bias 7), 3 mantissa bits, no infinities (largest value 448);
 *   CS_KV_E5M2  5 exponent bits (bias 15), 2 mantissa bits: the upper byte of an fp16.
 * Half the bytes, always library-owned (cs_kv_pool_bytes() / 2); pool layout as above except that V pages are
 * kept transposed, [head_dim][page_size].
 * It serves the decode-shaped use of the pass, where reading the cache bounds the time: cs_verify_steps accepts it
 * when every step has at most 32 query rows per kv head (step_lens[i] * n_q_heads / n_kv_heads <= 32; CS_EINVAL
 * otherwise), widens the codes to fp16 on the fly (exact) and computes as with the 16-bit cache. The format is
 * read-only for the pass: contexts come from cs_kv_fill (host arrays of uint8 codes instead of bf16 patterns);
 * cs_prefill and cs_append_accepted return CS_EINVAL on such a cache.
 */
#define CS_KV_E4M3 1
#define CS_KV_E5M2 2
int cs_kv_alloc_8bit(const cs_model* model, int num_pages, int page_size, int max_seqs, int max_pages_per_seq,
                     int format, cs_kv** out);
int cs_kv_free(cs_kv* kv);
/* Bytes of pool that cs_kv_alloc needs for this geometry (0 on bad arguments). */
uint64_t cs_kv_pool_bytes(const cs_model* model, int num_pages, int page_size);

/*
 * cs_kv_set_seq — define sequence `seq`: its pages, in order, and its cached length.
 *   page_ids           host int32[n_pages], each in [0, num_pages). Pages may be shared by several
 *                      sequences (k candidate steps verified on one context).
 *   ctx_len            cached tokens, 0 <= ctx_len <= n_pages * page_size.
 * Host-side only; the table is uploaded by the next call that reads it.
 */
int cs_kv_set_seq(cs_kv* kv, int seq, const int32_t* page_ids, int n_pages, int ctx_len);

/*
 * cs_kv_fill — write given K/V into the pages of sequence `seq` for one layer (synthetic contexts in
 * tests and benchmarks).
 *   host_k, host_v     host bf16 [ctx_len, n_kv_heads, head_dim] (uint8 codes of the same shape for a cache from
 *                      cs_kv_alloc_8bit); K already rotated.
 * Synchronous on `stream`.
 */
int cs_kv_fill(cs_kv* kv, int seq, int layer, const uint16_t* host_k, const uint16_t* host_v, void* stream);

/*
 * cs_prefill — run tokens through the model and APPEND their K/V to the sequences' pages
 * (context management of Algorithm 1, Stage 3: accepted steps become context). The sequences must have
 * enough pages set for ctx_len + lens[i]. On success each sequence's ctx_len grows by lens[i]. The pass ends with
 * the last layer's K/V projection: nothing reads what would follow it.
 *   seq_ids, lens      host int32[B];  tokens  host int32[sum lens], concatenated per sequence.
 */
int cs_prefill(cs_model* model, cs_kv* kv, const int32_t* seq_ids, const int32_t* tokens,
               const int32_t* lens, int B, void* stream);

/*
 * cs_append_accepted - context management of Algorithm 1, Stage 3, in terms of the cache: for every request r whose
 * accept-prefix length m_r (out_prefix_len of cs_cascade_select) is positive,
 *     context_r <- context_r (+) s^_1 (+) ... (+) s^_m,
 * i.e. the tokens of its first m_r drafted steps run through the model on top of the cached context and their K/V
 * are appended to the pages of the request's sequence (one cs_prefill over all such requests). Requests with
 * m_r = 0 are left alone: their next step comes from the target model's generation, which is outside this library.
 * The k candidates of a request are verified on the request's own sequence id (cs_verify_steps takes the same
 * sequence several times), so they share its pages; nothing is copied per candidate, and after this call the next
 * iteration's candidates see the longer context under the same id.
 *   kv                 cache of `model`; call once per model that caches the contexts (draft and target).
 *   req_seq_ids        host int32[R], distinct: the sequence holding request r's context. It must already own
 *                      pages for the appended tokens (cs_kv_set_seq), else CS_EINVAL and nothing is appended.
 *   req_offsets        host int32[R + 1]: the steps of request r are [req_offsets[r], req_offsets[r+1]) of the batch.
 *   dev_prefix_len     DEVICE int32[R], each in [0, number of steps of the request]; read back inside the call
 *                      (4 R bytes, blocks the host once).
 *   step_tokens, step_lens   host, as given to cs_verify_steps (the whole verification spans).
 *   draft_lens         host int32[B]: how many leading tokens of span i are the drafted step s^_i itself
 *                      (0 <= draft_lens[i] <= step_lens[i]); the rest of the span (the target's step, the
 *                      verification prompt) never enters the context.
 *   host_prefix_len    host int32[R] or NULL: receives the m_r that were read.
 * Errors: CS_EINVAL, CS_ESTATE (unset sequence) before any launch; then as cs_prefill.
 */
int cs_append_accepted(cs_model* model, cs_kv* kv, int R, const int32_t* req_seq_ids, const int32_t* req_offsets,
                       const int32_t* dev_prefix_len, const int32_t* step_tokens, const int32_t* step_lens,
                       const int32_t* draft_lens, int32_t* host_prefix_len, void* stream);

/*
 * cs_verify_steps — the verification pass itself (M.verify of Algorithm 1, Stage 2; Eqs. 2-4).
 * For step i, the new tokens step_tokens[cu[i] .. cu[i]+step_lens[i]) (draft step, target step and the
 * verification prompt, as one opaque span) are placed at positions ctx_len .. ctx_len+step_lens[i]-1 after
 * the cached context of sequence seq_ids[i]; the last position's logits z give
 *     conf = max_j exp(z[verdict_ids[j]] - logsumexp_v z[v]),   verdict = first j attaining it,
 *     accept = (conf >= tau)     (fp32 comparison; NaN never accepts).
 * The cache is read-only here: K/V of the new tokens live in the model's workspace and are discarded.
 * Only the last position of a step reaches the LM head, so the MLP half of the last layer is computed for those
 * B rows alone (same arithmetic per row).
 *   ctx_kv             cache handle whose sequences seq_ids[i] have been set.
 *   seq_ids            host int32[B]. The same sequence may appear several times.
 *   step_tokens        int32[sum step_lens]; host when tokens_on_device == 0 (copied on `stream`), else
 *                      device. Ids must lie in [0, vocab) (host tokens are checked; device tokens are clamped).
 *   step_lens          host int32[B], each >= 1 (verification suffix included).
 *   verdict_ids        host int32[n_verdict], 1 <= n_verdict <= 8, ids in [0, vocab).
 *   tau                threshold gamma of Eq. 4; NaN is rejected with CS_EINVAL.
 *   out_conf           device float[B].
 *   out_accept         device uint8[B]: 1 = the draft decision is trusted, 0 = escalate.
 *   out_verdict        device int32[B] or NULL: index into verdict_ids of the decision r_D.
 * Asynchronous on `stream`. Deterministic: the same call on the same inputs gives bit-identical out_conf, out_accept,
 * out_verdict (and logits) every time - every reduction of the pass has a fixed order (see cs_set_deterministic).
 * A model's calls must be issued on one stream at a time: they share its workspace and ordering words.
 * Errors: CS_EINVAL before any launch; CS_ESTATE for an unset sequence; CS_ENOMEM / CS_ECUDA.
 */
int cs_verify_steps(cs_model* model, const cs_kv* ctx_kv, const int32_t* seq_ids, int B,
                    const int32_t* step_tokens, int tokens_on_device, const int32_t* step_lens,
                    const int32_t* verdict_ids, int n_verdict, float tau,
                    float* out_conf, uint8_t* out_accept, int32_t* out_verdict, void* stream);

/*
 * cs_escalate_mask — re-apply the rule of Eq. 4 to stored confidences for another threshold and list
 * the steps that must go to the target model, without leaving the device.
 *   conf               device float[B].
 *   out_accept         device uint8[B] or NULL.
 *   out_escalate_idx   device int32[B]: the first *out_escalate_count entries are the indices of the
 *                      escalated steps in ascending order; the rest is left untouched.
 *   out_escalate_count device int32[1].
 * B <= 65536. Asynchronous on `stream`.
 */
int cs_escalate_mask(const float* conf, int B, float tau, uint8_t* out_accept,
                     int32_t* out_escalate_idx, int32_t* out_escalate_count, void* stream);

/*
 * cs_verify_cascade - the two-tier verifier V_cascade of Eq. 4 (Algorithm 1, Stage 2) in one call: every step goes
 * through the draft model (cs_verify_steps); the steps whose confidence p_D is below gamma are listed on the device
 * (cs_escalate_mask) and go, as one smaller batch, through the target model; the final decision of a step is r_D
 * where p_D >= gamma and r_T otherwise. The target model therefore costs time in proportion to the cascade rate
 * (Section 4.4).
 *   draft, kv_d        draft model and its context cache; target, kv_t likewise (draft != target). Sequence
 *                      seq_ids[i] must be set in BOTH caches and hold the same reasoning context as each model
 *                      caches it. The models may differ in every dimension; token and verdict ids must be valid in both.
 *   seq_ids, step_lens host int32[B];  step_tokens  HOST int32[sum step_lens] (the second batch is laid out on
 *                      the host from the list of escalated steps).
 *   out_conf_d, out_trusted, out_verdict_d   device float[B], uint8[B], int32[B]: the draft tier's p_D,
 *                      (p_D >= tau), r_D as an index into verdict_ids. All required.
 *   out_conf_t, out_verdict_t   device float[B], int32[B] or NULL: the target tier's p_T and r_T at the steps it
 *                      verified, (0, -1) at all others.
 *   out_verdict, out_conf   device int32[B], float[B]: final decision and the confidence of the verifier that
 *                      took it. Required.
 *   req_offsets, R, accept_index   linear drafting (Algorithm 1): host int32[R + 1], the steps of request r are
 *                      [req_offsets[r], req_offsets[r+1]) of the batch in drafting order, req_offsets[R] == B;
 *                      accept_index = index into verdict_ids of the "accept" decision. The loop of Algorithm 1 over a
 *                      request's steps breaks at the first rejection, so a step behind a TRUSTED draft rejection
 *                      of its request is not sent to the target model even when its own confidence is below tau;
 *                      it ends with out_verdict = -1, out_conf = 0 (cs_cascade_select counts it as rejected,
 *                      which leaves every accept-prefix length as it would be with all steps verified).
 *                      req_offsets == NULL (tree drafting, Section 4.3: every candidate counts): every step
 *                      below tau goes to the target; R and accept_index are ignored.
 *   host_n_escalated   host int32[1] or NULL: number of steps sent to the target model, valid on return.
 * The call blocks the host once between the tiers (it reads the list back: 4 (B + 1) bytes); the target pass and
 * the final scatter are asynchronous on `stream`. Arguments are checked for both tiers before anything is
 * launched. B <= 65536.
 * Errors: as cs_verify_steps.
 */
int cs_verify_cascade(cs_model* draft, const cs_kv* kv_d, cs_model* target, const cs_kv* kv_t,
                      const int32_t* seq_ids, int B, const int32_t* step_tokens, const int32_t* step_lens,
                      const int32_t* verdict_ids, int n_verdict, float tau,
                      float* out_conf_d, uint8_t* out_trusted, int32_t* out_verdict_d,
                      float* out_conf_t, int32_t* out_verdict_t, int32_t* out_verdict, float* out_conf,
                      const int32_t* req_offsets, int R, int accept_index, int32_t* host_n_escalated, void* stream);

/*
 * cs_cascade_select - what the drafting loop does with the verification results of one iteration, on the device.
 * Final decision of step i (Algorithm 1, Stage 2; Eq. 4): the draft verifier's decision when it was trusted
 * (trusted[i] != 0, i.e. p_D >= gamma), else the target verifier's; an escalated step without a target result
 * (verdict_t == NULL) counts as rejected. Its confidence is that of the verifier whose decision was taken.
 * Per request r, whose steps are [req_offsets[r], req_offsets[r+1]) of the batch:
 *   out_prefix_len[r]  m of Algorithm 1: the number of leading steps whose final decision is "accept" (the loop
 *                      over the drafted steps breaks at the first rejection);
 *   out_best[r]        tree drafting (Section 4.3, Eq. 5): batch index of the accepted candidate with the highest
 *                      confidence, the earliest on ties, or -1 if none was accepted.
 *   trusted            device uint8[B]  (out_accept of the draft pass).
 *   verdict_d, conf_d  device int32[B], float[B] (out_verdict, out_conf of the draft pass).
 *   verdict_t, conf_t  device int32[B], float[B], read only where trusted[i] == 0, or both NULL.
 *   req_offsets        device int32[R+1], ascending, req_offsets[0] .. req_offsets[R] within [0, B].
 *   accept_index       which entry of verdict_ids means "accept" (0..7).
 *   out_pass, out_conf device uint8[B], float[B] or NULL: the final decision (1 = accept) and confidence per step.
 * Asynchronous on `stream`. Errors: CS_EINVAL.
 */
int cs_cascade_select(const uint8_t* trusted, const int32_t* verdict_d, const float* conf_d, const int32_t* verdict_t,
                      const float* conf_t, const int32_t* req_offsets, int R, int accept_index, int32_t* out_prefix_len,
                      int32_t* out_best, uint8_t* out_pass, float* out_conf, void* stream);

/*
 * Debug / test access. cs_set_keep_logits(model, 1) makes every later cs_verify_steps also write the full
 * last-position logits (fp32 [B, vocab]) into the workspace; cs_get_last_logits copies them to
 * dev_out (device float[B*vocab]) on `stream`. cs_get_last_lse copies the per-step logsumexp
 * (device float[B]). cs_last_status synchronises `stream` and returns CS_ETIMEOUT if any kernel since the
 * previous query gave up on a bounded wait, else CS_OK.
 */
int cs_set_keep_logits(cs_model* model, int keep);
/*
 * cs_set_deterministic - choose how the residual projections (x += o Wo^T, x += h Wd^T) add the pieces of a long k
 * range that is cut over several SMs. on != 0 (the default): in a fixed order, one piece of a tile after the other, so
 * that a pass is bit-identical from run to run - the cascade rule of Eq. 4 is a threshold, and a last-bit difference
 * in a confidence next to tau would change which steps escalate. on == 0: pieces add as they finish; a little faster,
 * results agree to rounding only.
 */
int cs_set_deterministic(cs_model* model, int on);
int cs_get_last_logits(cs_model* model, float* dev_out, int B, void* stream);
int cs_get_last_lse(cs_model* model, float* dev_out, int B, void* stream);
int cs_last_status(cs_model* model, void* stream);

/*
 * cs_selftest_wait_timeout - failure detection, exercised without a fault: every wait inside the library's kernels
 * (on a copy's arrival, on a tensor-core commit) is bounded; a kernel whose wait runs out raises a bit in the
 * model's status word, stops issuing work, lets its copies land, frees its tensor memory and returns, and the next
 * cs_last_status reports CS_ETIMEOUT. This call launches a one-thread kernel that runs that same bounded wait, with a
 * limit of `polls` polls (1 .. 2^20; a few milliseconds at most), on a barrier nothing ever arrives at, so that the
 * path from a starved wait to the host can be tested on a healthy GPU. The context stays usable.
 * Returns CS_OK when the wait gave up as it should (the model's status word now holds the time-out bit: the next
 * cs_last_status returns CS_ETIMEOUT and clears it), CS_ESTATE if the wait returned as satisfied. Synchronises `stream`.
 */
int cs_selftest_wait_timeout(cs_model* model, int polls, void* stream);
/*
 * Debugging aids (there is no memory checker to run the kernels under).
 *  - A library compiled with -DCS_DEBUG (cs_debug_build() returns 1) tests page ids, token rows and tensor-memory
 *    columns on the device where they are used. A failed test raises a bit of the model's status word, the access is
 *    skipped or clamped, nothing traps; the next cs_last_status returns CS_ERANGE once. The release build has none of
 *    these tests (the host validates every argument before a launch).
 *  - cs_selftest_range_check launches a kernel whose one range test fails by construction without touching memory:
 *    afterwards cs_last_status returns CS_ERANGE in a debug build and CS_OK in a release build.
 *  - Every workspace of a model (activations, staging, partial results) is followed by 256 guard bytes of a fixed
 *    pattern. cs_check_workspace reads them back (synchronising `stream`): CS_ERANGE if any was written, in any build.
 */
int cs_debug_build(void);
int cs_selftest_range_check(cs_model* model, void* stream);
int cs_check_workspace(cs_model* model, void* stream);

/*
 * Per-stage entry points. They run single kernels of the pass on caller-provided device buffers so that
 * each can be checked against the oracle's corresponding block, and timed, in isolation.
 */
/* out[M,N] (+)= a[M,K] * w[N,K]^T on the tcgen05 tensor cores. a, w fp16 row-major (device), fp32 accumulate.
 *   epilogue 0: out fp16 [M,N] = result.
 *   epilogue 1: out fp32 [M,N] += result. Long k ranges are split over the SMs and the pieces of a tile are added in a
 *               fixed order (bit-identical from run to run); calls that overlap on the GPU share the ordering words
 *               and must be kept on one stream.
 *   epilogue 3: as 1 without the fixed order (pieces add as they finish; results agree to rounding only).
 *   epilogue 2: w2 is a second [N,K] matrix; out fp16 [M,N] = silu(a*w^T) * (a*w2^T).
 * K and N multiples of 8. Asynchronous on `stream`. */
int cs_gemm_f16(const uint16_t* a, const uint16_t* w, const uint16_t* w2, void* out,
                 int M, int N, int K, int epilogue, void* stream);
/* The last stage of the pass on its own (Section 4.2, Eqs. 2-4): logits z = w_lm h for B steps, logsumexp over the
 * whole vocabulary fused into the product (the logits are never written), conf = max_j exp(z[verdict_ids[j]] - lse),
 * verdict = first j attaining it, accept = (conf >= tau).
 *   w_lm               device fp16 [vocab, d_model], row-major.
 *   h                  device fp16 [B, d_model]: the final-normed hidden state of each step's last position.
 *   verdict_ids        host int32[n_verdict], 1 <= n_verdict <= 8.
 *   out_conf, out_accept, out_verdict (or NULL), out_lse (or NULL)   device arrays of B entries.
 * d_model a multiple of 8. The per-CTA partial sums live in a scratch buffer that the library allocates on first use
 * (cudaMalloc) and keeps; calls on different streams that overlap on the GPU would share it and race.
 * Asynchronous on `stream`. */
int cs_lm_head_gate(const uint16_t* w_lm, const uint16_t* h, int B, int d_model, int vocab, const int32_t* verdict_ids,
                    int n_verdict, float tau, float* out_conf, uint8_t* out_accept, int32_t* out_verdict, float* out_lse,
                    void* stream);
/*
 * cs_lm_head_gate_static - the same stage as cs_lm_head_gate, for callers that cannot allocate device memory.
 * (The paper has no counterpart: this entry point exists for the sake of its callers, not of the method.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits. Examples are a serving process whose memory pool owns
 * all of the device memory and forbids side allocations, a real-time loop that may not take the allocator's locks or
 * its implicit device synchronisation, and a plug-in loaded into a host application that hands out buffers itself.
 * cs_lm_head_gate would call cudaMalloc on its first use; this function never calls cudaMalloc, cudaFree or any
 * routine that allocates.
 *
 * Instead its scratch (per-CTA partial maxima and sums, the verdict logits, a status word: about 78 KB) is a fixed
 * array inside the library image. Consequences the caller must know:
 *   - every GPU on which the library is loaded holds that array until the process exits;
 *   - capacity is fixed: B <= CS_LM_HEAD_STATIC_MAX_STEPS, else CS_ELIMIT is returned and nothing is launched (larger
 *     batches: call it in chunks, one after the other on one stream);
 *   - all calls share the one array per GPU: two calls that overlap on the GPU (different streams, or different
 *     threads) race on it and give wrong results. Calls on one stream are ordered and safe. The function clears the
 *     part of the array that must start at zero on every call, so leftovers of an earlier call do no harm;
 *   - the first call on each device looks up the array's device address (with that device current). Make that first
 *     call outside any stream capture.
 * If the LM-head kernel gives up on a bounded wait, every out_conf is set to NaN and every out_accept to 0.
 * Arguments, layouts and asynchrony are those of cs_lm_head_gate.
 * Errors: CS_EINVAL (arguments), CS_ELIMIT (B too large), CS_ECUDA.
 */
#define CS_LM_HEAD_STATIC_MAX_STEPS 64
int cs_lm_head_gate_static(const uint16_t* w_lm, const uint16_t* h, int B, int d_model, int vocab,
                           const int32_t* verdict_ids, int n_verdict, float tau, float* out_conf, uint8_t* out_accept,
                           int32_t* out_verdict, float* out_lse, void* stream);
/* out fp16 [rows, d] = RMSNorm(x fp32 [rows, d]; gain fp32 [d], eps). */
int cs_rmsnorm(const float* x, const float* gain, uint16_t* out, int rows, int d, float eps, void* stream);
/*
 * Per-kernel-class timing of the pass. cs_profile(model, 1) makes cs_verify_steps / cs_prefill record a pair
 * of CUDA events around each kernel launch (on the call's stream); cs_profile_read waits for the recorded
 * events, adds the elapsed milliseconds and the number of timed launches per class into ms_out / calls_out
 * (host arrays of n_classes >= CS_PROF_CLASSES entries) and clears the record. Classes, in order: embedding,
 * RMSNorm, QKV GEMM (rotary turn in its epilogue), rotary (unused: always 0), attention, O GEMM, gate/up GEMM (SwiGLU),
 * down GEMM, LM head, gate, other. The events keep consecutive kernels from overlapping and cost a little host and
 * device time, so throughput is measured with profiling off.
 */
#define CS_PROF_CLASSES 11
int cs_profile(cs_model* model, int enable);
int cs_profile_read(cs_model* model, float* ms_out, int32_t* calls_out, int n_classes);
/* Bytes that the last cs_verify_steps / cs_prefill call on this model copied from the host to the device: the batch
 * metadata (offsets, positions, attention work items) and, when the tokens were given on the host, the tokens. */
int64_t cs_last_h2d_bytes(const cs_model* model);
/* Number of kernels the library has launched on this host thread since the last call of this function. */
int64_t cs_take_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* CONFSPEC_H */
