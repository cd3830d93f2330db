"""CPU oracle of the batched draft-verification pass. TEST INFRASTRUCTURE ONLY.

Nothing in the product path may import this file: it exists so that tests, the
smoke check and the benchmark's CPU-baseline leg can compare the CUDA kernels
with a slow, plain statement of what the paper defines. It shares no code with
the CUDA path and never imports it.

What it states (paper Section 4.2, "Draft Verification" and "Cascaded Decision
Rule"; Algorithm 1, Stage 2): the verifier model reads the cached reasoning
context followed by the step's new tokens (draft step, target step, prompt
suffix), emits one decision token, and the confidence p_D is the softmax
probability of that decision token (Eqs. 2-3); the draft's decision is trusted
when p_D >= gamma and escalated to the target model otherwise (Eq. 4).

The model itself is not defined by the paper beyond its family (decoder-only,
RMSNorm, rotary positions, grouped-query attention, SwiGLU MLP); those blocks
are written here from their textbook definitions. All arithmetic is float64 on
the exactly widened bf16 weights and bf16 context K/V. No tiling, no online
softmax, no split reductions: each function is the definition written out,
with numpy matmul as the only library step.

Parity pins (tests/test_oracle_*.py): closed forms for each block, the 8-bit cache format's decoding against
hand-decoded codes and a library's table, brute-force
attention with scalar loops, cache-extend == full causal recompute, rotary
shift invariance, GQA == MHA with repeated heads, softmax sums to one, gate
end points of Table 3 (gamma = 0 never escalates, gamma > 1 always does),
batch-permutation equivariance, the whole forward against the
`transformers` Qwen2 architecture (and, with per-head query/key normalisation, its Qwen3 architecture) used
as a black-box library routine, and hand-worked iterations of
Algorithm 1 / Eq. 5 for the selection bookkeeping (tests/golden/cascade_cases.txt); for the two-tier
verifier, its reduction to one tier at either end of the threshold and the rule of Eq. 4 applied step by step
to two independent full-batch runs; for the append of accepted steps (Stage 3), its equality with a prefill
of the concatenated tokens from an empty cache (tests/test_oracle_cascade.py).
"""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple

import numpy as np


# ----------------------------------------------------------------------------------------------
# storage formats
# ----------------------------------------------------------------------------------------------

def widen_bf16(bits: np.ndarray) -> np.ndarray:
    """uint16 bf16 bit patterns -> float64, exactly (bf16 is the upper half of an fp32)."""
    u = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """float64 -> nearest bf16 value (ties to even, via fp32), returned as float64. Used only where the
    cache format is bf16: the K/V a prefill writes are stored rounded."""
    u = np.ascontiguousarray(x, dtype=np.float64).astype(np.float32).view(np.uint32)
    r = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    r &= np.uint32(0xFFFF0000)
    return r.view(np.float32).astype(np.float64)


def widen_e4m3(codes: np.ndarray) -> np.ndarray:
    """uint8 codes of the 8-bit float with 4 exponent bits (bias 7) and 3 mantissa bits, in the variant without
    infinities (the optional 8-bit cache format) -> float64, exactly: sign s, exponent field e, mantissa field m
    give (-1)^s 2^(e-7) (1 + m/8) for e >= 1, (-1)^s 2^-6 (m/8) for e = 0; e = 15 with m = 7 is NaN, so the
    largest finite value is 448."""
    c = np.ascontiguousarray(codes, dtype=np.uint8).astype(np.int64)
    s, e, m = (c >> 7) & 1, (c >> 3) & 15, c & 7
    mag = np.where(e == 0, np.ldexp(m / 8.0, -6), np.ldexp(1.0 + m / 8.0, e - 7))
    mag = np.where((e == 15) & (m == 7), np.nan, mag)
    return np.where(s == 1, -mag, mag)


def widen_e5m2(codes: np.ndarray) -> np.ndarray:
    """uint8 codes of the 8-bit float with 5 exponent bits (bias 15) and 2 mantissa bits (the other optional 8-bit
    cache format; it is the upper byte of an fp16) -> float64, exactly: (-1)^s 2^(e-15) (1 + m/4) for 1 <= e <= 30,
    (-1)^s 2^-14 (m/4) for e = 0; e = 31 is infinity (m = 0) or NaN."""
    c = np.ascontiguousarray(codes, dtype=np.uint8).astype(np.int64)
    s, e, m = (c >> 7) & 1, (c >> 2) & 31, c & 3
    mag = np.where(e == 0, np.ldexp(m / 4.0, -14), np.ldexp(1.0 + m / 4.0, e - 15))
    mag = np.where(e == 31, np.where(m == 0, np.inf, np.nan), mag)
    return np.where(s == 1, -mag, mag)


# ----------------------------------------------------------------------------------------------
# model blocks (textbook definitions)
# ----------------------------------------------------------------------------------------------

def rmsnorm(x: np.ndarray, gain: np.ndarray, eps: float) -> np.ndarray:
    """x / sqrt(mean(x^2) + eps) * gain, row-wise."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * gain


def rope(y: np.ndarray, positions: np.ndarray, theta: float) -> np.ndarray:
    """Rotary position embedding, "rotate-half" pairing. y: [n, heads, hd]; positions: [n].
    Pair (j, j + hd/2) is rotated by the angle pos * theta^(-2j/hd)."""
    n, _, hd = y.shape
    half = hd // 2
    inv_freq = theta ** (-2.0 * np.arange(half, dtype=np.float64) / hd)
    ang = positions.astype(np.float64)[:, None] * inv_freq[None, :]          # [n, half]
    c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    a, b = y[..., :half], y[..., half:]
    return np.concatenate([a * c - b * s, b * c + a * s], axis=-1)


def silu(z: np.ndarray) -> np.ndarray:
    return z / (1.0 + np.exp(-z))


def attention_extend(q: np.ndarray, k_ctx: np.ndarray, v_ctx: np.ndarray,
                     k_new: np.ndarray, v_new: np.ndarray) -> np.ndarray:
    """Grouped-query attention of n new positions over c cached positions (all visible) and over the
    new positions themselves (causal). q: [n, Hq, hd]; k_ctx, v_ctx: [c, Hkv, hd]; k_new, v_new:
    [n, Hkv, hd]. Query head h reads kv head h // (Hq // Hkv). Returns [n, Hq, hd]."""
    n, hq, hd = q.shape
    c = k_ctx.shape[0]
    group = hq // k_new.shape[1]
    keys = np.concatenate([k_ctx, k_new], axis=0)        # [c + n, Hkv, hd]
    vals = np.concatenate([v_ctx, v_new], axis=0)
    # new position p (absolute index c + p) may see absolute key indices 0 .. c + p
    visible = np.arange(c + n)[None, :] <= (c + np.arange(n))[:, None]
    out = np.empty_like(q)
    for h in range(hq):
        kh = h // group
        s = (q[:, h, :] @ keys[:, kh, :].T) / np.sqrt(float(hd))           # [n, c + n]
        s = np.where(visible, s, -np.inf)
        s = s - np.max(s, axis=-1, keepdims=True)
        p = np.exp(s)
        p = p / np.sum(p, axis=-1, keepdims=True)
        out[:, h, :] = p @ vals[:, kh, :]
    return out


class LayerWeights:
    """One decoder layer's matrices widened to float64 ([out_features, in_features])."""

    def __init__(self, layer: dict):
        for name in ("wq", "wk", "wv", "wo", "wg", "wu", "wd"):
            setattr(self, name, widen_bf16(layer[name]))
        self.norm1 = np.asarray(layer["norm1"], dtype=np.float64)
        self.norm2 = np.asarray(layer["norm2"], dtype=np.float64)
        # per-head RMSNorm gains of the query and key vectors ([hd] each); absent in the first model family
        self.q_norm = np.asarray(layer["q_norm"], dtype=np.float64) if "q_norm" in layer else None
        self.k_norm = np.asarray(layer["k_norm"], dtype=np.float64) if "k_norm" in layer else None


def decoder_layer_extend(x: np.ndarray, lw: LayerWeights, shape, ctx_len: int,
                         k_ctx: np.ndarray, v_ctx: np.ndarray
                         ) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """One pre-norm decoder layer over the n new positions of one step whose cached context has ctx_len
    positions. x: [n, d]. Returns (x_out, k_new, v_new) with k_new rotated, both [n, Hkv, hd]."""
    n = x.shape[0]
    hq, hkv, hd = shape.n_q_heads, shape.n_kv_heads, shape.head_dim
    if n == 0:  # no new position: nothing to compute, nothing to cache
        return x, np.zeros((0, hkv, hd)), np.zeros((0, hkv, hd))
    pos = ctx_len + np.arange(n)
    a = rmsnorm(x, lw.norm1, shape.rms_eps)
    q = (a @ lw.wq.T).reshape(n, hq, hd)
    k = (a @ lw.wk.T).reshape(n, hkv, hd)
    v = (a @ lw.wv.T).reshape(n, hkv, hd)
    if lw.q_norm is not None:
        # second model family of the paper's experiments (Section 5.1): every head's query and key vector is
        # RMS-normalised over its hd entries, with one gain vector shared by all heads, before the rotary turn
        q = rmsnorm(q, lw.q_norm, shape.rms_eps)
        k = rmsnorm(k, lw.k_norm, shape.rms_eps)
    q = rope(q, pos, shape.rope_theta)
    k = rope(k, pos, shape.rope_theta)
    o = attention_extend(q, k_ctx, v_ctx, k, v).reshape(n, hq * hd)
    x = x + o @ lw.wo.T
    b = rmsnorm(x, lw.norm2, shape.rms_eps)
    x = x + (silu(b @ lw.wg.T) * (b @ lw.wu.T)) @ lw.wd.T
    return x, k, v


# ----------------------------------------------------------------------------------------------
# confidence and gate (paper Eqs. 2-4)
# ----------------------------------------------------------------------------------------------

def logsumexp_full_vocab(logits: np.ndarray) -> np.ndarray:
    """log sum_v exp(z_v) over the whole vocabulary (last axis), shifted by the row maximum."""
    m = np.max(logits, axis=-1, keepdims=True)
    return (m + np.log(np.sum(np.exp(logits - m), axis=-1, keepdims=True)))[..., 0]


def log_softmax_full_vocab(logits: np.ndarray) -> np.ndarray:
    """log of the softmax over the whole vocabulary (last axis)."""
    return logits - logsumexp_full_vocab(logits)[..., None]


def verdict_confidence(logits: np.ndarray, verdict_ids: Sequence[int]
                       ) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Decision r_D and confidence p_D of Eqs. 2-3. The decision is the verdict token (one of
    `verdict_ids`) with the largest probability under the full-vocabulary softmax and p_D is that
    probability; ties go to the earliest entry of `verdict_ids`. logits: [B, V].
    Returns (conf [B] float64, verdict index [B] int32, log-sum-exp [B] float64)."""
    lse = logsumexp_full_vocab(logits)
    pv = np.exp(logits[:, list(verdict_ids)] - lse[:, None])   # [B, n_verdict]
    verdict = np.argmax(pv, axis=-1).astype(np.int32)   # first maximum
    conf = pv[np.arange(pv.shape[0]), verdict]
    return conf, verdict, lse


def gate(conf: np.ndarray, tau: float) -> np.ndarray:
    """Cascade rule of Eq. 4: 1 where the draft verifier's decision is trusted (p_D >= gamma), 0 where
    the step is escalated to the target model. The comparison is taken in fp32, the precision in which
    the confidence is stored; a NaN confidence escalates."""
    c32 = np.asarray(conf, dtype=np.float64).astype(np.float32)
    return (c32 >= np.float32(tau)).astype(np.uint8)


def escalate_list(conf: np.ndarray, tau: float) -> Tuple[np.ndarray, np.ndarray, int]:
    """Re-gate stored confidences and list the escalated steps in ascending order.
    Returns (accept mask uint8 [B], escalated step indices int32 [count], count)."""
    acc = gate(conf, tau)
    idx = np.nonzero(acc == 0)[0].astype(np.int32)
    return acc, idx, int(idx.shape[0])


def cascade_select(trusted: Sequence[int], verdict_d: Sequence[int], conf_d: Sequence[float],
                   verdict_t: Optional[Sequence[int]], conf_t: Optional[Sequence[float]],
                   req_offsets: Sequence[int], accept_index: int = 0
                   ) -> Tuple[np.ndarray, np.ndarray, np.ndarray, np.ndarray]:
    """What the drafting loop does with the verification results of one iteration, per request (the steps of
    request r are [req_offsets[r], req_offsets[r+1]) of the batch).

    Final decision of a step (Algorithm 1, Stage 2; Eq. 4): the draft verifier's decision r_D when it was
    trusted (p_D >= gamma), else the target verifier's decision; a step that was escalated but has no target
    result counts as rejected. Its confidence is that of the verifier whose decision was taken (Section 4.3).
    Linear drafting (Algorithm 1, the loop over j with `break`): m = number of leading steps of the request
    whose final decision is "accept". Tree drafting (Section 4.3, Eq. 5): among the request's candidates that
    pass verification, the one with the highest confidence (the earliest on ties); -1 if none passes.

    Returns (passed uint8 [B], final confidence float32 [B], m int32 [R], best int32 [R] batch index or -1).
    Written as plain loops: this is bookkeeping, not arithmetic."""
    B = len(trusted)
    passed = np.zeros(B, dtype=np.uint8)
    conf = np.zeros(B, dtype=np.float32)
    for i in range(B):
        if trusted[i]:
            passed[i] = 1 if verdict_d[i] == accept_index else 0
            conf[i] = np.float32(conf_d[i])
        elif verdict_t is not None:
            passed[i] = 1 if verdict_t[i] == accept_index else 0
            conf[i] = np.float32(conf_t[i])
        else:
            passed[i] = 0
            conf[i] = np.float32(conf_d[i])
    R = len(req_offsets) - 1
    m = np.zeros(R, dtype=np.int32)
    best = np.full(R, -1, dtype=np.int32)
    for r in range(R):
        lo, hi = int(req_offsets[r]), int(req_offsets[r + 1])
        j = lo
        while j < hi and passed[j]:
            j += 1
        m[r] = j - lo
        for i in range(lo, hi):
            if passed[i] and not np.isnan(conf[i]) and (best[r] < 0 or conf[i] > conf[best[r]]):
                best[r] = i
    return passed, conf, m, best


# ----------------------------------------------------------------------------------------------
# whole pass
# ----------------------------------------------------------------------------------------------

def forward_extend(weights: dict, tokens_per_step: List[np.ndarray], ctx_lens: Sequence[int],
                   ctx_kv_fn, collect_new_kv: bool = False):
    """Run every step's new tokens through all layers on top of its cached context.

    ctx_kv_fn(step, layer) -> (K, V) float64 arrays [c_i, Hkv, hd] (K already rotated).
    Steps never interact (the paper verifies candidates independently, Section 4.3); the layer loop is
    outermost only so that each layer's weights are widened once.
    Returns (hidden states per step [n_i, d] before the final norm, optional per-step per-layer new K/V).
    """
    shape = weights["shape"]
    emb = weights["embed"]
    xs = [widen_bf16(emb[np.asarray(t, dtype=np.int64)]) for t in tokens_per_step]
    new_kv = [[None] * shape.n_layers for _ in xs] if collect_new_kv else None
    for li in range(shape.n_layers):
        lw = LayerWeights(weights["layers"][li])
        for i in range(len(xs)):
            k_ctx, v_ctx = ctx_kv_fn(i, li)
            xs[i], k, v = decoder_layer_extend(xs[i], lw, shape, int(ctx_lens[i]), k_ctx, v_ctx)
            if collect_new_kv:
                new_kv[i][li] = (k, v)
    return xs, new_kv


def last_position_logits(weights: dict, xs: List[np.ndarray]) -> np.ndarray:
    """Final RMSNorm of each step's last new position, then the LM head. Returns [B, V] float64."""
    shape = weights["shape"]
    g = np.asarray(weights["final_norm"], dtype=np.float64)
    h = np.stack([rmsnorm(x[-1:, :], g, shape.rms_eps)[0] for x in xs], axis=0)
    return h @ widen_bf16(weights["lm_head"]).T


def prefill_context(weights: dict, ctx_tokens: List[np.ndarray], store_bf16: bool):
    """Build each sequence's context K/V by running its context tokens through the model from an empty
    cache. Returns kv[i][layer] = (K, V), each [c_i, Hkv, hd] float64; rounded to bf16 values when
    `store_bf16` (the cache format), exact otherwise."""
    shape = weights["shape"]
    empty = np.zeros((0, shape.n_kv_heads, shape.head_dim))
    _, kv = forward_extend(weights, ctx_tokens, [0] * len(ctx_tokens),
                           lambda i, l: (empty, empty), collect_new_kv=True)
    if store_bf16:
        kv = [[(round_to_bf16(k), round_to_bf16(v)) for (k, v) in per_layer] for per_layer in kv]
    return kv


def verify_steps(weights: dict, tokens_per_step: List[np.ndarray], ctx_lens: Sequence[int],
                 ctx_kv_fn, verdict_ids: Sequence[int], tau: float) -> dict:
    """The whole verification pass for a batch of steps (Algorithm 1, Stage 2, draft tier).
    Returns logits [B, V], conf [B], verdict [B], lse [B], accept [B] (1 = trusted, 0 = escalate)."""
    xs, _ = forward_extend(weights, tokens_per_step, ctx_lens, ctx_kv_fn)
    logits = last_position_logits(weights, xs)
    conf, verdict, lse = verdict_confidence(logits, verdict_ids)
    return {"logits": logits, "conf": conf, "verdict": verdict, "lse": lse, "accept": gate(conf, tau)}


def verify_cascade(weights_d: dict, weights_t: dict, tokens_per_step: List[np.ndarray],
                   ctx_lens: Sequence[int], ctx_kv_fn_d, ctx_kv_fn_t,
                   verdict_ids: Sequence[int], tau: float,
                   req_offsets: Optional[Sequence[int]] = None, accept_index: int = 0) -> dict:
    """The two-tier verifier V_cascade (Eq. 4; Algorithm 1, Stage 2): every step goes through the draft
    model; the steps whose draft confidence is below gamma, and only those, go through the target model;
    the final decision of a step is r_D where p_D >= gamma and r_T otherwise.

    With `req_offsets` (linear drafting: the steps of request r are req_offsets[r] .. req_offsets[r+1]-1, in
    drafting order) the loop of Algorithm 1 over a request's steps ends at the first rejection, so a step that
    follows a TRUSTED draft rejection in its request is never looked at again: such a step is not sent to the
    target model even if its own confidence is below gamma, and it has no final decision (verdict -1,
    confidence 0). Steps after an escalated step stay in, since the target may still accept that step.

    ctx_kv_fn_d / ctx_kv_fn_t (step, layer) -> (K, V): the same reasoning context as cached by each model,
    indexed by the step's position in the full batch.
    Returns the draft tier's dict under "draft", the target tier's under "target" (its arrays run over the
    escalated steps only, in ascending step order; None when nothing was escalated), "escalated" (their
    step indices), and per step of the batch "verdict" (final decision) and "conf" (confidence of the
    verifier whose decision was taken)."""
    draft = verify_steps(weights_d, tokens_per_step, ctx_lens, ctx_kv_fn_d, verdict_ids, tau)
    B = len(tokens_per_step)
    live = [True] * B
    if req_offsets is not None:
        for r in range(len(req_offsets) - 1):
            alive = True
            for i in range(int(req_offsets[r]), int(req_offsets[r + 1])):
                live[i] = alive
                if draft["accept"][i] and draft["verdict"][i] != accept_index:
                    alive = False            # the loop over this request's steps breaks here
    escalated = [i for i in range(B) if not draft["accept"][i] and live[i]]
    verdict = np.array(draft["verdict"], dtype=np.int32)
    conf = np.array(draft["conf"], dtype=np.float64)
    for i in range(B):
        if not draft["accept"][i]:
            verdict[i], conf[i] = -1, 0.0
    target = None
    if escalated:
        target = verify_steps(weights_t, [tokens_per_step[i] for i in escalated],
                              [ctx_lens[i] for i in escalated],
                              lambda j, l: ctx_kv_fn_t(escalated[j], l), verdict_ids, tau)
        for j, i in enumerate(escalated):
            verdict[i] = target["verdict"][j]
            conf[i] = target["conf"][j]
    return {"draft": draft, "target": target, "escalated": np.array(escalated, dtype=np.int32),
            "verdict": verdict, "conf": conf}


def append_accepted_steps(weights: dict, ctx_kv: list, m: Sequence[int], req_offsets: Sequence[int],
                          draft_steps: List[np.ndarray], store_bf16: bool) -> list:
    """Context management of Algorithm 1, Stage 3: context <- context (+) s^_1 (+) ... (+) s^_m for every request
    with m > 0, in terms of the cache. ctx_kv[r][layer] = (K, V) of request r's context; draft_steps[i] holds the
    token ids of drafted step i (the candidates of request r are steps req_offsets[r] .. req_offsets[r+1]-1).
    The accepted tokens run through the model on top of the cached context, and their K/V (rounded to bf16
    values when `store_bf16`, the cache format) are appended; requests with m = 0 keep their context as it is
    (their next step comes from the target model's generation, which is outside this pass).
    Returns the new ctx_kv (same structure; untouched requests share their arrays with the input)."""
    out = list(ctx_kv)
    grow = [r for r in range(len(m)) if m[r] > 0]
    if not grow:
        return out
    toks = [np.concatenate([np.asarray(draft_steps[req_offsets[r] + j]) for j in range(int(m[r]))]) for r in grow]
    lens = [ctx_kv[r][0][0].shape[0] for r in grow]
    _, new = forward_extend(weights, toks, lens, lambda j, l: ctx_kv[grow[j]][l], collect_new_kv=True)
    for j, r in enumerate(grow):
        layers = []
        for l, (k, v) in enumerate(new[j]):
            if store_bf16:
                k, v = round_to_bf16(k), round_to_bf16(v)
            layers.append((np.concatenate([ctx_kv[r][l][0], k], axis=0), np.concatenate([ctx_kv[r][l][1], v], axis=0)))
        out[r] = layers
    return out
