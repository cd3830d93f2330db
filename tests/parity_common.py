"""Shared driver of the end-to-end parity checks: run the CUDA path through the C ABI and the CPU oracle on
the same seeded inputs and compare with the tolerances the pass is specified to:
  last-position logits  max-abs <= 3e-2
  confidence            abs     <= 5e-3
  accept/escalate mask  bit-exact except where |conf - tau| < 5e-3
  verdict index         equal unless the two best verdict probabilities are within 5e-3 of each other
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import numpy as np

from oracle import confspec_oracle as O
from workloads import context_kv, make_batch, model_weights, page_assignment, plant_verdict_rows

LOGIT_TOL = 3e-2
CONF_TOL = 5e-3


def steps_of(batch) -> List[np.ndarray]:
    return [batch.step_tokens[batch.cu_new[i]:batch.cu_new[i + 1]] for i in range(batch.n_steps)]


def build_session(cfg, weights, batch, keep_logits=True):
    """GPU side: model, cache and contexts for one workload."""
    from paper_2602_18447_b200 import VerifySession, binding as B
    ses = VerifySession(cfg, weights, batch)
    B.cs_set_keep_logits(ses.model, keep_logits)
    if cfg.ctx_kv == "prefill":
        need = [(int(c) + cfg.page_size - 1) // cfg.page_size for c in batch.ctx_lens]
        total, pages = page_assignment(cfg, batch.ctx_lens)
        ses.alloc_cache(pages, total, batch.ctx_lens, room_for_prefill=True)
        ses.prefill_context(batch.ctx_tokens)
    else:
        total, pages = page_assignment(cfg, batch.ctx_lens)
        ses.alloc_cache(pages, total, batch.ctx_lens)
        ses.fill_synthetic_context(lambda i, l: context_kv(cfg, i, l, int(batch.ctx_lens[i])))
    return ses


def oracle_outputs(cfg, weights, batch, steps: Optional[Sequence[int]] = None, tau: Optional[float] = None) -> dict:
    """CPU side, for all steps or a sample of them (steps are independent)."""
    idx = list(range(batch.n_steps)) if steps is None else list(steps)
    toks = steps_of(batch)
    tau = cfg.tau if tau is None else tau
    if cfg.ctx_kv == "prefill":
        kv = O.prefill_context(weights, [batch.ctx_tokens[i] for i in idx], store_bf16=True)
        fn = lambda j, l: kv[j][l]
    else:
        def fn(j, l):
            k, v = context_kv(cfg, idx[j], l, int(batch.ctx_lens[idx[j]]))
            widen = {"e4m3": O.widen_e4m3, "e5m2": O.widen_e5m2}.get(cfg.kv_format, O.widen_bf16)
            return widen(k), widen(v)
    return O.verify_steps(weights, [toks[i] for i in idx], [int(batch.ctx_lens[i]) for i in idx], fn,
                          cfg.verdict_ids, tau)


def compare(gpu: dict, gpu_logits: Optional[np.ndarray], ref: dict, tau: float, steps: Optional[Sequence[int]] = None,
            gpu_lse: Optional[np.ndarray] = None) -> dict:
    """Assert the specified tolerances (workloads as written); returns the observed maxima for reporting."""
    sel = slice(None) if steps is None else list(steps)
    conf = gpu["conf"][sel].astype(np.float64)
    stats = {"conf_err": float(np.max(np.abs(conf - ref["conf"])))}
    assert np.all(np.isfinite(conf)), conf
    assert stats["conf_err"] <= CONF_TOL, stats
    if gpu_logits is not None:
        stats["logit_err"] = float(np.max(np.abs(gpu_logits[sel].astype(np.float64) - ref["logits"])))
        assert stats["logit_err"] <= LOGIT_TOL, stats
    if gpu_lse is not None:
        stats["lse_err"] = float(np.max(np.abs(gpu_lse[sel].astype(np.float64) - ref["lse"])))
        assert stats["lse_err"] <= LOGIT_TOL, stats
    near = np.abs(ref["conf"] - tau) < CONF_TOL
    acc = gpu["accept"][sel]
    assert np.array_equal(acc[~near], ref["accept"][~near]), (acc, ref["accept"], ref["conf"])
    assert np.all((acc == 0) | (acc == 1))
    stats["n_near_tau"] = int(near.sum())
    stats["n_accept"] = int(ref["accept"].sum())
    record_stats("base", stats)
    return stats


# Planted-verdict variant: tolerances of the two planted LM-head rows and of the confidence they produce.
#
# The planted rows have norm beta ~ ln V + 0.5 instead of init_std * sqrt(d), so the same direction error of the last
# hidden state (the fp16 rounding of the activations, accumulated over the layers) moves their logits further than an
# ordinary row's. The bounds below are not derived from that worst case: they are at most three times the largest
# error observed on the GPU for the class of model (the tests record the maxima when CS_PARITY_STATS is set), so a
# regression of the forward pass by a small factor fails them. Keys: (shallow, deep) = (up to 3 layers, more).
# Observed worst cases: planted-row logit 2.1e-2 (shallow) / 4.8e-2 (deep), confidence 4.0e-3 / 1.1e-2.
PLANTED_LOGIT_TOL = {"shallow": 6e-2, "deep": 1.2e-1}
PLANTED_CONF_TOL = {"shallow": 1e-2, "deep": 3e-2}


def planted_tols(cfg):
    k = "shallow" if cfg.model.n_layers <= 3 else "deep"
    return PLANTED_LOGIT_TOL[k], PLANTED_CONF_TOL[k]


def record_stats(name: str, stats: dict) -> None:
    """Append the observed maxima of one comparison to the file named by CS_PARITY_STATS (if set)."""
    import json
    import os
    path = os.environ.get("CS_PARITY_STATS")
    if path:
        with open(path, "a") as f:
            f.write(json.dumps({"case": name, **{k: (float(v) if isinstance(v, (float, np.floating)) else v)
                                                 for k, v in stats.items()}}) + "\n")


def compare_planted(gpu: dict, gpu_logits: np.ndarray, ref: dict, tau: float, cfg, weights=None,
                    steps: Optional[Sequence[int]] = None, gpu_lse: Optional[np.ndarray] = None,
                    need_both_sides: bool = False, case: str = "") -> dict:
    """Planted-verdict variant of a workload against the oracle: ordinary logits and lse at the specified 3e-2, the two
    planted rows and the confidence at the tightened bounds above, and the accept/escalate mask against the ORACLE's
    mask for every step whose oracle confidence is further from tau than the confidence bound - trusted steps included.
    `need_both_sides` additionally demands that at least one trusted and one escalated step were so compared."""
    sel = slice(None) if steps is None else list(steps)
    vids = list(cfg.verdict_ids)
    logit_tol, conf_tol = planted_tols(cfg)
    z = gpu_logits[sel].astype(np.float64)
    d = np.abs(z - ref["logits"])
    stats = {"planted_logit_err": float(d[:, vids].max()), "logit_err": float(np.delete(d, vids, axis=1).max())}
    conf = gpu["conf"][sel].astype(np.float64)
    stats["conf_err"] = float(np.max(np.abs(conf - ref["conf"])))
    if gpu_lse is not None:
        stats["lse_err"] = float(np.max(np.abs(gpu_lse[sel].astype(np.float64) - ref["lse"])))
    # softmax + confidence + gate, given the GPU's own logits: tight
    conf_z, verdict_z, _ = O.verdict_confidence(z, vids)
    stats["conf_err_given_logits"] = float(np.max(np.abs(conf - conf_z)))
    acc = gpu["accept"][sel]
    far = np.abs(ref["conf"] - tau) > conf_tol
    stats["n_cmp_trusted"] = int((far & (ref["accept"] == 1)).sum())
    stats["n_cmp_escalated"] = int((far & (ref["accept"] == 0)).sum())
    stats["n_in_band"] = int((~far).sum())
    stats["tau"] = float(tau)
    record_stats(case or cfg.name, stats)
    assert np.all(np.isfinite(conf)), conf
    assert stats["logit_err"] <= LOGIT_TOL, stats
    assert stats["planted_logit_err"] <= logit_tol, stats
    assert stats["conf_err"] <= conf_tol, stats
    if gpu_lse is not None:
        # where the planted logit dominates the sum, the logsumexp is that logit and moves with it
        assert stats["lse_err"] <= logit_tol, stats
    assert stats["conf_err_given_logits"] <= 1e-4, stats
    sure = np.abs(conf_z - tau) > 1e-4
    assert np.array_equal(acc[sure], O.gate(conf_z, tau)[sure])
    assert np.all((acc == 0) | (acc == 1))
    # the mask against the oracle's, on both sides of the threshold
    assert np.array_equal(acc[far], ref["accept"][far]), (acc, ref["accept"], ref["conf"], tau)
    if need_both_sides:
        assert stats["n_cmp_trusted"] >= 1 and stats["n_cmp_escalated"] >= 1, stats
    stats["n_accept"] = int(ref["accept"].sum())
    return stats


def check_verdict(gpu: dict, ref: dict, verdict_ids: Sequence[int], steps: Optional[Sequence[int]] = None) -> None:
    sel = slice(None) if steps is None else list(steps)
    pv = np.exp(ref["logits"][:, list(verdict_ids)] - ref["lse"][:, None])
    srt = np.sort(pv, axis=-1)
    clear = (srt[:, -1] - srt[:, -2]) > CONF_TOL if pv.shape[1] > 1 else np.ones(pv.shape[0], bool)
    assert np.array_equal(gpu["verdict"][sel][clear], ref["verdict"][clear])
    assert np.all((gpu["verdict"][sel] >= 0) & (gpu["verdict"][sel] < len(verdict_ids)))


def planted_weights(cfg, seed=None):
    w = model_weights(cfg.model, cfg.seed if seed is None else seed)
    plant_verdict_rows(w, cfg.verdict_ids, beta=float(np.log(cfg.model.vocab) + 0.5), seed=cfg.seed)
    return w


def planted_copy(cfg, weights: dict) -> dict:
    """The same weights with the planted verdict rows, sharing every tensor but the LM head."""
    w = dict(weights, lm_head=weights["lm_head"].copy())
    plant_verdict_rows(w, cfg.verdict_ids, beta=float(np.log(cfg.model.vocab) + 0.5), seed=cfg.seed)
    return w


def sample_both_sides(conf: np.ndarray, tau: float, band: float, n: int, always: Sequence[int] = ()) -> List[int]:
    """Which steps of a full-size batch the oracle recomputes: picked from the confidences of the pass under test so
    that the sample has trusted and escalated steps outside the band around tau, the closest ones first (those are
    the ones a small error would flip), then the extremes. The oracle's own confidences decide the comparison."""
    conf = np.asarray(conf, dtype=np.float64)
    above = [int(i) for i in np.argsort(conf) if conf[i] >= tau + band]            # ascending: closest to tau first
    below = [int(i) for i in np.argsort(-conf) if conf[i] < tau - band]            # descending: closest first
    picks: List[int] = list(dict.fromkeys(int(i) for i in always))
    order = []
    for k in range(max(len(above), len(below))):
        if k < len(above):
            order.append(above[k])
        if k < len(below):
            order.append(below[k])
    if above:
        order.insert(2, above[-1])      # the most confident step
    if below:
        order.insert(3, below[-1])      # the least confident step
    for i in order:
        if len(picks) >= n:
            break
        if i not in picks:
            picks.append(i)
    return sorted(picks)
