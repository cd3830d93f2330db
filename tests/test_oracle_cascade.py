"""Pins for the oracle's two-tier verifier (Eq. 4; Algorithm 1, Stage 2): the end points of the threshold,
where the cascade reduces to one of its tiers, and, in between, the rule written per step on two independent
full-batch runs, which fixes the bookkeeping of the smaller target batch (which steps, which contexts, where
the results go back)."""
from dataclasses import replace

import numpy as np
import pytest

from oracle import confspec_oracle as O
from workloads import get_config, make_batch, model_weights, plant_verdict_rows


def _steps(batch):
    return [batch.step_tokens[batch.cu_new[i]:batch.cu_new[i + 1]] for i in range(batch.n_steps)]


class _Untouchable(dict):
    """Stands in for the target model where the rule says it is not consulted."""
    def __getitem__(self, key):
        raise AssertionError("the target model was read although no step was escalated")


@pytest.fixture(scope="module")
def two_models():
    cfg = replace(get_config("cfg1_tiny"), batch=12)
    beta = float(np.log(cfg.model.vocab) + 0.5)
    wd = model_weights(cfg.model, cfg.seed)
    plant_verdict_rows(wd, cfg.verdict_ids, beta=beta, seed=cfg.seed)
    wt = model_weights(cfg.model, cfg.seed + 1)
    plant_verdict_rows(wt, cfg.verdict_ids, beta=beta, seed=cfg.seed + 1)
    b = make_batch(cfg)
    kvd = O.prefill_context(wd, b.ctx_tokens, store_bf16=True)
    kvt = O.prefill_context(wt, b.ctx_tokens, store_bf16=True)
    fd, ft = (lambda i, l: kvd[i][l]), (lambda i, l: kvt[i][l])
    full_d = O.verify_steps(wd, _steps(b), b.ctx_lens, fd, cfg.verdict_ids, 0.5)
    full_t = O.verify_steps(wt, _steps(b), b.ctx_lens, ft, cfg.verdict_ids, 0.5)
    return cfg, b, wd, wt, fd, ft, full_d, full_t


def test_threshold_zero_is_the_draft_verifier_alone(two_models):
    cfg, b, wd, wt, fd, ft, full_d, full_t = two_models
    r = O.verify_cascade(wd, _Untouchable(), _steps(b), b.ctx_lens, fd, ft, cfg.verdict_ids, 0.0)
    assert r["target"] is None and r["escalated"].size == 0
    assert np.array_equal(r["verdict"], full_d["verdict"]) and np.array_equal(r["conf"], full_d["conf"])


def test_threshold_above_one_is_the_target_verifier_alone(two_models):
    cfg, b, wd, wt, fd, ft, full_d, full_t = two_models
    r = O.verify_cascade(wd, wt, _steps(b), b.ctx_lens, fd, ft, cfg.verdict_ids, 1.5)
    assert r["escalated"].tolist() == list(range(b.n_steps))
    assert np.array_equal(r["verdict"], full_t["verdict"])
    assert np.max(np.abs(r["conf"] - full_t["conf"])) < 1e-12
    assert np.max(np.abs(r["target"]["logits"] - full_t["logits"])) < 1e-9


def test_rule_per_step_between_the_end_points(two_models):
    cfg, b, wd, wt, fd, ft, full_d, full_t = two_models
    srt = np.sort(full_d["conf"])
    tau = float(0.5 * (srt[b.n_steps // 2 - 1] + srt[b.n_steps // 2]))     # half of the steps on either side
    r = O.verify_cascade(wd, wt, _steps(b), b.ctx_lens, fd, ft, cfg.verdict_ids, tau)
    esc = r["escalated"].tolist()
    assert 0 < len(esc) < b.n_steps and esc == sorted(esc)
    assert r["target"]["conf"].shape == (len(esc),)              # the target's cost is per escalated step (Section 4.4)
    for i in range(b.n_steps):
        if full_d["conf"][i] >= tau:
            assert i not in esc
            assert r["verdict"][i] == full_d["verdict"][i] and r["conf"][i] == full_d["conf"][i]
        else:
            assert i in esc
            assert r["verdict"][i] == full_t["verdict"][i] and abs(r["conf"][i] - full_t["conf"][i]) < 1e-12
    # not vacuous: the tiers disagree on the escalated steps, and the steps differ from one another
    assert max(abs(full_t["conf"][i] - full_d["conf"][i]) for i in esc) > 1e-2
    assert np.ptp(full_t["conf"][esc]) > 1e-2
    # the selection bookkeeping sees the same final decisions
    vt = np.full(b.n_steps, -1, np.int32)
    ct = np.zeros(b.n_steps, np.float32)
    vt[esc], ct[esc] = r["target"]["verdict"], r["target"]["conf"]
    passed, conf, m, best = O.cascade_select(r["draft"]["accept"], r["draft"]["verdict"], r["draft"]["conf"], vt, ct,
                                             [0, b.n_steps], accept_index=0)
    assert np.array_equal(passed, (r["verdict"] == 0).astype(np.uint8))
    assert np.array_equal(conf, r["conf"].astype(np.float32))


def test_single_escalated_step_uses_its_own_context(two_models):
    """One step below the threshold, and not the first of the batch: the target must see that step's tokens and
    that step's context."""
    cfg, b, wd, wt, fd, ft, full_d, full_t = two_models
    order = np.argsort(full_d["conf"])
    lowest = int(order[0])
    tau = float(0.5 * (full_d["conf"][order[0]] + full_d["conf"][order[1]]))
    r = O.verify_cascade(wd, wt, _steps(b), b.ctx_lens, fd, ft, cfg.verdict_ids, tau)
    assert lowest != 0 and r["escalated"].tolist() == [lowest]
    assert np.max(np.abs(r["target"]["logits"][0] - full_t["logits"][lowest])) < 1e-9
    others = [i for i in range(b.n_steps) if i != lowest]
    assert min(np.max(np.abs(full_t["logits"][i] - full_t["logits"][lowest])) for i in others) > 1e-3


def test_appending_accepted_steps_equals_prefilling_the_longer_context():
    """Stage 3 of Algorithm 1 in terms of the cache: context (+) accepted steps, built by appending, is the cache a
    prefill of the concatenated tokens builds from nothing; a request with m = 0 keeps its cache."""
    cfg = get_config("cfg1_tiny")
    w = model_weights(cfg.model, cfg.seed)
    g = np.random.default_rng(9)
    V = cfg.model.vocab
    ctx = [g.integers(3, V, size=n).astype(np.int32) for n in (19, 33, 7)]
    req_offsets = [0, 3, 5, 8]                                   # 3, 2 and 3 candidate steps
    steps = [g.integers(3, V, size=n).astype(np.int32) for n in (4, 9, 2, 5, 5, 1, 6, 3)]
    m = [2, 0, 3]
    kv = O.prefill_context(w, ctx, store_bf16=False)
    new = O.append_accepted_steps(w, kv, m, req_offsets, steps, store_bf16=False)
    longer = [np.concatenate([ctx[0], steps[0], steps[1]]), ctx[1], np.concatenate([ctx[2], steps[5], steps[6], steps[7]])]
    want = O.prefill_context(w, longer, store_bf16=False)
    for r in range(3):
        for l in range(cfg.model.n_layers):
            for a, b in zip(new[r][l], want[r][l]):
                assert a.shape == b.shape and np.max(np.abs(a - b)) < 1e-10
    assert new[1] is kv[1]
    assert new[0][0][0].shape[0] == 19 + 4 + 9 and new[2][1][1].shape[0] == 7 + 1 + 6 + 3
    # cache format: the appended rows are bf16 values, the earlier rows are the earlier bits
    kvb = O.prefill_context(w, ctx, store_bf16=True)
    newb = O.append_accepted_steps(w, kvb, m, req_offsets, steps, store_bf16=True)
    k_new = newb[0][1][0]
    assert np.array_equal(k_new[:19], kvb[0][1][0]) and np.array_equal(O.round_to_bf16(k_new), k_new)
    assert np.max(np.abs(k_new[19:] - new[0][1][0][19:])) < 0.05 and np.max(np.abs(k_new[19:] - new[0][1][0][19:])) > 0


def test_steps_behind_a_trusted_rejection_are_not_escalated_and_m_does_not_change(two_models):
    """Linear drafting: Algorithm 1's loop over a request's steps breaks at the first rejection, so the target model
    never needs the steps behind a trusted draft rejection. Leaving them out must not change any accept-prefix
    length m, and must leave out exactly those steps."""
    cfg, b, wd, wt, fd, ft, full_d, full_t = two_models
    req_offsets = [0, 5, 8, 12]
    n_pruned = 0
    for tau in (0.05, 0.2, 0.5, 0.8):
        allv = O.verify_cascade(wd, wt, _steps(b), b.ctx_lens, fd, ft, cfg.verdict_ids, tau)
        live = O.verify_cascade(wd, wt, _steps(b), b.ctx_lens, fd, ft, cfg.verdict_ids, tau, req_offsets=req_offsets)
        trusted, vd = allv["draft"]["accept"], allv["draft"]["verdict"]
        expect = []
        for r in range(3):
            seen_reject = False
            for i in range(req_offsets[r], req_offsets[r + 1]):
                if not trusted[i] and not seen_reject:
                    expect.append(i)
                if trusted[i] and vd[i] != 0:
                    seen_reject = True
        assert live["escalated"].tolist() == expect
        assert set(expect) <= set(allv["escalated"].tolist())
        n_pruned += len(allv["escalated"]) - len(expect)

        def m_of(res):
            vt = np.full(b.n_steps, -1, np.int32)
            ct = np.zeros(b.n_steps, np.float32)
            if res["target"] is not None:
                vt[res["escalated"]], ct[res["escalated"]] = res["target"]["verdict"], res["target"]["conf"]
            return O.cascade_select(trusted, vd, allv["draft"]["conf"], vt, ct, req_offsets, accept_index=0)[2]

        assert np.array_equal(m_of(allv), m_of(live))
        for i in range(b.n_steps):
            if trusted[i]:
                assert live["verdict"][i] == vd[i]
            elif i in expect:
                assert live["verdict"][i] == allv["verdict"][i] and abs(live["conf"][i] - allv["conf"][i]) < 1e-12
            else:
                assert live["verdict"][i] == -1 and live["conf"][i] == 0.0
    assert n_pruned > 0                                  # the rule left something out on this case
