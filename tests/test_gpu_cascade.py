"""Parity of cs_verify_cascade (the two-tier verifier of Eq. 4: draft pass, list of escalated steps, target pass over
those steps only, final decision per step) with the CPU oracle: element by element on a small pair of models, on
sampled steps for the 1.5B-shaped draft with the 7B-shaped target, and the end points and argument errors."""
import numpy as np
import pytest

from workloads import get_cascade, make_batch

import parity_common as P

pytestmark = pytest.mark.gpu


def _sessions(casc, wd, wt, batch):
    from paper_2602_18447_b200.runner import CascadeSession
    sd = P.build_session(casc.draft, wd, batch)
    try:
        st = P.build_session(casc.target, wt, batch)
    except BaseException:
        sd.close()
        raise
    return CascadeSession(sd, st)


def _compact_logits(ses, n):
    import torch
    from paper_2602_18447_b200 import binding as B
    out = torch.empty(n, ses.shape.vocab, dtype=torch.float32, device=ses.device)
    B.cs_get_last_logits(ses.model, out, n)
    torch.cuda.synchronize()
    return out.cpu().numpy()


def _check_bookkeeping(g):
    """What must hold exactly between the outputs of one call, whatever the models compute."""
    esc = np.nonzero(g["trusted"] == 0)[0]
    assert g["n_escalated"] == esc.size
    tr = g["trusted"] != 0
    assert np.all(g["verdict_t"][tr] == -1) and np.all(g["conf_t"][tr] == 0.0)
    assert np.array_equal(g["verdict"], np.where(tr, g["verdict_d"], g["verdict_t"]))
    assert np.array_equal(g["conf"], np.where(tr, g["conf_d"], g["conf_t"]))
    assert np.all(g["verdict_t"][esc] >= 0) and np.all(g["conf_t"][esc] > 0)
    return esc


def _tau_in_widest_gap(conf):
    """A threshold with about half of the steps on either side, as far from the nearest confidence as possible."""
    srt = np.sort(conf)
    n = len(srt)
    lo, hi = n // 4, n - n // 4
    k = lo + int(np.argmax(srt[lo + 1:hi + 1] - srt[lo:hi]))
    return float(0.5 * (srt[k] + srt[k + 1])), float(srt[k + 1] - srt[k])


def test_small_models_every_step():
    casc = get_cascade("cascade_tiny")
    cfg_d, cfg_t = casc.draft, casc.target
    wd, wt = P.planted_weights(cfg_d), P.planted_weights(cfg_t)
    batch = make_batch(cfg_d)
    toks = P.steps_of(batch)
    kvd = P.O.prefill_context(wd, batch.ctx_tokens, store_bf16=True)
    kvt = P.O.prefill_context(wt, batch.ctx_tokens, store_bf16=True)
    probe = P.O.verify_steps(wd, toks, batch.ctx_lens, lambda i, l: kvd[i][l], cfg_d.verdict_ids, 0.5)
    tau, gap = _tau_in_widest_gap(probe["conf"])
    ref = P.O.verify_cascade(wd, wt, toks, batch.ctx_lens, lambda i, l: kvd[i][l], lambda i, l: kvt[i][l],
                             cfg_d.verdict_ids, tau)
    want = ref["escalated"]
    assert 0 < want.size < batch.n_steps
    cs = _sessions(casc, wd, wt, batch)
    try:
        cs.verify(tau=tau)
        g = cs.results()
        esc = _check_bookkeeping(g)
        # draft tier
        assert np.max(np.abs(g["conf_d"] - ref["draft"]["conf"])) < 0.45 * gap      # so that the lists must agree
        assert np.array_equal(esc, want)
        gd = {"conf": g["conf_d"], "accept": g["trusted"], "verdict": g["verdict_d"]}
        P.compare_planted(gd, _compact_logits(cs.draft, batch.n_steps), ref["draft"], tau, cfg_d, wd)
        # target tier: its batch is the escalated steps in ascending order
        gt = {"conf": g["conf_t"][esc], "accept": (g["conf_t"][esc] >= np.float32(tau)).astype(np.uint8),
              "verdict": g["verdict_t"][esc]}
        st = P.compare_planted(gt, _compact_logits(cs.target, esc.size), ref["target"], tau, cfg_t, wt)
        P.check_verdict({"verdict": g["verdict_t"][esc]}, ref["target"], cfg_d.verdict_ids)
        P.check_verdict({"verdict": g["verdict_d"]}, ref["draft"], cfg_d.verdict_ids)
        assert st["logit_err"] <= P.LOGIT_TOL
        # the end points: nothing, then everything, goes to the target
        assert cs.verify(tau=0.0) == 0
        g0 = cs.results()
        _check_bookkeeping(g0)
        assert np.all(g0["trusted"] == 1) and np.array_equal(g0["verdict"], g0["verdict_d"])
        assert cs.verify(tau=1.0001) == batch.n_steps
        g1 = cs.results()
        _check_bookkeeping(g1)
        full_t = P.O.verify_steps(wt, toks, batch.ctx_lens, lambda i, l: kvt[i][l], cfg_d.verdict_ids, tau)
        P.compare_planted({"conf": g1["conf"], "accept": (g1["conf"] >= np.float32(tau)).astype(np.uint8),
                           "verdict": g1["verdict"]}, _compact_logits(cs.target, batch.n_steps), full_t, tau, cfg_t, wt)
    finally:
        cs.close()


def test_argument_errors_are_reported_before_any_launch():
    import torch
    from paper_2602_18447_b200 import binding as B
    casc = get_cascade("cascade_tiny")
    cfg_d, cfg_t = casc.draft, casc.target
    from workloads import model_weights
    wd, wt = model_weights(cfg_d.model, cfg_d.seed), model_weights(cfg_t.model, cfg_t.seed)
    batch = make_batch(cfg_d)
    cs = _sessions(casc, wd, wt, batch)
    try:
        d, t = cs.draft, cs.target
        n = batch.n_steps
        B.cs_take_launch_count()

        def call(draft=d.model, kv_d=d.kv, target=t.model, kv_t=t.kv, seq=d.seq_ids, toks=batch.step_tokens,
                 lens=batch.step_lens, vids=cfg_d.verdict_ids, tau=0.5, req_offsets=None, accept_index=0):
            return B.cs_verify_cascade(draft, kv_d, target, kv_t, seq, toks, lens, vids, tau, d.out_conf, d.out_accept,
                                       d.out_verdict, cs.out_conf_t, cs.out_verdict_t, cs.out_verdict, cs.out_conf,
                                       req_offsets=req_offsets, accept_index=accept_index)

        for bad in (dict(target=d.model, kv_t=d.kv),            # one model in both tiers
                    dict(kv_t=d.kv),                            # the target's cache belongs to the draft
                    dict(tau=float("nan")),
                    dict(vids=(1, cfg_t.model.vocab)),
                    dict(seq=np.full(n, n + 5, np.int32)),
                    dict(req_offsets=np.array([0, 4, n - 1], np.int32)),     # the requests do not cover the batch
                    dict(req_offsets=np.array([0, 7, 4, n], np.int32)),
                    dict(req_offsets=np.array([0, n], np.int32), accept_index=2),
                    dict(lens=np.where(np.arange(n) == 3, 0, batch.step_lens).astype(np.int32)),
                    dict(toks=np.where(np.arange(batch.n_tokens) == 7, -1, batch.step_tokens).astype(np.int32))):
            with pytest.raises(B.ConfSpecError) as e:
                call(**bad)
            assert e.value.status == B.CS_EINVAL, bad
        # a sequence the target's cache does not know
        B.cs_kv_free(t.kv)
        t.kv = B.cs_kv_alloc(t.model, 64, cfg_t.page_size, n, 16)
        with pytest.raises(B.ConfSpecError) as e:
            call(kv_t=t.kv)
        assert e.value.status == B.CS_ESTATE
        assert B.cs_take_launch_count() == 0                    # none of the above reached the device
        # an empty batch is a successful no-op
        assert B.cs_verify_cascade(d.model, d.kv, t.model, t.kv, np.zeros(0, np.int32), np.zeros(0, np.int32),
                                   np.zeros(0, np.int32), cfg_d.verdict_ids, 0.5, d.out_conf, d.out_accept, d.out_verdict,
                                   None, None, cs.out_verdict, cs.out_conf) == 0
        torch.cuda.synchronize()
    finally:
        cs.close()


def _full_size(target_layers, sample):
    casc = get_cascade("cascade_1p5b_7b", target_layers=target_layers)
    cfg_d, cfg_t = casc.draft, casc.target
    wd, wt = P.planted_weights(cfg_d), P.planted_weights(cfg_t)
    batch = make_batch(cfg_d)
    tau = cfg_d.tau
    cs = _sessions(casc, wd, wt, batch)
    try:
        n_esc = cs.verify(tau=tau)
        g = cs.results()
        esc = _check_bookkeeping(g)
        assert 0 < n_esc < batch.n_steps, g["conf_d"]            # both branches of the rule are exercised
        logits_t = _compact_logits(cs.target, n_esc)
        # every escalated step, not only the sampled ones, against the target model run over the whole batch:
        # the smaller batch must pair each step with its own tokens and context
        cs.target.verify(tau=tau)
        whole = cs.target.results()
        assert np.max(np.abs(whole["conf"][esc] - g["conf_t"][esc])) < 2e-2
        # sampled steps against the oracle: each tier on its own (tolerances of the planted-verdict workloads) ...
        ref_d = P.oracle_outputs(cfg_d, wd, batch, steps=sample, tau=tau)
        ref_t = P.oracle_outputs(cfg_t, wt, batch, steps=sample, tau=tau)
        gd = {"conf": g["conf_d"], "accept": g["trusted"], "verdict": g["verdict_d"]}
        P.compare_planted(gd, _compact_logits(cs.draft, batch.n_steps), ref_d, tau, cfg_d, wd, steps=sample)
        js = [j for j, i in enumerate(sample) if not g["trusted"][i]]
        if js:
            ks = [int(np.nonzero(esc == sample[j])[0][0]) for j in js]       # their places in the target's batch
            gt = {"conf": g["conf_t"][esc], "accept": (g["conf_t"][esc] >= np.float32(tau)).astype(np.uint8),
                  "verdict": g["verdict_t"][esc]}
            ref_sub = {k: v[js] for k, v in ref_t.items()}
            P.compare_planted(gt, logits_t, ref_sub, tau, cfg_t, wt, steps=ks)
        # ... then the rule, on the oracle's own numbers wherever they are clear of the threshold
        vids = list(cfg_d.verdict_ids)
        m = cfg_d.model
        row_scale = np.sqrt((P.O.widen_bf16(wd["lm_head"][vids[0]]) ** 2).sum()) / (m.init_std * np.sqrt(m.d_model))
        clear = P.CONF_TOL + 0.5 * P.LOGIT_TOL * row_scale
        n_rule = 0
        for j, i in enumerate(sample):
            cd, ct = float(ref_d["conf"][j]), float(ref_t["conf"][j])
            if abs(cd - tau) <= clear:
                continue
            n_rule += 1
            assert g["trusted"][i] == (1 if cd >= tau else 0)
            want_v, want_c = (ref_d["verdict"][j], cd) if cd >= tau else (ref_t["verdict"][j], ct)
            assert abs(g["conf"][i] - want_c) <= clear
            if abs(2 * want_c - 1) > 2 * clear:             # the two verdict probabilities are clearly apart
                assert g["verdict"][i] == want_v
        assert n_rule > 0
        return g
    finally:
        cs.close()


def test_1p5b_draft_with_7b_shaped_target_full_depth():
    """Both models at all 28 layers (3 GB + 15 GB of weights resident together), the whole batch of 16 steps."""
    _full_size(target_layers=None, sample=[5, 14])
