"""One whole iteration of the verification side of Algorithm 1 on the GPU against the oracle: the k candidates of
each request verified on the request's shared context pages by both tiers (cs_verify_cascade), the accept-prefix
length m (cs_cascade_select), the accepted drafted steps appended to both models' caches (cs_append_accepted), and
the next iteration's verification on the longer contexts."""
import numpy as np
import pytest

from workloads import get_cascade

import parity_common as P

pytestmark = pytest.mark.gpu

REQ_OFFSETS = np.array([0, 4, 8, 12], dtype=np.int32)      # 3 requests x k = 4 drafted steps
CTX_LENS = (40, 100, 23)
PAGES_PER_REQ = 12                                           # room for the context and all four drafted steps


def _draw(cfg, seed):
    g = np.random.default_rng(seed)
    V = cfg.model.vocab
    B = int(REQ_OFFSETS[-1])
    draft_lens = g.integers(3, 12, size=B).astype(np.int32)
    rest = g.integers(4, 14, size=B).astype(np.int32)          # target's step + verification prompt
    spans = [g.integers(3, V, size=int(d + r)).astype(np.int32) for d, r in zip(draft_lens, rest)]
    return spans, draft_lens


def _gpu_tier(cfg, weights, ctx_tokens):
    """Model, cache with one sequence per request (its pages shared by the request's candidates), contexts prefilled."""
    from paper_2602_18447_b200 import binding as B
    model = B.cs_model_load(cfg.model, weights)
    R = len(ctx_tokens)
    kv = B.cs_kv_alloc(model, R * PAGES_PER_REQ, cfg.page_size, R, PAGES_PER_REQ)
    perm = np.random.default_rng(3).permutation(R * PAGES_PER_REQ).astype(np.int32)
    for r in range(R):
        B.cs_kv_set_seq(kv, r, perm[r * PAGES_PER_REQ:(r + 1) * PAGES_PER_REQ], 0)
    B.cs_prefill(model, kv, np.arange(R, dtype=np.int32), np.concatenate(ctx_tokens).astype(np.int32),
                 np.array([len(t) for t in ctx_tokens], dtype=np.int32))
    return model, kv


def test_verify_select_append_verify():
    import torch
    from paper_2602_18447_b200 import binding as B
    casc = get_cascade("cascade_tiny")
    cfg_d, cfg_t = casc.draft, casc.target
    wd, wt = P.planted_weights(cfg_d), P.planted_weights(cfg_t)
    g = np.random.default_rng(77)
    ctx = [g.integers(3, cfg_d.model.vocab, size=n).astype(np.int32) for n in CTX_LENS]
    R, nB = len(ctx), int(REQ_OFFSETS[-1])
    req_of = np.repeat(np.arange(R), np.diff(REQ_OFFSETS)).astype(np.int32)
    spans1, dl1 = _draw(cfg_d, 7)       # gives m = (0, 1, 4): nothing, part and all of a request's steps
    spans2, dl2 = _draw(cfg_d, 2)
    vids = cfg_d.verdict_ids

    # ---- oracle: iteration 1, selection, append, iteration 2
    kvd = P.O.prefill_context(wd, ctx, store_bf16=True)
    kvt = P.O.prefill_context(wt, ctx, store_bf16=True)
    lens1 = [len(ctx[r]) for r in req_of]
    probe = P.O.verify_steps(wd, spans1, lens1, lambda i, l: kvd[req_of[i]][l], vids, 0.5)
    srt = np.sort(probe["conf"])
    k = 2 + int(np.argmax(srt[3:nB - 1] - srt[2:nB - 2]))
    tau, gap = float(0.5 * (srt[k] + srt[k + 1])), float(srt[k + 1] - srt[k])
    ref1 = P.O.verify_cascade(wd, wt, spans1, lens1, lambda i, l: kvd[req_of[i]][l], lambda i, l: kvt[req_of[i]][l],
                              vids, tau, req_offsets=REQ_OFFSETS, accept_index=0)
    esc = ref1["escalated"]
    # linear drafting: steps behind a trusted rejection of their request are not sent to the target model
    n_below = int((ref1["draft"]["accept"] == 0).sum())
    assert 0 < esc.size < n_below
    vt, ct = np.full(nB, -1, np.int32), np.zeros(nB, np.float32)
    if esc.size:
        vt[esc], ct[esc] = ref1["target"]["verdict"], ref1["target"]["conf"]
    _, _, m_ref, _ = P.O.cascade_select(ref1["draft"]["accept"], ref1["draft"]["verdict"], ref1["draft"]["conf"], vt, ct,
                                        REQ_OFFSETS, accept_index=0)
    assert m_ref.tolist() == [0, 1, 4]
    drafts1 = [s[:d] for s, d in zip(spans1, dl1)]
    kvd2 = P.O.append_accepted_steps(wd, kvd, m_ref, REQ_OFFSETS, drafts1, store_bf16=True)
    kvt2 = P.O.append_accepted_steps(wt, kvt, m_ref, REQ_OFFSETS, drafts1, store_bf16=True)
    ctx2 = [kvd2[r][0][0].shape[0] for r in range(R)]
    lens2 = [ctx2[r] for r in req_of]
    ref2 = P.O.verify_cascade(wd, wt, spans2, lens2, lambda i, l: kvd2[req_of[i]][l], lambda i, l: kvt2[req_of[i]][l],
                              vids, 1.0001)                 # every step through both tiers

    # ---- GPU
    md, kd = _gpu_tier(cfg_d, wd, ctx)
    mt, kt = _gpu_tier(cfg_t, wt, ctx)
    try:
        dev = "cuda"
        f32 = lambda: torch.empty(nB, dtype=torch.float32, device=dev)
        i32 = lambda n=nB: torch.empty(n, dtype=torch.int32, device=dev)
        conf_d, conf_t, conf = f32(), f32(), f32()
        trusted = torch.empty(nB, dtype=torch.uint8, device=dev)
        ver_d, ver_t, ver = i32(), i32(), i32()
        for mdl in (md, mt):
            B.cs_set_keep_logits(mdl, True)

        def cascade(spans, tau_, req_offsets=None):
            toks = np.concatenate(spans).astype(np.int32)
            lens = np.array([len(s) for s in spans], dtype=np.int32)
            n = B.cs_verify_cascade(md, kd, mt, kt, req_of, toks, lens, vids, tau_, conf_d, trusted, ver_d, conf_t,
                                    ver_t, ver, conf, req_offsets=req_offsets, accept_index=0)
            torch.cuda.synchronize()
            B.cs_last_status(md), B.cs_last_status(mt)
            return n, toks, lens

        n1, toks1, lens_1 = cascade(spans1, tau, REQ_OFFSETS)
        assert np.max(np.abs(conf_d.cpu().numpy() - ref1["draft"]["conf"])) < 0.45 * gap
        assert np.array_equal(trusted.cpu().numpy(), ref1["draft"]["accept"])
        assert n1 == esc.size and np.array_equal(np.nonzero(ver_t.cpu().numpy() >= 0)[0], esc)
        left_out = (trusted.cpu().numpy() == 0) & (ver_t.cpu().numpy() < 0)
        assert left_out.sum() == n_below - esc.size
        assert np.all(ver.cpu().numpy()[left_out] == -1) and np.all(conf.cpu().numpy()[left_out] == 0.0)
        m_dev, best = i32(R), i32(R)
        B.cs_cascade_select(trusted, ver_d, conf_d, ver_t, conf_t, torch.from_numpy(REQ_OFFSETS).to(dev), 0, m_dev, best)
        torch.cuda.synchronize()
        # the decisions may differ from the oracle's only where the two verdict probabilities are nearly equal
        pv_d = np.exp(ref1["draft"]["logits"][:, list(vids)] - ref1["draft"]["lse"][:, None])
        clear = (np.abs(pv_d[:, 0] - pv_d[:, 1]) > 0.03) | (ref1["draft"]["accept"] == 0)   # only decisions that are used
        if esc.size:
            pv_t = np.exp(ref1["target"]["logits"][:, list(vids)] - ref1["target"]["lse"][:, None])
            clear[esc] = np.abs(pv_t[:, 0] - pv_t[:, 1]) > 0.03
        assert clear.all()
        assert np.array_equal(m_dev.cpu().numpy(), m_ref)
        # append what the oracle accepted, to both caches, and verify the next candidates on the longer contexts
        m_in = torch.from_numpy(m_ref.astype(np.int32)).to(dev)
        for mdl, kv in ((md, kd), (mt, kt)):
            got = B.cs_append_accepted(mdl, kv, np.arange(R, dtype=np.int32), REQ_OFFSETS, m_in, toks1, lens_1, dl1)
            assert np.array_equal(got, m_ref)
        n2, _, _ = cascade(spans2, 1.0001)
        assert n2 == nB
        out_d = torch.empty(nB, cfg_d.model.vocab, dtype=torch.float32, device=dev)
        out_t = torch.empty(nB, cfg_t.model.vocab, dtype=torch.float32, device=dev)
        B.cs_get_last_logits(md, out_d, nB)
        B.cs_get_last_logits(mt, out_t, nB)
        torch.cuda.synchronize()
        gd = {"conf": conf_d.cpu().numpy(), "accept": trusted.cpu().numpy(), "verdict": ver_d.cpu().numpy()}
        gt = {"conf": conf_t.cpu().numpy(), "accept": np.zeros(nB, np.uint8), "verdict": ver_t.cpu().numpy()}
        sd = P.compare_planted(gd, out_d.cpu().numpy(), ref2["draft"], 1.0001, cfg_d, wd)
        st = P.compare_planted(gt, out_t.cpu().numpy(), ref2["target"], 1.0001, cfg_t, wt)
        assert sd["logit_err"] <= P.LOGIT_TOL and st["logit_err"] <= P.LOGIT_TOL
        # the appended context matters: the same candidates on the OLD contexts give other logits
        old = P.O.verify_steps(wd, spans2, lens1, lambda i, l: kvd[req_of[i]][l], vids, 0.5)
        grown = [i for i in range(nB) if m_ref[req_of[i]] > 0]
        assert min(np.max(np.abs(old["logits"][i] - ref2["draft"]["logits"][i])) for i in grown) > 10 * P.LOGIT_TOL
        # a request without room for the accepted tokens is refused before anything is appended
        tight = B.cs_kv_alloc(md, 8, cfg_d.page_size, 1, 3)
        try:
            B.cs_kv_set_seq(tight, 0, np.arange(3, dtype=np.int32), 45)
            one = torch.tensor([4], dtype=torch.int32, device=dev)
            with pytest.raises(B.ConfSpecError) as e:
                B.cs_append_accepted(md, tight, np.zeros(1, np.int32), np.array([0, 4], np.int32), one, toks1[:int(lens_1[:4].sum())],
                                     lens_1[:4], dl1[:4])
            assert e.value.status == B.CS_EINVAL and dl1[:4].sum() > 3
        finally:
            B.cs_kv_free(tight)
    finally:
        for kv in (kd, kt):
            B.cs_kv_free(kv)
        for mdl in (md, mt):
            B.cs_model_free(mdl)
