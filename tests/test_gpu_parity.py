"""End-to-end parity of cs_verify_steps with the CPU oracle at sizes the oracle finishes in seconds: the tiny
workload (real prefill through cs_prefill), reduced-depth variants of the 1.5B- and 7B-shaped workloads (same
widths, ragged contexts and steps, scattered pages), planted-verdict variants that put confidences on both
sides of the threshold, and the edge cases of the batch structure."""
from dataclasses import replace

import numpy as np
import pytest

from workloads import get_config, make_batch, model_weights, scaled_config

import parity_common as P

pytestmark = pytest.mark.gpu


def _run(cfg, weights, batch, taus=None, planted=False, both_sides=False):
    """One pass at cfg.tau and one per extra threshold, each against the oracle. With `both_sides` the planted runs
    must, over all thresholds together, have compared at least one trusted and one escalated step with the oracle's
    mask outside the confidence bound."""
    ses = P.build_session(cfg, weights, batch)
    try:
        ses.verify()
        gpu = ses.results()
        logits, lse = ses.last_logits(), ses.last_lse()
        ref = P.oracle_outputs(cfg, weights, batch)
        n_tr = n_es = 0
        if planted:
            stats = P.compare_planted(gpu, logits, ref, cfg.tau, cfg, weights, gpu_lse=lse)
            n_tr, n_es = stats["n_cmp_trusted"], stats["n_cmp_escalated"]
        else:
            stats = P.compare(gpu, logits, ref, cfg.tau, gpu_lse=lse)
            P.check_verdict(gpu, ref, cfg.verdict_ids)
        for tau in taus or ():
            ses.verify(tau=tau)
            g2 = ses.results()
            r2 = dict(ref, accept=P.O.gate(ref["conf"], tau))
            if planted:
                st = P.compare_planted(g2, ses.last_logits(), r2, tau, cfg, weights, gpu_lse=ses.last_lse())
                n_tr += st["n_cmp_trusted"]
                n_es += st["n_cmp_escalated"]
            else:
                P.compare(g2, None, r2, tau)
        if both_sides:
            assert n_tr >= 1 and n_es >= 1, (n_tr, n_es, ref["conf"])
        # nothing wrote past the end of a workspace (guard bytes behind every buffer)
        from paper_2602_18447_b200 import binding as B
        B.cs_check_workspace(ses.model)
        # host-token entry (tokens copied inside the call): the same pass, bit for bit (every reduction of the pass has
        # a fixed order), logits included
        ses.verify(host_tokens=True)
        g3 = ses.results()
        assert np.array_equal(g3["conf"].view(np.uint32), gpu["conf"].view(np.uint32))
        assert np.array_equal(g3["accept"], gpu["accept"]) and np.array_equal(g3["verdict"], gpu["verdict"])
        assert np.array_equal(ses.last_logits().view(np.uint32), logits.view(np.uint32))
        return stats, gpu, ref
    finally:
        ses.close()


def test_cfg1_tiny_with_real_prefill():
    cfg = get_config("cfg1_tiny")
    stats, gpu, ref = _run(cfg, model_weights(cfg.model, cfg.seed), make_batch(cfg))
    assert gpu["accept"].tolist() == [0] * cfg.batch      # random-init weights: conf ~ 1/V, all escalate
    assert stats["logit_err"] < 3e-2


def test_cfg1_tiny_planted_verdict_rows_and_tau_sweep():
    cfg = replace(get_config("cfg1_tiny"), batch=24)
    stats, gpu, ref = _run(cfg, P.planted_weights(cfg), make_batch(cfg), taus=(0.0, 0.5, 0.7, 0.9, 0.95, 0.99, 1.0001),
                           planted=True, both_sides=True)
    assert 0 < ref["accept"].sum() < cfg.batch           # the gate is exercised on both sides
    assert ref["conf"].max() > 0.9 and ref["conf"].min() < 0.5


@pytest.mark.parametrize("name,layers,batch", [("cfg2_1p5b_b16", 2, 8), ("cfg3_1p5b_b64", 1, 9), ("cfg5_7b_b32", 1, 8)])
def test_reduced_depth_large_shapes(name, layers, batch):
    cfg = scaled_config(name, n_layers=layers, batch=batch, vocab=20480 + 8)   # ragged vocabulary tail
    stats, gpu, ref = _run(cfg, P.planted_weights(cfg), make_batch(cfg), taus=(0.3, 0.5, 0.99), planted=True,
                           both_sides=True)
    assert stats["logit_err"] < 3e-2
    # the same shapes with the weights as specified (random init): the specified tolerances
    _run(cfg, model_weights(cfg.model, cfg.seed), make_batch(cfg))


def test_long_context_split_kv():
    cfg = scaled_config("cfg4_1p5b_long", n_layers=1, batch=2, vocab=8192)
    _run(cfg, P.planted_weights(cfg), make_batch(cfg), planted=True)
    _run(cfg, model_weights(cfg.model, cfg.seed), make_batch(cfg))


@pytest.mark.parametrize("ctx,step", [(0, 1), (1, 1), (15, 3), (16, 64), (17, 65), (63, 129), (64, 200), (65, 7)])
def test_context_and_step_length_edges(ctx, step):
    """Empty context, single-token step, page and tile boundaries +-1."""
    base = get_config("cfg1_tiny")
    cfg = replace(base, batch=3, ctx_dist=("fixed", ctx), step_dist=("fixed", step), suffix_len=0)
    batch = make_batch(cfg)
    _run(cfg, P.planted_weights(cfg), batch, planted=True)


def test_batch_permutation_permutes_outputs():
    cfg = replace(get_config("cfg1_tiny"), batch=6, ctx_dist=("uniform", 20, 150), step_dist=("uniform", 5, 60))
    w = P.planted_weights(cfg)
    batch = make_batch(cfg)
    ses = P.build_session(cfg, w, batch)
    try:
        ses.verify()
        base = ses.results()
        perm = np.array([3, 0, 5, 1, 4, 2])
        from paper_2602_18447_b200 import binding as B
        import torch
        toks = np.concatenate([P.steps_of(batch)[p] for p in perm]).astype(np.int32)
        conf = torch.empty(6, dtype=torch.float32, device="cuda")
        acc = torch.empty(6, dtype=torch.uint8, device="cuda")
        B.cs_verify_steps(ses.model, ses.kv, perm.astype(np.int32), toks, batch.step_lens[perm], cfg.verdict_ids,
                          cfg.tau, conf, acc)
        torch.cuda.synchronize()
        # a step's arithmetic does not depend on its place in the batch, except for which pieces a residual tile's k
        # range is cut into (the cut depends on the token count before it): equal to rounding, which the planted rows magnify
        assert np.max(np.abs(conf.cpu().numpy() - base["conf"][perm])) <= 2.5e-3
    finally:
        ses.close()


def test_invalid_arguments_are_rejected_before_any_launch():
    import torch
    from paper_2602_18447_b200 import binding as B
    cfg = replace(get_config("cfg1_tiny"), batch=2)
    batch = make_batch(cfg)
    ses = P.build_session(cfg, model_weights(cfg.model, cfg.seed), batch)
    try:
        B.cs_take_launch_count()
        conf = torch.empty(2, dtype=torch.float32, device="cuda")
        acc = torch.empty(2, dtype=torch.uint8, device="cuda")

        def call(**kw):
            a = dict(seq=ses.seq_ids, toks=batch.step_tokens, lens=batch.step_lens, vids=cfg.verdict_ids, tau=0.9)
            a.update(kw)
            B.cs_verify_steps(ses.model, ses.kv, a["seq"], a["toks"], a["lens"], a["vids"], a["tau"], conf, acc)

        for bad in (dict(tau=float("nan")), dict(lens=np.array([0, 5], np.int32)), dict(vids=[cfg.model.vocab]),
                    dict(vids=[]), dict(seq=np.array([0, 7], np.int32)),
                    dict(toks=np.full_like(batch.step_tokens, cfg.model.vocab))):
            with pytest.raises(B.ConfSpecError) as e:
                call(**bad)
            assert e.value.status == B.CS_EINVAL
        assert B.cs_take_launch_count() == 0
        # an empty batch is a no-op
        B.cs_verify_steps(ses.model, ses.kv, np.zeros(0, np.int32), np.zeros(0, np.int32), np.zeros(0, np.int32),
                          cfg.verdict_ids, 0.9, conf, acc)
        assert B.cs_take_launch_count() == 0
    finally:
        ses.close()


def test_qk_norm_family_tiny_with_real_prefill():
    """Per-head query/key RMSNorm before the rotary turn (fused into the QKV projection's epilogue), through a real
    prefill and a verification pass; the planted variant puts the gate on both sides."""
    cfg = get_config("cfg8_tiny_qknorm")
    stats, gpu, ref = _run(cfg, model_weights(cfg.model, cfg.seed), make_batch(cfg))
    assert stats["logit_err"] < 3e-2
    _run(cfg, P.planted_weights(cfg), make_batch(cfg), taus=(0.5, 0.9), planted=True)
    # the gains matter: the oracle without them is far away
    w = model_weights(cfg.model, cfg.seed)
    plain = dict(w, layers=[{k: v for k, v in l.items() if k not in ("q_norm", "k_norm")} for l in w["layers"]])
    other = P.oracle_outputs(cfg, plain, make_batch(cfg))
    assert np.max(np.abs(other["logits"] - ref["logits"])) > 10 * P.LOGIT_TOL


@pytest.mark.parametrize("name,layers,batch", [("cfg6_q3_b16", 2, 4), ("cfg7_q3_short", 2, 9)])
def test_qk_norm_family_reduced_depth(name, layers, batch):
    cfg = scaled_config(name, n_layers=layers, batch=batch, vocab=20480 + 8)
    stats, gpu, ref = _run(cfg, P.planted_weights(cfg), make_batch(cfg), taus=(0.5,), planted=True)
    assert stats["logit_err"] < 3e-2
    _run(cfg, model_weights(cfg.model, cfg.seed), make_batch(cfg))


def test_more_steps_than_one_lm_head_pass_takes():
    """70 steps: the LM head runs in two passes of at most 64 steps, the last layer's MLP on 70 rows."""
    cfg = replace(get_config("cfg1_tiny"), batch=70, ctx_dist=("uniform", 0, 90), step_dist=("uniform", 1, 12), suffix_len=2)
    stats, gpu, ref = _run(cfg, P.planted_weights(cfg), make_batch(cfg), planted=True)
    assert stats["logit_err"] < 3e-2 and 0 < ref["accept"].sum() < cfg.batch


def test_without_the_fixed_order_passes_agree_to_rounding():
    """cs_set_deterministic(model, 0): the residual projections add their pieces as they finish."""
    from paper_2602_18447_b200 import binding as B
    cfg = scaled_config("cfg2_1p5b_b16", n_layers=2, batch=8, vocab=20480 + 8)
    w, batch = P.planted_weights(cfg), make_batch(cfg)
    ses = P.build_session(cfg, w, batch)
    try:
        ses.verify()
        a = ses.results()
        B.cs_set_deterministic(ses.model, False)
        ses.verify()
        b = ses.results()
        assert np.max(np.abs(a["conf"] - b["conf"])) <= 2.5e-3
        ref = P.oracle_outputs(cfg, w, batch)
        P.compare_planted(b, ses.last_logits(), ref, cfg.tau, cfg, gpu_lse=ses.last_lse())
    finally:
        ses.close()


def test_splitting_the_batch_changes_nothing_beyond_rounding():
    """Steps are verified independently (Section 4.3): one call over the batch and two calls over its halves give the
    same confidences up to the rounding order of the residual projections (whose pieces depend on the token count)."""
    import torch
    from paper_2602_18447_b200 import binding as B
    cfg = replace(get_config("cfg1_tiny"), batch=10, ctx_dist=("uniform", 20, 150), step_dist=("uniform", 5, 60))
    w, batch = P.planted_weights(cfg), make_batch(cfg)
    ses = P.build_session(cfg, w, batch)
    try:
        ses.verify()
        whole = ses.results()
        parts = []
        for lo, hi in ((0, 4), (4, 10)):
            toks = np.concatenate(P.steps_of(batch)[lo:hi]).astype(np.int32)
            conf = torch.empty(hi - lo, dtype=torch.float32, device="cuda")
            acc = torch.empty(hi - lo, dtype=torch.uint8, device="cuda")
            B.cs_verify_steps(ses.model, ses.kv, np.arange(lo, hi, dtype=np.int32), toks, batch.step_lens[lo:hi],
                              cfg.verdict_ids, cfg.tau, conf, acc)
            torch.cuda.synchronize()
            parts.append((conf.cpu().numpy(), acc.cpu().numpy()))
        conf2 = np.concatenate([p[0] for p in parts])
        acc2 = np.concatenate([p[1] for p in parts])
        assert np.max(np.abs(conf2 - whole["conf"])) <= 2.5e-3
        sure = np.abs(whole["conf"] - cfg.tau) > 2.5e-3
        assert np.array_equal(acc2[sure], whole["accept"][sure])
    finally:
        ses.close()
