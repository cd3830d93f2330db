"""Parity at the full sizes of the workloads (all 28 layers, the whole batch, the launch configuration the benchmark
times): the CUDA path runs the complete batch, the CPU oracle recomputes a sample of its steps one by one (steps are
independent), and the two are compared with the specified tolerances. Every workload runs as written (random-init
weights: every confidence is ~ 1/V and every step escalates) and in its planted-verdict variant, whose confidences
lie on both sides of the threshold: there the sampled steps include trusted and escalated ones and the mask is held to
the oracle's. The tau sweep of the batch-64 workload goes through cs_escalate_mask on the planted confidences."""
import numpy as np
import pytest

from workloads import context_kv, get_config, make_batch, model_weights

import parity_common as P

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def weights_1p5b():
    cfg = get_config("cfg2_1p5b_b16")
    return model_weights(cfg.model, cfg.seed)


def _planted_rows(cfg, weights):
    """(row ids, bf16 rows) of the planted LM head that differ from the given one."""
    wp = P.planted_copy(cfg, weights)
    ids = [int(v) for v in cfg.verdict_ids[:2]]
    return wp, ids, np.stack([wp["lm_head"][i] for i in ids])


def _run_full(name, weights, n_sample, always=()):
    """The whole batch at full depth, twice in one session: with the weights as specified (random init: every
    confidence ~ 1/V) and with the two verdict rows of the LM head replaced by the planted ones, which spreads the
    confidences over (0, 1). The oracle runs its forward once over a sample of steps taken from both sides of the
    threshold and applies either LM head to it."""
    from paper_2602_18447_b200 import binding as B
    cfg = get_config(name)
    if weights is None:
        weights = model_weights(cfg.model, cfg.seed)
    batch = make_batch(cfg)
    ses = P.build_session(cfg, weights, batch)
    try:
        ses.verify()
        gpu = ses.results()
        logits, lse = ses.last_logits(), ses.last_lse()
        # properties that hold for every step of the batch, sampled or not
        assert np.all(np.isfinite(gpu["conf"])) and np.all(gpu["conf"] > 0) and np.all(gpu["conf"] <= 1)
        assert np.array_equal(gpu["accept"], (gpu["conf"] >= np.float32(cfg.tau)).astype(np.uint8))
        z = logits.astype(np.float64)
        lse_from_logits = np.log(np.exp(z - z.max(axis=1, keepdims=True)).sum(axis=1)) + z.max(axis=1)
        assert np.max(np.abs(lse_from_logits - lse)) < 1e-4          # fused logsumexp == logsumexp of the logits
        vid = list(cfg.verdict_ids)
        assert np.max(np.abs(np.exp(z[:, vid] - lse_from_logits[:, None]).max(axis=1) - gpu["conf"])) < 1e-6
        del z
        B.cs_check_workspace(ses.model)          # guard bytes behind every workspace are intact
        # the pass is deterministic: a second run gives the same bits (logits of all steps, confidences, mask)
        ses.verify()
        again = ses.results()
        assert np.array_equal(again["conf"].view(np.uint32), gpu["conf"].view(np.uint32))
        assert np.array_equal(again["accept"], gpu["accept"]) and np.array_equal(again["verdict"], gpu["verdict"])
        assert np.array_equal(ses.last_logits().view(np.uint32), logits.view(np.uint32))

        # ---- planted verdict rows, same session
        wp, ids, rows = _planted_rows(cfg, weights)
        B.cs_model_set_lm_head_rows(ses.model, ids, rows)
        ses.verify()
        gpu_p = ses.results()
        logits_p, lse_p = ses.last_logits(), ses.last_lse()
        assert np.array_equal(gpu_p["accept"], (gpu_p["conf"] >= np.float32(cfg.tau)).astype(np.uint8))
        _, conf_tol = P.planted_tols(cfg)
        sample = P.sample_both_sides(gpu_p["conf"], cfg.tau, conf_tol, n_sample, always=always)

        # ---- the oracle: one forward over the sample, both LM heads
        toks = P.steps_of(batch)

        def kv_fn(j, l):
            k, v = context_kv(cfg, sample[j], l, int(batch.ctx_lens[sample[j]]))
            return P.O.widen_bf16(k), P.O.widen_bf16(v)

        xs, _ = P.O.forward_extend(weights, [toks[i] for i in sample], [int(batch.ctx_lens[i]) for i in sample], kv_fn)

        def head(w):
            zz = P.O.last_position_logits(w, xs)
            conf, verdict, l = P.O.verdict_confidence(zz, cfg.verdict_ids)
            return {"logits": zz, "conf": conf, "verdict": verdict, "lse": l, "accept": P.O.gate(conf, cfg.tau)}

        ref = head(weights)
        stats = P.compare(gpu, logits, ref, cfg.tau, steps=sample, gpu_lse=lse)
        P.check_verdict(gpu, ref, cfg.verdict_ids, steps=sample)
        ref_p = head(wp)
        stats_p = P.compare_planted(gpu_p, logits_p, ref_p, cfg.tau, cfg, steps=sample, gpu_lse=lse_p,
                                    need_both_sides=True, case=name + "/full-depth planted")
        P.check_verdict(gpu_p, ref_p, cfg.verdict_ids, steps=sample)
        P.record_stats(name + "/full-depth base", stats)
        return cfg, ses, gpu_p, ref_p, sample, stats, stats_p
    except BaseException:
        ses.close()
        raise


def test_cfg2_batch16_full_depth(weights_1p5b):
    cfg, ses, gpu_p, ref_p, sample, stats, stats_p = _run_full("cfg2_1p5b_b16", weights_1p5b, 8, always=(0, 15))
    ses.close()
    assert stats["logit_err"] <= P.LOGIT_TOL and stats["conf_err"] <= P.CONF_TOL


def test_cfg3_batch64_full_depth_and_tau_sweep(weights_1p5b):
    """The threshold sweep of the batch-64 workload goes through cs_escalate_mask on the stored confidences of the
    planted variant, so the escalation list changes with tau; the sampled steps are held to the oracle's mask at every
    tau at which they lie outside the confidence bound."""
    import torch
    from paper_2602_18447_b200 import binding as B
    cfg, ses, gpu_p, ref_p, sample, stats, stats_p = _run_full("cfg3_1p5b_b64", weights_1p5b, 8, always=(3, 40))
    try:
        n = cfg.batch
        _, conf_tol = P.planted_tols(cfg)
        counts, n_tr, n_es = [], 0, 0
        for tau in cfg.taus:
            acc = torch.zeros(n, dtype=torch.uint8, device="cuda")
            idx = torch.full((n,), -1, dtype=torch.int32, device="cuda")
            cnt = torch.zeros(1, dtype=torch.int32, device="cuda")
            B.cs_escalate_mask(ses.out_conf, tau, acc, idx, cnt)
            torch.cuda.synchronize()
            want_acc, want_idx, want_cnt = P.O.escalate_list(gpu_p["conf"], tau)
            got_acc = acc.cpu().numpy()
            assert int(cnt.item()) == want_cnt and np.array_equal(got_acc, want_acc)
            assert np.array_equal(idx.cpu().numpy()[:want_cnt], want_idx)
            counts.append(want_cnt)
            # against the oracle's own confidences, for the sampled steps outside the bound around this tau
            far = np.abs(ref_p["conf"] - tau) > conf_tol
            want = P.O.gate(ref_p["conf"], tau)
            assert np.array_equal(got_acc[sample][far], want[far])
            n_tr += int((far & (want == 1)).sum())
            n_es += int((far & (want == 0)).sum())
        assert counts == sorted(counts) and counts[0] < counts[-1]     # a higher threshold escalates more steps
        assert 0 < counts[0] and counts[-1] <= n and n_tr >= 1 and n_es >= 1
    finally:
        ses.close()


def test_cfg4_long_context_full_depth(weights_1p5b):
    cfg, ses, gpu_p, ref_p, sample, stats, stats_p = _run_full("cfg4_1p5b_long", weights_1p5b, 4)
    ses.close()
    assert stats["logit_err"] <= P.LOGIT_TOL


def test_cfg5_7b_shape_full_batch_reduced_depth():
    """The 7B-shaped escalation verifier with its whole batch of 32 steps, full width and vocabulary, at 3 of its 28
    layers (drawing all 15 GB of its weights on the host takes minutes): every kernel runs in the launch shapes of
    the full model, only the loop over layers is shorter."""
    from workloads import scaled_config
    cfg = scaled_config("cfg5_7b_b32", n_layers=3)
    weights = model_weights(cfg.model, cfg.seed)
    batch = make_batch(cfg)
    sample = [2, 17, 31]
    ses = P.build_session(cfg, weights, batch)
    try:
        ses.verify()
        gpu = ses.results()
        ref = P.oracle_outputs(cfg, weights, batch, steps=sample)
        stats = P.compare(gpu, ses.last_logits(), ref, cfg.tau, steps=sample, gpu_lse=ses.last_lse())
        P.check_verdict(gpu, ref, cfg.verdict_ids, steps=sample)
        assert stats["logit_err"] <= P.LOGIT_TOL
    finally:
        ses.close()


def test_cfg5_7b_shape_full_depth():
    """All 28 layers of the 7B-shaped verifier (15 GB of weights), whole batch; the oracle recomputes two steps."""
    cfg, ses, gpu_p, ref_p, sample, stats, stats_p = _run_full("cfg5_7b_b32", None, 4)
    ses.close()
    assert stats["logit_err"] <= P.LOGIT_TOL and stats["conf_err"] <= P.CONF_TOL


@pytest.fixture(scope="module")
def weights_q3():
    cfg = get_config("cfg6_q3_b16")
    return model_weights(cfg.model, cfg.seed)


def test_cfg6_second_family_full_depth(weights_q3):
    """The 1.7B-shaped model of the second family (query/key normalisation, 8 KV heads), all 28 layers."""
    cfg, ses, gpu_p, ref_p, sample, stats, stats_p = _run_full("cfg6_q3_b16", weights_q3, 4, always=(2,))
    ses.close()
    assert stats["logit_err"] <= P.LOGIT_TOL and stats["conf_err"] <= P.CONF_TOL


def test_cfg7_cfg9_short_steps_on_long_contexts_full_depth(weights_q3):
    """Decode-shaped batch: 64 steps of 5 to 8 new tokens on contexts of 2K to 8K tokens, all 28 layers, over the
    16-bit cache (cfg7) and over the 8-bit cache holding the same draws rounded to 8 bits (cfg9). The two caches are
    filled side by side so that the 20 G context values are drawn once."""
    from concurrent.futures import ThreadPoolExecutor
    from workloads import context_kv, e4m3_codes_from_f32, page_assignment
    from paper_2602_18447_b200 import VerifySession, binding as B
    cfg7, cfg9 = get_config("cfg7_q3_short"), get_config("cfg9_q3_short_fp8")
    assert cfg7.seed == cfg9.seed and cfg7.model == cfg9.model
    batch = make_batch(cfg7)
    sample = [0, 33, 63]
    sessions = []
    try:
        for cfg in (cfg7, cfg9):
            ses = VerifySession(cfg, weights_q3, batch)
            sessions.append(ses)
            B.cs_set_keep_logits(ses.model, True)
            total, pages = page_assignment(cfg, batch.ctx_lens)
            ses.alloc_cache(pages, total, batch.ctx_lens)
        widen = lambda b: (b.astype(np.uint32) << np.uint32(16)).view(np.float32)

        def draw(job):
            i, l = job
            k, v = context_kv(cfg7, i, l, int(batch.ctx_lens[i]))
            return k, v, e4m3_codes_from_f32(widen(k)), e4m3_codes_from_f32(widen(v))

        jobs = [(i, l) for i in range(batch.n_steps) for l in range(cfg7.model.n_layers)]
        import os
        workers = min(16, os.cpu_count() or 8)
        with ThreadPoolExecutor(max_workers=workers) as pool:
            for o in range(0, len(jobs), 4 * workers):
                part = jobs[o:o + 4 * workers]
                for (i, l), (k, v, k8, v8) in zip(part, pool.map(draw, part)):
                    B.cs_kv_fill(sessions[0].kv, i, l, k, v)
                    B.cs_kv_fill(sessions[1].kv, i, l, k8, v8)
        # the generator's own 8-bit path gives the same codes as the ones filled above
        k8, v8 = context_kv(cfg9, 5, 3, int(batch.ctx_lens[5]))
        k, v = context_kv(cfg7, 5, 3, int(batch.ctx_lens[5]))
        assert np.array_equal(k8, e4m3_codes_from_f32(widen(k))) and np.array_equal(v8, e4m3_codes_from_f32(widen(v)))
        for cfg, ses in zip((cfg7, cfg9), sessions):
            ses.verify()
            gpu = ses.results()
            ref = P.oracle_outputs(cfg, weights_q3, batch, steps=sample)
            stats = P.compare(gpu, ses.last_logits(), ref, cfg.tau, steps=sample, gpu_lse=ses.last_lse())
            P.check_verdict(gpu, ref, cfg.verdict_ids, steps=sample)
            assert stats["logit_err"] <= P.LOGIT_TOL and stats["conf_err"] <= P.CONF_TOL
            assert np.all(np.isfinite(gpu["conf"])) and np.all(gpu["conf"] > 0) and np.all(gpu["conf"] <= 1)
    finally:
        for ses in sessions:
            ses.close()
