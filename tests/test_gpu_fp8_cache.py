"""Parity of the verification pass over the optional 8-bit cache (short steps; codes widened on the fly) with the
oracle, which reads the same codes through its own decoder: small models every step, the decode-shaped 1.7B-shaped
workload at reduced and full depth, contexts cut into pieces, the edges of the page structure, and what the format
refuses."""
from dataclasses import replace

import numpy as np
import pytest

from workloads import get_config, make_batch, model_weights, scaled_config

import parity_common as P

pytestmark = pytest.mark.gpu


def _run(cfg, weights, batch, planted=False):
    ses = P.build_session(cfg, weights, batch)
    try:
        ses.verify()
        gpu = ses.results()
        logits, lse = ses.last_logits(), ses.last_lse()
        ref = P.oracle_outputs(cfg, weights, batch)
        if planted:
            return P.compare_planted(gpu, logits, ref, cfg.tau, cfg, weights), gpu, ref
        stats = P.compare(gpu, logits, ref, cfg.tau, gpu_lse=lse)
        P.check_verdict(gpu, ref, cfg.verdict_ids)
        return stats, gpu, ref
    finally:
        ses.close()


def _tiny(name, **kw):
    base = dict(ctx_kv="synthetic", kv_format="e4m3", suffix_len=0)     # kw may choose the other format
    base.update(kw)
    return replace(get_config(name), **base)


@pytest.mark.parametrize("fmt", ["e4m3", "e5m2"])
@pytest.mark.parametrize("name,steps", [("cfg1_tiny", ("uniform", 1, 32)), ("cfg8_tiny_qknorm", ("uniform", 1, 16))])
def test_small_models_every_step(name, steps, fmt):
    cfg = _tiny(name, batch=7, ctx_dist=("uniform", 1, 300), step_dist=steps, kv_format=fmt)
    stats, gpu, ref = _run(cfg, P.planted_weights(cfg), make_batch(cfg), planted=True)
    assert stats["logit_err"] < 3e-2
    _run(cfg, model_weights(cfg.model, cfg.seed), make_batch(cfg))
    # the 8-bit rounding of the cache is part of the input, and it matters: the oracle on the unrounded draws differs
    other = P.oracle_outputs(replace(cfg, kv_format="bf16"), model_weights(cfg.model, cfg.seed), make_batch(cfg))
    mine = P.oracle_outputs(cfg, model_weights(cfg.model, cfg.seed), make_batch(cfg))
    assert np.max(np.abs(other["logits"] - mine["logits"])) > 1e-4


@pytest.mark.parametrize("ctx,step", [(0, 1), (1, 1), (15, 3), (16, 16), (17, 32), (63, 5), (64, 8), (65, 7), (257, 2)])
def test_context_and_step_length_edges(ctx, step):
    cfg = _tiny("cfg1_tiny", batch=3, ctx_dist=("fixed", ctx), step_dist=("fixed", step))
    _run(cfg, P.planted_weights(cfg), make_batch(cfg), planted=True)


@pytest.mark.parametrize("fmt", ["e4m3", "e5m2"])
def test_long_contexts_cut_into_pieces(fmt):
    """Two steps on contexts of thousands of tokens: every (step, kv head) range is cut into pieces whose partial
    results a second kernel combines."""
    cfg = _tiny("cfg8_tiny_qknorm", batch=2, ctx_dist=("uniform", 5000, 9000), step_dist=("uniform", 3, 9), kv_format=fmt)
    stats, gpu, ref = _run(cfg, P.planted_weights(cfg), make_batch(cfg), planted=True)
    assert stats["logit_err"] < 3e-2


@pytest.mark.parametrize("name", ["cfg9_q3_short_fp8", "cfg10_q3_short_e5m2"])
def test_decode_shaped_workload_reduced_depth(name):
    cfg = scaled_config(name, n_layers=2, batch=9, vocab=20480 + 8)
    stats, gpu, ref = _run(cfg, P.planted_weights(cfg), make_batch(cfg), planted=True)
    assert stats["logit_err"] < 3e-2
    _run(cfg, model_weights(cfg.model, cfg.seed), make_batch(cfg))


def test_what_the_format_refuses():
    from paper_2602_18447_b200 import binding as B
    cfg = _tiny("cfg1_tiny", batch=2, ctx_dist=("fixed", 40), step_dist=("fixed", 33))      # 33 query rows: too long
    w = model_weights(cfg.model, cfg.seed)
    batch = make_batch(cfg)
    ses = P.build_session(cfg, w, batch)
    try:
        B.cs_take_launch_count()
        with pytest.raises(B.ConfSpecError) as e:
            ses.verify()
        assert e.value.status == B.CS_EINVAL
        with pytest.raises(B.ConfSpecError) as e:
            B.cs_prefill(ses.model, ses.kv, np.array([0], np.int32), np.arange(3, 8, dtype=np.int32), np.array([5], np.int32))
        assert e.value.status == B.CS_EINVAL
        assert B.cs_take_launch_count() == 0
    finally:
        ses.close()


@pytest.mark.parametrize("fmt", ["e4m3", "e5m2"])
def test_seven_heads_per_group_two_row_tiles(fmt):
    """The 7B shape has 7 query heads per kv head: steps of up to 4 tokens fill two 16-row tiles (28 rows) at head
    dimension 128."""
    cfg = scaled_config("cfg5_7b_b32", n_layers=1, batch=5, vocab=8192)
    cfg = replace(cfg, kv_format=fmt, ctx_dist=("uniform", 100, 700), step_dist=("uniform", 1, 2), suffix_len=2)
    stats, gpu, ref = _run(cfg, P.planted_weights(cfg), make_batch(cfg), planted=True)
    assert stats["logit_err"] < 3e-2
