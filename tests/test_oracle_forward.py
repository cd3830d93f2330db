"""Pins for the oracle's whole forward: invariants that hold for any decoder, and an external library
(the `transformers` Qwen2 architecture, called as a black box on the same weights) that fixes the
conventions the paper inherits from its model families (rotary pairing, GQA head mapping, SwiGLU order,
pre-norm residual wiring, final norm before the LM head)."""
import numpy as np
import pytest

from oracle import confspec_oracle as O
from workloads import ModelShape, VerifyConfig, get_config, make_batch, model_weights, plant_verdict_rows

SMALL = ModelShape("pin-small", 2, 64, 4, 2, 16, 96, 512, 1.0e4)


def _steps(batch):
    return [batch.step_tokens[batch.cu_new[i]:batch.cu_new[i + 1]] for i in range(batch.n_steps)]


def _rand_gains(w, seed):
    g = np.random.default_rng(seed)
    w["final_norm"] = (1.0 + 0.2 * g.standard_normal(w["final_norm"].shape)).astype(np.float32)
    for l in w["layers"]:
        l["norm1"] = (1.0 + 0.2 * g.standard_normal(l["norm1"].shape)).astype(np.float32)
        l["norm2"] = (1.0 + 0.2 * g.standard_normal(l["norm2"].shape)).astype(np.float32)


@pytest.fixture(scope="module")
def small_case():
    w = model_weights(SMALL, seed=11)
    # larger weights than the 0.02 init so that attention and the MLP are far from linear
    g = np.random.default_rng(5)
    from workloads import bf16_bits_from_f32
    for l in w["layers"]:
        for name in ("wq", "wk", "wv", "wo", "wg", "wu", "wd"):
            l[name] = bf16_bits_from_f32((0.25 * g.standard_normal(l[name].shape)).astype(np.float32))
    w["lm_head"] = bf16_bits_from_f32((0.3 * g.standard_normal(w["lm_head"].shape)).astype(np.float32))
    w["embed"] = bf16_bits_from_f32((1.0 * g.standard_normal(w["embed"].shape)).astype(np.float32))
    _rand_gains(w, 6)
    ctx = [g.integers(3, SMALL.vocab, size=c).astype(np.int32) for c in (11, 1, 24)]
    new = [g.integers(3, SMALL.vocab, size=n).astype(np.int32) for n in (5, 9, 1)]
    return w, ctx, new


def test_cache_extend_equals_full_causal_recompute(small_case):
    w, ctx, new = small_case
    kv = O.prefill_context(w, ctx, store_bf16=False)
    ext = O.verify_steps(w, new, [len(c) for c in ctx], lambda i, l: kv[i][l], (1, 2), 0.5)
    full = [np.concatenate([c, n]) for c, n in zip(ctx, new)]
    empty = np.zeros((0, SMALL.n_kv_heads, SMALL.head_dim))
    rec = O.verify_steps(w, full, [0, 0, 0], lambda i, l: (empty, empty), (1, 2), 0.5)
    assert np.max(np.abs(ext["logits"] - rec["logits"])) < 1e-5
    assert np.max(np.abs(ext["logits"] - rec["logits"])) < 1e-10
    assert np.std(rec["logits"]) > 0.5  # not a vacuous comparison


def test_batch_permutation_and_split_invariance(small_case):
    w, ctx, new = small_case
    kv = O.prefill_context(w, ctx, store_bf16=True)
    cl = [len(c) for c in ctx]
    base = O.verify_steps(w, new, cl, lambda i, l: kv[i][l], (1, 2), 0.5)
    perm = [2, 0, 1]
    pr = O.verify_steps(w, [new[p] for p in perm], [cl[p] for p in perm], lambda i, l: kv[perm[i]][l], (1, 2), 0.5)
    assert np.max(np.abs(pr["logits"] - base["logits"][perm])) < 1e-12
    assert np.max(np.abs(pr["conf"] - base["conf"][perm])) < 1e-14
    assert np.array_equal(pr["accept"], base["accept"][perm])
    one = O.verify_steps(w, new[1:2], cl[1:2], lambda i, l: kv[1][l], (1, 2), 0.5)
    # a one-step batch goes through a different BLAS shape in the LM head: equal up to rounding order
    assert np.max(np.abs(one["logits"][0] - base["logits"][1])) < 1e-12


def test_position_shift_invariance_when_cache_is_rerotated(small_case):
    """Rotary attention depends on relative positions only: moving the whole sequence by delta positions
    (cached keys re-rotated by delta, new tokens placed delta later) leaves the logits unchanged."""
    w, ctx, new = small_case
    kv = O.prefill_context(w, ctx, store_bf16=False)
    cl = [len(c) for c in ctx]
    base = O.verify_steps(w, new, cl, lambda i, l: kv[i][l], (1, 2), 0.5)
    delta = 1000

    # ctx_len as seen by the position arithmetic is c + delta; the cache still holds c entries
    def kv_shift(i, l):
        k, v = kv[i][l]
        return O.rope(k, np.full(k.shape[0], delta), SMALL.rope_theta), v
    sh = O.verify_steps(w, new, [c + delta for c in cl], kv_shift, (1, 2), 0.5)
    assert np.max(np.abs(sh["logits"] - base["logits"])) < 1e-4
    assert np.max(np.abs(sh["logits"] - base["logits"])) < 1e-9
    # without re-rotating the cache the answer does change (the test can fail)
    bad = O.verify_steps(w, new, [c + delta for c in cl], lambda i, l: kv[i][l], (1, 2), 0.5)
    assert np.max(np.abs(bad["logits"][0] - base["logits"][0])) > 1e-3


def _library_qwen2(w, m):
    """The `transformers` Qwen2 architecture in float64 with the given weights loaded: a black box."""
    import torch
    import transformers as tr
    cfg = tr.Qwen2Config(vocab_size=m.vocab, hidden_size=m.d_model, intermediate_size=m.d_ffn,
                         num_hidden_layers=m.n_layers, num_attention_heads=m.n_q_heads,
                         num_key_value_heads=m.n_kv_heads, rms_norm_eps=m.rms_eps, rope_theta=m.rope_theta,
                         tie_word_embeddings=False, max_position_embeddings=4096,
                         attn_implementation="eager", use_sliding_window=False)
    assert cfg.rope_parameters["rope_theta"] == m.rope_theta
    assert getattr(cfg, "head_dim", m.head_dim) == m.head_dim
    model = tr.Qwen2ForCausalLM(cfg).double().eval()
    t = lambda bits: torch.from_numpy(O.widen_bf16(bits))
    sd = {"model.embed_tokens.weight": t(w["embed"]), "lm_head.weight": t(w["lm_head"]),
          "model.norm.weight": torch.from_numpy(w["final_norm"].astype(np.float64))}
    names = {"wq": "self_attn.q_proj", "wk": "self_attn.k_proj", "wv": "self_attn.v_proj",
             "wo": "self_attn.o_proj", "wg": "mlp.gate_proj", "wu": "mlp.up_proj", "wd": "mlp.down_proj"}
    for li, l in enumerate(w["layers"]):
        for k, hf in names.items():
            sd[f"model.layers.{li}.{hf}.weight"] = t(l[k])
        for k in ("q_proj", "k_proj", "v_proj"):   # this architecture carries QKV biases; ours has none
            n = m.q_dim if k == "q_proj" else m.kv_dim
            sd[f"model.layers.{li}.self_attn.{k}.bias"] = torch.zeros(n, dtype=torch.float64)
        sd[f"model.layers.{li}.input_layernorm.weight"] = torch.from_numpy(l["norm1"].astype(np.float64))
        sd[f"model.layers.{li}.post_attention_layernorm.weight"] = torch.from_numpy(l["norm2"].astype(np.float64))
    missing, unexpected = model.load_state_dict(sd, strict=False)
    assert not unexpected and all("rotary" in k or "inv_freq" in k for k in missing), (missing, unexpected)
    return model


def test_two_layers_of_the_1p5b_shape_against_transformers_qwen2():
    """The oracle at the widths of the benchmarked model - d_model 1536, 12 query heads on 2 kv heads (6 per group),
    head_dim 128, d_ffn 8960, rotary base 1e6 - against the library, on two layers and a reduced vocabulary: a head
    mapping or rotary pairing that only holds for the small pin shape (head_dim 16, 2 heads per group) would show."""
    torch = pytest.importorskip("torch")
    pytest.importorskip("transformers")
    from workloads import bf16_bits_from_f32
    m = ModelShape("pin-1p5b-2l", 2, 1536, 12, 2, 128, 8960, 2048, 1.0e6)
    w = model_weights(m, seed=31)
    g = np.random.default_rng(32)
    for l in w["layers"]:      # weights large enough that attention and the MLP are far from linear
        for name in ("wq", "wk", "wv", "wo", "wg", "wu", "wd"):
            std = 1.5 / np.sqrt(l[name].shape[1])
            l[name] = bf16_bits_from_f32((std * g.standard_normal(l[name].shape)).astype(np.float32))
    w["lm_head"] = bf16_bits_from_f32((0.05 * g.standard_normal(w["lm_head"].shape)).astype(np.float32))
    w["embed"] = bf16_bits_from_f32(g.standard_normal(w["embed"].shape).astype(np.float32))
    _rand_gains(w, 33)
    ctx = [g.integers(3, m.vocab, size=c).astype(np.int32) for c in (37, 150)]
    new = [g.integers(3, m.vocab, size=n).astype(np.int32) for n in (9, 20)]
    model = _library_qwen2(w, m)
    kv = O.prefill_context(w, ctx, store_bf16=False)
    ours = O.verify_steps(w, new, [len(c) for c in ctx], lambda i, l: kv[i][l], (1, 2), 0.5)
    for i in range(len(ctx)):
        ids = torch.from_numpy(np.concatenate([ctx[i], new[i]]).astype(np.int64))[None]
        with torch.no_grad():
            ref = model(input_ids=ids).logits[0, -1].numpy()
        assert np.max(np.abs(ref - ours["logits"][i])) < 2e-5      # fp32 rotary tables inside the library
        p = torch.softmax(torch.from_numpy(ref), -1).numpy()
        assert abs(max(p[1], p[2]) - ours["conf"][i]) < 1e-6
    assert np.std(ours["logits"]) > 0.5


def test_whole_forward_against_transformers_qwen2(small_case):
    torch = pytest.importorskip("torch")
    pytest.importorskip("transformers")
    w, ctx, new = small_case
    m = SMALL
    model = _library_qwen2(w, m)

    kv = O.prefill_context(w, ctx, store_bf16=False)
    ours = O.verify_steps(w, new, [len(c) for c in ctx], lambda i, l: kv[i][l], (1, 2), 0.5)
    for i in range(len(ctx)):
        ids = torch.from_numpy(np.concatenate([ctx[i], new[i]]).astype(np.int64))[None]
        with torch.no_grad():
            ref = model(input_ids=ids).logits[0, -1].numpy()
        # the library keeps its rotary cos/sin tables in fp32 even for a float64 model, hence 1e-5 not 1e-12;
        # a wrong convention anywhere moves logits of std ~2 by O(1)
        assert np.max(np.abs(ref - ours["logits"][i])) < 1e-5
        # confidence from the library's own softmax
        p = torch.softmax(torch.from_numpy(ref), -1).numpy()
        assert abs(max(p[1], p[2]) - ours["conf"][i]) < 1e-6
    assert np.std(ours["logits"]) > 0.5


def test_tiny_config_runs_and_planted_rows_spread_the_confidence():
    cfg = get_config("cfg1_tiny")
    w = model_weights(cfg.model, cfg.seed)
    b = make_batch(cfg)
    kv = O.prefill_context(w, b.ctx_tokens, store_bf16=True)
    r = O.verify_steps(w, _steps(b), b.ctx_lens, lambda i, l: kv[i][l], cfg.verdict_ids, cfg.tau)
    # random-init weights: every probability is about 1/V, everything escalates
    assert np.all(r["conf"] < 5.0 / cfg.model.vocab) and r["accept"].tolist() == [0] * cfg.batch
    assert np.all(np.abs(np.exp(O.log_softmax_full_vocab(r["logits"])).sum(-1) - 1.0) < 1e-6)
    plant_verdict_rows(w, cfg.verdict_ids, beta=float(np.log(cfg.model.vocab) + 0.5), seed=cfg.seed)
    big = get_config("cfg1_tiny")
    from dataclasses import replace
    big = replace(big, batch=48)
    bb = make_batch(big)
    kv = O.prefill_context(w, bb.ctx_tokens, store_bf16=True)
    r = O.verify_steps(w, _steps(bb), bb.ctx_lens, lambda i, l: kv[i][l], cfg.verdict_ids, cfg.tau)
    assert r["conf"].min() < 0.3 and r["conf"].max() > 0.9      # both sides of the thresholds in use
    assert 0 < r["accept"].sum() < big.batch
    assert set(r["verdict"].tolist()) == {0, 1}


def test_whole_forward_with_qk_norm_against_transformers_qwen3(small_case):
    """The second model family normalises every head's query and key vector before the rotary turn; the library's
    Qwen3 architecture, as a black box on the same weights, fixes where that norm sits and what it is taken over."""
    torch = pytest.importorskip("torch")
    tr = pytest.importorskip("transformers")
    w0, ctx, new = small_case
    m = SMALL
    g = np.random.default_rng(21)
    w = dict(w0, layers=[dict(l, q_norm=(1.0 + 0.3 * g.standard_normal(m.head_dim)).astype(np.float32),
                              k_norm=(1.0 + 0.3 * g.standard_normal(m.head_dim)).astype(np.float32))
                         for l in w0["layers"]])
    cfg = tr.Qwen3Config(vocab_size=m.vocab, hidden_size=m.d_model, intermediate_size=m.d_ffn,
                         num_hidden_layers=m.n_layers, num_attention_heads=m.n_q_heads,
                         num_key_value_heads=m.n_kv_heads, head_dim=m.head_dim, rms_norm_eps=m.rms_eps,
                         rope_theta=m.rope_theta, tie_word_embeddings=False, max_position_embeddings=4096,
                         attn_implementation="eager", use_sliding_window=False, attention_bias=False)
    assert cfg.rope_parameters["rope_theta"] == m.rope_theta
    model = tr.Qwen3ForCausalLM(cfg).double().eval()
    t = lambda bits: torch.from_numpy(O.widen_bf16(bits))
    f = lambda a: torch.from_numpy(np.asarray(a, dtype=np.float64))
    sd = {"model.embed_tokens.weight": t(w["embed"]), "lm_head.weight": t(w["lm_head"]),
          "model.norm.weight": f(w["final_norm"])}
    names = {"wq": "self_attn.q_proj", "wk": "self_attn.k_proj", "wv": "self_attn.v_proj",
             "wo": "self_attn.o_proj", "wg": "mlp.gate_proj", "wu": "mlp.up_proj", "wd": "mlp.down_proj"}
    for li, l in enumerate(w["layers"]):
        for k, hf in names.items():
            sd[f"model.layers.{li}.{hf}.weight"] = t(l[k])
        sd[f"model.layers.{li}.self_attn.q_norm.weight"] = f(l["q_norm"])
        sd[f"model.layers.{li}.self_attn.k_norm.weight"] = f(l["k_norm"])
        sd[f"model.layers.{li}.input_layernorm.weight"] = f(l["norm1"])
        sd[f"model.layers.{li}.post_attention_layernorm.weight"] = f(l["norm2"])
    missing, unexpected = model.load_state_dict(sd, strict=False)
    assert not unexpected and all("rotary" in k or "inv_freq" in k for k in missing), (missing, unexpected)
    kv = O.prefill_context(w, ctx, store_bf16=False)
    ours = O.verify_steps(w, new, [len(c) for c in ctx], lambda i, l: kv[i][l], (1, 2), 0.5)
    kv0 = O.prefill_context(w0, ctx, store_bf16=False)
    plain = O.verify_steps(w0, new, [len(c) for c in ctx], lambda i, l: kv0[i][l], (1, 2), 0.5)
    for i in range(len(ctx)):
        ids = torch.from_numpy(np.concatenate([ctx[i], new[i]]).astype(np.int64))[None]
        with torch.no_grad():
            ref = model(input_ids=ids).logits[0, -1].numpy()
        assert np.max(np.abs(ref - ours["logits"][i])) < 1e-5
    # the norm is not a no-op on this case
    assert np.max(np.abs(plain["logits"] - ours["logits"])) > 0.1
