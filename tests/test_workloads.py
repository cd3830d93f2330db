"""Host-side checks of the seeded input generators and of the golden gate cases."""
import os

import numpy as np
import pytest

from oracle import confspec_oracle as O
from workloads import CONFIGS, context_kv, get_config, make_batch, model_weights, page_assignment, scaled_config


def test_gate_golden_cases():
    path = os.path.join(os.path.dirname(__file__), "golden", "gate_cases.txt")
    rows = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    assert len(rows) >= 10
    for conf, tau, want in rows:
        assert O.gate(np.array([float(conf)]), float(tau)).tolist() == [int(want)], (conf, tau)


def test_batches_follow_the_config_recipes():
    for name, cfg in CONFIGS.items():
        b = make_batch(cfg)
        assert b.n_steps == cfg.batch and b.cu_new[-1] == b.step_lens.sum() == b.step_tokens.shape[0]
        body = b.step_lens - cfg.suffix_len
        if cfg.step_dist[0] == "uniform":
            assert body.min() >= cfg.step_dist[1] and body.max() <= cfg.step_dist[2]
        if cfg.ctx_dist[0] == "uniform":
            assert b.ctx_lens.min() >= cfg.ctx_dist[1] and b.ctx_lens.max() <= cfg.ctx_dist[2]
        if cfg.ctx_dist[0] == "lognormal":
            assert b.ctx_lens.min() >= cfg.ctx_dist[3] and b.ctx_lens.max() <= cfg.ctx_dist[4]
        assert b.step_tokens.min() >= 3 and b.step_tokens.max() < cfg.model.vocab
        for i in range(b.n_steps):   # every step ends with the shared verify suffix
            assert np.array_equal(b.step_tokens[b.cu_new[i + 1] - cfg.suffix_len:b.cu_new[i + 1]], b.suffix)
        b2 = make_batch(cfg)
        assert np.array_equal(b.step_tokens, b2.step_tokens) and np.array_equal(b.ctx_lens, b2.ctx_lens)


def test_weights_are_seeded_bf16_normals():
    cfg = get_config("cfg1_tiny")
    w1, w2 = model_weights(cfg.model, 5, threads=1), model_weights(cfg.model, 5, threads=4)
    assert np.array_equal(w1["layers"][1]["wd"], w2["layers"][1]["wd"])
    assert np.array_equal(w1["lm_head"], w2["lm_head"])
    assert not np.array_equal(w1["lm_head"], w1["embed"])           # untied
    x = O.widen_bf16(w1["lm_head"])
    assert abs(x.std() - 0.02) < 5e-4 and abs(x.mean()) < 2e-4
    assert w1["layers"][0]["wq"].shape == (256, 256) and w1["layers"][0]["wg"].shape == (688, 256)
    assert np.all(w1["final_norm"] == 1.0)


def test_context_kv_and_pages():
    cfg = scaled_config("cfg2_1p5b_b16", n_layers=2, batch=3)
    b = make_batch(cfg)
    k, v = context_kv(cfg, 1, 0, int(b.ctx_lens[1]))
    assert k.shape == (b.ctx_lens[1], 2, 128) and k.dtype == np.uint16
    k2, _ = context_kv(cfg, 1, 0, int(b.ctx_lens[1]))
    assert np.array_equal(k, k2)
    assert abs(O.widen_bf16(k).std() - cfg.kv_std) < 0.01
    total, pages = page_assignment(cfg, b.ctx_lens)
    allp = np.concatenate(pages)
    assert len(set(allp.tolist())) == allp.shape[0] and allp.max() < total
    assert [len(p) for p in pages] == [(int(c) + 15) // 16 for c in b.ctx_lens]
    assert not np.array_equal(pages[0], np.sort(pages[0]))          # scattered, not contiguous


def test_e4m3_encoding_rounds_to_nearest_even_and_saturates():
    from workloads import e4m3_codes_from_f32
    torch = pytest.importorskip("torch")
    g = np.random.default_rng(0)
    x = np.concatenate([g.standard_normal(20000) * 0.78, g.standard_normal(2000) * 100, [0.0, -0.0, 448.0, 449.0, -1e9,
                        2.0 ** -10, 3 * 2.0 ** -10, 1.0625, 1.1875, 2.0 ** -9, 1e-12]]).astype(np.float32)
    ours = e4m3_codes_from_f32(x)
    lib = torch.from_numpy(x).clamp(-448, 448).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    same = ours == lib
    zero = (ours & 0x7F) == 0                      # the sign of a zero result is storage detail
    assert np.all(same | (zero & ((lib & 0x7F) == 0)))
    # ties go to the even code: 1.0625 is halfway between 1.0 (0x38) and 1.125 (0x39); 1.1875 between 0x39 and 0x3A
    assert e4m3_codes_from_f32(np.array([1.0625, 1.1875, 449.0, 1e9], np.float32)).tolist() == [0x38, 0x3A, 0x7E, 0x7E]


def test_e5m2_encoding_rounds_to_nearest_even_and_saturates():
    from workloads import e5m2_codes_from_f32
    torch = pytest.importorskip("torch")
    g = np.random.default_rng(1)
    x = np.concatenate([g.standard_normal(20000) * 0.78, g.standard_normal(2000) * 1000, [0.0, -0.0, 57344.0, 60000.0,
                        -1e9, 2.0 ** -17, 3 * 2.0 ** -17, 1.125, 1.375, 2.0 ** -16, 1e-12]]).astype(np.float32)
    ours = e5m2_codes_from_f32(x)
    lib = torch.from_numpy(x).clamp(-57344, 57344).to(torch.float8_e5m2).view(torch.uint8).numpy()
    zero = (ours & 0x7F) == 0
    assert np.all((ours == lib) | (zero & ((lib & 0x7F) == 0)))
    # ties to the even code: 1.125 is halfway between 1.0 (0x3C) and 1.25 (0x3D); 1.375 between 0x3D and 0x3E
    assert e5m2_codes_from_f32(np.array([1.125, 1.375, 60000.0, 1e9], np.float32)).tolist() == [0x3C, 0x3E, 0x7B, 0x7B]


def test_sample_of_a_full_size_batch_has_both_sides_of_the_threshold():
    """Host logic of the full-size parity tests: which steps the oracle recomputes."""
    import parity_common as P
    conf = np.array([0.05, 0.93, 0.999, 0.87, 0.5, 0.91, 0.2, 0.97, 0.895, 0.0001])
    s = P.sample_both_sides(conf, 0.9, 0.02, 6, always=(4,))
    assert len(s) == 6 and s == sorted(s) and 4 in s
    assert 1 in s and 3 in s            # the trusted and the escalated step closest to the band come first
    assert 2 in s and 9 in s            # then the extremes
    assert 8 not in s and 5 not in s    # inside the band around tau: never picked
    assert P.sample_both_sides(np.full(4, 1e-5), 0.9, 0.02, 3) == [0, 1, 2]    # one-sided batches still give a sample
