"""Pins for the CPU oracle's building blocks: closed forms, invariants and scalar-loop brute force.

Each check is chosen so that a plausible slip in the oracle (dropped scale, wrong sign in the rotation,
transposed operand, wrong head mapping, off-by-one in the causal mask) fails it.
"""
import math

import numpy as np
import pytest

from oracle import confspec_oracle as O


def _rng(seed):
    return np.random.default_rng(seed)


# ---------------------------------------------------------------- storage formats
def test_widen_bf16_known_patterns():
    bits = np.array([0x3F80, 0xBF80, 0x4000, 0x3F00, 0x0000, 0x3DCC], dtype=np.uint16)
    got = O.widen_bf16(bits)
    assert got.tolist()[:5] == [1.0, -1.0, 2.0, 0.5, 0.0]
    assert got[5] == 0.099609375  # 0x3DCC = 1.59375 * 2^-4


def test_round_to_bf16_ties_to_even():
    # 1 + 2^-8 lies exactly between bf16 neighbours 1.0 and 1 + 2^-7: ties go to the even mantissa (1.0)
    assert O.round_to_bf16(np.array([1.0 + 2.0 ** -8]))[0] == 1.0
    # 1 + 3 * 2^-8 lies between 1 + 2^-7 (odd) and 1 + 2^-6 (even)
    assert O.round_to_bf16(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 1.0 + 2.0 ** -6
    x = _rng(0).standard_normal(1000)
    r = O.round_to_bf16(x)
    assert np.all(np.abs(r - x) <= np.abs(x) * 2.0 ** -8)
    assert np.array_equal(O.round_to_bf16(r), r)


# ---------------------------------------------------------------- RMSNorm / SiLU
def test_rmsnorm_closed_forms():
    d = 64
    x = np.full((1, d), 3.0)
    out = O.rmsnorm(x, np.ones(d), 0.0)
    assert np.allclose(out, 1.0, atol=1e-15)
    g = np.linspace(0.5, 2.0, d)
    assert np.allclose(O.rmsnorm(-7.0 * np.ones((2, d)), g, 0.0), -g[None, :], atol=1e-14)
    # eps enters under the square root, added to the mean square
    assert np.allclose(O.rmsnorm(x, np.ones(d), 7.0), 3.0 / 4.0, atol=1e-15)
    y = _rng(1).standard_normal((5, d))
    out = O.rmsnorm(y, np.ones(d), 0.0)
    assert np.allclose(np.mean(out * out, axis=-1), 1.0, atol=1e-12)
    # scale invariance of the direction
    assert np.allclose(O.rmsnorm(10.0 * y, np.ones(d), 0.0), out, atol=1e-12)


def test_silu_closed_forms():
    assert O.silu(np.array([0.0]))[0] == 0.0
    z = np.array([1.0, -1.0, 20.0, -20.0])
    want = [1 / (1 + math.exp(-1)), -1 / (1 + math.exp(1)), 20 / (1 + math.exp(-20)), -20 / (1 + math.exp(20))]
    assert np.allclose(O.silu(z), want, rtol=1e-14)
    # silu(z) - silu(-z) = z
    t = _rng(2).standard_normal(100)
    assert np.allclose(O.silu(t) - O.silu(-t), t, atol=1e-14)


# ---------------------------------------------------------------- rotary
def test_rope_identity_norm_and_pairing():
    n, h, hd = 6, 3, 16
    y = _rng(3).standard_normal((n, h, hd))
    assert np.array_equal(O.rope(y, np.zeros(n, dtype=np.int64), 1e4), y)
    r = O.rope(y, np.arange(n) * 37 + 5, 1e4)
    assert np.allclose(np.sum(r * r, -1), np.sum(y * y, -1), rtol=1e-13)
    # each (j, j + hd/2) pair keeps its own length: the rotation couples exactly those two slots
    half = hd // 2
    assert np.allclose(r[..., :half] ** 2 + r[..., half:] ** 2, y[..., :half] ** 2 + y[..., half:] ** 2, rtol=1e-12)


def test_rope_explicit_angle():
    # one head, hd = 4, theta = 100: frequencies 1 and 100^(-1/2) = 0.1; position 3
    y = np.array([[[1.0, 2.0, 3.0, 4.0]]])
    r = O.rope(y, np.array([3]), 100.0)[0, 0]
    a0, a1 = 3.0 * 1.0, 3.0 * 0.1
    want = [1 * math.cos(a0) - 3 * math.sin(a0), 2 * math.cos(a1) - 4 * math.sin(a1),
            3 * math.cos(a0) + 1 * math.sin(a0), 4 * math.cos(a1) + 2 * math.sin(a1)]
    assert np.allclose(r, want, rtol=1e-14)


def test_rope_scores_depend_on_relative_position_only():
    hd = 32
    g = _rng(4)
    q, k = g.standard_normal((1, 1, hd)), g.standard_normal((1, 1, hd))
    def score(pq, pk):
        return float(np.sum(O.rope(q, np.array([pq]), 1e4) * O.rope(k, np.array([pk]), 1e4)))
    assert abs(score(10, 3) - score(110, 103)) < 1e-12
    assert abs(score(10, 3) - score(3, 10)) > 1e-3  # direction matters


# ---------------------------------------------------------------- attention
def _attention_scalar_loops(q, k_ctx, v_ctx, k_new, v_new):
    """Brute force with python floats: for each query, loop over each visible key."""
    n, hq, hd = q.shape
    c = k_ctx.shape[0]
    hkv = k_new.shape[1]
    grp = hq // hkv
    out = np.zeros_like(q)
    for p in range(n):
        for h in range(hq):
            kh = h // grp
            ks = [k_ctx[t, kh] for t in range(c)] + [k_new[t, kh] for t in range(p + 1)]
            vs = [v_ctx[t, kh] for t in range(c)] + [v_new[t, kh] for t in range(p + 1)]
            sc = [sum(float(q[p, h, j]) * float(kk[j]) for j in range(hd)) / math.sqrt(hd) for kk in ks]
            mx = max(sc)
            w = [math.exp(s - mx) for s in sc]
            z = sum(w)
            for j in range(hd):
                out[p, h, j] = sum(w[t] * float(vs[t][j]) for t in range(len(vs))) / z
    return out


@pytest.mark.parametrize("c,n,hq,hkv", [(0, 1, 2, 2), (5, 3, 4, 2), (3, 6, 6, 2), (7, 1, 3, 1), (0, 5, 2, 1)])
def test_attention_matches_scalar_brute_force(c, n, hq, hkv):
    hd = 8
    g = _rng(100 + c * 7 + n)
    q = g.standard_normal((n, hq, hd))
    kc, vc = g.standard_normal((c, hkv, hd)), g.standard_normal((c, hkv, hd))
    kn, vn = g.standard_normal((n, hkv, hd)), g.standard_normal((n, hkv, hd))
    got = O.attention_extend(q, kc, vc, kn, vn)
    want = _attention_scalar_loops(q, kc, vc, kn, vn)
    assert np.allclose(got, want, atol=1e-13)


def test_attention_degenerate_cases():
    hd = 16
    g = _rng(5)
    # a single new token with no context attends only to itself: output is its own value
    q, k, v = g.standard_normal((1, 2, hd)), g.standard_normal((1, 2, hd)), g.standard_normal((1, 2, hd))
    e = np.zeros((0, 2, hd))
    assert np.allclose(O.attention_extend(q, e, e, k, v), v, atol=1e-15)
    # all keys identical: uniform weights, output of position p = mean of the values it can see
    c, n = 4, 3
    kc = np.tile(g.standard_normal((1, 1, hd)), (c, 1, 1))
    kn = np.tile(kc[:1], (n, 1, 1))
    vc, vn = g.standard_normal((c, 1, hd)), g.standard_normal((n, 1, hd))
    q = g.standard_normal((n, 2, hd))
    out = O.attention_extend(q, kc, vc, kn, vn)
    allv = np.concatenate([vc, vn], 0)[:, 0]
    for p in range(n):
        assert np.allclose(out[p, 0], allv[:c + p + 1].mean(0), atol=1e-14)
        assert np.allclose(out[p, 1], allv[:c + p + 1].mean(0), atol=1e-14)
    # the first new token never sees later new tokens: perturbing them changes nothing for it
    vn2 = vn.copy(); vn2[1:] += 5.0
    kn2 = kn.copy(); kn2[1:] -= 3.0
    out2 = O.attention_extend(q, kc, vc, kn2, vn2)
    assert np.array_equal(out2[0], out[0])


def test_gqa_equals_mha_with_repeated_heads():
    g = _rng(6)
    c, n, hq, hkv, hd = 9, 4, 6, 2, 8
    q = g.standard_normal((n, hq, hd))
    kc, vc = g.standard_normal((c, hkv, hd)), g.standard_normal((c, hkv, hd))
    kn, vn = g.standard_normal((n, hkv, hd)), g.standard_normal((n, hkv, hd))
    rep = lambda a: np.repeat(a, hq // hkv, axis=1)  # head h of the MHA copy = kv head h // group
    a = O.attention_extend(q, kc, vc, kn, vn)
    b = O.attention_extend(q, rep(kc), rep(vc), rep(kn), rep(vn))
    assert np.allclose(a, b, atol=1e-15)


# ---------------------------------------------------------------- confidence and gate
def test_softmax_sums_to_one_and_uniform_case():
    g = _rng(7)
    z = g.standard_normal((5, 4096)) * 3.0
    p = np.exp(O.log_softmax_full_vocab(z))
    assert np.all(np.abs(p.sum(-1) - 1.0) < 1e-6)
    assert np.all(np.abs(p.sum(-1) - 1.0) < 1e-12)
    # zero LM head: every token equally likely, confidence exactly 1/V
    conf, verdict, lse = O.verdict_confidence(np.zeros((3, 4096)), (1, 2))
    assert np.allclose(conf, 1.0 / 4096, rtol=1e-14)
    assert np.allclose(lse, math.log(4096), rtol=1e-14)
    assert verdict.tolist() == [0, 0, 0]  # tie -> earliest verdict id
    # shifting all logits by a constant changes nothing
    c1, v1, _ = O.verdict_confidence(z, (1, 2))
    c2, v2, _ = O.verdict_confidence(z + 1000.0, (1, 2))
    assert np.allclose(c1, c2, rtol=1e-9) and np.array_equal(v1, v2)


def test_confidence_picks_best_verdict_token_under_full_vocab_softmax():
    V = 50
    z = np.zeros((2, V))
    z[0, 1], z[0, 2], z[0, 7] = 2.0, 3.0, 4.0      # token 7 is not a verdict token: it only dilutes
    z[1, 1], z[1, 2] = 50.0, -50.0
    conf, verdict, lse = O.verdict_confidence(z, (1, 2))
    denom0 = (V - 3) + math.exp(2) + math.exp(3) + math.exp(4)
    assert abs(conf[0] - math.exp(3) / denom0) < 1e-15
    assert verdict[0] == 1
    assert verdict[1] == 0 and 1.0 - conf[1] < 1e-19 + 60 * math.exp(-50)
    assert abs(lse[0] - math.log(denom0)) < 1e-14
    # two-token renormalisation would give e^3/(e^2+e^3) = 0.731...; make sure that is NOT what we compute
    assert abs(conf[0] - math.exp(3) / (math.exp(2) + math.exp(3))) > 0.3


def test_gate_rule_endpoints_boundary_and_monotonicity():
    conf = np.array([0.0, 1e-6, 0.3, 0.8999999, 0.9, 0.95, 1.0, np.nan])
    # gamma = 0: the draft verifier is always trusted (Table 3, "Draft Verification")
    assert O.gate(conf[:-1], 0.0).tolist() == [1] * 7
    # gamma > 1: everything is escalated (Table 3, "Target Verification")
    assert O.gate(conf, 1.0001).tolist() == [0] * 8
    # Eq. 4 uses >=: a confidence equal to the threshold (in fp32) is trusted
    assert O.gate(np.array([np.float32(0.9)]), 0.9).tolist() == [1]
    assert O.gate(np.array([np.nextafter(np.float32(0.9), np.float32(0))]), 0.9).tolist() == [0]
    assert O.gate(conf, 0.9).tolist() == [0, 0, 0, 0, 1, 1, 1, 0]   # NaN escalates
    prev = None
    for tau in np.linspace(0, 1.01, 60):
        a = O.gate(conf[:-1], float(tau))
        if prev is not None:
            assert np.all(a <= prev)  # raising the threshold never un-escalates a step
        prev = a


def test_escalate_list_is_complement_in_order():
    conf = np.array([0.95, 0.2, 0.91, 0.5, 0.1])
    acc, idx, cnt = O.escalate_list(conf, 0.9)
    assert acc.tolist() == [1, 0, 1, 0, 0] and idx.tolist() == [1, 3, 4] and cnt == 3
    acc, idx, cnt = O.escalate_list(conf, 0.0)
    assert cnt == 0 and idx.shape == (0,)


def test_cascade_select_hand_worked_iterations():
    """Algorithm 1's sequential accept loop and Eq. 5's choice, against cases worked by hand."""
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "cascade_cases.txt")
    rows = [l for l in open(path) if l.strip() and not l.startswith("#")]
    assert len(rows) >= 8
    trusted, vd, cd, vt, ct, offs, want_m, want_best = [], [], [], [], [], [0], [], []
    for line in rows:
        steps, exp = line.split("|")
        for tok in steps.split():
            t, dec, p = tok[0] == "T", 0 if tok[1] == "a" else 1, float(tok[2:])
            trusted.append(1 if t else 0)
            # the verifier that does not count says the opposite with another confidence: it must be ignored
            vd.append(dec if t else 1 - dec); cd.append(p if t else 0.123)
            vt.append(dec if not t else 1 - dec); ct.append(p if not t else 0.999)
        m, best = exp.split()
        want_m.append(int(m))
        want_best.append(-1 if int(best) < 0 else offs[-1] + int(best))
        offs.append(len(trusted))
    passed, conf, m, best = O.cascade_select(trusted, vd, cd, vt, ct, offs, accept_index=0)
    assert m.tolist() == want_m and best.tolist() == want_best
    # invariants: m never exceeds the request's length; all accepted -> m = length; best is an accepted step
    for r in range(len(want_m)):
        k = offs[r + 1] - offs[r]
        assert 0 <= m[r] <= k and (m[r] == k) == bool(passed[offs[r]:offs[r + 1]].all())
        assert best[r] == -1 or passed[best[r]]
    # without target results every escalated step is a rejection
    p2, _, m2, _ = O.cascade_select(trusted, vd, cd, None, None, offs)
    assert all(p2[i] == 0 for i in range(len(trusted)) if not trusted[i]) and np.all(m2 <= m)


def test_e4m3_decode_against_hand_values_and_a_library():
    """The 8-bit cache format: hand-decoded codes, order, and every code against torch's float8_e4m3fn."""
    hand = {0x00: 0.0, 0x01: 2.0 ** -9, 0x07: 7 * 2.0 ** -9, 0x08: 2.0 ** -6, 0x38: 1.0, 0x3C: 1.5, 0x40: 2.0,
            0x7E: 448.0, 0xB8: -1.0, 0xFE: -448.0, 0x30: 0.5, 0x39: 1.125}
    for code, want in hand.items():
        assert O.widen_e4m3(np.array([code], np.uint8))[0] == want, hex(code)
    assert np.isnan(O.widen_e4m3(np.array([0x7F, 0xFF], np.uint8))).all()
    pos = O.widen_e4m3(np.arange(0x7F, dtype=np.uint8))
    assert np.all(np.diff(pos) > 0)
    torch = pytest.importorskip("torch")
    lib = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    ours = O.widen_e4m3(np.arange(256, dtype=np.uint8))
    assert np.array_equal(np.isnan(lib), np.isnan(ours)) and np.array_equal(lib[~np.isnan(lib)], ours[~np.isnan(ours)])


def test_e5m2_decode_against_hand_values_and_a_library():
    hand = {0x00: 0.0, 0x01: 2.0 ** -16, 0x03: 3 * 2.0 ** -16, 0x04: 2.0 ** -14, 0x3C: 1.0, 0x3D: 1.25, 0x3E: 1.5,
            0x40: 2.0, 0x7B: 57344.0, 0xBC: -1.0, 0x38: 0.5}
    for code, want in hand.items():
        assert O.widen_e5m2(np.array([code], np.uint8))[0] == want, hex(code)
    assert np.isinf(O.widen_e5m2(np.array([0x7C], np.uint8))[0]) and np.isnan(O.widen_e5m2(np.array([0x7D], np.uint8))[0])
    torch = pytest.importorskip("torch")
    lib = torch.arange(256, dtype=torch.uint8).view(torch.float8_e5m2).to(torch.float64).numpy()
    ours = O.widen_e5m2(np.arange(256, dtype=np.uint8))
    assert np.array_equal(np.isnan(lib), np.isnan(ours)) and np.array_equal(lib[~np.isnan(lib)], ours[~np.isnan(ours)])
    # the upper byte of an fp16
    h = (np.arange(256, dtype=np.uint16) << 8).view(np.float16).astype(np.float64)
    ok = ~np.isnan(h)
    assert np.array_equal(h[ok], ours[ok])
