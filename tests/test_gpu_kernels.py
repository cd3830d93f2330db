"""Single-kernel parity: each CUDA kernel that has a C entry point of its own is compared, element by
element, with the oracle's corresponding block on the same seeded inputs. Sizes span several tiles, ragged
tails in every dimension and the degenerate one-row case."""
import numpy as np
import pytest

from oracle import confspec_oracle as O

pytestmark = pytest.mark.gpu


def _f16_randn(g, shape, std):
    return (std * g.standard_normal(shape)).astype(np.float16)


def _to_dev(a):
    import torch
    return torch.from_numpy(a).cuda()


GEMM_SHAPES = [
    # M, N, K
    (160, 768, 256),      # tiny-config QKV
    (1, 256, 256),        # one row
    (129, 264, 200),      # every dimension ragged (N, K multiples of 8 only)
    (300, 1536, 1536),    # O projection, 1.5B shape
    (1088, 2048, 1536),   # QKV, 1.5B shape, 8.5 row tiles
    (200, 1536, 8960),    # down projection K
]


@pytest.mark.parametrize("M,N,K", GEMM_SHAPES)
@pytest.mark.parametrize("epilogue", [0, 1, 2, 3])
def test_gemm_matches_oracle_matmul(M, N, K, epilogue):
    import torch
    from paper_2602_18447_b200 import binding as B
    g = np.random.default_rng(1000 + M + N + K + epilogue)
    a = _f16_randn(g, (M, K), 1.0)
    w = _f16_randn(g, (N, K), 0.05)
    w2 = _f16_randn(g, (N, K), 0.05)
    af, wf, w2f = a.astype(np.float64), w.astype(np.float64), w2.astype(np.float64)
    da, dw, dw2 = _to_dev(a), _to_dev(w), _to_dev(w2)
    if epilogue in (1, 3):      # x += a w^T, pieces of a split k range added in a fixed order (1) or as they finish (3)
        x0 = g.standard_normal((M, N)).astype(np.float32)
        out = torch.from_numpy(x0.copy()).cuda()
        want = x0.astype(np.float64) + af @ wf.T
    else:
        out = torch.full((M, N), -777.0, dtype=torch.float16, device="cuda")
        want = af @ wf.T if epilogue == 0 else O.silu(af @ wf.T) * (af @ w2f.T)
    B.cs_gemm_f16(da, dw, dw2 if epilogue == 2 else None, out, M, N, K, epilogue)
    torch.cuda.synchronize()
    got = out.float().cpu().numpy().astype(np.float64)
    scale = float(np.abs(want).max())
    # fp32 accumulation of exact fp16 products, then one rounding to the output type
    tol = (2.0 ** -11) * np.abs(want) + 2e-5 * scale * (1 + K / 1024) if epilogue not in (1, 3) else 3e-5 * scale * (1 + K / 1024)
    bad = np.abs(got - want) > tol
    assert not bad.any(), (int(bad.sum()), float(np.abs(got - want).max()), scale)


@pytest.mark.parametrize("M,N,K", [(1163, 1536, 8960), (16, 1536, 8960), (2038, 3584, 3584), (1163, 1536, 1536), (300, 264, 4104),
                                   (735, 1536, 8960), (64, 256, 16384), (129, 520, 2056), (1, 1536, 8960)])
def test_residual_gemm_is_bit_identical_from_run_to_run(M, N, K):
    """Long k ranges are cut over the SMs and several CTAs add pieces into the same elements of x; with the fixed order
    of those additions ten runs on the same inputs give the same bits, also with other work on the GPU in between."""
    import torch
    from paper_2602_18447_b200 import binding as B
    g = np.random.default_rng(M + N + K)
    da, dw = _to_dev(_f16_randn(g, (M, K), 1.0)), _to_dev(_f16_randn(g, (N, K), 0.05))
    x0 = torch.from_numpy(g.standard_normal((M, N)).astype(np.float32)).cuda()
    other = torch.randn(4096, 4096, device="cuda")
    runs = []
    for r in range(10):
        out = x0.clone()
        if r % 3 == 1:
            other @ other            # disturbs which CTAs start first
        B.cs_gemm_f16(da, dw, None, out, M, N, K, 1)
        torch.cuda.synchronize()
        runs.append(out.cpu().numpy().view(np.uint32))
    for r in runs[1:]:
        assert np.array_equal(r, runs[0])
    # ... and it is the right sum (several pieces per tile, each added exactly once)
    want = x0.cpu().numpy().astype(np.float64) + da.float().cpu().numpy().astype(np.float64) @ dw.float().cpu().numpy().astype(np.float64).T
    got = runs[0].view(np.float32).astype(np.float64)
    assert np.max(np.abs(got - want)) <= 3e-5 * float(np.abs(want).max()) * (1 + K / 1024)


@pytest.mark.parametrize("rows,d", [(1, 256), (37, 1536), (1088, 1536), (70, 3584)])
def test_rmsnorm_matches_oracle(rows, d):
    import torch
    from paper_2602_18447_b200 import binding as B
    g = np.random.default_rng(rows * 7 + d)
    x = (g.standard_normal((rows, d)) * g.uniform(0.01, 30.0, size=(rows, 1))).astype(np.float32)
    gain = (1.0 + 0.2 * g.standard_normal(d)).astype(np.float32)
    out = torch.empty((rows, d), dtype=torch.float16, device="cuda")
    B.cs_rmsnorm(torch.from_numpy(x).cuda(), torch.from_numpy(gain).cuda(), out, rows, d, 1e-6)
    torch.cuda.synchronize()
    want = O.rmsnorm(x.astype(np.float64), gain.astype(np.float64), 1e-6)
    got = out.float().cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got - want) <= (2.0 ** -11) * np.abs(want) + 1e-6)


def test_escalate_mask_matches_oracle_bit_exact():
    import torch
    from paper_2602_18447_b200 import binding as B
    g = np.random.default_rng(5)
    for n in (1, 31, 64, 1000, 5000):
        conf = g.uniform(0, 1, size=n).astype(np.float32)
        conf[::7] = np.float32(0.9)          # exactly on the threshold: trusted
        if n > 3:
            conf[3] = np.nan                 # never trusted
        dconf = torch.from_numpy(conf).cuda()
        for tau in (0.0, 0.5, 0.9, 1.0001):
            acc = torch.zeros(n, dtype=torch.uint8, device="cuda")
            idx = torch.full((n,), -1, dtype=torch.int32, device="cuda")
            cnt = torch.zeros(1, dtype=torch.int32, device="cuda")
            B.cs_escalate_mask(dconf, tau, acc, idx, cnt)
            torch.cuda.synchronize()
            want_acc, want_idx, want_cnt = O.escalate_list(conf, tau)
            assert int(cnt.item()) == want_cnt
            assert np.array_equal(acc.cpu().numpy(), want_acc)
            assert np.array_equal(idx.cpu().numpy()[:want_cnt], want_idx)
            assert np.all(idx.cpu().numpy()[want_cnt:] == -1)


@pytest.mark.parametrize("B,d,vocab", [(1, 256, 4096), (16, 1536, 151936), (33, 1536, 20488), (64, 3584, 30000),
                                       (100, 256, 4100)])
def test_lm_head_gate_matches_oracle(B, d, vocab):
    """Logits of B hidden states against the whole vocabulary, fused logsumexp, confidence and gate. Two LM-head rows
    are planted so that confidences land on both sides of the threshold; the vocabulary has a ragged last tile."""
    import torch
    from paper_2602_18447_b200 import binding as Bd
    g = np.random.default_rng(B * 31 + d + vocab)
    w = _f16_randn(g, (vocab, d), 0.02)
    h = _f16_randn(g, (B, d), 1.0)
    vids = [1, vocab - 1, 7]
    u = g.standard_normal(d)
    u /= np.linalg.norm(u)
    beta = np.log(vocab) + 0.5
    w[vids[0]] = (beta * u).astype(np.float16)      # h has unit-variance entries, so u.h ~ N(0, 1)
    w[vids[1]] = (-beta * u).astype(np.float16)
    z = h.astype(np.float64) @ w.astype(np.float64).T
    conf, verdict, lse = O.verdict_confidence(z, vids)
    out_conf = torch.empty(B, dtype=torch.float32, device="cuda")
    out_acc = torch.empty(B, dtype=torch.uint8, device="cuda")
    out_v = torch.empty(B, dtype=torch.int32, device="cuda")
    out_lse = torch.empty(B, dtype=torch.float32, device="cuda")
    for tau in (0.3, 0.9):
        Bd.cs_lm_head_gate(_to_dev(w), _to_dev(h), vids, tau, out_conf, out_acc, out_v, out_lse)
        torch.cuda.synchronize()
        got = out_conf.cpu().numpy().astype(np.float64)
        # fp32 accumulation of exact fp16 products, exponentials in fp32
        assert np.max(np.abs(out_lse.cpu().numpy() - lse)) < 2e-4
        assert np.max(np.abs(got - conf)) < 2e-4 * np.maximum(conf, 1e-3).max()
        sure = np.abs(conf - tau) > 1e-3
        assert np.array_equal(out_acc.cpu().numpy()[sure], O.gate(conf, tau)[sure])
        pv = np.sort(np.exp(z[:, vids] - lse[:, None]), axis=1)
        clear = (pv[:, -1] - pv[:, -2]) > 1e-4
        assert np.array_equal(out_v.cpu().numpy()[clear], verdict[clear])
    if B > 4:
        assert 0 < (conf >= 0.3).sum() < B


def test_cascade_select_matches_oracle_bit_exact():
    """Algorithm 1's accept-prefix length and Eq. 5's choice per request, on random iterations: requests of 0 to 70
    steps (more than one warp's worth), ties in the confidence, NaN confidences, with and without target results."""
    import torch
    from paper_2602_18447_b200 import binding as B
    g = np.random.default_rng(77)
    for trial in range(6):
        sizes = g.integers(0, 12, size=40).tolist() + [70, 33, 1, 0, 32]
        offs = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
        n = int(offs[-1])
        trusted = (g.uniform(size=n) < 0.6).astype(np.uint8)
        vd = (g.uniform(size=n) < 0.25).astype(np.int32)
        vt = (g.uniform(size=n) < 0.4).astype(np.int32)
        cd = np.round(g.uniform(0.5, 1.0, size=n), 1).astype(np.float32)     # coarse grid: many ties
        ct = np.round(g.uniform(0.5, 1.0, size=n), 1).astype(np.float32)
        cd[::17] = np.nan
        with_target = trial % 2 == 0
        want = O.cascade_select(trusted, vd, cd, vt if with_target else None, ct if with_target else None, offs, 0)
        dev = lambda a: torch.from_numpy(a).cuda()
        R = len(sizes)
        m = torch.full((R,), -7, dtype=torch.int32, device="cuda")
        best = torch.full((R,), -7, dtype=torch.int32, device="cuda")
        passed = torch.full((n,), 9, dtype=torch.uint8, device="cuda")
        conf = torch.full((n,), -1.0, dtype=torch.float32, device="cuda")
        B.cs_cascade_select(dev(trusted), dev(vd), dev(cd), dev(vt) if with_target else None,
                            dev(ct) if with_target else None, dev(offs), 0, m, best, passed, conf)
        torch.cuda.synchronize()
        assert np.array_equal(passed.cpu().numpy(), want[0])
        assert np.array_equal(conf.cpu().numpy(), want[1], equal_nan=True)
        assert np.array_equal(m.cpu().numpy(), want[2])
        assert np.array_equal(best.cpu().numpy(), want[3])

