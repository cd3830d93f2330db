"""The entry point for callers that cannot allocate device memory (a serving process whose pool owns the whole GPU,
a loop that must not take the allocator's locks): cs_lm_head_gate_static keeps its scratch in a fixed array inside
the library instead of calling cudaMalloc. Its results must equal those of cs_lm_head_gate, which allocates, on two
calls in a row: the second call finds the first call's leftovers in the shared array. Collected last on purpose, so
that a run that stops at the first failure has already run every other test."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

TOL = 2e-4      # the tolerance the LM-head stage is held to against the oracle


def _case(seed, B, d, vocab):
    g = np.random.default_rng(seed)
    w = (0.02 * g.standard_normal((vocab, d))).astype(np.float16)
    h = g.standard_normal((B, d)).astype(np.float16)
    u = g.standard_normal(d)
    u /= np.linalg.norm(u)
    beta = np.log(vocab) + 0.5
    w[1] = (beta * u).astype(np.float16)          # verdict rows that put confidences on both sides of tau
    w[2] = (-beta * u).astype(np.float16)
    return w, h


def _both(Bd, torch, w, h, tau, check_no_alloc):
    B = h.shape[0]
    dw, dh = torch.from_numpy(w).cuda(), torch.from_numpy(h).cuda()
    outs = []
    for fn in (Bd.cs_lm_head_gate, Bd.cs_lm_head_gate_static):
        conf = torch.full((B,), -1.0, dtype=torch.float32, device="cuda")
        acc = torch.full((B,), 7, dtype=torch.uint8, device="cuda")
        ver = torch.full((B,), -5, dtype=torch.int32, device="cuda")
        lse = torch.full((B,), -1.0, dtype=torch.float32, device="cuda")
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        fn(dw, dh, [1, 2], tau, conf, acc, ver, lse)
        torch.cuda.synchronize()
        if check_no_alloc and fn is Bd.cs_lm_head_gate_static:
            # the driver's own count of free device memory: the call took none (device allocations come in 2 MiB
            # granules; the first call on a device may load the kernel's code, so only a later call is held to this)
            assert free_before - torch.cuda.mem_get_info()[0] < (1 << 20)
        outs.append((conf.cpu().numpy(), acc.cpu().numpy(), ver.cpu().numpy(), lse.cpu().numpy()))
    return outs


def test_static_scratch_entry_matches_the_allocating_one_twice_in_a_row():
    import torch
    from paper_2602_18447_b200 import binding as Bd
    # first a large batch, then a smaller one with other values: stale partial sums or verdict logits would show
    for call, (seed, B, d, vocab, tau) in enumerate(((11, 64, 1536, 20488, 0.5), (12, 5, 1536, 20488, 0.9),
                                                     (14, 64, 1536, 20488, 0.7))):
        w, h = _case(seed, B, d, vocab)
        (c0, a0, v0, l0), (c1, a1, v1, l1) = _both(Bd, torch, w, h, tau, check_no_alloc=call == 2)
        assert np.all(np.isfinite(c1)) and np.all((c1 > 0) & (c1 <= 1))
        assert np.max(np.abs(c1 - c0)) <= TOL and np.max(np.abs(l1 - l0)) <= TOL
        sure = np.abs(c0 - tau) > TOL
        assert np.array_equal(a1[sure], a0[sure]) and np.all((a1 == 0) | (a1 == 1))
        assert np.array_equal(v1, v0)
        if B > 8:
            assert 0 < a0.sum() < B


def test_static_scratch_entry_rejects_batches_beyond_its_capacity():
    import torch
    from paper_2602_18447_b200 import binding as Bd
    w, h = _case(13, 65, 256, 4096)
    conf = torch.empty(65, dtype=torch.float32, device="cuda")
    acc = torch.empty(65, dtype=torch.uint8, device="cuda")
    Bd.cs_take_launch_count()
    with pytest.raises(Bd.ConfSpecError) as e:
        Bd.cs_lm_head_gate_static(torch.from_numpy(w).cuda(), torch.from_numpy(h).cuda(), [1, 2], 0.5, conf, acc)
    assert e.value.status == Bd.CS_ELIMIT and "capacity" in str(e.value)
    assert Bd.cs_take_launch_count() == 0
