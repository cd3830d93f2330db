"""Property tests of the oracle's decision stage (Section 4.2, Eqs. 2-4; Algorithm 1's accept loop; Eq. 5) on
generated inputs: what must hold for ANY logits, confidences and thresholds, stated independently of the oracle's own
formulas (a library logsumexp, set algebra, a second statement of the loop)."""
import numpy as np
import pytest

hyp = pytest.importorskip("hypothesis")
from hypothesis import given, settings, strategies as st   # noqa: E402
from hypothesis.extra import numpy as hnp                  # noqa: E402

from oracle import confspec_oracle as O                    # noqa: E402

conf_arrays = hnp.arrays(np.float32, st.integers(1, 40),
                         elements=st.one_of(st.floats(0.0, 1.0, width=32), st.just(np.float32("nan"))))
taus = st.one_of(st.floats(0.0, 1.0, width=32), st.sampled_from([0.0, 1.0, 1.0001, 0.5, 0.9]))


@settings(max_examples=200, deadline=None)
@given(conf_arrays, taus, taus)
def test_gate_is_monotone_in_tau_and_has_table_3s_end_points(conf, t1, t2):
    lo, hi = min(t1, t2), max(t1, t2)
    a_lo, a_hi = O.gate(conf, lo), O.gate(conf, hi)
    assert np.all(a_hi <= a_lo)                                  # raising the threshold never trusts more steps
    finite = ~np.isnan(conf)
    assert np.all(O.gate(conf, 0.0)[finite] == 1)                # gamma = 0: the draft verifier decides everything
    assert np.all(O.gate(conf, 1.0001) == 0)                     # gamma > 1: everything goes to the target
    assert np.all(O.gate(conf, lo)[~finite] == 0)                # a NaN confidence is never trusted
    # the comparison is >= in fp32: a threshold equal to a confidence trusts that step
    for c in conf[finite][:3]:
        assert O.gate(np.array([c]), float(c))[0] == 1


@settings(max_examples=200, deadline=None)
@given(conf_arrays, taus)
def test_escalation_list_is_the_ordered_complement_of_the_mask(conf, tau):
    acc, idx, cnt = O.escalate_list(conf, tau)
    assert cnt == len(idx) == int((acc == 0).sum())
    assert np.all(np.diff(idx) > 0)                              # ascending, no repeats
    assert set(idx.tolist()) == {i for i in range(len(conf)) if not (conf[i] >= np.float32(tau))}


@settings(max_examples=100, deadline=None)
@given(hnp.arrays(np.float64, st.tuples(st.integers(1, 5), st.integers(5, 60)), elements=st.floats(-30, 30)),
       st.integers(1, 3))
def test_confidence_is_the_largest_verdict_probability_of_the_full_softmax(logits, n_verdict):
    from scipy.special import logsumexp, softmax
    ids = list(range(1, 1 + n_verdict))
    conf, verdict, lse = O.verdict_confidence(logits, ids)
    assert np.allclose(lse, logsumexp(logits, axis=-1), rtol=0, atol=1e-12)
    p = softmax(logits, axis=-1)
    assert np.allclose(conf, p[:, ids].max(axis=-1), rtol=1e-12, atol=1e-300)
    assert np.all(conf <= 1.0) and np.all(conf >= 0.0)
    for b in range(logits.shape[0]):                             # earliest verdict id among equal probabilities
        assert verdict[b] == int(np.argmax(p[b, ids] >= p[b, ids].max()))
    # raising any non-verdict logit can only lower the confidence (dilution)
    z2 = logits.copy()
    z2[:, 0] += 3.0
    assert np.all(O.verdict_confidence(z2, ids)[0] <= conf + 1e-15)


@settings(max_examples=200, deadline=None)
@given(st.lists(st.integers(0, 6), min_size=1, max_size=5), st.data())
def test_accept_prefix_and_best_candidate_per_request(sizes, data):
    B = sum(sizes)
    offs = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    draw = lambda s: data.draw(s)
    trusted = np.array(draw(st.lists(st.integers(0, 1), min_size=B, max_size=B)), dtype=np.uint8)
    vd = np.array(draw(st.lists(st.integers(0, 1), min_size=B, max_size=B)), dtype=np.int32)
    vt = np.array(draw(st.lists(st.integers(0, 1), min_size=B, max_size=B)), dtype=np.int32)
    cd = np.array(draw(st.lists(st.floats(0, 1, width=32), min_size=B, max_size=B)), dtype=np.float32)
    ct = np.array(draw(st.lists(st.floats(0, 1, width=32), min_size=B, max_size=B)), dtype=np.float32)
    passed, conf, m, best = O.cascade_select(trusted, vd, cd, vt, ct, offs, accept_index=0)
    final = np.where(trusted == 1, vd, vt)                       # Eq. 4
    assert np.array_equal(passed, (final == 0).astype(np.uint8))
    assert np.array_equal(conf, np.where(trusted == 1, cd, ct))
    for r, n in enumerate(sizes):
        seg = passed[offs[r]:offs[r + 1]]
        # Algorithm 1: steps are accepted up to, not including, the first rejection
        assert m[r] == (n if seg.all() else int(np.argmin(seg)))
        ok = [i for i in range(offs[r], offs[r + 1]) if passed[i]]
        if not ok:
            assert best[r] == -1
        else:                                                    # Eq. 5: highest confidence among those that pass
            assert passed[best[r]] and conf[best[r]] == max(conf[i] for i in ok)
            assert best[r] == min(i for i in ok if conf[i] == conf[best[r]])
