"""Failure detection without a fault: a bounded wait is made to run out on a healthy GPU (a barrier nothing arrives
at), the kernel returns, the host sees CS_ETIMEOUT once, and the same model keeps verifying correctly."""
import numpy as np
import pytest

from workloads import get_config, make_batch

import parity_common as P

pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_is_reported_once_and_the_context_stays_usable():
    from paper_2602_18447_b200 import binding as B
    cfg = get_config("cfg1_tiny")
    w = P.planted_weights(cfg)
    batch = make_batch(cfg)
    ses = P.build_session(cfg, w, batch)
    try:
        ses.verify()
        before = ses.results()                      # results() queries the status word: clean so far
        B.cs_selftest_wait_timeout(ses.model, 4096)
        with pytest.raises(B.ConfSpecError) as e:
            B.cs_last_status(ses.model)
        assert e.value.status == B.CS_ETIMEOUT
        B.cs_last_status(ses.model)                 # reported once, then clear
        ses.verify()
        after = ses.results()
        assert np.max(np.abs(after["conf"] - before["conf"])) <= 2.5e-3
        assert np.array_equal(after["verdict"], before["verdict"])
        ref = P.oracle_outputs(cfg, w, batch)
        P.compare_planted(after, ses.last_logits(), ref, cfg.tau, cfg, w)
        for bad in (0, -3, (1 << 20) + 1):
            with pytest.raises(B.ConfSpecError) as e:
                B.cs_selftest_wait_timeout(ses.model, bad)
            assert e.value.status == B.CS_EINVAL
    finally:
        ses.close()
