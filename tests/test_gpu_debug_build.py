"""The library compiled with -DCS_DEBUG: device-side range checks on page ids, token rows and tensor-memory columns
that raise a status bit instead of trapping. The small cases - real prefill, ragged steps across page and tile
boundaries, a context cut into pieces, the 8-bit cache - must run through it without a range error and with the guard
bytes behind every workspace intact; the path from a failed check to the host is exercised by a kernel whose one check
fails by construction without touching memory."""
from dataclasses import replace

import numpy as np
import pytest

from workloads import get_config, make_batch, scaled_config

import parity_common as P

pytestmark = pytest.mark.gpu


@pytest.fixture()
def debug_binding():
    from paper_2602_18447_b200 import binding, build
    binding.load_library(build.build(debug=True))
    assert binding.cs_debug_build()
    yield binding
    binding.load_library(build.LIB_PATH)
    assert not binding.cs_debug_build()


def _run_checked(B, cfg, planted=True):
    w = P.planted_weights(cfg) if planted else None
    batch = make_batch(cfg)
    ses = P.build_session(cfg, w, batch)
    try:
        ses.verify()
        gpu = ses.results()                       # cs_last_status inside: raises on a time-out or a range error
        B.cs_check_workspace(ses.model)
        ref = P.oracle_outputs(cfg, w, batch)
        P.compare_planted(gpu, ses.last_logits(), ref, cfg.tau, cfg, gpu_lse=ses.last_lse())
        ses.verify(host_tokens=True)
        again = ses.results()
        assert np.array_equal(again["conf"].view(np.uint32), gpu["conf"].view(np.uint32))
        B.cs_check_workspace(ses.model)
    finally:
        ses.close()


def test_small_cases_pass_the_device_side_range_checks(debug_binding):
    B = debug_binding
    tiny = get_config("cfg1_tiny")
    _run_checked(B, replace(tiny, batch=6))                                                   # real prefill + verify
    _run_checked(B, replace(tiny, batch=3, ctx_dist=("fixed", 17), step_dist=("fixed", 65), suffix_len=0))
    _run_checked(B, replace(tiny, batch=5, ctx_dist=("uniform", 0, 90), step_dist=("uniform", 1, 12), suffix_len=2))
    _run_checked(B, get_config("cfg8_tiny_qknorm"))                                           # second family
    _run_checked(B, scaled_config("cfg4_1p5b_long", n_layers=1, batch=2, vocab=8192))         # context cut into pieces
    _run_checked(B, scaled_config("cfg9_q3_short_fp8", n_layers=1, batch=6, vocab=8192))      # 8-bit cache


def test_a_failed_range_check_reaches_the_host_and_leaves_the_context_usable(debug_binding):
    B = debug_binding
    cfg = replace(get_config("cfg1_tiny"), batch=3)
    w, batch = P.planted_weights(cfg), make_batch(cfg)
    ses = P.build_session(cfg, w, batch)
    try:
        ses.verify()
        before = ses.results()
        B.cs_selftest_range_check(ses.model)
        with pytest.raises(B.ConfSpecError) as e:
            B.cs_last_status(ses.model)
        assert e.value.status == B.CS_ERANGE
        B.cs_last_status(ses.model)               # reported once, then clear
        ses.verify()
        after = ses.results()
        assert np.array_equal(after["conf"].view(np.uint32), before["conf"].view(np.uint32))
    finally:
        ses.close()


def test_release_build_has_no_range_checks():
    from paper_2602_18447_b200 import binding as B
    assert not B.cs_debug_build()
    cfg = replace(get_config("cfg1_tiny"), batch=2)
    ses = P.build_session(cfg, P.planted_weights(cfg), make_batch(cfg))
    try:
        B.cs_selftest_range_check(ses.model)
        B.cs_last_status(ses.model)               # the check compiled away: nothing was raised
    finally:
        ses.close()
