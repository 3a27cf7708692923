"""Failure detection without a GPU fault: the bounded device-side wait gives up, reports through the status
word, and the context stays usable (a normal call right after it still matches the oracle)."""
import numpy as np
import pytest
import torch

import workloads as W
from oracle import verify as OV

pytestmark = pytest.mark.gpu


def test_bounded_wait_times_out_and_context_survives():
    import paper_2609_27396_b200 as dp
    status, waited_ns = dp.selftest_bounded_wait(limit_us=500)
    assert status & dp.STATUS_TIMEOUT
    assert 400_000 <= waited_ns < 50_000_000          # gave up after about the limit, long before "forever"
    # the context is intact: a real call works and is bit-exact
    sh = W.VerifyShape(3, 4, 5000, 2, 64, "greedy", 0.7, 1.0)
    v = W.make_verify_inputs(sh, 3)
    from gpu_util import run_verify, check_verify
    check_verify(run_verify(v, 0), OV.verify_greedy(v.target, v.draft_tokens, v.reps))


def test_selftest_rejects_bad_limits():
    import paper_2609_27396_b200 as dp
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    assert dp.lib.dpara_selftest_bounded_wait(st.data_ptr(), 0, None, None) == dp.ERR_INVALID_ARG
    assert dp.lib.dpara_selftest_bounded_wait(None, 10, None, None) == dp.ERR_INVALID_ARG
