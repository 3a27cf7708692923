"""The fixed-scratch verify/select entry point (dpara_verify_select_static) against the normal one.

That entry point exists for callers that cannot allocate device memory -- a server whose own pool
already owns all of it, or a decode loop that cannot afford the stall of an allocation -- so it keeps
its scratch in an array inside the library.  It must give exactly what dpara_verify_select gives, and what the CPU oracle gives.
Checked on two calls in a row (the shared array keeps the first call's contents, so the second call
proves that whatever must start at zero is cleared), for both modes, through the C ABI.
This file is collected last on purpose: a failure here cannot hide any other test's result.
"""
import ctypes as C

import numpy as np
import pytest
import torch

import workloads as W
from oracle import verify as OV

pytestmark = pytest.mark.gpu

KEYS = ("accept_len", "bonus", "gather_idx", "out_tokens", "selected")


def _dev_bf16(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def _run_both(sh, seed):
    import paper_2609_27396_b200 as dp
    mode = 1 if sh.mode == "sampling" else 0
    kw = dict(batch=sh.batch, n_boundaries=sh.n_boundaries, vocab=sh.vocab, block=sh.block, hidden=sh.hidden, mode=mode)
    ref_plan, st_plan = dp.VerifyPlan(**kw), dp.VerifyPlan(**kw)          # all allocation happens here, up front
    for rep in range(2):                                                   # two calls in a row, different inputs
        v = W.make_verify_inputs(sh, seed + rep)
        args = dict(target=torch.from_numpy(v.target).cuda(), draft_tokens=torch.from_numpy(v.draft_tokens).cuda(),
                    reps=_dev_bf16(v.reps))
        if mode == 1:
            args.update(draft_probs=torch.from_numpy(v.draft_probs).cuda(), uniforms=torch.from_numpy(v.uniforms).cuda())
        for k in KEYS:
            getattr(st_plan, k).fill_(-7)
        ref_plan(**args)
        torch.cuda.synchronize()
        before = (torch.cuda.memory_allocated(), torch.cuda.memory_reserved())
        dp.verify_select_static(st_plan, **args)
        torch.cuda.synchronize()
        assert (torch.cuda.memory_allocated(), torch.cuda.memory_reserved()) == before     # the call took no device memory
        for k in KEYS:                                                     # integer / bit-copy outputs: exact
            assert torch.equal(getattr(st_plan, k), getattr(ref_plan, k)), (k, rep)
        assert int(st_plan.status.item()) == int(ref_plan.status.item())
        # ... and against the CPU oracle, not only against the sibling entry point
        if mode == 0:
            orc = OV.verify_greedy(v.target, v.draft_tokens, v.reps)
        else:
            orc = OV.verify_sampling(v.target, v.draft_probs, v.draft_tokens, v.uniforms, v.reps)
        for k in ("accept_len", "bonus", "gather_idx", "out_tokens"):
            assert np.array_equal(getattr(st_plan, k).cpu().numpy(), orc[k]), (k, rep)
        assert np.array_equal(st_plan.selected.cpu().view(torch.int16).numpy().view(np.uint16), orc["selected"]), rep
        assert int(st_plan.status.item()) == orc["status"]


def test_static_matches_workspace_entry_greedy():
    _run_both(W.VerifyShape(6, 8, 40000, 4, 256, "greedy", 0.8, 2.0), 31)


def test_static_matches_workspace_entry_sampling():
    _run_both(W.VerifyShape(4, 6, 20000, 4, 256, "sampling", 0.0, 3.0), 47)


def test_static_rejects_oversize_request():
    import paper_2609_27396_b200 as dp
    # sampling scratch grows with batch * ceil(vocab / 4096) * 16 bytes: make it exceed the fixed array
    io = dp.VerifyIO(4096, 2, 4096 * 8, 1, 8, 1, 16, 16, 16, 16, None, 16, 16, 16, None, None)
    assert dp.lib.dpara_verify_workspace_bytes(C.byref(io)) > dp.VERIFY_STATIC_SCRATCH_BYTES
    assert dp.lib.dpara_verify_select_static(C.byref(io), None, None) == dp.ERR_STATIC_LIMIT
    assert b"scratch" in dp.lib.dpara_status_string(dp.ERR_STATIC_LIMIT)
