"""The C-ABI library loads, exports what include/dpara.h declares, and rejects bad arguments on the
host before any launch (no GPU needed)."""
import ctypes as C
import os
import re

import paper_2609_27396_b200 as dp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    txt = open(os.path.join(ROOT, "include", "dpara.h")).read()
    txt = re.sub(r"/\*.*?\*/", "", txt, flags=re.S)
    return sorted(set(re.findall(r"\b(dpara_[a-z_0-9]+)\s*\(", txt)))


def test_every_declared_symbol_is_exported():
    names = _declared()
    assert "dpara_draft_all_boundaries" in names and "dpara_verify_select" in names
    for n in names:
        assert hasattr(dp.lib, n), n
    assert set(dp.EXPORTED) <= set(names)


def test_status_strings_and_version():
    assert dp.lib.dpara_version() >= 1000
    for code in (0, -1, -2, -3, -4, -5):
        assert len(dp.lib.dpara_status_string(code)) > 0


def _shape(**kw):
    d = dict(batch=1, n_boundaries=3, block=2, n_q_heads=4, n_kv_heads=2, head_dim=64, prefix_base=1, n_spine=3,
             boundary_lo=0, boundary_hi=3, softmax_scale=0.0, spine_queries=0)
    d.update(kw)
    return dp.Shape(*[d[f[0]] for f in dp.Shape._fields_])


def test_draft_argument_validation():
    off = (C.c_int64 * 2)(0, 5)
    io = dp.AttnIO()
    call = lambda s, i: dp.lib.dpara_draft_all_boundaries(C.byref(s), C.byref(i) if i is not None else None, None, None, 0, None, None)
    assert call(_shape(head_dim=96), io) == dp.ERR_UNSUPPORTED
    assert call(_shape(n_q_heads=3), io) == dp.ERR_UNSUPPORTED
    assert call(_shape(batch=0), io) == dp.ERR_INVALID_ARG
    assert call(_shape(boundary_hi=4), io) == dp.ERR_INVALID_ARG
    assert call(_shape(spine_queries=2), io) == dp.ERR_INVALID_ARG
    assert call(_shape(spine_queries=1, boundary_lo=1), io) == dp.ERR_UNSUPPORTED    # spine rows need the full boundary range
    assert call(_shape(), None) == dp.ERR_INVALID_ARG
    assert call(_shape(), io) == dp.ERR_INVALID_ARG                     # no host offsets
    io.host_ctx_offsets = C.cast(off, C.c_void_p).value
    assert call(_shape(), io) == dp.ERR_INVALID_ARG                     # null device pointers
    bad = (C.c_int64 * 2)(5, 0)
    io.host_ctx_offsets = C.cast(bad, C.c_void_p).value
    assert call(_shape(), io) == dp.ERR_INVALID_ARG                     # decreasing offsets
    assert dp.lib.dpara_draft_workspace_bytes(C.byref(_shape(head_dim=7)), C.cast(off, C.c_void_p), None, 0) == 0


def test_verify_argument_validation():
    io = dp.VerifyIO(2, 4, 100, 2, 8, 0)
    assert dp.lib.dpara_verify_workspace_bytes(C.byref(io)) > 0
    assert dp.lib.dpara_verify_select(C.byref(io), None, 0, None, None) == dp.ERR_INVALID_ARG      # null tensors
    assert dp.lib.dpara_verify_select(None, None, 0, None, None) == dp.ERR_INVALID_ARG
    io2 = dp.VerifyIO(2, 100, 100, 2, 8, 0)
    assert dp.lib.dpara_verify_workspace_bytes(C.byref(io2)) == 0                                   # J > 64
    io3 = dp.VerifyIO(2, 4, 100, 2, 8, 0, 16, None, 16, None, None, 16, 16, 16, None, None)
    assert dp.lib.dpara_verify_select(C.byref(io3), None, 0, None, None) == dp.ERR_WORKSPACE
    io4 = dp.VerifyIO(2, 4, 100, 2, 8, 1, 16, None, 16, None, None, 16, 16, 16, None, None)
    assert dp.lib.dpara_verify_select(C.byref(io4), None, 0, None, None) == dp.ERR_INVALID_ARG      # sampling needs uniforms
    io5 = dp.VerifyIO(2, 4, 100, 2, 8, 7)
    assert dp.lib.dpara_verify_workspace_bytes(C.byref(io5)) == 0                                   # bad mode
