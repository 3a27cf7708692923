"""GPU parity of the full backbone block (dpara_draft_all_boundaries with a layer) against the oracle's
block, boundary by boundary.

Bound on the fp32 output y: |delta| <= 1e-2 * max(1, rms(y)), i.e. the stated 1e-2 at unit scale (the error
is additive noise of the down projection, independent of the element's own size).  Derivation:
the oracle mirrors the block's bf16 rounding points, but the tensor-core attention rounds probabilities to
bf16 before the PV product, so its output differs from the oracle's by ~1e-3 relative; that flips the bf16
rounding of `a` on a large share of elements, which perturbs h1 by ~3e-5, flips ~1 % of the bf16 `hn`
elements, moves gate/up by ~6e-4 relative and so flips the rounding of most `act` elements by one ulp:
sqrt(12288) * (2^-8 * 0.5) * 0.02 ~ 4e-3 rms on y (measured 3.2e-3 rms, y rms 2.5, |y| up to 11), whose
5-sigma tail over 65 536 outputs per boundary is ~1.6e-2.  The rms is asserted as well."""
import numpy as np
import pytest
import torch

import workloads as W
from oracle import layer as OL

pytestmark = pytest.mark.gpu
TOL = 1e-2


def _dev(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def _run_layer(ain, lin, qk_norm=True, use_rope=True):
    import paper_2609_27396_b200 as dp
    sh = ain.shape
    M = sh.batch * sh.n_boundaries * sh.block
    t = {k: _dev(getattr(lin, k)) for k in ("x", "w_qkv", "w_o", "w_gate_up", "w_down", "rms1_w", "rms2_w", "qnorm_w", "knorm_w")}
    y = torch.zeros((sh.batch, sh.n_boundaries, sh.block, lin.shape.hidden), dtype=torch.float32, device="cuda")
    y16 = torch.zeros_like(y, dtype=torch.bfloat16)
    lio = dp.make_layer_io(x=t["x"], w_qkv=t["w_qkv"], w_o=t["w_o"], w_gate_up=t["w_gate_up"], w_down=t["w_down"],
                           rms1_w=t["rms1_w"], rms2_w=t["rms2_w"], qnorm_w=t["qnorm_w"] if qk_norm else None,
                           knorm_w=t["knorm_w"] if qk_norm else None, rms_eps=lin.shape.rms_eps,
                           rope_theta=lin.shape.rope_theta, use_rope=use_rope, y_f32=y, y_bf16=y16)
    plan = dp.DraftPlan(ctx_offsets=[int(v) for v in ain.ctx_offsets], n_boundaries=sh.n_boundaries, block=sh.block,
                        n_q_heads=sh.n_q_heads, n_kv_heads=sh.n_kv_heads, head_dim=sh.head_dim, prefix_base=sh.prefix_base,
                        n_spine=sh.spine, layer=lio)
    keep = [_dev(v) for v in (ain.k_ctx, ain.v_ctx, ain.k_spine, ain.v_spine)]
    plan(k_ctx=keep[0], v_ctx=keep[1], k_spine=keep[2], v_spine=keep[3])
    torch.cuda.synchronize()
    assert int(plan.status.item()) == 0
    assert plan.workspace_bytes > 0
    return y.cpu().numpy(), y16.float().cpu().numpy()


@pytest.mark.parametrize("ashape,lshape,norm,rope", [
    (W.AttnShape((300, 77), 4, 2, 64, 4, 4), W.LayerShape(256, 384), True, True),
    (W.AttnShape((150, 260), 8, 2, 128, 3, 5), W.LayerShape(512, 768), True, True),
    (W.AttnShape((200,), 8, 4, 64, 5, 8), W.LayerShape(320, 448), False, False),
])
def test_layer_parity(ashape, lshape, norm, rope):
    import dataclasses
    lshape = dataclasses.replace(lshape, qk_norm=norm, use_rope=rope)
    ain = W.make_attn_inputs(ashape, 31, with_q=False, with_blk=False)
    lin = W.make_layer_inputs(lshape, ashape, 31)
    y, y16 = _run_layer(ain, lin, norm, rope)
    orc = OL.LayerOracle(lin, ain)
    worst = 0.0
    for n in range(ashape.batch):
        for j in range(ashape.n_boundaries):
            ref = orc.boundary(n, j)["y"].astype(np.float64)
            worst = max(worst, float(np.abs(y[n, j] - ref).max()))
            assert np.all(np.abs(y16[n, j] - ref) <= 2 ** -8 * np.abs(ref) + TOL)
    assert worst <= TOL, worst


def test_cfg5_full_size_sampled_boundaries():
    """The full-layer, long-context workload (b = 4, context 32768, M = 1024 rows) in the launch
    configuration the benchmark uses; the oracle evaluates a seeded sample of (request, boundary) blocks."""
    w = W.workload(5)
    ain = W.make_attn_inputs(w.attn, w.seed, with_q=False, with_blk=False)
    lin = W.make_layer_inputs(w.layer, w.attn, w.seed)
    y, y16 = _run_layer(ain, lin, True, True)
    assert np.isfinite(y).all()
    orc = OL.LayerOracle(lin, ain)
    rng = np.random.default_rng(5)
    picks = {(0, 0), (3, 15)} | {(int(rng.integers(4)), int(rng.integers(16))) for _ in range(4)}
    for (n, j) in sorted(picks):
        ref = orc.boundary(n, j)["y"].astype(np.float64)
        d = np.abs(y[n, j] - ref)
        assert np.all(d <= TOL * max(1.0, float(np.sqrt((ref * ref).mean())))), (n, j, float(d.max()))
        assert np.sqrt((d * d).mean()) <= 5e-3
