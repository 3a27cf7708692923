"""GPU parity of the backbone pass with the spine tokens as query rows (dpara_draft_backbone) against the oracle's block
over all rows of a request and its stack of blocks.

One block: every row (mask slots and spine) within the literal 1e-2 of the oracle's `request`.
Two blocks: checked TEACHER-FORCED -- the oracle's second block is fed the kernel's own first-block output (obtained from
a one-block call with the same weights), so that a single flipped bf16 rounding in the residual stream between the
blocks (one step is 1.6e-2 at |x| >= 2) is not mistaken for an error of the second block or of the stacking; the
free-running difference is printed and held to the rms-scaled bound of the long-context layer test."""
import numpy as np
import pytest
import torch

import workloads as W
from oracle import attention as OA
from oracle import layer as OL
from oracle import verify as OV

pytestmark = pytest.mark.gpu
TOL = 1e-2


def _dev(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def _setup(ashape, lshape, n_layers, seed):
    rng = np.random.default_rng(seed)
    R = ashape.n_boundaries * ashape.block + ashape.spine
    x_rows = W.f32_to_bf16_bits(rng.standard_normal((ashape.batch, R, lshape.hidden)).astype(np.float32))
    ains = [W.make_attn_inputs(ashape, seed + 10 * l, with_q=False, with_blk=False) for l in range(n_layers)]
    lins = [W.make_layer_inputs(lshape, ashape, seed + 10 * l) for l in range(n_layers)]
    return x_rows, ains, lins


def _run(ashape, x_rows, ains, lins):
    import paper_2609_27396_b200 as dp
    b, R, H = x_rows.shape
    y = torch.zeros((b, R, H), dtype=torch.float32, device="cuda")
    y16 = torch.zeros((b, R, H), dtype=torch.bfloat16, device="cuda")
    x = _dev(x_rows)
    keep, layers = [], []
    for l, lin in enumerate(lins):
        t = {k: _dev(getattr(lin, k)) for k in ("w_qkv", "w_o", "w_gate_up", "w_down", "rms1_w", "rms2_w", "qnorm_w", "knorm_w")}
        keep.append(t)
        layers.append(dp.make_layer_io(x=x, **t, rms_eps=lin.shape.rms_eps, rope_theta=lin.shape.rope_theta, use_rope=True, y_f32=y, y_bf16=y16))
    kc, vc = [_dev(a.k_ctx) for a in ains], [_dev(a.v_ctx) for a in ains]
    plan = dp.BackbonePlan(ctx_offsets=[int(v) for v in ains[0].ctx_offsets], n_boundaries=ashape.n_boundaries, block=ashape.block,
                           n_q_heads=ashape.n_q_heads, n_kv_heads=ashape.n_kv_heads, head_dim=ashape.head_dim, layers=layers,
                           k_ctx=kc, v_ctx=vc, prefix_base=ashape.prefix_base, n_spine=ashape.spine)
    plan()
    torch.cuda.synchronize()
    assert int(plan.status.item()) == 0
    return y.cpu().numpy().astype(np.float64), y16


SHAPES = [
    (W.AttnShape((150, 260), 8, 2, 128, 3, 5), W.LayerShape(512, 768)),
    (W.AttnShape((300, 77, 9), 4, 2, 64, 4, 4), W.LayerShape(256, 384)),
    (W.AttnShape((200,), 10, 2, 128, 8, 8), W.LayerShape(320, 448)),       # group size 5
]


@pytest.mark.parametrize("ashape,lshape", SHAPES)
def test_one_block_with_spine_rows(ashape, lshape):
    x_rows, ains, lins = _setup(ashape, lshape, 1, 61)
    y, _ = _run(ashape, x_rows, ains, lins)
    orc = OL.LayerOracle(lins[0], ains[0])
    worst = 0.0
    for n in range(ashape.batch):
        ref = orc.request(n, OA.bf16_bits_to_f64(x_rows[n]))["y"]
        worst = max(worst, float(np.abs(y[n] - ref).max()))
    print(f"one block, all rows: max |delta| {worst:.3e}")
    assert worst <= TOL


@pytest.mark.parametrize("ashape,lshape", SHAPES[:2])
def test_two_blocks_teacher_forced(ashape, lshape):
    x_rows, ains, lins = _setup(ashape, lshape, 2, 71)
    y2, _ = _run(ashape, x_rows, ains, lins)
    _, y1_16 = _run(ashape, x_rows, ains[:1], lins[:1])                    # the kernel's own first-block output (bf16)
    y1 = y1_16.float().cpu().numpy().astype(np.float64)
    l1, l2 = OL.LayerOracle(lins[0], ains[0]), OL.LayerOracle(lins[1], ains[1])
    forced, free = 0.0, 0.0
    for n in range(ashape.batch):
        ref = l2.request(n, y1[n], ains[1].k_ctx, ains[1].v_ctx)["y"]
        forced = max(forced, float(np.abs(y2[n] - ref).max()))
        full = OL.backbone([l1, l2], n, OA.bf16_bits_to_f64(x_rows[n]), caches=[(a.k_ctx, a.v_ctx) for a in ains])
        d = np.abs(y2[n] - full)
        free = max(free, float(d.max()))
        assert d.max() <= TOL * max(1.0, float(np.sqrt((full * full).mean()))) * 2 and np.sqrt((d * d).mean()) <= 5e-3
    print(f"two blocks: teacher-forced max |delta| {forced:.3e}, free-running {free:.3e}")
    assert forced <= TOL


def test_select_gathers_from_rows_with_a_request_stride():
    """The backbone's output keeps each request's spine rows behind its mask-slot rows; dpara_verify_select gathers the
    selected branch from it through rep_req_rows."""
    import paper_2609_27396_b200 as dp
    b, J, Bq, S, H, V = 3, 4, 4, 4, 64, 1000
    rng = np.random.default_rng(2)
    rows = W.f32_to_bf16_bits(rng.standard_normal((b, J * Bq + S, H)).astype(np.float32))
    v = W.make_verify_inputs(W.VerifyShape(b, J, V, Bq, H, "greedy", 0.7, 1.0), 5)
    plan = dp.VerifyPlan(batch=b, n_boundaries=J, vocab=V, block=Bq, hidden=H, mode=0, rep_req_rows=J * Bq + S)
    plan(target=torch.from_numpy(v.target).cuda(), draft_tokens=torch.from_numpy(v.draft_tokens).cuda(), reps=_dev(rows))
    torch.cuda.synchronize()
    packed = np.ascontiguousarray(rows[:, :J * Bq].reshape(b, J, Bq, H))
    ref = OV.verify_greedy(v.target, v.draft_tokens, packed)
    assert np.array_equal(plan.accept_len.cpu().numpy(), ref["accept_len"])
    assert np.array_equal(plan.selected.cpu().view(torch.int16).numpy().view(np.uint16), ref["selected"])
