"""GPU parity of dpara_cache_append against the oracle's row-by-row cache update, and of the draft call reading the
appended cache through ctx_lens.

Bounds: lengths, row placement and untouched rows are exact.  Values: the kernel's norm and GEMM work in fp32 (the oracle
in float64), so a bf16 rounding may fall the other way: values (rounded after the norm and after the product) within two
bf16 steps of the oracle's; keys (norm, product, head norm, rotation: four roundings, the rotation mixing the pair
(d, d + D/2)) within four steps of the larger member of the pair; plus an absolute floor (1e-3 on values, 4e-3 on the
normalised keys) because one flipped rounding of a normalised input moves the whole 320..512-term product by up to
ulp(x) * |w| ~ 1e-4..1e-3, which is many steps of a product that happens to be near zero; and nearly all elements must
be bit-equal."""
import numpy as np
import pytest
import torch

import workloads as W
from oracle import attention as OA
from oracle import cache as OC

pytestmark = pytest.mark.gpu
FINITE_SENTINEL = 0x4348      # bf16 200.0: unused cache rows must be finite (they pass through the tensor core with weight 0)


def _dev(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def _host(t):
    return t.cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def _run(ci, use_rope=True, knorm=True):
    import paper_2609_27396_b200 as dp
    for k in ci.k_cache + ci.v_cache:
        k[k == 0x7FC1] = FINITE_SENTINEL
    nl = len(ci.w_kv)
    kc, vc = [_dev(x) for x in ci.k_cache], [_dev(x) for x in ci.v_cache]
    lens = torch.from_numpy(ci.ctx_len.copy()).cuda()
    plan = dp.CachePlan(batch=ci.features.shape[0], n_rows=ci.features.shape[1], w_kv=[_dev(w) for w in ci.w_kv], k_ctx=kc, v_ctx=vc,
                        row_start=torch.from_numpy(ci.row_start).cuda(), capacity=torch.from_numpy(ci.capacity).cuda(), ctx_len=lens,
                        norm_w=[_dev(g) for g in ci.norm_w], knorm_w=[_dev(g) for g in ci.knorm_w] if knorm else None, use_rope=use_rope)
    plan.run(_dev(ci.features), torch.from_numpy(ci.accept_len).cuda())
    torch.cuda.synchronize()
    return [_host(k) for k in kc], [_host(v) for v in vc], lens.cpu().numpy(), int(plan.status.item())


def _check(ci, use_rope=True, knorm=True, capacity=None):
    cap = ci.capacity if capacity is None else capacity
    ci.capacity = cap
    gk, gv, glen, gst = _run(ci, use_rope, knorm)
    D = ci.k_cache[0].shape[2]
    for l in range(len(ci.w_kv)):
        rk, rv, rlen, rst = OC.append_verified(ci.k_cache[l], ci.v_cache[l], ci.row_start, cap, ci.ctx_len, ci.features, ci.accept_len,
                                               ci.w_kv[l], ci.norm_w[l], ci.knorm_w[l] if knorm else None, use_rope=use_rope)
        assert np.array_equal(glen, rlen) and gst == rst
        new = np.zeros(rk.shape[0], bool)
        for n in range(len(rlen)):
            new[ci.row_start[n] + ci.ctx_len[n]: ci.row_start[n] + rlen[n]] = True
        assert np.array_equal(gk[l][~new], ci.k_cache[l][~new]) and np.array_equal(gv[l][~new], ci.v_cache[l][~new])   # nothing else moved
        a, b = OA.bf16_bits_to_f64(gv[l][new]), OA.bf16_bits_to_f64(rv[new])
        assert np.all(np.abs(a - b) <= 2 * 2.0 ** -7 * np.abs(b) + 1e-3), float(np.abs(a - b).max())
        a, b = OA.bf16_bits_to_f64(gk[l][new]), OA.bf16_bits_to_f64(rk[new])
        pair = np.maximum(np.abs(b), np.abs(np.roll(b, D // 2, axis=-1)))
        assert np.all(np.abs(a - b) <= 4 * 2.0 ** -7 * pair + 4e-3), float(np.abs(a - b).max())
        assert (gv[l][new] == rv[new]).mean() > 0.98 and (gk[l][new] == rk[new]).mean() > 0.9     # flips are the exception
    return gk, gv, glen


@pytest.mark.parametrize("lens,J,F,Hkv,D,layers", [
    ((37, 0, 5, 130), 4, 256, 2, 64, 2),
    ((300, 12, 77), 8, 512, 8, 128, 3),
    ((64,) * 20, 16, 320, 4, 128, 1),          # 320 candidate rows: several GEMM row tiles
    ((50, 9, 31) * 6, 9, 512, 4, 128, 10),     # 162 rows x 10 layers: two grouped launches (8 + 2 layers), K ranges in parts
    ((40,) * 33, 8, 1024, 2, 64, 3),           # 264 rows: two row pairs per layer, three layers in one launch
    ((100, 37, 64, 12) * 4, 16, 5120, 8, 128, 5),   # the benchmark's shape: 256 candidate rows x 5120 features, 5 layers in one grouped launch
])
def test_append_parity(lens, J, F, Hkv, D, layers):
    ci = W.make_cache_inputs(lens, J, F, Hkv, D, layers, 21)
    ci.accept_len[0] = J - 1
    ci.accept_len[1] = 0
    _check(ci)


def test_append_without_rope_and_key_norm():
    _check(W.make_cache_inputs((9, 40), 5, 128, 2, 64, 1, 4), use_rope=False, knorm=False)


def test_full_cache_is_reported_and_left_alone():
    ci = W.make_cache_inputs((10, 10, 10), 6, 128, 2, 64, 2, 6, accept_len=[5, 2, 5])
    cap = ci.capacity.copy()
    cap[2] = 12                                   # 10 + 6 rows do not fit
    _, _, glen = _check(ci, capacity=cap)
    assert glen.tolist() == [16, 13, 10]


def test_two_rounds_then_draft_reads_the_grown_cache():
    """Two append rounds on one plan, then the all-boundary attention over the grown cache (ctx_lens) against the
    oracle's attention over the oracle's cache."""
    import paper_2609_27396_b200 as dp
    sh = W.AttnShape((150, 9, 260), 8, 2, 128, 4, 4)
    inp = W.make_attn_inputs(sh, 12)
    ci = W.make_cache_inputs(sh.ctx_lens, 4, 256, 2, 128, 1, 12, slack=4)
    for k in ci.k_cache + ci.v_cache:
        k[k == 0x7FC1] = FINITE_SENTINEL
    kc, vc = _dev(ci.k_cache[0]), _dev(ci.v_cache[0])
    lens = torch.from_numpy(ci.ctx_len.copy()).cuda()
    plan = dp.CachePlan(batch=3, n_rows=4, w_kv=[_dev(ci.w_kv[0])], k_ctx=[kc], v_ctx=[vc], row_start=torch.from_numpy(ci.row_start).cuda(),
                        capacity=torch.from_numpy(ci.capacity).cuda(), ctx_len=lens, norm_w=[_dev(ci.norm_w[0])], knorm_w=[_dev(ci.knorm_w[0])])
    rk, rv, rlen = ci.k_cache[0], ci.v_cache[0], ci.ctx_len
    rng = np.random.default_rng(3)
    for rnd in range(2):
        feats = W.make_cache_inputs(sh.ctx_lens, 4, 256, 2, 128, 1, 50 + rnd).features
        acc = rng.integers(0, 4, size=3).astype(np.int32)
        plan.run(_dev(feats), torch.from_numpy(acc).cuda())
        rk, rv, rlen, _ = OC.append_verified(rk, rv, ci.row_start, ci.capacity, rlen, feats, acc, ci.w_kv[0], ci.norm_w[0], ci.knorm_w[0])
    torch.cuda.synchronize()
    assert np.array_equal(lens.cpu().numpy(), rlen) and int(plan.status.item()) == 0
    starts = [int(x) for x in ci.row_start] + [int(ci.row_start[-1] + ci.capacity[-1])]
    dplan = dp.DraftPlan(ctx_offsets=starts, n_boundaries=4, block=4, n_q_heads=8, n_kv_heads=2, head_dim=128, ctx_lens=[int(x) for x in rlen])
    dplan.set_ctx_lens([int(x) for x in rlen], dev_lens=lens)
    out = torch.zeros((3, 4, 4, 8, 128), dtype=torch.float32, device="cuda")
    dplan(q=_dev(inp.q), k_ctx=kc, v_ctx=vc, k_spine=_dev(inp.k_spine), v_spine=_dev(inp.v_spine), k_blk=_dev(inp.k_blk), v_blk=_dev(inp.v_blk), out=out)
    torch.cuda.synchronize()
    # the oracle's attention over the KERNEL's cache (teacher-forced: rounding flips of single cache elements aside)
    ref, _ = OA.draft_all_boundaries(inp.q, _host(kc), _host(vc), np.array(starts), inp.k_spine, inp.v_spine, inp.k_blk, inp.v_blk, ctx_lens=rlen)
    assert np.abs(out.cpu().numpy() - ref).max() <= 1e-2
    ref2, _ = OA.draft_all_boundaries(inp.q, rk, rv, np.array(starts), inp.k_spine, inp.v_spine, inp.k_blk, inp.v_blk, ctx_lens=rlen)
    assert np.abs(out.cpu().numpy() - ref2).max() <= 1e-2
