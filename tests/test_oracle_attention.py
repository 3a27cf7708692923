"""Pins for oracle/attention.py against what the paper and the mathematics fix (CPU only)."""
import math
import os

import numpy as np
import pytest
import torch

import workloads as W
from oracle import attention as OA

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _gold_mask():
    rows = []
    with open(os.path.join(GOLD, "fig4_mask_d3.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            rows.append([int(t) for t in line.split()])
    return np.array(rows, dtype=bool)


def _paper_numbers():
    d = {}
    with open(os.path.join(GOLD, "paper_numbers.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            k, v = line.split()
            d[k] = int(v)
    return d


def _inputs(ctx_lens=(5,), Hq=2, Hkv=1, D=8, J=3, Bq=2, seed=1, pb=1):
    sh = W.AttnShape(tuple(ctx_lens), Hq, Hkv, D, J, Bq, pb)
    return W.make_attn_inputs(sh, seed)


def _run(inp, **kw):
    return OA.draft_all_boundaries(inp.q, inp.k_ctx, inp.v_ctx, inp.ctx_offsets, inp.k_spine, inp.v_spine,
                                   inp.k_blk, inp.v_blk, prefix_base=inp.shape.prefix_base, **kw)


def test_fig4_mask_literal():
    """oracle.tree_mask(d=3) is the figure's mask, cell by cell."""
    assert np.array_equal(OA.tree_mask(3, 3, prefix_base=1), _gold_mask())


def test_paper_counts():
    p = _paper_numbers()
    for d, key in ((3, "tokens_per_request_d3"), (7, "tokens_per_request_d7")):
        assert OA.tree_mask(d, d).shape[0] == p[key] == (d + 1) + (d + 1) * d
    # representation block layout [d+1][d][hidden] bf16
    d, hid = p["hidden_push_d"], p["hidden_push_hidden"]
    assert (d + 1) * d * hid * 2 == p["hidden_push_bytes"]
    assert round(151936 / hid) == p["logits_over_hidden_ratio"]
    # Fig. 3: r accepted drafts -> branch r reads r + 1 anchors
    m = OA.tree_mask(3, 3)
    r = p["fig3_accept_len"]
    row = 4 + p["fig3_branch"] * 3
    assert p["fig3_branch"] == r and m[row, :4].sum() == p["fig3_anchors"] == r + 1


def test_matches_tree_masked_sdpa_from_figure():
    """One pass of a library attention over [context | spine | all branches] under the FIGURE's mask
    (read from the fixture, not from the oracle) gives the oracle's per-boundary outputs."""
    d = 3
    L, Hq, Hkv, D = 7, 4, 2, 16
    inp = _inputs((L,), Hq, Hkv, D, J=d + 1, Bq=d, seed=11)
    out, _ = _run(inp)
    mask = _gold_mask()                                    # [16][16]
    S = d + 1
    dec = lambda a: torch.from_numpy(OA.bf16_bits_to_f64(a))
    # keys in the combined order: context, spine, branch 0..d
    K = torch.cat([dec(inp.k_ctx), dec(inp.k_spine[0]), dec(inp.k_blk[0]).reshape(S * d, Hkv, D)], 0)   # [T][Hkv][D]
    V = torch.cat([dec(inp.v_ctx), dec(inp.v_spine[0]), dec(inp.v_blk[0]).reshape(S * d, Hkv, D)], 0)
    Q = dec(inp.q[0]).reshape(S * d, Hq, D)                                                                # mask-token rows
    full = torch.cat([torch.ones(S * d, L, dtype=torch.bool), torch.from_numpy(mask[S:])], 1)              # rows of mask tokens
    o = torch.nn.functional.scaled_dot_product_attention(
        Q.permute(1, 0, 2)[None], K.permute(1, 0, 2)[None], V.permute(1, 0, 2)[None],
        attn_mask=full[None, None], enable_gqa=True)[0]                                                     # [Hq][S*d][D]
    ref = o.permute(1, 0, 2).reshape(S, d, Hq, D).numpy()
    assert np.abs(ref - out[0]).max() < 1e-12


@pytest.mark.parametrize("pb", [0, 1])
def test_one_hot_probe_closed_form(pb):
    """q = 0 makes every visible key weigh the same; with v_spine[s] = e_s and all other values 0 the
    output is 1/(L + n_anchor + Bq) on the visible anchors' coordinates and exactly 0 elsewhere."""
    L, J, Bq, D = 6, 4, 3, 8
    inp = _inputs((L,), 2, 1, D, J, Bq, seed=3, pb=pb)
    inp.q[:] = 0
    inp.v_ctx[:] = 0
    inp.v_blk[:] = 0
    inp.v_spine[:] = 0
    one = W.f32_to_bf16_bits(np.float32([1.0]))[0]
    for s in range(J):
        inp.v_spine[0, s, 0, s] = one
    out, lse = _run(inp)
    for j in range(J):
        na = min(j + pb, J)
        exp = np.zeros(D)
        exp[:na] = 1.0 / (L + na + Bq)
        assert np.allclose(out[0, j], exp[None, None, :], atol=1e-15)
        assert np.all(out[0, j][..., na:] == 0)
        assert np.allclose(lse[0, j], math.log(L + na + Bq))


def test_isolation_and_causality():
    """Changing later spine rows or another branch's block leaves boundary j bit-identical; changing a
    visible anchor or the own block does change it."""
    inp = _inputs((9, 4), 4, 2, 8, J=4, Bq=3, seed=5)
    base, _ = _run(inp)
    j = 1
    mod = _inputs((9, 4), 4, 2, 8, J=4, Bq=3, seed=5)
    mod.k_spine[:, j + 1:] ^= 0x1234
    mod.v_spine[:, j + 1:] ^= 0x0234
    for jj in range(4):
        if jj != j:
            mod.k_blk[:, jj] ^= 0x0111
            mod.v_blk[:, jj] ^= 0x0111
    out, _ = _run(mod)
    assert np.array_equal(out[:, j], base[:, j])
    mod2 = _inputs((9, 4), 4, 2, 8, J=4, Bq=3, seed=5)
    mod2.v_spine[:, j] ^= 0x0100
    assert not np.array_equal(_run(mod2)[0][:, j], base[:, j])
    mod3 = _inputs((9, 4), 4, 2, 8, J=4, Bq=3, seed=5)
    mod3.v_blk[:, j, 0] ^= 0x0100
    assert not np.array_equal(_run(mod3)[0][:, j], base[:, j])
    # requests are independent: request 0's outputs do not depend on request 1's context
    mod4 = _inputs((9, 4), 4, 2, 8, J=4, Bq=3, seed=5)
    mod4.v_ctx[9:] ^= 0x0100
    o4, _ = _run(mod4)
    assert np.array_equal(o4[0], base[0]) and not np.array_equal(o4[1], base[1])


def test_single_boundary_is_library_gqa_attention():
    """Boundary j alone == torch SDPA (enable_gqa) over the serial drafter's inputs: the context, the
    (j + 1)-anchor prefix and the block -- the 'standalone serial forward' the method generalises."""
    inp = _inputs((33, 17), 8, 2, 16, J=5, Bq=4, seed=7)
    out, lse = _run(inp)
    dec = lambda a: torch.from_numpy(OA.bf16_bits_to_f64(a))
    for n in range(2):
        lo, hi = int(inp.ctx_offsets[n]), int(inp.ctx_offsets[n + 1])
        for j in range(5):
            K = torch.cat([dec(inp.k_ctx[lo:hi]), dec(inp.k_spine[n, :j + 1]), dec(inp.k_blk[n, j])], 0)
            V = torch.cat([dec(inp.v_ctx[lo:hi]), dec(inp.v_spine[n, :j + 1]), dec(inp.v_blk[n, j])], 0)
            Q = dec(inp.q[n, j])
            o = torch.nn.functional.scaled_dot_product_attention(
                Q.permute(1, 0, 2)[None], K.permute(1, 0, 2)[None], V.permute(1, 0, 2)[None], enable_gqa=True)[0]
            assert np.abs(o.permute(1, 0, 2).numpy() - out[n, j]).max() < 1e-12
            # LSE against the library logsumexp
            s = torch.einsum("ihd,thd->iht", Q, K.repeat_interleave(4, dim=1)) / math.sqrt(16)
            assert np.abs(torch.logsumexp(s, -1).numpy() - lse[n, j]).max() < 1e-12
    # restricting the boundary range computes the same rows and leaves the rest untouched
    o1, l1 = _run(inp, boundary_lo=2, boundary_hi=3)
    assert np.array_equal(o1[:, 2], out[:, 2]) and np.all(o1[:, :2] == 0) and np.all(np.isinf(l1[:, 3:]))


def test_equal_values_and_scale():
    inp = _inputs((12,), 2, 2, 8, J=3, Bq=2, seed=9)
    v0 = inp.v_ctx[0, 0].copy()
    inp.v_ctx[:] = v0
    inp.v_spine[:] = v0
    inp.v_blk[:] = v0
    out, _ = _run(inp)
    assert np.allclose(out, OA.bf16_bits_to_f64(v0), atol=1e-15)      # convex combination of equal rows
    inp2 = _inputs((12,), 2, 2, 8, J=3, Bq=2, seed=9)
    a, _ = _run(inp2, scale=0.0)          # 0 selects the default 1/sqrt(D)
    b, _ = _run(inp2, scale=1.0 / math.sqrt(8))
    assert np.array_equal(a, b)
    c, _ = _run(inp2, scale=0.5)
    assert not np.allclose(a, c)


def test_brute_force_tiny():
    """Scalar Python loops with math.exp, no numpy linear algebra."""
    inp = _inputs((5, 3), 2, 1, 8, J=3, Bq=2, seed=13)
    out, _ = _run(inp)
    f = lambda a: OA.bf16_bits_to_f64(a)
    q, kc, vc, ks, vs, kb, vb = map(f, (inp.q, inp.k_ctx, inp.v_ctx, inp.k_spine, inp.v_spine, inp.k_blk, inp.v_blk))
    sc = 1.0 / math.sqrt(8)
    for n in range(2):
        lo, hi = int(inp.ctx_offsets[n]), int(inp.ctx_offsets[n + 1])
        for j in range(3):
            for i in range(2):
                for h in range(2):
                    keys = [(kc[t, 0], vc[t, 0]) for t in range(lo, hi)]
                    keys += [(ks[n, s, 0], vs[n, s, 0]) for s in range(j + 1)]
                    keys += [(kb[n, j, t, 0], vb[n, j, t, 0]) for t in range(2)]
                    sco = [sc * sum(q[n, j, i, h, d] * k[d] for d in range(8)) for k, _ in keys]
                    mx = max(sco)
                    e = [math.exp(s - mx) for s in sco]
                    tot = sum(e)
                    for d in range(8):
                        o = sum(e[t] * keys[t][1][d] for t in range(len(keys))) / tot
                        assert abs(o - out[n, j, i, h, d]) < 1e-13


def test_no_block_keys_and_empty_context():
    inp = _inputs((0, 4), 2, 1, 8, J=3, Bq=2, seed=17, pb=0)
    out, lse = OA.draft_all_boundaries(inp.q, inp.k_ctx, inp.v_ctx, inp.ctx_offsets, inp.k_spine, inp.v_spine,
                                       None, None, prefix_base=0)
    # request 0, boundary 0: no context, no anchors, no block keys -> nothing visible
    assert np.all(out[0, 0] == 0) and np.all(np.isinf(lse[0, 0]))
    # request 0, boundary 1: exactly one key (anchor 0) -> output is that value row
    assert np.allclose(out[0, 1], OA.bf16_bits_to_f64(inp.v_spine[0, 0, 0])[None, None, :])


def test_rows_sampler_matches_full():
    inp = _inputs((20, 9), 4, 2, 8, J=3, Bq=2, seed=21)
    out, _ = _run(inp)
    rows = [(0, 0, 0, 0), (1, 2, 1, 3), (0, 1, 1, 2)]
    r = OA.draft_rows(inp.q, inp.k_ctx, inp.v_ctx, inp.ctx_offsets, inp.k_spine, inp.v_spine, inp.k_blk, inp.v_blk, rows)
    for t, (n, j, i, h) in enumerate(rows):
        assert np.abs(r[t] - out[n, j, i, h]).max() < 1e-14      # same definition, BLAS summation order may differ


def test_bf16_rounding_helper():
    x = np.float32([1.0, 1.00390625, 1.005859375, -2.5, 3.0e38, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8])
    r = OA.round_to_bf16(x)
    t = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(r, t)
    assert np.array_equal(OA.bf16_bits_to_f64(W.f32_to_bf16_bits(x)), t.astype(np.float64))


# ----------------------------------------------------------------------------- spine tokens as query rows (next scope row)
def _spine_q(inp, seed):
    rng = np.random.Generator(np.random.Philox(seed))
    b, S, Hkv, D = inp.k_spine.shape
    Hq = inp.q.shape[3]
    return W.f32_to_bf16_bits(rng.standard_normal((b, S, Hq, D), dtype=np.float32))


def test_spine_rows_match_the_figures_mask():
    """Library attention over [context | spine] under the SPINE rows of the figure's mask (from the fixture)."""
    d = 3
    L, Hq, Hkv, D = 5, 4, 2, 16
    inp = _inputs((L,), Hq, Hkv, D, J=d + 1, Bq=d, seed=21)
    qs = _spine_q(inp, 5)
    got = OA.spine_rows(qs, inp.k_ctx, inp.v_ctx, inp.ctx_offsets, inp.k_spine, inp.v_spine)
    S = d + 1
    mask = _gold_mask()[:S, :S]                            # spine rows x spine columns of the figure
    dec = lambda a: torch.from_numpy(OA.bf16_bits_to_f64(a))
    K = torch.cat([dec(inp.k_ctx), dec(inp.k_spine[0])], 0)
    V = torch.cat([dec(inp.v_ctx), dec(inp.v_spine[0])], 0)
    full = torch.cat([torch.ones(S, L, dtype=torch.bool), torch.from_numpy(mask)], 1)
    o = torch.nn.functional.scaled_dot_product_attention(
        dec(qs[0]).permute(1, 0, 2)[None], K.permute(1, 0, 2)[None], V.permute(1, 0, 2)[None],
        attn_mask=full[None, None], enable_gqa=True)[0]
    assert np.abs(o.permute(1, 0, 2).numpy() - got[0]).max() < 1e-12


def test_spine_row_equals_boundary_row_with_the_same_query_and_no_block():
    """Anchor a reads exactly the key set of boundary j = a (prefix_base 1) without its block: putting the
    anchor's query into slot 0 of that boundary must give the same row from the pinned boundary function."""
    inp = _inputs((9, 0), 4, 2, 16, J=4, Bq=2, seed=8)
    qs = _spine_q(inp, 6)
    got = OA.spine_rows(qs, inp.k_ctx, inp.v_ctx, inp.ctx_offsets, inp.k_spine, inp.v_spine)
    q = inp.q.copy()
    q[:, :, 0] = qs                                        # [b][J = S][slot 0][Hq][D]
    ref, _ = OA.draft_all_boundaries(q, inp.k_ctx, inp.v_ctx, inp.ctx_offsets, inp.k_spine, inp.v_spine, None, None,
                                     prefix_base=1)
    assert np.abs(ref[:, :, 0] - got).max() < 1e-12


def test_first_anchor_without_context_returns_its_own_value():
    inp = _inputs((0,), 2, 1, 8, J=3, Bq=2, seed=4)
    qs = _spine_q(inp, 7)
    got = OA.spine_rows(qs, inp.k_ctx, inp.v_ctx, inp.ctx_offsets, inp.k_spine, inp.v_spine)
    v0 = OA.bf16_bits_to_f64(inp.v_spine[0, 0, 0])
    assert np.array_equal(got[0, 0, 0], v0) and np.array_equal(got[0, 0, 1], v0)

