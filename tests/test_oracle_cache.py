"""Pins for oracle/cache.py (CPU only): Alg. 1's cache update "C <- [C, C_new(0..r)]" as keys/values of a drafter layer.
What fixes the result: the update is a LIST APPEND of per-row projections -- so (a) the appended cache must equal the
projection of the longer history built from scratch (here with torch library routines, another code path), (b) two
rounds equal one round over the concatenated accepted rows, bit for bit, (c) nothing outside the r + 1 new rows of a
request changes, and (d) the attention over the appended cache equals the attention over a packed copy of it."""
import numpy as np
import torch
import torch.nn.functional as F

import workloads as W
from oracle import attention as OA
from oracle import cache as OC


def _library_projection(feat_bits, positions, w_bits, g_bits, gk_bits, Hkv, D, theta=1e6, eps=1e-6):
    """Keys/values of a whole history in float64 from torch routines, WITHOUT the bf16 rounding points; rotary
    embedding as a complex multiplication of the pair (d, d + D/2)."""
    d = lambda b: torch.from_numpy(OA.bf16_bits_to_f64(b))
    c = d(feat_bits)
    cn = F.rms_norm(c, (c.shape[-1],), d(g_bits), eps)
    kv = F.linear(cn, d(w_bits))
    R = c.shape[0]
    k = kv[:, : Hkv * D].reshape(R, Hkv, D)
    v = kv[:, Hkv * D:].reshape(R, Hkv, D)
    k = F.rms_norm(k, (D,), d(gk_bits), eps)
    z = torch.complex(k[..., : D // 2], k[..., D // 2:])
    ang = torch.tensor(positions, dtype=torch.float64)[:, None] * theta ** (-2.0 * torch.arange(D // 2, dtype=torch.float64) / D)
    z = z * torch.polar(torch.ones_like(ang), ang)[:, None, :]
    return torch.cat([z.real, z.imag], -1).numpy(), v.numpy()


def _setup(seed=3, accept=None, slack=0):
    return W.make_cache_inputs((9, 0, 5), 4, 32, 2, 16, 1, seed, accept_len=accept, slack=slack)


def test_append_equals_projection_of_the_longer_history():
    ci = _setup(accept=[2, 3, 0])
    k2, v2, new_len, st = OC.append_verified(ci.k_cache[0], ci.v_cache[0], ci.row_start, ci.capacity, ci.ctx_len, ci.features,
                                             ci.accept_len, ci.w_kv[0], ci.norm_w[0], ci.knorm_w[0])
    assert st == 0 and new_len.tolist() == [12, 4, 6]                     # L + r + 1 (r = 0: the previous bonus alone)
    for n, (L, r) in enumerate(zip(ci.ctx_len, ci.accept_len)):
        row0 = int(ci.row_start[n] + L)
        kl, vl = _library_projection(ci.features[n, : r + 1], list(range(L, L + r + 1)), ci.w_kv[0], ci.norm_w[0], ci.knorm_w[0], 2, 16)
        got_k, got_v = OA.bf16_bits_to_f64(k2[row0:row0 + r + 1]), OA.bf16_bits_to_f64(v2[row0:row0 + r + 1])
        # the library path has no rounding points: agreement within the three bf16 roundings of a key (two of a value)
        assert np.all(np.abs(got_k - kl) <= 3 * 2.0 ** -8 * np.abs(kl).max(-1, keepdims=True) + 1e-6)
        assert np.all(np.abs(got_v - vl) <= 2 * 2.0 ** -8 * np.abs(vl).max(-1, keepdims=True) + 1e-6)
    # everything else is untouched: other rows of k and v, including the sentinel rows behind the new length
    touched = np.zeros(k2.shape[0], bool)
    for n, (L, r) in enumerate(zip(ci.ctx_len, ci.accept_len)):
        touched[ci.row_start[n] + L: ci.row_start[n] + L + r + 1] = True
    assert np.array_equal(k2[~touched], ci.k_cache[0][~touched]) and np.array_equal(v2[~touched], ci.v_cache[0][~touched])
    assert not np.any(k2[touched] == 0x7FC1)


def test_two_rounds_equal_one_round_over_the_concatenation():
    ci = W.make_cache_inputs((7, 3), 6, 32, 2, 16, 1, 8, accept_len=[5, 5])
    args = (ci.w_kv[0], ci.norm_w[0], ci.knorm_w[0])
    # one round: rows 0..5 of both requests
    k1, v1, l1, _ = OC.append_verified(ci.k_cache[0], ci.v_cache[0], ci.row_start, ci.capacity, ci.ctx_len, ci.features, [5, 5], *args)
    # two rounds: rows 0..1 (r = 1), then the next four rows presented as a new block (r = 3)
    ka, va, la, _ = OC.append_verified(ci.k_cache[0], ci.v_cache[0], ci.row_start, ci.capacity, ci.ctx_len, ci.features, [1, 1], *args)
    kb, vb, lb, _ = OC.append_verified(ka, va, ci.row_start, ci.capacity, la, ci.features[:, 2:], [3, 3], *args)
    assert np.array_equal(l1, lb) and np.array_equal(k1, kb) and np.array_equal(v1, vb)
    # ... and a history projected from scratch in one call gives the same bits again (the positions are what matters)
    n = 1
    kk, vv = OC.project_rows(ci.features[n, :6], np.arange(3, 9), *args, 2, 16)
    assert np.array_equal(k1[ci.row_start[n] + 3: ci.row_start[n] + 9], kk)


def test_position_enters_through_the_rotation_only():
    """The same feature row appended behind histories of different length: values identical, keys rotated --
    a query rotated by the same offset scores it the same."""
    from oracle import layer as OL
    feats = W.make_cache_inputs((4,), 1, 32, 1, 16, 1, 5).features
    ci = W.make_cache_inputs((4,), 1, 32, 1, 16, 1, 5)
    ka, va = OC.project_rows(feats[0, :1], np.array([4]), ci.w_kv[0], ci.norm_w[0], None, 1, 16)
    kb, vb = OC.project_rows(feats[0, :1], np.array([11]), ci.w_kv[0], ci.norm_w[0], None, 1, 16)
    assert np.array_equal(va, vb) and not np.array_equal(ka, kb)
    q = np.random.default_rng(0).standard_normal((1, 1, 16))
    sa = (OL.rope(q, np.array([6]), 1e6) * OA.bf16_bits_to_f64(ka)).sum()
    sb = (OL.rope(q, np.array([13]), 1e6) * OA.bf16_bits_to_f64(kb)).sum()
    assert abs(sa - sb) < 0.05 * np.abs(OA.bf16_bits_to_f64(ka)).sum() * 2.0 ** -7 + 1e-2    # equal up to the key's bf16 rounding


def test_full_cache_is_left_alone_and_reported():
    ci = W.make_cache_inputs((5, 5), 3, 32, 2, 16, 1, 2, accept_len=[2, 2])
    cap = ci.capacity.copy(); cap[1] = 7                                 # 5 + 3 rows do not fit into 7
    k2, v2, new_len, st = OC.append_verified(ci.k_cache[0], ci.v_cache[0], ci.row_start, cap, ci.ctx_len, ci.features,
                                             ci.accept_len, ci.w_kv[0], ci.norm_w[0], ci.knorm_w[0])
    assert st == OC.STATUS_CACHE_FULL and new_len.tolist() == [8, 5]
    r1 = slice(int(ci.row_start[1]), int(ci.row_start[1] + ci.capacity[1]))
    assert np.array_equal(k2[r1], ci.k_cache[0][r1])


def test_attention_reads_the_appended_cache_like_a_packed_one():
    """The draft call's context = the filled rows of each request, wherever the cache keeps them."""
    sh = W.AttnShape((9, 5), 4, 2, 16, 3, 2)
    inp = W.make_attn_inputs(sh, 4)
    ci = W.make_cache_inputs(sh.ctx_lens, 3, 32, 2, 16, 1, 4, accept_len=[1, 2])
    k2, v2, new_len, _ = OC.append_verified(ci.k_cache[0], ci.v_cache[0], ci.row_start, ci.capacity, ci.ctx_len, ci.features,
                                            ci.accept_len, ci.w_kv[0], ci.norm_w[0], ci.knorm_w[0])
    starts = np.concatenate([ci.row_start, [ci.row_start[-1] + ci.capacity[-1]]])
    got, _ = OA.draft_all_boundaries(inp.q, k2, v2, starts, inp.k_spine, inp.v_spine, inp.k_blk, inp.v_blk, ctx_lens=new_len)
    packed_k = np.concatenate([k2[s:s + L] for s, L in zip(ci.row_start, new_len)])
    packed_v = np.concatenate([v2[s:s + L] for s, L in zip(ci.row_start, new_len)])
    off = np.concatenate([[0], np.cumsum(new_len)])
    want, _ = OA.draft_all_boundaries(inp.q, packed_k, packed_v, off, inp.k_spine, inp.v_spine, inp.k_blk, inp.v_blk)
    assert np.array_equal(got, want) and np.isfinite(got).all()          # a sentinel (NaN) row in the context would show
