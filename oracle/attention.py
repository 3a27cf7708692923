"""All-boundary attention, the plain way (test infrastructure; float64).

What is computed (paper Sec. 3.2 "Shared causal spine with isolated bidirectional branches" and the
caption of Fig. 4): the d+1 acceptance boundaries each own a block of mask slots.  A slot of
boundary j reads (a) every row of the cached target context, (b) the anchor prefix of that boundary
-- the first j + prefix_base rows of the feature-less spine (prefix_base = 1: the previous bonus
plus j accepted drafts, Sec. 3.1 "k = r + 1 anchor tokens") -- and (c) the slots of its own block,
bidirectionally.  It reads nothing of any other boundary's block and no later spine row.

Because the branches are isolated, the whole pass is d+1 independent softmax attentions.  This file
evaluates them exactly so: for each (request, boundary) it concatenates the visible keys and runs an
ordinary softmax attention.  The combined tree mask is never built here (tests build it, from the
figure, and check that this file agrees with it).
"""
from __future__ import annotations

import math
from typing import Iterable, Optional, Tuple

import numpy as np


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact value of bf16 bit patterns (uint16) as float64."""
    return (np.asarray(bits).astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round (via fp32, nearest-even) to the bf16 grid; returned as float32 holding bf16 values."""
    u = np.ascontiguousarray(np.asarray(x, dtype=np.float32)).view(np.uint32)
    r = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return (((u + r) >> np.uint32(16)) << np.uint32(16)).view(np.float32)


def softmax_attention(q: np.ndarray, k: np.ndarray, v: np.ndarray, scale: float) -> Tuple[np.ndarray, np.ndarray]:
    """Plain attention of query rows q [R, D] over keys k [T, D] / values v [T, D].

    s = scale * q k^T;  o = softmax_rows(s) v;  lse = log sum exp(s) (natural log).
    No visible key (T == 0): o = 0, lse = -inf.
    """
    R, D = q.shape
    if k.shape[0] == 0:
        return np.zeros((R, v.shape[1] if v.ndim == 2 else D)), np.full(R, -np.inf)
    s = scale * (q @ k.T)
    m = s.max(axis=1, keepdims=True)
    e = np.exp(s - m)
    l = e.sum(axis=1, keepdims=True)
    o = (e @ v) / l
    return o, (m + np.log(l))[:, 0]


def context_rows(n: int, ctx_offsets, ctx_lens=None) -> Tuple[int, int]:
    """Cache rows [lo, hi) that hold request n's context.  Packed layout (ctx_lens None): request n owns rows
    ctx_offsets[n] .. ctx_offsets[n + 1].  Layout with slack for in-place appends: rows ctx_offsets[n] ..
    ctx_offsets[n] + ctx_lens[n] are filled, whatever lies behind them is not part of the context."""
    lo = int(ctx_offsets[n])
    return lo, (int(ctx_offsets[n + 1]) if ctx_lens is None else lo + int(ctx_lens[n]))


def visible_keys(n: int, j: int, g: int, k_ctx, v_ctx, ctx_offsets, k_spine, v_spine, k_blk, v_blk,
                 prefix_base: int, ctx_lens=None) -> Tuple[np.ndarray, np.ndarray]:
    """Keys/values (float64) that boundary j of request n reads for KV head g, in the order
    context, anchor prefix, own block."""
    lo, hi = context_rows(n, ctx_offsets, ctx_lens)
    S = k_spine.shape[1]
    n_anchor = max(0, min(j + prefix_base, S))
    ks = [bf16_bits_to_f64(k_ctx[lo:hi, g]), bf16_bits_to_f64(k_spine[n, :n_anchor, g])]
    vs = [bf16_bits_to_f64(v_ctx[lo:hi, g]), bf16_bits_to_f64(v_spine[n, :n_anchor, g])]
    if k_blk is not None:
        ks.append(bf16_bits_to_f64(k_blk[n, j, :, g]))
        vs.append(bf16_bits_to_f64(v_blk[n, j, :, g]))
    return np.concatenate(ks, axis=0), np.concatenate(vs, axis=0)


def draft_all_boundaries(q, k_ctx, v_ctx, ctx_offsets, k_spine, v_spine, k_blk, v_blk,
                         prefix_base: int = 1, scale: Optional[float] = None,
                         boundary_lo: int = 0, boundary_hi: Optional[int] = None, ctx_lens=None):
    """Representations of every boundary in [boundary_lo, boundary_hi).

    q [b][J][Bq][Hq][D], k/v tensors as bf16 bit patterns (see workloads.AttnInputs); query head h
    reads KV head h // (Hq // Hkv).  Returns (out [b][J][Bq][Hq][D] float64, lse [b][J][Bq][Hq]);
    boundaries outside the range are left at 0 / -inf.
    """
    b, J, Bq, Hq, D = q.shape
    Hkv = k_spine.shape[2]
    G = Hq // Hkv
    if scale is None or scale == 0:
        scale = 1.0 / math.sqrt(D)
    if boundary_hi is None:
        boundary_hi = J
    out = np.zeros((b, J, Bq, Hq, D))
    lse = np.full((b, J, Bq, Hq), -np.inf)
    for n in range(b):
        for j in range(boundary_lo, boundary_hi):
            for g in range(Hkv):
                keys, vals = visible_keys(n, j, g, k_ctx, v_ctx, ctx_offsets, k_spine, v_spine, k_blk, v_blk,
                                          prefix_base, ctx_lens)
                for h in range(g * G, (g + 1) * G):
                    o, l = softmax_attention(bf16_bits_to_f64(q[n, j, :, h]), keys, vals, scale)
                    out[n, j, :, h] = o
                    lse[n, j, :, h] = l
    return out, lse


def draft_rows(q, k_ctx, v_ctx, ctx_offsets, k_spine, v_spine, k_blk, v_blk,
               rows: Iterable[Tuple[int, int, int, int]], prefix_base: int = 1, scale: Optional[float] = None):
    """The same definition evaluated only for the listed (n, j, i, h) query rows -> [len(rows)][D].
    Used to check full-size runs on a sample of outputs."""
    b, J, Bq, Hq, D = q.shape
    G = Hq // k_spine.shape[2]
    if scale is None or scale == 0:
        scale = 1.0 / math.sqrt(D)
    res = []
    for (n, j, i, h) in rows:
        keys, vals = visible_keys(n, j, h // G, k_ctx, v_ctx, ctx_offsets, k_spine, v_spine, k_blk, v_blk, prefix_base)
        o, _ = softmax_attention(bf16_bits_to_f64(q[n, j, i:i + 1, h]), keys, vals, scale)
        res.append(o[0])
    return np.stack(res) if res else np.zeros((0, D))


def spine_rows(q_spine, k_ctx, v_ctx, ctx_offsets, k_spine, v_spine, scale: Optional[float] = None, ctx_lens=None):
    """The spine tokens as query rows (Sec. 3.2, Fig. 4: the anchors run causally among themselves and see the
    whole cached context): anchor a of request n attends the context and spine rows 0..a, itself included.
    q_spine [b][S][Hq][D], k_spine / v_spine [b][S][Hkv][D] (bf16 bit patterns).  Returns float64 [b][S][Hq][D].
    Not part of the call that is built so far (there the spine's K/V are inputs); kept here, pinned, for the
    backbone pass that produces them itself."""
    b, S, Hq, D = q_spine.shape
    G = Hq // k_spine.shape[2]
    if scale is None or scale == 0:
        scale = 1.0 / math.sqrt(D)
    out = np.zeros((b, S, Hq, D))
    for n in range(b):
        lo, hi = context_rows(n, ctx_offsets, ctx_lens)
        for a in range(S):
            for h in range(Hq):
                g = h // G
                keys = np.concatenate([bf16_bits_to_f64(k_ctx[lo:hi, g]), bf16_bits_to_f64(k_spine[n, :a + 1, g])], axis=0)
                vals = np.concatenate([bf16_bits_to_f64(v_ctx[lo:hi, g]), bf16_bits_to_f64(v_spine[n, :a + 1, g])], axis=0)
                o, _ = softmax_attention(bf16_bits_to_f64(q_spine[n, a:a + 1, h]), keys, vals, scale)
                out[n, a, h] = o[0]
    return out


def tree_mask(d: int, n_slots: int, prefix_base: int = 1) -> np.ndarray:
    """Visibility among the non-context tokens for draft length d: rows/cols ordered as the d+1 spine
    tokens followed by d+1 branches of n_slots mask tokens (Fig. 4 uses n_slots = d).  True = visible.
    Spine row s sees spine columns <= s; a slot of branch j sees spine columns < j + prefix_base and
    the columns of branch j.  (Every row additionally sees all context columns, not part of this
    matrix.)  Exists so that tests can compare it with the figure; the attention above never uses it.
    """
    S = d + 1
    T = S + S * n_slots
    m = np.zeros((T, T), dtype=bool)
    for s in range(S):
        m[s, : s + 1] = True
    for j in range(S):
        r0 = S + j * n_slots
        m[r0:r0 + n_slots, : min(j + prefix_base, S)] = True
        m[r0:r0 + n_slots, r0:r0 + n_slots] = True
    return m
