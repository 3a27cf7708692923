"""Verification outcome and branch selection, the plain way (test infrastructure).

Paper Sec. 2.1: the target scores the draft block in one pass; an accepted prefix is kept and a bonus
token is appended -- a correction drawn at the first rejection, or one more target sample after full
acceptance.  Alg. 1 (lines 2-3): verification yields the accepted length r and the bonus b, then the
precomputed branch r is selected.  App. C: under sampling the standard speculative-sampling
rejection rule applies, so a draft can be rejected although it is the target's most likely token.

Indexing used throughout (the paper only says the target "forwards t_{0:d}"): target row i is the
target's prediction for the token after t_0..t_i, so draft t_{i+1} is judged by row i and the bonus
comes from row r.

Everything that decides an integer is done in a stated precision so that a second implementation can
reproduce it bit for bit: comparisons of fp32 inputs as they are, one fp32 multiply for the accept
test, and integer fixed-point weights for the bonus draw.
"""
from __future__ import annotations

from typing import Optional

import numpy as np

STATUS_BAD_TOKEN = 1  # a draft token outside [0, V): treated as rejected at that position


def row_argmax(row: np.ndarray) -> int:
    """Lowest index holding the row maximum.  -0.0 equals +0.0; NaN ranks below every number
    (an all-NaN row gives index 0)."""
    row = np.asarray(row)
    ok = ~np.isnan(row)
    if not ok.any():
        return 0
    mx = row[ok].max()
    return int(np.flatnonzero(ok & (row == mx))[0])


def _finish(n, r, bonus, tokens, reps, accept_len, bonus_out, gather_idx, out_tokens, selected):
    accept_len[n] = r
    bonus_out[n] = bonus
    gather_idx[n] = r
    out_tokens[n, :] = -1
    out_tokens[n, :r] = tokens[n, :r]
    out_tokens[n, r] = bonus
    if reps is not None:
        selected[n] = reps[n, r]          # bit copy of branch r: [Bq][hidden]


def verify_greedy(logits: np.ndarray, draft_tokens: np.ndarray, reps: Optional[np.ndarray] = None):
    """Greedy verification (the setting of the paper's Table 1).

    logits [b][J][V] fp32, draft_tokens [b][J-1] (t_1..t_gamma), reps [b][J][Bq][hidden] (any dtype,
    copied bitwise).  a_i = row_argmax(logits[n][i]); r = number of leading drafts with
    t_i == a_{i-1}; bonus = a_r.  Returns dict(accept_len, bonus, gather_idx, out_tokens, selected,
    status).
    """
    b, J, V = logits.shape
    accept_len = np.zeros(b, np.int32)
    bonus = np.zeros(b, np.int32)
    gather_idx = np.zeros(b, np.int32)
    out_tokens = np.full((b, J), -1, np.int32)
    selected = None if reps is None else np.zeros((b,) + reps.shape[2:], reps.dtype)
    status = 0
    for n in range(b):
        a = [row_argmax(logits[n, i]) for i in range(J)]
        r = 0
        while r < J - 1:
            t = int(draft_tokens[n, r])
            if t < 0 or t >= V:
                status |= STATUS_BAD_TOKEN
                break
            if t != a[r]:
                break
            r += 1
        _finish(n, r, a[r], draft_tokens, reps, accept_len, bonus, gather_idx, out_tokens, selected)
    return dict(accept_len=accept_len, bonus=bonus, gather_idx=gather_idx, out_tokens=out_tokens,
                selected=selected, status=status)


def fixed_point_weights(p_row: np.ndarray, q_row: Optional[np.ndarray]) -> np.ndarray:
    """Integer sampling weights: trunc(max(fl32(p - q), 0) * 2^32) per token (q_row None: trunc(p * 2^32)).
    The fp32 subtraction is a single rounded operation; scaling by 2^32 is exact."""
    p = np.asarray(p_row, dtype=np.float32)
    if q_row is None:
        d = p
    else:
        d = (p - np.asarray(q_row, dtype=np.float32)).astype(np.float32)
    d = np.where(d > 0, d, np.float32(0)).astype(np.float64)      # NaN and negatives -> 0
    return np.floor(d * 4294967296.0).astype(np.uint64)


def draw_from_weights(w: np.ndarray, m: int) -> int:
    """Inverse-CDF draw in vocabulary order with the uniform m * 2^-24 (m integer in [0, 2^24)):
    threshold T = (m * W) >> 24 with W = sum w; result = lowest v whose inclusive prefix sum exceeds T."""
    W = int(w.sum(dtype=np.uint64))
    T = (int(m) * W) >> 24
    c = np.cumsum(w, dtype=np.uint64)
    return int(np.searchsorted(c, np.uint64(T), side="right"))


def verify_sampling(target_probs: np.ndarray, draft_probs: np.ndarray, draft_tokens: np.ndarray,
                    uniforms: np.ndarray, reps: Optional[np.ndarray] = None):
    """Speculative-sampling verification (paper App. C: temperature 1, top-p 1).

    target_probs [b][J][V] fp32, draft_probs [b][J-1][V] fp32, draft_tokens [b][J-1], uniforms [b][J]
    fp32 with uniforms = m * 2^-24.  Draft t_i (i = 1..gamma) is accepted iff
    fl32(u[i-1] * q_{i-1}(t_i)) < p_{i-1}(t_i) -- i.e. with probability min(1, p/q); the scan stops at
    the first rejection (r = i - 1) or accepts all (r = gamma).  The bonus is drawn with u[gamma] from
    the residual max(p_r - q_r, 0) when r < gamma, from p_gamma when r = gamma.  If the residual has no
    weight the draw falls back to p_r, and if that has none either to the lowest-index maximum of p_r.
    """
    b, J, V = target_probs.shape
    g = J - 1
    accept_len = np.zeros(b, np.int32)
    bonus = np.zeros(b, np.int32)
    gather_idx = np.zeros(b, np.int32)
    out_tokens = np.full((b, J), -1, np.int32)
    selected = None if reps is None else np.zeros((b,) + reps.shape[2:], reps.dtype)
    status = 0
    for n in range(b):
        r = 0
        while r < g:
            t = int(draft_tokens[n, r])
            if t < 0 or t >= V:
                status |= STATUS_BAD_TOKEN
                break
            lhs = np.float32(uniforms[n, r]) * np.float32(draft_probs[n, r, t])   # one fp32 multiply
            if not (lhs < np.float32(target_probs[n, r, t])):
                break
            r += 1
        # a uniform is m * 2^-24 with m < 2^24 (App. C draws from [0, 1)); a value of 1 or more is read as the
        # largest uniform, so that the threshold stays below the total weight and the draw inside the vocabulary
        m = min(int(round(float(uniforms[n, g]) * (1 << 24))), (1 << 24) - 1)
        w = fixed_point_weights(target_probs[n, r], draft_probs[n, r] if r < g else None)
        if int(w.sum(dtype=np.uint64)) == 0:
            w = fixed_point_weights(target_probs[n, r], None)
        if int(w.sum(dtype=np.uint64)) == 0:
            tok = row_argmax(target_probs[n, r])
        else:
            tok = draw_from_weights(w, m)
        _finish(n, r, tok, draft_tokens, reps, accept_len, bonus, gather_idx, out_tokens, selected)
    return dict(accept_len=accept_len, bonus=bonus, gather_idx=gather_idx, out_tokens=out_tokens,
                selected=selected, status=status)
