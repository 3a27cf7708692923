"""The critical-path remainder T_Head, the plain way (test infrastructure).

Alg. 1, after the barrier: the precomputed branch r is selected, y_0 = b (the bonus token), and for
i = 1..d the frozen autoregressive head adds to the branch's base logits a correction that depends only
on the previously produced token,
    z_i = l_i + W E(y_{i-1}),        y_i ~ softmax(z_i)
(Sec. 3.2 "Loss": E is the head's own low-rank token embedding, W projects it to the vocabulary).
The base logits are the language-model head applied to the selected branch's final hidden states
(App. D: the drafting side can ship hidden states and the language-model head runs where the head loop runs).

Greedy decoding (the setting of Table 1) takes y_i = argmax z_i, lowest index on ties.  Sampling (App. C: temperature 1,
top-p 1) draws y_i from softmax(z_i) with a SUPPLIED uniform u = m * 2^-24 by the inverse CDF in vocabulary order:
y_i = min{ v : sum_{v' <= v} w_{v'} > u * sum_v w_v },  w_v = exp(z_v - max z)  (NaN logits carry no weight).  Everything is
computed in float64 from the exact values of the bf16 inputs; a second implementation that accumulates
in fp32 can differ only where two logits are closer than its rounding error, which the tests allow for.
"""
from __future__ import annotations

import numpy as np

from .attention import bf16_bits_to_f64
from .verify import row_argmax


def lm_head(hidden_bits: np.ndarray, w_lm_bits: np.ndarray, cols=None) -> np.ndarray:
    """Base logits l = h W_lm^T.  hidden_bits [M][hidden], w_lm_bits [V][hidden] (bf16 bit patterns,
    weights stored [out][in]); `cols` restricts the result to those vocabulary entries.  float64 [M][len]."""
    h = bf16_bits_to_f64(hidden_bits)
    w = w_lm_bits if cols is None else w_lm_bits[np.asarray(cols)]
    return h @ bf16_bits_to_f64(w).T


def ar_logits(base_row: np.ndarray, ar_w_bits: np.ndarray, ar_e_bits: np.ndarray, y_prev: int) -> np.ndarray:
    """z = l + W E(y_prev): base_row [V] float64, ar_w_bits [V][rank] (W), ar_e_bits [V][rank] (E, one
    row per token).  float64 [V]."""
    e = bf16_bits_to_f64(ar_e_bits[y_prev])
    return np.asarray(base_row, np.float64) + bf16_bits_to_f64(ar_w_bits) @ e


def ar_head_greedy(base_logits: np.ndarray, ar_w_bits: np.ndarray, ar_e_bits: np.ndarray, bonus: int) -> np.ndarray:
    """The head loop of one request: base_logits [d][V] (rows l_1..l_d of the selected branch), y_0 = bonus;
    returns y_1..y_d (int32)."""
    d = base_logits.shape[0]
    out = np.zeros(d, np.int32)
    y = int(bonus)
    for i in range(d):
        y = row_argmax(ar_logits(base_logits[i], ar_w_bits, ar_e_bits, y))
        out[i] = y
    return out


def sample_from_logits(z: np.ndarray, u: float) -> int:
    """Inverse-CDF draw from softmax(z) in vocabulary order with the uniform u in [0, 1): the lowest v whose inclusive
    cumulative weight exceeds u times the total.  float64 throughout; NaN logits weigh nothing; a row without any
    weight (all NaN / -inf) gives token 0."""
    z = np.asarray(z, np.float64)
    finite_max = np.nanmax(np.where(np.isnan(z), -np.inf, z)) if z.size else -np.inf
    if not np.isfinite(finite_max):
        return 0
    w = np.where(np.isnan(z), 0.0, np.exp(z - finite_max))
    c = np.cumsum(w)
    v = int(np.searchsorted(c, float(u) * c[-1], side="right"))
    return min(v, int(np.nonzero(w > 0)[0][-1]))      # u * total rounding up to the total: the last token with weight


def ar_head_sampling(base_logits: np.ndarray, ar_w_bits: np.ndarray, ar_e_bits: np.ndarray, bonus: int,
                     uniforms: np.ndarray) -> np.ndarray:
    """The sampling head loop of one request: y_0 = bonus, y_i drawn from softmax(l_i + W E(y_{i-1})) with uniforms[i-1]."""
    d = base_logits.shape[0]
    out = np.zeros(d, np.int32)
    y = int(bonus)
    for i in range(d):
        y = sample_from_logits(ar_logits(base_logits[i], ar_w_bits, ar_e_bits, y), float(uniforms[i]))
        out[i] = y
    return out


def draft_head_sampling(sel_reps_bits: np.ndarray, w_lm_bits: np.ndarray, ar_w_bits: np.ndarray, ar_e_bits: np.ndarray,
                        bonus: np.ndarray, uniforms: np.ndarray) -> np.ndarray:
    """All requests: uniforms [b][d] (each m * 2^-24); returns [b][d] int32."""
    b, d, _ = sel_reps_bits.shape
    out = np.zeros((b, d), np.int32)
    for n in range(b):
        out[n] = ar_head_sampling(lm_head(sel_reps_bits[n], w_lm_bits), ar_w_bits, ar_e_bits, int(bonus[n]), uniforms[n])
    return out


def draft_head_greedy(sel_reps_bits: np.ndarray, w_lm_bits: np.ndarray, ar_w_bits: np.ndarray, ar_e_bits: np.ndarray,
                      bonus: np.ndarray) -> np.ndarray:
    """All requests: sel_reps_bits [b][d][hidden] (the selected branches), bonus [b]; returns [b][d] int32."""
    b, d, _ = sel_reps_bits.shape
    out = np.zeros((b, d), np.int32)
    for n in range(b):
        out[n] = ar_head_greedy(lm_head(sel_reps_bits[n], w_lm_bits), ar_w_bits, ar_e_bits, int(bonus[n]))
    return out
