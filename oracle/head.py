"""The critical-path remainder T_Head, the plain way (test infrastructure).

Alg. 1, after the barrier: the precomputed branch r is selected, y_0 = b (the bonus token), and for
i = 1..d the frozen autoregressive head adds to the branch's base logits a correction that depends only
on the previously produced token,
    z_i = l_i + W E(y_{i-1}),        y_i ~ softmax(z_i)
(Sec. 3.2 "Loss": E is the head's own low-rank token embedding, W projects it to the vocabulary).
The base logits are the language-model head applied to the selected branch's final hidden states
(App. D: the drafting side can ship hidden states and the language-model head runs where the head loop runs).

Greedy decoding (the setting of Table 1) takes y_i = argmax z_i, lowest index on ties.  Everything is
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


def draft_head_greedy(sel_reps_bits: np.ndarray, w_lm_bits: np.ndarray, ar_w_bits: np.ndarray, ar_e_bits: np.ndarray,
                      bonus: np.ndarray) -> np.ndarray:
    """All requests: sel_reps_bits [b][d][hidden] (the selected branches), bonus [b]; returns [b][d] int32."""
    b, d, _ = sel_reps_bits.shape
    out = np.zeros((b, d), np.int32)
    for n in range(b):
        out[n] = ar_head_greedy(lm_head(sel_reps_bits[n], w_lm_bits), ar_w_bits, ar_e_bits, int(bonus[n]))
    return out
