"""Feature-cache append, the plain way (test infrastructure; float64 with the bf16 rounding points written out).

What is computed (paper Alg. 1, the cache update after the head loop: the verified features of t_0..t_r join the
cache C and the rejected suffix t_{r+1..d} is dropped; Sec. 3.3 "Only the head stays on the critical path" says the
same in words; App. D, single-GPU paragraph: the history's features are projected incrementally, never again).

The drafter layers do not read C itself but its projection to keys and values.  Reading taken here (the paper gives
no equations): for every drafter layer, a feature row c at absolute position p becomes

    cn   = bf16( rmsnorm(c) * g )                       input norm of the layer (g = None: no gain)
    k|v  = bf16( cn W_kv^T )                            W_kv rows = [Hkv*D keys | Hkv*D values]
    k    = bf16( rmsnorm_over_D(k) * gk )               per head, when the layer uses QK-norm
    k    = bf16( rope(k, p) )                           rotate-half, when the layer uses RoPE

and the layer's context cache holds one such (k, v) row per history position.  Request n owns cache rows
[row_start[n], row_start[n] + capacity[n]); the first ctx_len[n] of them are filled.  The append writes the rows of
t_0..t_r (r = accept_len[n], r + 1 rows; t_i sits at position ctx_len[n] + i) right behind the filled part and adds
r + 1 to ctx_len[n].  A request whose rows would not fit is left untouched and reported (STATUS_CACHE_FULL).
Each row depends only on its own feature and position, so appending is the same as projecting the longer history
from scratch -- the tests check exactly that.
"""
from __future__ import annotations

from typing import Optional, Sequence

import numpy as np

from .attention import bf16_bits_to_f64, round_to_bf16
from .layer import linear, rmsnorm, rope

STATUS_CACHE_FULL = 4


def _bits(x: np.ndarray) -> np.ndarray:
    """float values on the bf16 grid -> uint16 bit patterns."""
    return (np.ascontiguousarray(round_to_bf16(x)).view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def project_rows(features: np.ndarray, positions: np.ndarray, w_kv: np.ndarray, norm_w: Optional[np.ndarray],
                 knorm_w: Optional[np.ndarray], n_kv_heads: int, head_dim: int, rms_eps: float = 1e-6,
                 rope_theta: float = 1e6, use_rope: bool = True):
    """Keys and values of feature rows.  features [R][F] bf16 bits, positions [R] ints, w_kv [2*Hkv*D][F] bf16 bits,
    gains bf16 bits or None.  Returns (k, v) as bf16 bit patterns [R][Hkv][D]."""
    R = features.shape[0]
    Hkv, D = n_kv_heads, head_dim
    r16 = lambda a: round_to_bf16(a).astype(np.float64)
    c = bf16_bits_to_f64(features)
    cn = r16(rmsnorm(c, None if norm_w is None else bf16_bits_to_f64(norm_w), rms_eps))
    kv = r16(linear(cn, bf16_bits_to_f64(w_kv)))
    k = kv[:, : Hkv * D].reshape(R, Hkv, D)
    v = kv[:, Hkv * D:].reshape(R, Hkv, D)
    if knorm_w is not None:
        k = r16(rmsnorm(k, bf16_bits_to_f64(knorm_w), rms_eps))
    if use_rope:
        k = r16(rope(k.transpose(1, 0, 2), np.asarray(positions), rope_theta)).transpose(1, 0, 2)
    return _bits(k), _bits(v)


def append_verified(k_cache: np.ndarray, v_cache: np.ndarray, row_start: Sequence[int], capacity: Sequence[int],
                    ctx_len: Sequence[int], features: np.ndarray, accept_len: Sequence[int], w_kv: np.ndarray,
                    norm_w: Optional[np.ndarray], knorm_w: Optional[np.ndarray], rms_eps: float = 1e-6,
                    rope_theta: float = 1e6, use_rope: bool = True):
    """One layer's cache update.  k_cache / v_cache [rows][Hkv][D] bf16 bits (copies are returned, the inputs are left
    alone), features [b][J][F] bf16 bits (row i = target feature of t_i; rows above accept_len[n] are ignored).
    Returns (k_cache, v_cache, new ctx_len [b] int64, status)."""
    k_out, v_out = k_cache.copy(), v_cache.copy()
    Hkv, D = k_cache.shape[1], k_cache.shape[2]
    new_len = np.asarray(ctx_len, dtype=np.int64).copy()
    status = 0
    for n in range(features.shape[0]):
        r = int(accept_len[n])
        L = int(ctx_len[n])
        if r < 0 or r >= features.shape[1] or L + r + 1 > int(capacity[n]):
            status |= STATUS_CACHE_FULL
            continue
        pos = L + np.arange(r + 1)
        k, v = project_rows(features[n, : r + 1], pos, w_kv, norm_w, knorm_w, Hkv, D, rms_eps, rope_theta, use_rope)
        row0 = int(row_start[n]) + L
        k_out[row0:row0 + r + 1] = k
        v_out[row0:row0 + r + 1] = v
        new_len[n] = L + r + 1
    return k_out, v_out, new_len, status
