"""One drafter backbone block around the all-boundary attention (test infrastructure).

PARITY UNPINNED (structure): the paper lists the parts of a backbone block (Sec. 3.1, trainable/frozen
split: the attention, the MLP and the norms around them) and fixes no layer equations.  The block below is
this build's reading -- the pre-norm block of the Qwen3 family the drafters are trained for:

    xn  = bf16( rmsnorm(x) * g1 )
    qkv = bf16( xn W_qkv^T )                      rows split as [Hq*D | Hkv*D | Hkv*D]
    q,k = bf16( rmsnorm_over_D(.) * gain )        per head, when QK-norm is on
    q,k = bf16( rope(., position) )               rotate-half, when RoPE is on
    a   = bf16( all-boundary attention )          the mask slots' own k, v are the block keys/values;
                                                  context and spine K/V are inputs (already projected)
    h1  = fp32( x + a W_o^T )
    hn  = bf16( rmsnorm(h1) * g2 )
    act = bf16( silu(hn W_gate^T) * (hn W_up^T) )
    y   = fp32( h1 + act W_down^T )

The bf16 roundings are part of the definition ("bf16 inputs, fp32 accumulate" for every product); the
sums themselves are taken in float64 here.  Positions: spine row s of request n sits at L_n + s; the
unknown bonus of boundary j would sit at L_n + j + 1; mask slot i of boundary j therefore sits at
L_n + j + 2 + i.  The individual pieces (rmsnorm, silu, rope, matmul) are pinned by closed forms in
the tests (linear / swiglu_linear by integer-exact scalar loops that a transposed weight or swapped
gate/up halves would fail); the composition is pinned by nothing but this text.
"""
from __future__ import annotations

import math
from typing import Optional

import numpy as np

from .attention import bf16_bits_to_f64, round_to_bf16, softmax_attention


def _r16(x):
    """Round to bf16, keep as float64 values."""
    return round_to_bf16(x).astype(np.float64)


def rmsnorm(x: np.ndarray, gain: Optional[np.ndarray], eps: float) -> np.ndarray:
    """x / sqrt(mean(x^2) + eps) * gain over the last axis (float64)."""
    ms = (x * x).mean(axis=-1, keepdims=True)
    y = x / np.sqrt(ms + eps)
    return y if gain is None else y * gain


def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


def linear(x: np.ndarray, w: np.ndarray) -> np.ndarray:
    """x [M][K] times w [N][K] transposed (weights stored [out][in]), float64."""
    return x @ w.T


def swiglu_linear(x: np.ndarray, w_gate_up: np.ndarray) -> np.ndarray:
    """silu(x Wg^T) * (x Wu^T) with w_gate_up rows [0, I) = gate and [I, 2I) = up; rounded to bf16."""
    I = w_gate_up.shape[0] // 2
    gu = linear(x, w_gate_up)
    return _r16(silu(gu[:, :I]) * gu[:, I:])


def rope(x: np.ndarray, pos: np.ndarray, theta: float) -> np.ndarray:
    """Rotate-half rotary embedding.  x [..., R, D] with one position per row R (pos [R]).
    Pair (d, d + D/2) is rotated by angle pos * theta^(-2d/D)."""
    D = x.shape[-1]
    half = D // 2
    inv = theta ** (-2.0 * np.arange(half) / D)
    ang = pos[:, None].astype(np.float64) * inv[None, :]
    c, s = np.cos(ang), np.sin(ang)
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


class LayerOracle:
    """Holds the decoded weights so that several boundaries can be evaluated without re-decoding.

    `boundary(n, j)` is the block for the mask slots of one boundary with the spine's keys/values SUPPLIED (the call
    that takes them as inputs).  `request(n, x_rows)` is the block for ALL rows of a request -- the d+1 spine tokens as
    causal query rows (Sec. 3.2, Fig. 4: every anchor reads the cache, itself and the earlier anchors) followed by
    nothing else changed for the mask slots -- with the spine's keys/values PRODUCED by the block itself, which is what
    lets blocks be stacked (`backbone`)."""

    def __init__(self, lin, attn_in, prefix_base: int = 1, scale: Optional[float] = None):
        sh = attn_in.shape
        self.sh, self.lsh, self.ain = sh, lin.shape, attn_in
        self.prefix_base = prefix_base
        self.scale = scale if scale else 1.0 / math.sqrt(sh.head_dim)
        self.x = lin.x
        self.w_qkv = bf16_bits_to_f64(lin.w_qkv)
        self.w_o = bf16_bits_to_f64(lin.w_o)
        self.w_gu = bf16_bits_to_f64(lin.w_gate_up)
        self.w_down = bf16_bits_to_f64(lin.w_down)
        self.g1 = bf16_bits_to_f64(lin.rms1_w)
        self.g2 = bf16_bits_to_f64(lin.rms2_w)
        self.gq = bf16_bits_to_f64(lin.qnorm_w) if self.lsh.qk_norm else None
        self.gk = bf16_bits_to_f64(lin.knorm_w) if self.lsh.qk_norm else None

    def qkv_rows(self, n: int, j: int):
        """q [Bq][Hq][D], k [Bq][Hkv][D], v [Bq][Hkv][D] of boundary j's mask slots (bf16 values, float64)."""
        sh, L = self.sh, self.lsh
        Hq, Hkv, D, Bq = sh.n_q_heads, sh.n_kv_heads, sh.head_dim, sh.block
        x = bf16_bits_to_f64(self.x[n, j])                                   # [Bq][hidden]
        xn = _r16(rmsnorm(x, self.g1, L.rms_eps))
        qkv = _r16(linear(xn, self.w_qkv))
        q = qkv[:, : Hq * D].reshape(Bq, Hq, D)
        k = qkv[:, Hq * D:(Hq + Hkv) * D].reshape(Bq, Hkv, D)
        v = qkv[:, (Hq + Hkv) * D:].reshape(Bq, Hkv, D)
        if L.qk_norm:
            q = _r16(rmsnorm(q, self.gq, L.rms_eps))
            k = _r16(rmsnorm(k, self.gk, L.rms_eps))
        if L.use_rope:
            pos = sh.ctx_lens[n] + j + 2 + np.arange(Bq)
            q = _r16(rope(q.transpose(1, 0, 2), pos, L.rope_theta)).transpose(1, 0, 2)
            k = _r16(rope(k.transpose(1, 0, 2), pos, L.rope_theta)).transpose(1, 0, 2)
        return x, q, k, v

    def boundary(self, n: int, j: int):
        """Forward of boundary j of request n.  Returns dict with y [Bq][hidden] (fp32 values) and the
        intermediates q, k, v, a, h1."""
        sh, L, A = self.sh, self.lsh, self.ain
        Hq, Hkv, D, Bq = sh.n_q_heads, sh.n_kv_heads, sh.head_dim, sh.block
        G = Hq // Hkv
        x, q, k, v = self.qkv_rows(n, j)
        lo, hi = int(A.ctx_offsets[n]), int(A.ctx_offsets[n + 1])
        n_anchor = max(0, min(j + self.prefix_base, sh.spine))
        a = np.zeros((Bq, Hq, D))
        for g in range(Hkv):
            keys = np.concatenate([bf16_bits_to_f64(A.k_ctx[lo:hi, g]), bf16_bits_to_f64(A.k_spine[n, :n_anchor, g]), k[:, g]])
            vals = np.concatenate([bf16_bits_to_f64(A.v_ctx[lo:hi, g]), bf16_bits_to_f64(A.v_spine[n, :n_anchor, g]), v[:, g]])
            for h in range(g * G, (g + 1) * G):
                a[:, h], _ = softmax_attention(q[:, h], keys, vals, self.scale)
        a = _r16(a).reshape(Bq, Hq * D)
        h1 = (x + linear(a, self.w_o)).astype(np.float32).astype(np.float64)
        hn = _r16(rmsnorm(h1, self.g2, L.rms_eps))
        act = swiglu_linear(hn, self.w_gu)
        y = (h1 + linear(act, self.w_down)).astype(np.float32)
        return dict(y=y, q=q, k=k, v=v, a=a, h1=h1.astype(np.float32))

    # ------------------------------------------------------------------ all rows of a request, spine included
    def request(self, n: int, x_rows: np.ndarray, k_ctx=None, v_ctx=None, ctx_lens=None):
        """x_rows [J*Bq + S][hidden] float64 (bf16 values): the request's mask-slot rows in (boundary, slot) order, then
        its S spine rows.  Context keys/values default to the ones this oracle was built with.  Returns y [J*Bq + S][hidden]
        (fp32 values, float64 array) and the intermediates.  Positions: spine row s at L + s, slot i of boundary j at
        L + j + 2 + i."""
        sh, L, A = self.sh, self.lsh, self.ain
        Hq, Hkv, D, Bq, J, S = sh.n_q_heads, sh.n_kv_heads, sh.head_dim, sh.block, sh.n_boundaries, sh.spine
        G = Hq // Hkv
        k_ctx = A.k_ctx if k_ctx is None else k_ctx
        v_ctx = A.v_ctx if v_ctx is None else v_ctx
        lo = int(A.ctx_offsets[n])
        Ln = int(A.ctx_offsets[n + 1]) - lo if ctx_lens is None else int(ctx_lens[n])
        R = J * Bq + S
        assert x_rows.shape[0] == R
        x = np.asarray(x_rows, dtype=np.float64)
        xn = _r16(rmsnorm(x, self.g1, L.rms_eps))
        qkv = _r16(linear(xn, self.w_qkv))
        q = qkv[:, : Hq * D].reshape(R, Hq, D)
        k = qkv[:, Hq * D:(Hq + Hkv) * D].reshape(R, Hkv, D)
        v = qkv[:, (Hq + Hkv) * D:].reshape(R, Hkv, D)
        if L.qk_norm:
            q = _r16(rmsnorm(q, self.gq, L.rms_eps))
            k = _r16(rmsnorm(k, self.gk, L.rms_eps))
        if L.use_rope:
            pos = np.concatenate([Ln + j + 2 + np.arange(Bq) for j in range(J)] + [Ln + np.arange(S)])
            q = _r16(rope(q.transpose(1, 0, 2), pos, L.rope_theta)).transpose(1, 0, 2)
            k = _r16(rope(k.transpose(1, 0, 2), pos, L.rope_theta)).transpose(1, 0, 2)
        ks, vs = k[J * Bq:], v[J * Bq:]                       # the spine's own keys/values, produced here
        a = np.zeros((R, Hq, D))
        for g in range(Hkv):
            kc, vc = bf16_bits_to_f64(k_ctx[lo:lo + Ln, g]), bf16_bits_to_f64(v_ctx[lo:lo + Ln, g])
            for h in range(g * G, (g + 1) * G):
                for j in range(J):                            # a branch: cache, its anchor prefix, its own block
                    na = max(0, min(j + self.prefix_base, S))
                    r0 = j * Bq
                    keys = np.concatenate([kc, ks[:na, g], k[r0:r0 + Bq, g]])
                    vals = np.concatenate([vc, vs[:na, g], v[r0:r0 + Bq, g]])
                    a[r0:r0 + Bq, h], _ = softmax_attention(q[r0:r0 + Bq, h], keys, vals, self.scale)
                for s_ in range(S):                           # an anchor: cache, the earlier anchors, itself
                    keys = np.concatenate([kc, ks[: s_ + 1, g]])
                    vals = np.concatenate([vc, vs[: s_ + 1, g]])
                    a[J * Bq + s_, h], _ = softmax_attention(q[J * Bq + s_: J * Bq + s_ + 1, h], keys, vals, self.scale)
        a = _r16(a).reshape(R, Hq * D)
        h1 = (x + linear(a, self.w_o)).astype(np.float32).astype(np.float64)
        hn = _r16(rmsnorm(h1, self.g2, L.rms_eps))
        act = swiglu_linear(hn, self.w_gu)
        y = (h1 + linear(act, self.w_down)).astype(np.float32).astype(np.float64)
        return dict(y=y, q=q, k=k, v=v, a=a, h1=h1)


def backbone(layers, n: int, x_rows: np.ndarray, caches=None, ctx_lens=None) -> np.ndarray:
    """A stack of blocks on one request's rows: block l reads block l-1's output rounded to bf16 (the residual
    stream between blocks is bf16) and its own context cache.  layers: LayerOracle objects; caches: optional list of
    (k_ctx, v_ctx) per layer.  Returns the last block's y [J*Bq + S][hidden] (fp32 values)."""
    x = np.asarray(x_rows, dtype=np.float64)
    y = None
    for l, lay in enumerate(layers):
        kc, vc = caches[l] if caches is not None else (None, None)
        y = lay.request(n, x, kc, vc, ctx_lens)["y"]
        x = _r16(y)
    return y
