"""Seeded synthetic inputs for the all-boundary draft step.

This module only draws random numbers and lays them out; it contains none of
the method's arithmetic (no attention, no acceptance rule, no selection).  Both
the CPU oracle's tests and the CUDA path's tests/bench feed on the same bits
produced here.

Tensors that the method consumes as bf16 are returned as ``uint16`` bit
patterns (numpy has no bf16 type); fp32 tensors are plain ``float32``.

The five named workloads mirror the Qwen3-shaped configurations this build is
measured on (paper setting: draft length d = 7 in Table 1, batch sizes 1..16 in
Table 2; the larger draft lengths and contexts come from the benchmark
definition, not from the paper).
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Optional, Sequence

import numpy as np

SEED_BASE = 27396 * 10


# --------------------------------------------------------------------------- bf16 bit helpers (input prep only)
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16, returned as uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + r) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def _normal_bf16(rng: np.random.Generator, shape, sigma: float = 1.0, chunk: int = 1 << 24) -> np.ndarray:
    """N(0, sigma^2) rounded once to bf16; generated in chunks to bound transient memory."""
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.uint16)
    for s in range(0, n, chunk):
        e = min(n, s + chunk)
        x = rng.standard_normal(e - s, dtype=np.float32)
        if sigma != 1.0:
            x *= np.float32(sigma)
        out[s:e] = f32_to_bf16_bits(x)
    return out.reshape(shape)


# --------------------------------------------------------------------------- shapes
@dataclass(frozen=True)
class AttnShape:
    """Shapes of one all-boundary attention call (J = gamma + 1 boundaries)."""
    ctx_lens: tuple            # per-request context lengths L_n
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    n_boundaries: int          # J
    block: int                 # Bq query slots per boundary
    prefix_base: int = 1       # boundary j sees spine rows [0, j + prefix_base)
    n_spine: Optional[int] = None  # S, defaults to J

    @property
    def batch(self) -> int:
        return len(self.ctx_lens)

    @property
    def spine(self) -> int:
        return self.n_boundaries if self.n_spine is None else self.n_spine

    @property
    def hidden(self) -> int:
        return self.n_q_heads * self.head_dim


@dataclass(frozen=True)
class VerifyShape:
    batch: int
    n_boundaries: int          # J = gamma + 1 target rows per request
    vocab: int
    block: int
    hidden: int
    mode: str = "greedy"       # "greedy" | "sampling"
    agreement: float = 0.8     # greedy: P(draft token == target argmax)
    logit_sigma: float = 1.0


@dataclass(frozen=True)
class LayerShape:
    hidden: int
    intermediate: int
    rms_eps: float = 1e-6
    rope_theta: float = 1e6
    use_rope: bool = True
    qk_norm: bool = True
    weight_sigma: float = 0.02


@dataclass(frozen=True)
class HeadShape:
    """Critical-path remainder: LM head on the selected branch + the autoregressive head loop."""
    batch: int
    block: int                 # d = draft length = rows per selected branch
    hidden: int
    vocab: int
    rank: int = 256            # width of the head's low-rank token embedding (the paper gives no number)
    lm_sigma: float = 0.02
    ar_sigma: float = 0.05


@dataclass(frozen=True)
class Workload:
    name: str
    index: int
    attn: Optional[AttnShape]
    verify: VerifyShape
    layer: Optional[LayerShape] = None

    @property
    def seed(self) -> int:
        return SEED_BASE + self.index


def _ragged_lens(seed: int, b: int, lo: int, hi: int) -> tuple:
    rng = np.random.Generator(np.random.Philox(seed))
    return tuple(int(x) for x in rng.integers(lo, hi + 1, size=b))


def workload(index: int) -> Workload:
    """The five benchmark configurations (1-based index)."""
    if index == 1:
        a = AttnShape((128,), 4, 2, 64, 5, 4)
        return Workload("cfg1_tiny", 1, a, VerifyShape(1, 5, 1000, 4, a.hidden, "greedy", 0.8, 1.0))
    if index == 2:
        a = AttnShape((2048,), 32, 8, 128, 8, 8)
        return Workload("cfg2_qwen3_8b_b1", 2, a, VerifyShape(1, 8, 151936, 8, 4096, "greedy", 0.8, 2.0))
    if index == 3:
        lens = _ragged_lens(SEED_BASE + 3, 16, 512, 4096)
        a = AttnShape(lens, 40, 8, 128, 16, 16)
        return Workload("cfg3_qwen3_14b_b16", 3, a, VerifyShape(16, 16, 151936, 16, 5120, "greedy", 0.75, 2.0))
    if index == 4:
        return Workload("cfg4_sampling_b8", 4, None, VerifyShape(8, 16, 151936, 16, 4096, "sampling", 0.0, 3.0))
    if index == 5:
        a = AttnShape((32768,) * 4, 32, 8, 128, 16, 16)
        return Workload("cfg5_layer_long", 5, a, VerifyShape(4, 16, 151936, 16, 4096, "greedy", 0.8, 2.0),
                        LayerShape(4096, 12288))
    raise ValueError(f"no workload {index}")


# --------------------------------------------------------------------------- generators
@dataclass
class AttnInputs:
    shape: AttnShape
    q: np.ndarray            # [b][J][Bq][Hq][D] bf16 bits
    k_ctx: np.ndarray        # [sum L][Hkv][D]
    v_ctx: np.ndarray
    ctx_offsets: np.ndarray  # [b+1] int64
    k_spine: np.ndarray      # [b][S][Hkv][D]
    v_spine: np.ndarray
    k_blk: np.ndarray        # [b][J][Bq][Hkv][D]
    v_blk: np.ndarray


def make_attn_inputs(shape: AttnShape, seed: int, with_q: bool = True, with_blk: bool = True) -> AttnInputs:
    rng = np.random.Generator(np.random.Philox(seed))
    b, J, Bq, S = shape.batch, shape.n_boundaries, shape.block, shape.spine
    Hq, Hkv, D = shape.n_q_heads, shape.n_kv_heads, shape.head_dim
    off = np.zeros(b + 1, dtype=np.int64)
    off[1:] = np.cumsum(np.asarray(shape.ctx_lens, dtype=np.int64))
    tot = int(off[-1])
    q = _normal_bf16(rng, (b, J, Bq, Hq, D)) if with_q else np.zeros((b, J, Bq, Hq, D), np.uint16)
    k_ctx = _normal_bf16(rng, (tot, Hkv, D))
    v_ctx = _normal_bf16(rng, (tot, Hkv, D))
    k_spine = _normal_bf16(rng, (b, S, Hkv, D))
    v_spine = _normal_bf16(rng, (b, S, Hkv, D))
    if with_blk:
        k_blk = _normal_bf16(rng, (b, J, Bq, Hkv, D))
        v_blk = _normal_bf16(rng, (b, J, Bq, Hkv, D))
    else:
        k_blk = np.zeros((b, J, Bq, Hkv, D), np.uint16)
        v_blk = np.zeros((b, J, Bq, Hkv, D), np.uint16)
    return AttnInputs(shape, q, k_ctx, v_ctx, off, k_spine, v_spine, k_blk, v_blk)


@dataclass
class VerifyInputs:
    shape: VerifyShape
    target: np.ndarray                 # [b][J][V] fp32: logits (greedy) or probabilities (sampling)
    draft_tokens: np.ndarray           # [b][J-1] int32
    reps: np.ndarray                   # [b][J][Bq][hidden] bf16 bits
    draft_probs: Optional[np.ndarray] = None   # [b][J-1][V] fp32 (sampling)
    uniforms: Optional[np.ndarray] = None      # [b][J] fp32 = m * 2^-24 (sampling)


def _softmax64_to_f32(z: np.ndarray) -> np.ndarray:
    """Row softmax of fp32 logits evaluated in float64 and rounded to fp32 (input prep:
    the verify call consumes probabilities, temperature 1 / top-p 1 as in the paper's App. C)."""
    z = z.astype(np.float64)
    z -= z.max(axis=-1, keepdims=True)
    e = np.exp(z)
    return (e / e.sum(axis=-1, keepdims=True)).astype(np.float32)


def make_verify_inputs(shape: VerifyShape, seed: int, reps: Optional[np.ndarray] = None,
                       force_full: Sequence[int] = (), force_zero: Sequence[int] = ()) -> VerifyInputs:
    """Verification-side inputs.

    greedy: logits ~ N(0, sigma^2); draft token i equals the row-(i-1) maximum's position with
    probability `agreement`, else is uniform over the vocabulary.  Requests listed in `force_full`
    agree everywhere (accepted length gamma); those in `force_zero` disagree at the first draft.
    sampling: draft logits ~ N(0, sigma^2), target logits = draft + N(0,1); both turned into
    probabilities; draft token i drawn from draft row i-1; uniforms are m * 2^-24.
    """
    rng = np.random.Generator(np.random.Philox(seed ^ 0x5EED))
    b, J, V = shape.batch, shape.n_boundaries, shape.vocab
    g = J - 1
    if reps is None:
        reps = _normal_bf16(rng, (b, J, shape.block, shape.hidden))
    if shape.mode == "greedy":
        logits = rng.standard_normal((b, J, V), dtype=np.float32)
        if shape.logit_sigma != 1.0:
            logits *= np.float32(shape.logit_sigma)
        top = logits.argmax(axis=-1).astype(np.int32)          # position of each row's maximum (first on ties)
        agree = rng.random((b, g)) < shape.agreement
        rnd = rng.integers(0, V, size=(b, g), dtype=np.int64).astype(np.int32)
        for n in force_full:
            agree[n, :] = True
        tokens = np.where(agree, top[:, :g], rnd).astype(np.int32)
        for n in force_zero:
            tokens[n, 0] = (top[n, 0] + 1) % V
        return VerifyInputs(shape, logits, tokens, reps)
    if shape.mode == "sampling":
        zq = rng.standard_normal((b, J, V), dtype=np.float32) * np.float32(shape.logit_sigma)
        zp = zq + rng.standard_normal((b, J, V), dtype=np.float32)
        p = _softmax64_to_f32(zp)
        q = _softmax64_to_f32(zq[:, :g])
        del zq, zp
        tokens = np.empty((b, g), dtype=np.int32)
        for n in range(b):
            for i in range(g):
                c = np.cumsum(q[n, i].astype(np.float64))
                tokens[n, i] = min(int(np.searchsorted(c, rng.random() * c[-1], side="right")), V - 1)
        m = rng.integers(0, 1 << 24, size=(b, J), dtype=np.int64)
        u = (m.astype(np.float64) * 2.0 ** -24).astype(np.float32)
        for n in force_full:          # drafts identical to what the target would certainly accept: q := p
            q[n] = p[n, :g]
        return VerifyInputs(shape, p, tokens, reps, q, u)
    raise ValueError(shape.mode)


@dataclass
class LayerInputs:
    shape: LayerShape
    x: np.ndarray          # [b][J][Bq][hidden] bf16 bits
    w_qkv: np.ndarray      # [(Hq + 2 Hkv) * D][hidden]
    w_o: np.ndarray        # [hidden][Hq * D]
    w_gate_up: np.ndarray  # [2 * inter][hidden]; rows [0,inter) = gate, [inter, 2 inter) = up
    w_down: np.ndarray     # [hidden][inter]
    rms1_w: np.ndarray     # [hidden]
    rms2_w: np.ndarray     # [hidden]
    qnorm_w: np.ndarray    # [D]
    knorm_w: np.ndarray    # [D]


def make_layer_inputs(layer: LayerShape, attn: AttnShape, seed: int) -> LayerInputs:
    rng = np.random.Generator(np.random.Philox(seed ^ 0x1A7E5))
    b, J, Bq = attn.batch, attn.n_boundaries, attn.block
    Hq, Hkv, D = attn.n_q_heads, attn.n_kv_heads, attn.head_dim
    H, I = layer.hidden, layer.intermediate
    s = layer.weight_sigma
    x = _normal_bf16(rng, (b, J, Bq, H))
    w_qkv = _normal_bf16(rng, ((Hq + 2 * Hkv) * D, H), s)
    w_o = _normal_bf16(rng, (H, Hq * D), s)
    w_gate_up = _normal_bf16(rng, (2 * I, H), s)
    w_down = _normal_bf16(rng, (H, I), s)
    gains = [f32_to_bf16_bits(1.0 + 0.1 * rng.standard_normal(n, dtype=np.float32)) for n in (H, H, D, D)]
    return LayerInputs(layer, x, w_qkv, w_o, w_gate_up, w_down, *gains)


@dataclass
class HeadInputs:
    shape: HeadShape
    sel_reps: np.ndarray   # [b][d][hidden] bf16 bits: the selected branches' final hidden states
    w_lm: np.ndarray       # [V][hidden] bf16 bits
    ar_w: np.ndarray       # [V][rank] bf16 bits (W)
    ar_e: np.ndarray       # [V][rank] bf16 bits (E)
    bonus: np.ndarray      # [b] int32


def head_shape(w: Workload, rank: int = 256) -> HeadShape:
    v = w.verify
    return HeadShape(v.batch, v.block, v.hidden, v.vocab, rank)


def make_head_inputs(shape: HeadShape, seed: int) -> HeadInputs:
    """Unit-variance hidden states; N(0, lm_sigma^2) head weights (base logits with standard deviation
    lm_sigma * sqrt(hidden), 1.4 at hidden 5120); W ~ N(0, 1), E ~ N(0, ar_sigma^2), so the correction W E(y) has
    standard deviation ar_sigma * sqrt(rank) (0.8 at rank 256): comparable to the base logits' spread, the
    previous token really changes the argmax."""
    rng = np.random.Generator(np.random.Philox(seed ^ 0x4EAD))
    reps = _normal_bf16(rng, (shape.batch, shape.block, shape.hidden))
    w_lm = _normal_bf16(rng, (shape.vocab, shape.hidden), shape.lm_sigma)
    ar_w = _normal_bf16(rng, (shape.vocab, shape.rank), 1.0)
    ar_e = _normal_bf16(rng, (shape.vocab, shape.rank), shape.ar_sigma)
    bonus = rng.integers(0, shape.vocab, size=shape.batch).astype(np.int32)
    return HeadInputs(shape, reps, w_lm, ar_w, ar_e, bonus)


@dataclass
class CacheInputs:
    """One round of the feature-cache update for `n_layers` drafter layers (caches laid out with slack)."""
    row_start: np.ndarray    # [b] int64: first cache row of request n
    capacity: np.ndarray     # [b] int64: rows request n owns
    ctx_len: np.ndarray      # [b] int64: rows filled before the update
    features: np.ndarray     # [b][J][F] bf16 bits: target features of t_0..t_d
    accept_len: np.ndarray   # [b] int32
    w_kv: list               # per layer [2 * Hkv * D][F] bf16 bits (rows = [keys | values])
    norm_w: list             # per layer [F] bf16 bits
    knorm_w: list            # per layer [D] bf16 bits
    k_cache: list            # per layer [rows][Hkv][D] bf16 bits (filled part random, the rest a sentinel pattern)
    v_cache: list


def make_cache_inputs(ctx_lens: Sequence[int], n_rows: int, feat_dim: int, n_kv_heads: int, head_dim: int,
                      n_layers: int, seed: int, accept_len: Optional[Sequence[int]] = None, slack: int = 0,
                      weight_sigma: float = 0.02) -> CacheInputs:
    """Caches with `n_rows + slack` spare rows per request behind the filled part; accepted lengths uniform in
    [0, n_rows) unless given; unfilled rows hold the bit pattern 0x7FC1 (a NaN) so that a stray write or read shows."""
    rng = np.random.Generator(np.random.Philox(seed ^ 0xCAC4E))
    b = len(ctx_lens)
    cap = np.asarray([int(L) + n_rows + slack for L in ctx_lens], dtype=np.int64)
    start = np.zeros(b, dtype=np.int64)
    start[1:] = np.cumsum(cap)[:-1]
    rows = int(cap.sum())
    feats = _normal_bf16(rng, (b, n_rows, feat_dim))
    acc = (rng.integers(0, n_rows, size=b) if accept_len is None else np.asarray(accept_len)).astype(np.int32)
    w_kv, g1, gk, kc, vc = [], [], [], [], []
    for _ in range(n_layers):
        w_kv.append(_normal_bf16(rng, (2 * n_kv_heads * head_dim, feat_dim), weight_sigma))
        g1.append(f32_to_bf16_bits(1.0 + 0.1 * rng.standard_normal(feat_dim, dtype=np.float32)))
        gk.append(f32_to_bf16_bits(1.0 + 0.1 * rng.standard_normal(head_dim, dtype=np.float32)))
        k = np.full((rows, n_kv_heads, head_dim), 0x7FC1, np.uint16)
        v = np.full((rows, n_kv_heads, head_dim), 0x7FC1, np.uint16)
        for n, L in enumerate(ctx_lens):
            k[start[n]:start[n] + L] = _normal_bf16(rng, (int(L), n_kv_heads, head_dim))
            v[start[n]:start[n] + L] = _normal_bf16(rng, (int(L), n_kv_heads, head_dim))
        kc.append(k); vc.append(v)
    return CacheInputs(start, cap, np.asarray(ctx_lens, dtype=np.int64), feats, acc, w_kv, g1, gk, kc, vc)


def scaled(w: Workload, **kw) -> Workload:
    """A smaller variant of a named workload (same structure) for tests; kw override AttnShape/VerifyShape fields."""
    a = w.attn
    v = w.verify
    if a is not None:
        a = replace(a, **{k: kw[k] for k in kw if k in AttnShape.__dataclass_fields__})
    v = replace(v, **{k: kw[k] for k in kw if k in VerifyShape.__dataclass_fields__})
    if a is not None:
        v = replace(v, batch=a.batch, n_boundaries=a.n_boundaries, block=a.block)
    return Workload(w.name + "_scaled", w.index, a, v, w.layer)
