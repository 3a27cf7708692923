"""Pins for oracle/layer.py pieces (closed forms, library routines) and the input generators (CPU only).
The block STRUCTURE is this build's reading of the paper (Sec. 3.1 lists a block's parts only)
and stays unpinned by the paper; the library-composed check below only guards against slips."""
import math

import numpy as np
import torch
import torch.nn.functional as F

import workloads as W
from oracle import attention as OA
from oracle import layer as OL


def test_rmsnorm_closed_form_and_library():
    x = np.full((2, 8), 3.0)
    g = np.arange(1, 9, dtype=np.float64)
    assert np.allclose(OL.rmsnorm(x, g, 1e-6), 3.0 / math.sqrt(9.0 + 1e-6) * g)
    r = np.random.default_rng(0).standard_normal((5, 64))
    ref = F.rms_norm(torch.from_numpy(r), (64,), torch.from_numpy(np.ones(64)), 1e-6).numpy()
    assert np.allclose(OL.rmsnorm(r, None, 1e-6), ref, atol=1e-14)


def test_silu():
    x = np.linspace(-6, 6, 25)
    assert OL.silu(np.zeros(1))[0] == 0
    assert np.allclose(OL.silu(x), F.silu(torch.from_numpy(x)).numpy(), atol=1e-15)


def test_rope_properties():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((3, 4, 16))
    pos = np.array([0, 5, 1000, 40000])
    y = OL.rope(x, pos, 1e6)
    assert np.allclose(y[:, 0], x[:, 0])                                         # position 0: identity
    assert np.allclose((y * y).sum(-1), (x * x).sum(-1))                           # a rotation
    # D = 2 is a plain planar rotation by the position (frequency 1)
    v = np.array([[[1.0, 0.0]]])
    r = OL.rope(v, np.array([math.pi / 2]), 1e6)
    assert np.allclose(r[0, 0], [0.0, 1.0], atol=1e-15)
    # scores depend on the position difference only
    q, k = rng.standard_normal((1, 1, 16)), rng.standard_normal((1, 1, 16))
    s1 = (OL.rope(q, np.array([17]), 1e4) * OL.rope(k, np.array([11]), 1e4)).sum()
    s2 = (OL.rope(q, np.array([1017]), 1e4) * OL.rope(k, np.array([1011]), 1e4)).sum()
    assert abs(s1 - s2) < 1e-9
    # pair (d, d + D/2) turns with frequency theta^(-2d/D)
    e = np.zeros((1, 1, 8)); e[0, 0, 1] = 1
    r = OL.rope(e, np.array([3]), 100.0)
    ang = 3 * 100.0 ** (-2 / 8)
    assert np.allclose(r[0, 0, [1, 5]], [math.cos(ang), math.sin(ang)])


def _small():
    a = W.AttnShape((19, 7), 4, 2, 16, 3, 2)
    l = W.LayerShape(64, 96)
    return W.make_attn_inputs(a, 5), W.make_layer_inputs(l, a, 5)


def test_layer_identity_when_projections_vanish():
    ain, lin = _small()
    lin.w_o[:] = 0
    lin.w_down[:] = 0
    orc = OL.LayerOracle(lin, ain)
    y = orc.boundary(1, 2)["y"]
    assert np.array_equal(y, OA.bf16_bits_to_f64(lin.x[1, 2]).astype(np.float32))


def test_layer_against_library_composition():
    """Same block assembled from torch library routines in float64 without the bf16 roundings."""
    ain, lin = _small()
    orc = OL.LayerOracle(lin, ain)
    sh = ain.shape
    Hq, Hkv, D, Bq = 4, 2, 16, 2
    d = lambda b: torch.from_numpy(OA.bf16_bits_to_f64(b))
    for (n, j) in [(0, 0), (1, 2)]:
        got = orc.boundary(n, j)
        x = d(lin.x[n, j])
        xn = F.rms_norm(x, (64,), d(lin.rms1_w), 1e-6)
        qkv = F.linear(xn, d(lin.w_qkv))
        q = qkv[:, :64].reshape(Bq, Hq, D); k = qkv[:, 64:96].reshape(Bq, Hkv, D); v = qkv[:, 96:].reshape(Bq, Hkv, D)
        q = F.rms_norm(q, (D,), d(lin.qnorm_w), 1e-6); k = F.rms_norm(k, (D,), d(lin.knorm_w), 1e-6)
        pos = torch.tensor([sh.ctx_lens[n] + j + 2 + i for i in range(Bq)], dtype=torch.float64)
        inv = 1e6 ** (-torch.arange(0, D, 2, dtype=torch.float64) / D)
        ang = pos[:, None] * inv[None]
        cos, sin = torch.cat([ang.cos(), ang.cos()], -1)[:, None], torch.cat([ang.sin(), ang.sin()], -1)[:, None]
        rot = lambda t: torch.cat([-t[..., D // 2:], t[..., :D // 2]], -1)
        q = q * cos + rot(q) * sin; k = k * cos + rot(k) * sin
        lo, hi = int(ain.ctx_offsets[n]), int(ain.ctx_offsets[n + 1])
        K = torch.cat([d(ain.k_ctx[lo:hi]), d(ain.k_spine[n, :j + 1]), k], 0)
        V = torch.cat([d(ain.v_ctx[lo:hi]), d(ain.v_spine[n, :j + 1]), v], 0)
        a = F.scaled_dot_product_attention(q.permute(1, 0, 2)[None], K.permute(1, 0, 2)[None], V.permute(1, 0, 2)[None],
                                           enable_gqa=True)[0].permute(1, 0, 2).reshape(Bq, Hq * D)
        h1 = x + F.linear(a, d(lin.w_o))
        hn = F.rms_norm(h1, (64,), d(lin.rms2_w), 1e-6)
        gu = F.linear(hn, d(lin.w_gate_up))
        y = h1 + F.linear(F.silu(gu[:, :96]) * gu[:, 96:], d(lin.w_down))
        assert np.abs(y.numpy() - got["y"]).max() < 2e-2          # only the bf16 rounding points differ
        assert np.abs(a.numpy() - got["a"]).max() < 2e-2


def test_generators_are_seeded_and_shaped():
    w3 = W.workload(3)
    assert w3.attn.batch == 16 and all(512 <= L <= 4096 for L in w3.attn.ctx_lens)
    assert W.workload(3).attn.ctx_lens == w3.attn.ctx_lens
    w1 = W.workload(1)
    a = W.make_attn_inputs(w1.attn, w1.seed)
    b = W.make_attn_inputs(w1.attn, w1.seed)
    assert np.array_equal(a.q, b.q) and a.q.shape == (1, 5, 4, 4, 64) and a.k_ctx.shape == (128, 2, 64)
    assert a.k_spine.shape == (1, 5, 2, 64) and a.k_blk.shape == (1, 5, 4, 2, 64)
    x = W.bf16_bits_to_f32(a.k_ctx).astype(np.float64)
    assert abs(x.mean()) < 0.05 and abs(x.std() - 1) < 0.05
    v = W.make_verify_inputs(w1.verify, w1.seed)
    assert v.target.shape == (1, 5, 1000) and v.draft_tokens.shape == (1, 4)
    sv = W.VerifyShape(3, 4, 64, 2, 8, "sampling", 0.0, 3.0)
    s = W.make_verify_inputs(sv, 9)
    assert np.allclose(s.target.sum(-1), 1, atol=1e-5) and np.allclose(s.draft_probs.sum(-1), 1, atol=1e-5)
    m = s.uniforms.astype(np.float64) * 2 ** 24
    assert np.array_equal(m, np.round(m)) and m.max() < 2 ** 24 and m.min() >= 0


def test_linear_against_scalar_loops_integer_exact():
    """`linear` is x [M][K] times w [N][K] transposed.  Small integers make every product and sum exact, so
    the scalar triple loop must be reproduced bit for bit; M, N, K all differ and w is not symmetric, so a
    transposed operand either fails to broadcast or changes the numbers."""
    rng = np.random.default_rng(2)
    M, N, K = 3, 5, 4
    x = rng.integers(-7, 8, (M, K)).astype(np.float64)
    w = rng.integers(-7, 8, (N, K)).astype(np.float64)
    want = np.zeros((M, N))
    for m in range(M):
        for n in range(N):
            acc = 0
            for k in range(K):
                acc += int(x[m, k]) * int(w[n, k])
            want[m, n] = acc
    got = OL.linear(x, w)
    assert got.shape == (M, N) and np.array_equal(got, want)
    # square case (a silent transposition would still broadcast): w[n][k] = 1 only at (0, 1) picks x[:, 1] into column 0
    xs = np.arange(9, dtype=np.float64).reshape(3, 3)
    ws = np.zeros((3, 3)); ws[0, 1] = 1
    assert np.array_equal(OL.linear(xs, ws)[:, 0], xs[:, 1]) and not OL.linear(xs, ws)[:, 1:].any()


def test_swiglu_linear_halves_and_closed_form():
    """Rows [0, I) of the stacked weight are the gate (through SiLU), rows [I, 2I) the plain `up` factor."""
    K, I = 4, 3
    x = np.array([[1.0, 2.0, -1.0, 0.5], [0.0, -3.0, 2.0, 1.0]])
    rng = np.random.default_rng(3)
    wg = rng.integers(-2, 3, (I, K)).astype(np.float64)
    wu = rng.integers(-2, 3, (I, K)).astype(np.float64)
    got = OL.swiglu_linear(x, np.concatenate([wg, wu]))
    want = np.zeros((2, I))
    for m in range(2):
        for c in range(I):
            g = sum(x[m, k] * wg[c, k] for k in range(K))
            u = sum(x[m, k] * wu[c, k] for k in range(K))
            want[m, c] = g / (1.0 + math.exp(-g)) * u
    assert np.array_equal(got, OA.round_to_bf16(want).astype(np.float64))
    swapped = OL.swiglu_linear(x, np.concatenate([wu, wg]))
    assert not np.array_equal(got, swapped)                      # SiLU is applied to the FIRST half only
    # a zero gate silences the unit whatever `up` is; a zero `up` likewise
    assert not OL.swiglu_linear(x, np.concatenate([np.zeros((I, K)), wu])).any()
    assert not OL.swiglu_linear(x, np.concatenate([wg, np.zeros((I, K))])).any()
    # gate pre-activation 0 < g: silu(g) * 1 with up = e_0 row-sum selector -> closed form g * sigmoid(g)
    one = np.zeros((1, K)); one[0, 0] = 1
    y = OL.swiglu_linear(np.array([[2.0, 0, 0, 0]]), np.concatenate([one, 0.5 * one]))
    assert y[0, 0] == OA.round_to_bf16(np.array(2.0 / (1 + math.exp(-2.0)) * 1.0)).astype(np.float64)


# ----------------------------------------------------------------------------- all rows of a request: spine tokens as queries
def _rows(ain, lin, n, seed=0):
    """x of request n in the combined order: mask-slot rows (boundary, slot), then spine rows (drawn here)."""
    sh = ain.shape
    xm = OA.bf16_bits_to_f64(lin.x[n]).reshape(sh.n_boundaries * sh.block, -1)
    xs = OA.round_to_bf16(np.random.default_rng(seed).standard_normal((sh.spine, xm.shape[1]))).astype(np.float64)
    return np.concatenate([xm, xs])


def test_request_rows_reduce_to_the_supplied_spine_block():
    """With the spine's keys/values taken from `request` and handed to `boundary` as inputs, the mask-slot rows agree
    bit for bit: producing the spine inside the block changes nothing for the branches."""
    ain, lin = _small()
    sh = ain.shape
    orc = OL.LayerOracle(lin, ain)
    n = 1
    full = orc.request(n, _rows(ain, lin, n))
    JB = sh.n_boundaries * sh.block
    ain.k_spine[n] = W.f32_to_bf16_bits(full["k"][JB:].astype(np.float32))
    ain.v_spine[n] = W.f32_to_bf16_bits(full["v"][JB:].astype(np.float32))
    orc2 = OL.LayerOracle(lin, ain)
    for j in range(sh.n_boundaries):
        assert np.array_equal(orc2.boundary(n, j)["y"].astype(np.float64), full["y"][j * sh.block:(j + 1) * sh.block])


def test_spine_rows_of_the_block_follow_the_figures_mask():
    """Fig. 4 through a whole block: anchor s reads the cache, itself and earlier anchors only; branch j reads anchors
    < j + 1 and its own slots only.  Perturbing a row must leave every row that cannot see it bit-identical."""
    ain, lin = _small()
    sh = ain.shape
    J, Bq, S = sh.n_boundaries, sh.block, sh.spine
    JB = J * Bq
    orc = OL.LayerOracle(lin, ain)
    x = _rows(ain, lin, 0)
    base = orc.request(0, x)["y"]
    # change spine token 2 (of 3): anchors 0, 1 and branches 0, 1 (prefix 1, 2 anchors) must not move; anchor 2 and branch 2 must
    x2 = x.copy(); x2[JB + 2] += 1.0
    y2 = orc.request(0, x2)["y"]
    same = list(range(0, 2 * Bq)) + [JB, JB + 1]
    assert np.array_equal(y2[same], base[same])
    assert not np.array_equal(y2[JB + 2], base[JB + 2]) and not np.array_equal(y2[2 * Bq:3 * Bq], base[2 * Bq:3 * Bq])
    # change a mask slot of branch 1: only branch 1's rows move (bidirectional inside the branch, invisible elsewhere)
    x3 = x.copy(); x3[1 * Bq] += 1.0
    y3 = orc.request(0, x3)["y"]
    others = [r for r in range(JB + S) if not (Bq <= r < 2 * Bq)]
    assert np.array_equal(y3[others], base[others])
    assert not np.array_equal(y3[Bq + 1], base[Bq + 1])
    # the anchors' attention output equals the stand-alone spine attention on the block's own q, k, v
    r = orc.request(0, x)
    q = W.f32_to_bf16_bits(r["q"][JB:].astype(np.float32))[None]
    k = W.f32_to_bf16_bits(r["k"][JB:].astype(np.float32))[None]
    v = W.f32_to_bf16_bits(r["v"][JB:].astype(np.float32))[None]
    lo, hi = int(ain.ctx_offsets[0]), int(ain.ctx_offsets[1])
    want = OA.spine_rows(q, ain.k_ctx[lo:hi], ain.v_ctx[lo:hi], np.array([0, hi - lo]), k, v)[0]
    assert np.array_equal(OA.round_to_bf16(want.reshape(S, -1)).astype(np.float64), r["a"][JB:])


def test_stacked_blocks_keep_causality_and_isolation():
    """Two blocks: the second reads the first one's rows (bf16).  What Fig. 4 forbids at one block stays forbidden through
    the stack; and a second block with zero output projections passes the first block's result through."""
    ain, lin = _small()
    sh = ain.shape
    J, Bq, S = sh.n_boundaries, sh.block, sh.spine
    JB = J * Bq
    lin2 = W.make_layer_inputs(W.LayerShape(64, 96), sh, 77)
    l1, l2 = OL.LayerOracle(lin, ain), OL.LayerOracle(lin2, ain)
    x = _rows(ain, lin, 0)
    base = OL.backbone([l1, l2], 0, x)
    x2 = x.copy(); x2[JB + 1] -= 0.5                                   # spine token 1
    y2 = OL.backbone([l1, l2], 0, x2)
    same = list(range(0, Bq)) + [JB]                                   # branch 0 (reads anchor 0 only) and anchor 0
    assert np.array_equal(y2[same], base[same])
    assert not np.array_equal(y2[Bq:2 * Bq], base[Bq:2 * Bq])           # branch 1 reads anchors 0, 1
    lin2.w_o[:] = 0; lin2.w_down[:] = 0
    y1 = l1.request(0, x)["y"]
    thru = OL.backbone([l1, OL.LayerOracle(lin2, ain)], 0, x)
    assert np.array_equal(thru, OA.round_to_bf16(y1).astype(np.float64))
