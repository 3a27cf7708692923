"""Pins for the head oracle (LM head + autoregressive head loop; Alg. 1 after the barrier, Sec. 3.2 "Loss")."""
import numpy as np

import workloads as W
from oracle import head as H


def _bits(x):
    return W.f32_to_bf16_bits(np.asarray(x, np.float32))


def test_lm_head_exact_on_small_integers():
    """Small integers are exact in bf16 and in every accumulation order: the result must equal integer matmul."""
    rng = np.random.default_rng(1)
    h = rng.integers(-4, 5, size=(5, 24))
    w = rng.integers(-4, 5, size=(37, 24))
    got = H.lm_head(_bits(h), _bits(w))
    assert got.shape == (5, 37)
    assert np.array_equal(got, (h @ w.T).astype(np.float64))
    cols = [3, 36, 0]
    assert np.array_equal(H.lm_head(_bits(h), _bits(w), cols), (h @ w.T)[:, cols].astype(np.float64))


def test_ar_logits_brute_force_loops():
    """z[v] = l[v] + sum_k W[v][k] E[y][k], written out with Python loops on a tiny case (catches a transposed
    operand or the wrong embedding row)."""
    rng = np.random.default_rng(2)
    V, r = 11, 3
    base = rng.standard_normal(V)
    Wm = rng.integers(-3, 4, size=(V, r)).astype(np.float64)
    Em = rng.integers(-3, 4, size=(V, r)).astype(np.float64)
    for y in (0, 4, 10):
        want = [base[v] + sum(Wm[v][k] * Em[y][k] for k in range(r)) for v in range(V)]
        assert np.allclose(H.ar_logits(base, _bits(Wm), _bits(Em), y), want, rtol=0, atol=1e-12)
    # W and E are not interchangeable
    assert not np.allclose(H.ar_logits(base, _bits(Wm), _bits(Em), 4), H.ar_logits(base, _bits(Em), _bits(Wm), 4))


def test_zero_correction_gives_per_row_argmax_independent_of_bonus():
    rng = np.random.default_rng(3)
    V, r, d = 50, 4, 6
    base = rng.standard_normal((d, V))
    z = np.zeros((V, r))
    e = rng.standard_normal((V, r))
    want = base.argmax(axis=1)
    for bonus in (0, 17, 49):
        assert np.array_equal(H.ar_head_greedy(base, _bits(z), _bits(e), bonus), want)


def test_constructed_chain_follows_the_previous_token():
    """Rank-V one-hot embedding and a shift matrix: the correction puts +10 on token (y + 1) mod V, the base
    logits are flat, so the head must walk bonus + 1, bonus + 2, ...; and a base-logit spike larger than the
    correction must win at its position (the base term is really added)."""
    V, d = 9, 5
    E = np.eye(V)
    Wm = np.zeros((V, V))
    for y in range(V):
        Wm[(y + 1) % V][y] = 10.0
    base = np.zeros((d, V))
    got = H.ar_head_greedy(base, _bits(Wm), _bits(E), bonus=6)
    assert list(got) == [7, 8, 0, 1, 2]
    base[2][5] = 11.0   # beats the +10 correction at step 3; the chain continues from 5
    got = H.ar_head_greedy(base, _bits(Wm), _bits(E), bonus=6)
    assert list(got) == [7, 8, 5, 6, 7]


def test_ties_take_the_lowest_index():
    V, d = 6, 2
    base = np.zeros((d, V))
    base[0][[2, 4]] = 1.0
    got = H.ar_head_greedy(base, _bits(np.zeros((V, 2))), _bits(np.zeros((V, 2))), 0)
    assert list(got) == [2, 0]


def test_draft_head_matches_composition_and_bf16_inputs_are_taken_exactly():
    sh = W.HeadShape(3, 4, 32, 101, 8)
    inp = W.make_head_inputs(sh, 11)
    got = H.draft_head_greedy(inp.sel_reps, inp.w_lm, inp.ar_w, inp.ar_e, inp.bonus)
    assert got.shape == (3, 4) and got.dtype == np.int32
    h = W.bf16_bits_to_f32(inp.sel_reps).astype(np.float64)
    wl = W.bf16_bits_to_f32(inp.w_lm).astype(np.float64)
    aw = W.bf16_bits_to_f32(inp.ar_w).astype(np.float64)
    ae = W.bf16_bits_to_f32(inp.ar_e).astype(np.float64)
    for n in range(3):
        y = int(inp.bonus[n])
        for i in range(4):
            z = wl @ h[n, i] + aw @ ae[y]
            y = int(np.argmax(z))
            assert got[n, i] == y
    # the generator's correction really matters: without it some token differs
    base_only = np.stack([np.argmax(wl @ h[n].T, axis=0) for n in range(3)])
    assert (base_only != got).any()


# ----------------------------------------------------------------------------- sampling head loop (App. C setting: T = 1, top-p = 1)
def test_sample_from_logits_closed_forms():
    """Two tokens with logits (0, ln 3): probabilities 1/4 and 3/4 -- token 0 iff u < 1/4.  A one-hot row always gives its
    token.  Adding a constant to every logit changes nothing.  NaN logits are never drawn."""
    z = np.array([0.0, np.log(3.0)])
    assert H.sample_from_logits(z, 0.0) == 0 and H.sample_from_logits(z, 0.2499) == 0
    assert H.sample_from_logits(z, 0.25) == 1 and H.sample_from_logits(z, 0.999999) == 1
    one_hot = np.array([-np.inf, -np.inf, 2.0, -np.inf])
    assert all(H.sample_from_logits(one_hot, u) == 2 for u in (0.0, 0.5, 1 - 2.0 ** -24))
    rng = np.random.default_rng(0)
    z = rng.standard_normal(50)
    for u in rng.random(20):
        assert H.sample_from_logits(z, u) == H.sample_from_logits(z + 7.5, u)
    z[3] = np.nan
    assert all(H.sample_from_logits(z, u) != 3 for u in np.linspace(0, 0.9999, 200))
    assert H.sample_from_logits(np.full(5, np.nan), 0.3) == 0
    # monotone in u: the draw is the inverse of a non-decreasing function
    draws = [H.sample_from_logits(z, u) for u in np.linspace(0, 0.9999, 300)]
    assert draws == sorted(draws)


def test_sampling_reproduces_softmax_chi_square():
    """2e5 seeded uniforms m * 2^-24 over a 16-token vocabulary: the draws follow softmax(z) (15 dof, p > 0.001 <=> chi2 < 37.7)."""
    rng = np.random.default_rng(4)
    z = rng.standard_normal(16) * 1.5
    p = np.exp(z - z.max()); p /= p.sum()
    m = rng.integers(0, 1 << 24, size=200000)
    c = np.cumsum(np.exp(z - z.max()))
    toks = np.searchsorted(c, m * 2.0 ** -24 * c[-1], side="right")         # vectorised copy of the definition ...
    assert all(H.sample_from_logits(z, mm * 2.0 ** -24) == t for mm, t in zip(m[:500], toks[:500]))   # ... checked against the function
    counts = np.bincount(toks, minlength=16)
    chi2 = float(((counts - p * len(m)) ** 2 / (p * len(m))).sum())
    assert chi2 < 37.7, chi2


def test_sampling_chain_feeds_the_previous_token():
    """Same construction as the greedy chain: a +30 correction on (y + 1) mod V makes softmax a point mass, so the sampled
    chain walks bonus + 1, bonus + 2, ... whatever the uniforms; with zero correction the draws depend on the uniforms only
    and equal independent draws from the base rows."""
    V, d = 9, 5
    E = np.eye(V)
    Wm = np.zeros((V, V))
    for y in range(V):
        Wm[(y + 1) % V][y] = 30.0
    u = np.random.default_rng(1).random(d)
    got = H.ar_head_sampling(np.zeros((d, V)), _bits(Wm), _bits(E), 6, u)
    assert got.tolist() == [(6 + i + 1) % V for i in range(d)]
    base = np.random.default_rng(2).standard_normal((d, V))
    got = H.ar_head_sampling(base, _bits(np.zeros((V, V))), _bits(E), 3, u)
    assert got.tolist() == [H.sample_from_logits(base[i], u[i]) for i in range(d)]
    # a very peaked distribution: sampling equals greedy
    sharp = base * 200.0
    assert np.array_equal(H.ar_head_sampling(sharp, _bits(np.zeros((V, V))), _bits(E), 3, u),
                          H.ar_head_greedy(sharp, _bits(np.zeros((V, V))), _bits(E), 3))
