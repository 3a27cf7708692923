"""Pins for oracle/verify.py: target-argmax prefix, brute force, distribution preservation (CPU only)."""
import itertools

import numpy as np
import pytest

import workloads as W
from oracle import verify as OV


# ----------------------------------------------------------------------------- greedy
def test_row_argmax_rules():
    assert OV.row_argmax(np.float32([1, 3, 3, 2])) == 1                     # lowest index on ties
    assert OV.row_argmax(np.float32([-0.0, 0.0, -1])) == 0                  # -0 == +0
    assert OV.row_argmax(np.float32([0.0, -0.0, -1])) == 0
    assert OV.row_argmax(np.float32([np.nan, -np.inf, np.nan])) == 1        # NaN below everything
    assert OV.row_argmax(np.float32([np.nan, np.nan])) == 0
    assert OV.row_argmax(np.float32([np.nan, 5, np.inf, np.inf])) == 2
    x = np.random.default_rng(0).standard_normal(1000).astype(np.float32)
    assert OV.row_argmax(x) == int(np.argmax(x))


def test_greedy_emits_target_argmax_prefix():
    """Whatever the drafts, the emitted tokens (accepted drafts + bonus) are the target's own greedy
    choices a_0..a_r; the accepted length is the longest agreeing prefix."""
    sh = W.VerifyShape(12, 6, 50, 2, 8, "greedy", 0.7, 1.0)
    v = W.make_verify_inputs(sh, 3, force_full=[0], force_zero=[1])
    res = OV.verify_greedy(v.target, v.draft_tokens, v.reps)
    a = v.target.argmax(-1)
    seen = set()
    for n in range(sh.batch):
        r = int(res["accept_len"][n])
        seen.add(r)
        emitted = res["out_tokens"][n, : r + 1]
        assert np.array_equal(emitted, a[n, : r + 1])
        assert np.all(res["out_tokens"][n, r + 1:] == -1)
        assert res["bonus"][n] == a[n, r] and res["gather_idx"][n] == r
        if r < sh.n_boundaries - 1:
            assert v.draft_tokens[n, r] != a[n, r]                 # maximal: the next draft disagrees
        assert np.array_equal(res["selected"][n], v.reps[n, r])    # bit copy of branch r
    assert res["accept_len"][0] == sh.n_boundaries - 1 and res["accept_len"][1] == 0
    assert len(seen) >= 3
    assert res["status"] == 0


def test_greedy_exhaustive_tiny():
    """All draft strings for V = 3, gamma = 2 and a grid of logits with ties, against a direct scan."""
    vals = [0.0, 1.0]
    gamma, V = 2, 3
    for rows in itertools.product(itertools.product(vals, repeat=V), repeat=gamma + 1):
        logits = np.float32(rows)[None]
        a = [min(i for i in range(V) if row[i] == max(row)) for row in rows]
        for toks in itertools.product(range(V), repeat=gamma):
            res = OV.verify_greedy(logits, np.int32([toks]))
            r = 0
            for i in range(gamma):
                if toks[i] == a[i]:
                    r += 1
                else:
                    break
            assert res["accept_len"][0] == r and res["bonus"][0] == a[r]


def test_greedy_bad_token_rejected():
    logits = np.float32([[[0, 1, 0], [0, 0, 1], [1, 0, 0]]])
    res = OV.verify_greedy(logits, np.int32([[1, 7]]))
    assert res["accept_len"][0] == 1 and res["bonus"][0] == 2 and res["status"] == OV.STATUS_BAD_TOKEN
    res = OV.verify_greedy(logits, np.int32([[-1, 2]]))
    assert res["accept_len"][0] == 0 and res["bonus"][0] == 1 and res["status"] == OV.STATUS_BAD_TOKEN


# ----------------------------------------------------------------------------- sampling: integer draw
def test_draw_from_weights_brute_force():
    rng = np.random.default_rng(5)
    for _ in range(200):
        V = int(rng.integers(1, 9))
        w = rng.integers(0, 5, size=V).astype(np.uint64) * np.uint64(rng.integers(1, 1 << 30))
        if w.sum() == 0:
            continue
        m = int(rng.integers(0, 1 << 24))
        Wt = sum(int(x) for x in w)
        T = (m * Wt) >> 24
        acc, exp = 0, None
        for v in range(V):
            acc += int(w[v])
            if acc > T:
                exp = v
                break
        got = OV.draw_from_weights(w, m)
        assert got == exp and w[got] > 0          # never lands on a zero-weight token


def test_fixed_point_weights():
    p = np.float32([0.5, 0.25, 0.25, 0.0])
    q = np.float32([0.25, 0.5, 0.25, 0.0])
    assert list(OV.fixed_point_weights(p, q)) == [1 << 30, 0, 0, 0]
    assert list(OV.fixed_point_weights(p, None)) == [1 << 31, 1 << 30, 1 << 30, 0]
    assert OV.fixed_point_weights(np.float32([1.0]), None)[0] == 1 << 32
    # truncation, not rounding; and the subtraction is the fp32 one
    a, b = np.float32(0.1), np.float32(0.03)
    d = np.float32(a - b)
    assert OV.fixed_point_weights(np.float32([a]), np.float32([b]))[0] == int(float(d) * 2 ** 32)


# ----------------------------------------------------------------------------- sampling: distribution
def _trial_batch(p_rows, q_rows, n_trials, seed):
    """n_trials independent verifications of the same (p, q) rows: tokens drawn from q by numpy,
    uniforms m * 2^-24."""
    rng = np.random.default_rng(seed)
    J, V = p_rows.shape
    g = J - 1
    toks = np.stack([rng.choice(V, size=n_trials, p=q_rows[i].astype(np.float64) / q_rows[i].astype(np.float64).sum())
                     for i in range(g)], 1).astype(np.int32)
    u = (rng.integers(0, 1 << 24, size=(n_trials, J)).astype(np.float64) * 2.0 ** -24).astype(np.float32)
    P = np.broadcast_to(p_rows, (n_trials, J, V))
    Q = np.broadcast_to(q_rows, (n_trials, g, V))
    return P, Q, toks, u


def _softmax(z):
    e = np.exp(z - z.max(-1, keepdims=True))
    return (e / e.sum(-1, keepdims=True)).astype(np.float32)


def _chi2(counts, probs):
    n = counts.sum()
    e = probs.astype(np.float64) / probs.astype(np.float64).sum() * n
    return float(((counts - e) ** 2 / e).sum())


N_TRIALS = 1_000_000


@pytest.fixture(scope="module")
def sampling_run():
    rng = np.random.default_rng(42)
    V, J = 16, 3
    zq = rng.standard_normal((J, V)) * 1.5
    p = _softmax(zq + rng.standard_normal((J, V)))
    q = _softmax(zq[: J - 1])
    P, Q, toks, u = _trial_batch(p, q, N_TRIALS, 7)
    res = OV.verify_sampling(P, Q, toks, u)
    return p, q, toks, res


def test_sampling_preserves_target_distribution(sampling_run):
    """Chi-square (15 dof; 37.7 is the 0.1 % point) of the first emitted token against target row 0 and
    of the second emitted token, given that there is one, against target row 1 -- 1e6 seeded trials on
    a 16-token vocabulary."""
    p, q, toks, res = sampling_run
    first = res["out_tokens"][:, 0]
    c0 = np.bincount(first, minlength=16).astype(np.float64)
    assert _chi2(c0, p[0]) < 37.7
    has2 = res["accept_len"] >= 1
    second = res["out_tokens"][has2, 1]
    c1 = np.bincount(second, minlength=16).astype(np.float64)
    assert has2.sum() > 100_000 and _chi2(c1, p[1]) < 37.7
    # and it is NOT the drafter's distribution (the test has power)
    assert _chi2(c0, q[0]) > 1000


def test_sampling_acceptance_rate_closed_form(sampling_run):
    """P(first draft accepted) = sum_v min(p, q) = 1 - TV(p, q)."""
    p, q, toks, res = sampling_run
    rate = (res["accept_len"] >= 1).mean()
    exp = np.minimum(p[0].astype(np.float64), q[0].astype(np.float64)).sum()
    sigma = np.sqrt(exp * (1 - exp) / N_TRIALS)
    assert abs(rate - exp) < 4 * sigma
    # second draft, given the first was accepted
    got2 = (res["accept_len"][res["accept_len"] >= 1] >= 2).mean()
    exp2 = np.minimum(p[1].astype(np.float64), q[1].astype(np.float64)).sum()
    assert abs(got2 - exp2) < 4 * np.sqrt(exp2 * (1 - exp2) / (res["accept_len"] >= 1).sum())


def test_sampling_special_cases():
    rng = np.random.default_rng(1)
    V, J = 16, 4
    p = _softmax(rng.standard_normal((J, V)))
    # p == q: always accepted (u * q < q for u < 1), r = gamma, bonus ~ p_gamma
    P, Q, toks, u = _trial_batch(p, p[: J - 1], 20000, 3)
    res = OV.verify_sampling(P, Q, toks, u)
    assert np.all(res["accept_len"] == J - 1)
    assert _chi2(np.bincount(res["bonus"], minlength=V).astype(float), p[J - 1]) < 37.7
    # drafter is certain of a token the target gives zero mass: always rejected, bonus ~ p_0 (residual = p_0)
    p2 = p.copy()
    p2[0, 5] = 0
    p2[0] /= p2[0].sum()
    q2 = np.zeros((J - 1, V), np.float32)
    q2[:, 5] = 1
    P, Q, toks, u = _trial_batch(p2, q2, 20000, 4)
    res = OV.verify_sampling(P, Q, toks, u)
    assert np.all(res["accept_len"] == 0) and np.all(res["bonus"] != 5)
    assert _chi2(np.bincount(res["bonus"], minlength=V).astype(float)[np.arange(V) != 5], p2[0][np.arange(V) != 5]) < 36.1


def test_argmax_draft_can_be_rejected():
    """The paper's App. C remark: a draft equal to the target's most likely token is still rejected
    with probability 1 - p/q when the drafter is more confident than the target."""
    V, J = 16, 2
    p = np.full((J, V), 0.4 / 15, np.float32)
    p[:, 3] = 0.6                                   # target argmax = 3 with p = 0.6
    q = np.full((1, V), 0.1 / 15, np.float32)
    q[:, 3] = 0.9                                   # drafter says 3 with q = 0.9
    n = 200000
    rng = np.random.default_rng(9)
    u = (rng.integers(0, 1 << 24, size=(n, J)).astype(np.float64) * 2.0 ** -24).astype(np.float32)
    toks = np.full((n, 1), 3, np.int32)
    res = OV.verify_sampling(np.broadcast_to(p, (n, J, V)), np.broadcast_to(q, (n, 1, V)), toks, u)
    rej = (res["accept_len"] == 0).mean()
    exp = 1 - 0.6 / 0.9
    assert abs(rej - exp) < 4 * np.sqrt(exp * (1 - exp) / n)
    # a rejected draft is never re-emitted as the bonus when p(t) < q(t): residual at t is zero
    assert np.all(res["bonus"][res["accept_len"] == 0] != 3)


def test_sampling_fallbacks_and_boundaries():
    # residual identically zero with a rejection impossible -> p == q accepted; force the W == 0 path by
    # handing a rejected position whose residual vanishes: p = q except the draft token has q > p is
    # impossible with sums equal, so use unnormalised rows (the call does not require normalisation).
    p = np.float32([[[0.5, 0.25, 0.0, 0.0], [0.1, 0.2, 0.3, 0.4]]])
    q = np.float32([[[0.5, 0.5, 0.0, 0.0]]])
    toks = np.int32([[1]])
    u = np.float32([[0.75, 0.75]])                   # 0.75 * 0.5 = 0.375 >= 0.25 -> reject
    res = OV.verify_sampling(p, q, toks, u)
    # residual max(p - q, 0) = 0 everywhere -> fall back to p_0 = (0.5, 0.25): T = 0.75 * W = 0.5625 >= 0.5 -> token 1
    assert res["accept_len"][0] == 0 and res["bonus"][0] == 1
    # all-zero target row -> lowest-index maximum
    res = OV.verify_sampling(np.zeros((1, 2, 4), np.float32), q, toks, u)
    assert res["accept_len"][0] == 0 and res["bonus"][0] == 0
    # u = 0 always accepts when p > 0; q(t) = 0 accepts iff p > 0
    res = OV.verify_sampling(p, np.float32([[[0.5, 0.0, 0.0, 0.5]]]), toks, np.float32([[0.999, 0.0]]))
    assert res["accept_len"][0] == 1 and res["bonus"][0] == 0     # m = 0 -> T = 0 -> first positive weight
    # largest uniform lands on the last positive-weight token
    umax = np.float32((2 ** 24 - 1) * 2.0 ** -24)
    res = OV.verify_sampling(p, np.float32([[[0.5, 0.0, 0.0, 0.5]]]), toks, np.float32([[0.0, umax]]))
    assert res["bonus"][0] == 3
    # out-of-range draft
    res = OV.verify_sampling(p, q, np.int32([[9]]), u)
    assert res["accept_len"][0] == 0 and res["status"] == OV.STATUS_BAD_TOKEN


def test_bonus_uniform_of_one_stays_inside_the_vocabulary():
    """A bonus uniform of exactly 1.0 (m = 2^24, outside [0, 1)) is read as the largest uniform: the threshold
    stays below the total weight, so the draw is the LAST token that carries weight, never an index = V."""
    p = np.zeros((1, 1, 8), np.float32)
    p[0, 0, [1, 5]] = 0.5                                  # J = 1: no drafts, bonus drawn from p_0
    toks = np.zeros((1, 0), np.int32)
    q = np.zeros((1, 0, 8), np.float32)
    for u, want in ((1.0, 5), (float(np.float32(1 - 2 ** -24)), 5), (0.0, 1), (0.5, 5), (0.5 - 2 ** -24, 1)):
        r = OV.verify_sampling(p, q, toks, np.array([[u]], np.float32))
        assert r["bonus"][0] == want and r["accept_len"][0] == 0, (u, r["bonus"])
