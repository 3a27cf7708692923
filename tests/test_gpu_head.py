"""GPU parity of dpara_draft_head (LM head on the selected branch + autoregressive head loop) against the oracle.

The kernels accumulate bf16 products in fp32, the oracle in float64, so a token may differ only where two logits
are closer than the fp32 rounding error; the head loop is sequential, so the comparison is step by step with the
kernel's own previous token: the kernel's token must be the oracle's argmax, or hold an oracle logit within TIE of
it.  TIE: fp32 accumulation of K = hidden + rank products of magnitude <= |h||w| gives an absolute error of about
sqrt(K) * 2^-24 * |z|_max (3e-6 * |z|_max at K = 5376); 1e-4 * max(1, |z|_max) leaves a wide margin and still
separates neighbouring logits (spacing of the top two of 150k Gaussians is ~0.1 sigma).
"""
import numpy as np
import pytest
import torch

import workloads as W
from oracle import head as H
from gpu_util import dev_bf16

import paper_2609_27396_b200 as dp

pytestmark = pytest.mark.gpu
TIE = 1e-4


def _run(inp):
    sh = inp.shape
    t = [dev_bf16(x) for x in (inp.sel_reps, inp.w_lm, inp.ar_w, inp.ar_e)]
    bonus = torch.from_numpy(inp.bonus).cuda()
    toks, plan = dp.draft_head(t[0], t[1], t[2], t[3], bonus)
    torch.cuda.synchronize()
    assert plan.status.item() == 0
    return toks.cpu().numpy(), plan.base_logits().cpu().numpy().astype(np.float64)


def _check(inp, toks, logits, rows=None):
    sh = inp.shape
    base = H.lm_head(inp.sel_reps.reshape(-1, sh.hidden), inp.w_lm) if rows is None else None
    exact = 0
    for n in (range(sh.batch) if rows is None else rows):
        y = int(inp.bonus[n])
        for i in range(sh.block):
            row = base[n * sh.block + i] if base is not None else H.lm_head(inp.sel_reps[n, i][None], inp.w_lm)[0]
            got_l = logits[n * sh.block + i]
            scale = max(1.0, float(np.abs(row).max()))
            assert np.abs(got_l - row).max() <= TIE * scale          # base logits element by element
            z = H.ar_logits(row, inp.ar_w, inp.ar_e, y)
            want = int(np.argmax(z))
            got = int(toks[n, i])
            assert 0 <= got < sh.vocab
            assert got == want or z[got] >= z[want] - TIE * max(1.0, float(np.abs(z).max())), (n, i, got, want)
            exact += got == want
            y = got                                                  # teacher-forced with the kernel's own token
    return exact


@pytest.mark.parametrize("shape", [
    W.HeadShape(3, 4, 128, 1000, 64),          # one partial tile row range, 16-column accumulator
    W.HeadShape(16, 16, 512, 20000 + 8, 256),  # several tiles per CTA and a ragged last tile
    W.HeadShape(20, 5, 256, 4096, 128),        # batch above 16: 32-column accumulator
    W.HeadShape(1, 8, 1024, 33000, 192),       # b = 1, rank not a power of two
])
def test_head_matches_oracle(shape):
    inp = W.make_head_inputs(shape, 41)
    toks, logits = _run(inp)
    exact = _check(inp, toks, logits)
    assert exact >= 0.99 * shape.batch * shape.block
    # and the whole chain equals the oracle's own chain wherever no near-tie intervened
    ref = H.draft_head_greedy(inp.sel_reps, inp.w_lm, inp.ar_w, inp.ar_e, inp.bonus)
    assert (ref == toks).mean() >= 0.9


def test_head_constructed_chain_and_ties():
    """Identity-like embedding with a shift matrix (exact in bf16): y_i = bonus + i; equal logits take the lowest index."""
    V, d, r, hid = 256, 6, 256, 64
    E = np.eye(V, r, dtype=np.float32)
    Wm = np.zeros((V, r), np.float32)
    for y in range(V):
        Wm[(y + 1) % V][y] = 10.0
    reps = np.zeros((2, d, hid), np.float32)
    w_lm = np.zeros((V, hid), np.float32)
    inp = W.HeadInputs(W.HeadShape(2, d, hid, V, r), W.f32_to_bf16_bits(reps), W.f32_to_bf16_bits(w_lm),
                       W.f32_to_bf16_bits(Wm), W.f32_to_bf16_bits(E), np.array([250, 3], np.int32))
    toks, _ = _run(inp)
    assert toks[0].tolist() == [251, 252, 253, 254, 255, 0]
    assert toks[1].tolist() == [4, 5, 6, 7, 8, 9]
    # all logits equal (zero weights, zero correction): index 0 everywhere
    inp0 = W.HeadInputs(inp.shape, inp.sel_reps, inp.w_lm, W.f32_to_bf16_bits(np.zeros((V, r), np.float32)), inp.ar_e, inp.bonus)
    toks0, _ = _run(inp0)
    assert (toks0 == 0).all()


def test_head_rejects_bad_arguments():
    sh = W.HeadShape(2, 4, 128, 1000, 64)
    inp = W.make_head_inputs(sh, 5)
    t = [dev_bf16(x) for x in (inp.sel_reps, inp.w_lm, inp.ar_w, inp.ar_e)]
    bonus = torch.from_numpy(inp.bonus).cuda()
    plan = dp.HeadPlan(2, 4, 128, 1000, 64)
    plan.rank = 96                      # not a multiple of 64
    with pytest.raises(dp.DparaError):
        plan.run(t[0], t[1], t[2], t[3], bonus)
    plan = dp.HeadPlan(2, 4, 128, 1000, 64)
    plan.workspace_bytes = 16           # too small
    with pytest.raises(dp.DparaError):
        plan.run(t[0], t[1], t[2], t[3], bonus)
    # an out-of-range bonus is reported, not followed
    plan = dp.HeadPlan(2, 4, 128, 1000, 64)
    bad = torch.tensor([5, 100000], dtype=torch.int32, device="cuda")
    plan.run(t[0], t[1], t[2], t[3], bad)
    torch.cuda.synchronize()
    assert plan.status.item() & 1


def test_head_full_size_sampled():
    """The benchmark shape (b = 16, d = 16, hidden 5120, vocab 151 936, rank 256) in the launch configuration the
    bench times; the oracle checks sampled (request, step) pairs one by one, teacher-forced with the kernel's
    own previous token, and the base logits of those rows element by element."""
    sh = W.head_shape(W.workload(3))
    inp = W.make_head_inputs(sh, W.workload(3).seed)
    toks, logits = _run(inp)
    assert ((toks >= 0) & (toks < sh.vocab)).all()
    rng = np.random.default_rng(7)
    for n, i in [(0, 0), (15, 15)] + [(int(rng.integers(sh.batch)), int(rng.integers(1, sh.block))) for _ in range(2)]:
        row = np.concatenate([H.lm_head(inp.sel_reps[n, i][None], inp.w_lm, cols=range(c, min(c + 16384, sh.vocab)))[0]
                              for c in range(0, sh.vocab, 16384)])
        scale = max(1.0, float(np.abs(row).max()))
        assert np.abs(logits[n * sh.block + i] - row).max() <= TIE * scale
        y_prev = int(inp.bonus[n]) if i == 0 else int(toks[n, i - 1])
        z = H.ar_logits(row, inp.ar_w, inp.ar_e, y_prev)
        want, got = int(np.argmax(z)), int(toks[n, i])
        assert got == want or z[got] >= z[want] - TIE * max(1.0, float(np.abs(z).max())), (n, i, got, want)


# ----------------------------------------------------------------------------- sampling head loop
def _check_sampling(inp, toks, logits, uniforms, eps=2e-5):
    """Step by step with the kernel's own previous token: the kernel's token v must satisfy the oracle's inverse-CDF rule
    up to rounding -- u inside [C(v-1) - eps, C(v) + eps] of the oracle's float64 cumulative softmax (the kernel's logits are
    fp32 accumulations, relative error ~3e-6, which moves every cumulative value by about that much)."""
    sh = inp.shape
    exact = 0
    for n in range(sh.batch):
        y = int(inp.bonus[n])
        base = H.lm_head(inp.sel_reps[n], inp.w_lm)
        for i in range(sh.block):
            assert np.abs(logits[n * sh.block + i] - base[i]).max() <= TIE * max(1.0, float(np.abs(base[i]).max()))
            z = H.ar_logits(base[i], inp.ar_w, inp.ar_e, y)
            u = float(uniforms[n, i])
            want = H.sample_from_logits(z, u)
            got = int(toks[n, i])
            assert 0 <= got < sh.vocab
            w = np.exp(z - z.max())
            c = np.cumsum(w) / w.sum()
            lo = c[got - 1] if got > 0 else 0.0
            assert lo - eps <= u <= c[got] + eps, (n, i, got, want, u, lo, c[got])
            exact += got == want
            y = got
    return exact


@pytest.mark.parametrize("shape", [
    W.HeadShape(3, 4, 128, 1000, 64),
    W.HeadShape(16, 8, 512, 20000 + 8, 256),
    W.HeadShape(20, 5, 256, 4096, 128),
    W.HeadShape(2, 6, 1024, 151936, 256),      # the full vocabulary
])
def test_head_sampling_parity(shape):
    inp = W.make_head_inputs(shape, 31)
    rng = np.random.default_rng(8)
    uniforms = (rng.integers(0, 1 << 24, size=(shape.batch, shape.block)) * 2.0 ** -24).astype(np.float32)
    uniforms[0, 0] = 0.0
    uniforms[-1, -1] = np.float32(1 - 2.0 ** -24)
    t = [dev_bf16(x) for x in (inp.sel_reps, inp.w_lm, inp.ar_w, inp.ar_e)]
    toks, plan = dp.draft_head(t[0], t[1], t[2], t[3], torch.from_numpy(inp.bonus).cuda(), uniforms=torch.from_numpy(uniforms).cuda())
    torch.cuda.synchronize()
    assert plan.status.item() == 0
    exact = _check_sampling(inp, toks.cpu().numpy(), plan.base_logits().cpu().numpy().astype(np.float64), uniforms)
    assert exact >= 0.98 * shape.batch * shape.block        # a different token than the oracle's is the rare boundary case


def test_head_sampling_repeats_and_leaves_greedy_unchanged():
    """Two runs with the same uniforms give the same tokens, and a greedy run on the same plan's workspace after a sampling
    run gives what it gave before (the sampling path leaves no state behind)."""
    sh = W.HeadShape(4, 6, 256, 8192, 64)
    inp = W.make_head_inputs(sh, 5)
    t = [dev_bf16(x) for x in (inp.sel_reps, inp.w_lm, inp.ar_w, inp.ar_e)]
    bonus = torch.from_numpy(inp.bonus).cuda()
    u = torch.rand(4, 6, device="cuda") * (1 - 2.0 ** -20)
    g, plan = dp.draft_head(t[0], t[1], t[2], t[3], bonus)
    g = g.clone()
    s1 = plan.run(t[0], t[1], t[2], t[3], bonus, uniforms=u).clone()
    s2 = plan.run(t[0], t[1], t[2], t[3], bonus, uniforms=u).clone()
    g2 = plan.run(t[0], t[1], t[2], t[3], bonus).clone()
    torch.cuda.synchronize()
    assert plan.status.item() == 0
    assert torch.equal(s1, s2)
    assert torch.equal(g, g2)
    assert not torch.equal(s1, g)
