"""GPU parity of dpara_verify_select against the oracle: bit-exact integers and bit-exact gathered rows."""
import numpy as np
import pytest
import torch

import workloads as W
from oracle import verify as OV

pytestmark = pytest.mark.gpu


def _check(v, mode):
    from gpu_util import run_verify, check_verify
    res = run_verify(v, mode)
    if mode == 0:
        ref = OV.verify_greedy(v.target, v.draft_tokens, v.reps)
    else:
        ref = OV.verify_sampling(v.target, v.draft_probs, v.draft_tokens, v.uniforms, v.reps)
    check_verify(res, ref)
    return ref


@pytest.mark.parametrize("V", [1000, 1001, 8192, 8196, 40000, 151936])
def test_greedy_parity_sizes(V):
    sh = W.VerifyShape(5, 6, V, 4, 256, "greedy", 0.7, 1.0)
    v = W.make_verify_inputs(sh, 100 + V, force_full=[0], force_zero=[1])
    ref = _check(v, 0)
    assert ref["accept_len"][0] == 5 and ref["accept_len"][1] == 0


def test_greedy_cfg1_and_cfg2():
    for idx in (1, 2):
        w = W.workload(idx)
        _check(W.make_verify_inputs(w.verify, w.seed), 0)


def test_greedy_cfg3_full_size():
    w = W.workload(3)
    v = W.make_verify_inputs(w.verify, w.seed, force_full=[3], force_zero=[5])
    ref = _check(v, 0)
    assert len(set(ref["accept_len"].tolist())) >= 4


def test_greedy_ties_and_specials():
    """Duplicate maxima inside one 16-byte vector, across threads, across CTAs (chunks), at the first and
    last vocabulary index; -0/+0; NaN and -inf rows."""
    V, J = 20000, 8
    rng = np.random.default_rng(3)
    logits = rng.standard_normal((2, J, V)).astype(np.float32)
    big = np.float32(50.0)
    logits[0, 0, [5, 6]] = big                    # same float4
    logits[0, 1, [100, 9000]] = big               # different CTAs (chunk = 8192)
    logits[0, 2, [V - 1, 3]] = big                # last index vs early index
    logits[0, 3, [0, V - 1]] = big                # first and last
    logits[0, 4, :] = -np.inf                     # all -inf -> 0
    logits[0, 5, :] = np.nan                      # all NaN -> 0
    logits[0, 6, :] = np.nan
    logits[0, 6, 777] = -np.inf                   # -inf beats NaN
    logits[0, 7, :] = -1.0
    logits[0, 7, 4097] = -0.0
    logits[0, 7, 12000] = 0.0                     # -0 == +0: lower index wins
    logits[1, 0, 8191] = big
    logits[1, 0, 8192] = big                      # chunk edge
    a0 = [5, 100, 3, 0, 0, 0, 777, 4097]
    toks = np.zeros((2, J - 1), np.int32)
    toks[0] = a0[:J - 1]
    toks[1] = -5                                   # out of range -> rejected, status bit
    v = W.VerifyInputs(W.VerifyShape(2, J, V, 2, 64), logits, toks, W.make_verify_inputs(W.VerifyShape(2, J, V, 2, 64), 1).reps)
    ref = _check(v, 0)
    assert ref["accept_len"][0] == J - 1 and ref["bonus"][0] == 4097
    assert ref["accept_len"][1] == 0 and ref["bonus"][1] == 8191 and ref["status"] == 1


def test_greedy_single_boundary_and_repeat():
    from gpu_util import run_verify, check_verify
    sh = W.VerifyShape(3, 1, 5000, 2, 64, "greedy", 0.5, 1.0)
    v = W.make_verify_inputs(sh, 9)
    ref = _check(v, 0)
    assert np.all(ref["accept_len"] == 0)
    # two runs give identical bits (no race on the ticket/atomic path)
    sh = W.VerifyShape(8, 16, 30000, 4, 128, "greedy", 0.8, 2.0)
    v = W.make_verify_inputs(sh, 10)
    r1, r2 = run_verify(v, 0), run_verify(v, 0)
    for k in ("accept_len", "bonus", "out_tokens", "selected"):
        assert torch.equal(r1[k], r2[k])


@pytest.mark.parametrize("V", [16, 1001, 4096, 5000, 151936])
def test_sampling_parity_sizes(V):
    sh = W.VerifyShape(6, 5, V, 4, 128, "sampling", 0.0, 3.0)
    v = W.make_verify_inputs(sh, 200 + V, force_full=[2])
    ref = _check(v, 1)
    assert ref["accept_len"][2] == 4


def test_sampling_cfg4_full_size():
    w = W.workload(4)
    v = W.make_verify_inputs(w.verify, w.seed, force_full=[1])
    ref = _check(v, 1)
    assert ref["accept_len"][1] == 15 and len(set(ref["accept_len"].tolist())) >= 3


def test_sampling_fallbacks():
    # rejected position with an empty residual -> p_r; all-zero target row -> lowest-index maximum;
    # extreme uniforms; out-of-range token
    V, J = 6000, 3
    p = np.zeros((4, J, V), np.float32)
    q = np.zeros((4, J - 1, V), np.float32)
    p[:, :, 10] = 0.5; p[:, :, 4500] = 0.25
    q[:, :, 10] = 0.5; q[:, :, 4500] = 0.5
    toks = np.full((4, J - 1), 4500, np.int32)
    u = np.full((4, J), 0.75, np.float32)
    p[1, 0, :] = 0                                  # request 1: row 0 all zero -> rejected (0 < 0 false), argmax fallback
    u[2, :] = 0.0                                   # request 2: u = 0 accepts while p > 0; bonus with m = 0
    u[2, J - 1] = np.float32((2 ** 24 - 1) * 2.0 ** -24)
    toks[3, 0] = V + 3                              # request 3: bad token
    reps = W.make_verify_inputs(W.VerifyShape(4, J, V, 2, 64), 1).reps
    v = W.VerifyInputs(W.VerifyShape(4, J, V, 2, 64, "sampling"), p, toks, reps, q, u)
    ref = _check(v, 1)
    assert ref["accept_len"].tolist() == [0, 0, 2, 0] and ref["bonus"][0] == 4500 and ref["bonus"][1] == 0
    assert ref["bonus"][2] == 4500 and ref["status"] == 1


def test_workspace_is_left_zeroed_and_reusable_across_modes_and_shapes():
    """One zero-filled workspace serves calls of both modes and several shapes back to back with no clearing in
    between: every call restores the zeros it consumed.  Covers each of the greedy kernel's chunk sizes
    (the chunk is chosen from rows x vocabulary so that the grid fills the GPU)."""
    import paper_2609_27396_b200 as dp
    from gpu_util import dev_bf16, host_bits
    shapes = [W.VerifyShape(1, 8, 151936, 8, 256, "greedy", 0.8, 2.0),       # few rows: small chunks
              W.VerifyShape(16, 16, 151936, 4, 64, "greedy", 0.75, 1.0),     # many rows: 16 K-float chunks
              W.VerifyShape(4, 6, 20000, 4, 128, "sampling", 0.0, 3.0),
              W.VerifyShape(3, 16, 151936, 4, 64, "greedy", 0.8, 1.0),
              W.VerifyShape(6, 16, 151936, 4, 64, "greedy", 0.8, 1.0),
              W.VerifyShape(2, 3, 50000, 4, 64, "sampling", 0.0, 3.0),
              W.VerifyShape(40, 16, 60000, 2, 64, "greedy", 0.8, 1.0)]
    plans = [dp.VerifyPlan(batch=s.batch, n_boundaries=s.n_boundaries, vocab=s.vocab, block=s.block, hidden=s.hidden,
                           mode=1 if s.mode == "sampling" else 0) for s in shapes]
    shared = torch.zeros(max(p.workspace.numel() for p in plans), dtype=torch.uint8, device="cuda")
    for rep in range(2):
        for k, (s, plan) in enumerate(zip(shapes, plans)):
            plan.workspace = shared
            v = W.make_verify_inputs(s, 300 + 10 * rep + k)
            kw = dict(target=torch.from_numpy(v.target).cuda(), draft_tokens=torch.from_numpy(v.draft_tokens).cuda(), reps=dev_bf16(v.reps))
            if s.mode == "sampling":
                kw.update(draft_probs=torch.from_numpy(v.draft_probs).cuda(), uniforms=torch.from_numpy(v.uniforms).cuda())
                ref = OV.verify_sampling(v.target, v.draft_probs, v.draft_tokens, v.uniforms, v.reps)
            else:
                ref = OV.verify_greedy(v.target, v.draft_tokens, v.reps)
            plan(**kw)
            torch.cuda.synchronize()
            for key in ("accept_len", "bonus", "gather_idx", "out_tokens"):
                assert np.array_equal(getattr(plan, key).cpu().numpy(), ref[key]), (key, k, rep)
            assert np.array_equal(host_bits(plan.selected), ref["selected"]), (k, rep)
            assert int(shared.count_nonzero().item()) == 0, (k, rep)       # left as it was found


def test_sampling_uniform_of_one_is_clamped():
    V, J = 5000, 2
    p = np.zeros((1, J, V), np.float32); q = np.zeros((1, J - 1, V), np.float32)
    p[0, :, [7, 4100]] = 0.5
    q[0, :, 7] = 1.0
    toks = np.full((1, J - 1), 7, np.int32)          # accepted iff u * 1 < 0.5
    u = np.array([[0.75, 1.0]], np.float32)          # rejected at once; bonus uniform exactly 1.0
    v = W.VerifyInputs(W.VerifyShape(1, J, V, 2, 64, "sampling"), p, toks, None, q, u)
    ref = _check(v, 1)
    assert ref["accept_len"][0] == 0 and ref["bonus"][0] == 4100


@pytest.mark.parametrize("mode", [0, 1])
def test_early_start_behind_the_attention_kernel(mode):
    """DPARA_VERIFY_EARLY_START: queued right behind the attention call that produces `reps`, the call starts on its other
    inputs at once and waits for the attention only before the gather -- same outputs as the plain call, bit for bit,
    every time (eight rounds with fresh attention inputs, so a gather that ran ahead would read the round before)."""
    import paper_2609_27396_b200 as dp
    from gpu_util import dev_bf16
    w = W.workload(2)
    a, v = w.attn, w.verify
    plain = dp.VerifyPlan(batch=v.batch, n_boundaries=v.n_boundaries, vocab=v.vocab, block=v.block, hidden=v.hidden, mode=mode)
    early = dp.VerifyPlan(batch=v.batch, n_boundaries=v.n_boundaries, vocab=v.vocab, block=v.block, hidden=v.hidden, mode=mode, early_start=True)
    out = torch.zeros((a.batch, a.n_boundaries, a.block, a.n_q_heads, a.head_dim), dtype=torch.bfloat16, device="cuda")
    reps = out.view(a.batch, a.n_boundaries, a.block, a.n_q_heads * a.head_dim)
    for rnd in range(8):
        inp = W.make_attn_inputs(a, 100 + rnd)
        t = {k: dev_bf16(getattr(inp, k)) for k in ("q", "k_ctx", "v_ctx", "k_spine", "v_spine", "k_blk", "v_blk")}
        plan = dp.DraftPlan(ctx_offsets=[int(x) for x in inp.ctx_offsets], n_boundaries=a.n_boundaries, block=a.block, n_q_heads=a.n_q_heads,
                            n_kv_heads=a.n_kv_heads, head_dim=a.head_dim, prefix_base=a.prefix_base, n_spine=a.spine)
        ver = W.make_verify_inputs(W.VerifyShape(v.batch, v.n_boundaries, v.vocab, v.block, v.hidden, "greedy" if mode == 0 else "sampling", v.agreement,
                                                 v.logit_sigma), 200 + rnd)
        kw = dict(target=torch.from_numpy(ver.target).cuda(), draft_tokens=torch.from_numpy(ver.draft_tokens).cuda())
        if mode == 1:
            kw.update(draft_probs=torch.from_numpy(ver.draft_probs).cuda(), uniforms=torch.from_numpy(ver.uniforms).cuda())
        plan(**t, out=out)
        early(reps=reps, **kw)
        torch.cuda.synchronize()
        plain(reps=reps, **kw)
        torch.cuda.synchronize()
        for f in ("accept_len", "bonus", "gather_idx", "out_tokens", "selected"):
            assert torch.equal(getattr(plain, f), getattr(early, f)), (rnd, f)
        assert plain.status.item() == early.status.item() == 0
