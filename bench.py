#!/usr/bin/env python
"""Benchmark of the all-boundary draft step (one process per GPU).

A step = one pass of the whole hot path over one synthetic batch: the all-boundary attention
(dpara_draft_all_boundaries) followed by greedy verify/select with the fused branch gather
(dpara_verify_select) on the attention's own output.  Default workload: the Qwen3-14B-shaped b = 16
ragged batch (cfg3); the b = 1 Qwen3-8B-shaped step (cfg2) is timed as well and reported under "b1".

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload cfg3|cfg2]

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle on the host cores instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import workloads as W  # noqa: E402

METRIC = "all_boundary_draft_step_us"
L2_FLUSH_BYTES = 256 << 20


def ncu_dram_traffic(workload: str):
    """dram__bytes_read.sum + dram__bytes_write.sum of one attention launch of this workload, as recorded from an ncu
    capture in profiles/traffic.json (bytes per launch; None where no capture exists)."""
    try:
        return json.load(open(os.path.join(ROOT, "profiles", "traffic.json")))["attention"][workload]["dram_bytes_per_launch"]
    except Exception:
        return None


# ----------------------------------------------------------------------------- algorithmic work (flops and bytes every launch must do)
def attention_flops(sh: W.AttnShape) -> float:
    """4 * D flops per (query row, visible key): QK^T and PV."""
    rows_per_boundary = sh.block * sh.n_q_heads
    tot = 0.0
    for L in sh.ctx_lens:
        for j in range(sh.n_boundaries):
            keys = L + min(j + sh.prefix_base, sh.spine) + sh.block
            tot += 4.0 * sh.head_dim * rows_per_boundary * keys
    return tot


def attention_bytes(sh: W.AttnShape, out_bytes: int = 2) -> float:
    """Every input read once, every output written once."""
    kv = 2 * 2 * sh.n_kv_heads * sh.head_dim
    b, J, Bq = sh.batch, sh.n_boundaries, sh.block
    q = b * J * Bq * sh.n_q_heads * sh.head_dim
    return sum(sh.ctx_lens) * kv + b * sh.spine * kv + b * J * Bq * kv + q * 2 + q * out_bytes


def verify_bytes(v: W.VerifyShape) -> float:
    gather = v.batch * v.block * v.hidden * 2
    return v.batch * v.n_boundaries * v.vocab * 4 + 2 * gather


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d["bf16_tflops"], bf16_tflops_sustained=d.get("bf16_tflops_sustained"),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


# ----------------------------------------------------------------------------- clocks sampler
class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "100"], stdout=subprocess.PIPE, text=True)
            threading.Thread(target=self._pump, daemon=True).start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], None, set()
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx = float(r[1])
            except Exception:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        busy = [x for x in sm if mx and x > 0.5 * mx] or sm
        return {"sm_mhz": statistics.median(busy) if busy else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


# ----------------------------------------------------------------------------- the CUDA arm
class StepRunner:
    """Owns device-resident inputs, fixed plans and (for the end-to-end leg) pinned host copies."""

    def __init__(self, wl: W.Workload, seed: int):
        import torch
        import paper_2609_27396_b200 as dp
        self.torch, self.dp, self.wl = torch, dp, wl
        a, v = wl.attn, wl.verify
        self.inp = W.make_attn_inputs(a, seed)
        self.ver = W.make_verify_inputs(v, seed, reps=np.zeros((1,), np.uint16))
        bf = lambda bits: torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16)
        i = self.inp
        self.host = dict(q=bf(i.q), k_ctx=bf(i.k_ctx), v_ctx=bf(i.v_ctx), k_spine=bf(i.k_spine), v_spine=bf(i.v_spine),
                         k_blk=bf(i.k_blk), v_blk=bf(i.v_blk), target=torch.from_numpy(self.ver.target),
                         draft_tokens=torch.from_numpy(self.ver.draft_tokens))
        self.dev = {k: t.cuda() for k, t in self.host.items()}
        self.out = torch.zeros((a.batch, a.n_boundaries, a.block, a.n_q_heads, a.head_dim), dtype=torch.bfloat16, device="cuda")
        self.plan = dp.DraftPlan(ctx_offsets=[int(x) for x in i.ctx_offsets], n_boundaries=a.n_boundaries, block=a.block,
                                 n_q_heads=a.n_q_heads, n_kv_heads=a.n_kv_heads, head_dim=a.head_dim,
                                 prefix_base=a.prefix_base, n_spine=a.spine)
        self.plan1 = dp.DraftPlan(ctx_offsets=[int(x) for x in i.ctx_offsets], n_boundaries=a.n_boundaries, block=a.block,
                                  n_q_heads=a.n_q_heads, n_kv_heads=a.n_kv_heads, head_dim=a.head_dim,
                                  prefix_base=a.prefix_base, n_spine=a.spine, boundary_lo=a.n_boundaries - 1)
        self.vplan = dp.VerifyPlan(batch=v.batch, n_boundaries=v.n_boundaries, vocab=v.vocab, block=v.block,
                                   hidden=v.hidden, mode=0)
        # the same call allowed to start while the attention kernel in front of it is still running (it waits for it only
        # before it gathers the selected branch): the case where verification has resolved before the precompute ends
        self.vplan_early = dp.VerifyPlan(batch=v.batch, n_boundaries=v.n_boundaries, vocab=v.vocab, block=v.block,
                                         hidden=v.hidden, mode=0, early_start=True)
        self.reps = self.out.view(a.batch, a.n_boundaries, a.block, a.hidden)
        self.flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device="cuda")
        self.pinned = None

    def attention(self, plan=None, src=None):
        d = src or self.dev
        (plan or self.plan)(q=d["q"], k_ctx=d["k_ctx"], v_ctx=d["v_ctx"], k_spine=d["k_spine"], v_spine=d["v_spine"],
                            k_blk=d["k_blk"], v_blk=d["v_blk"], out=self.out)

    def verify(self, src=None):
        d = src or self.dev
        self.vplan(target=d["target"], draft_tokens=d["draft_tokens"], reps=self.reps)

    def step(self):
        self.attention()
        self.verify()

    def step_early(self):
        d = self.dev
        self.attention()
        self.vplan_early(target=d["target"], draft_tokens=d["draft_tokens"], reps=self.reps)

    def timed_early_steps(self, k: int):
        """k steps with the early-start verify/select (ms each), and a check that it selects what the plain call selects."""
        torch = self.torch
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(k)]
        for s in range(k):
            self.flush.zero_()
            ev[s][0].record()
            self.step_early()
            ev[s][1].record()
        torch.cuda.synchronize()
        self.step()
        torch.cuda.synchronize()
        same = all(bool(torch.equal(getattr(self.vplan, f), getattr(self.vplan_early, f))) for f in ("accept_len", "bonus", "out_tokens", "selected"))
        return [e[0].elapsed_time(e[1]) for e in ev], same

    def timed_steps(self, k: int, single_boundary: bool = False, parts: bool = True):
        """k steps, each bracketed by CUDA events on the launching stream, L2 flushed in between.
        Returns per-step (total_ms, attention_ms, verify_ms); the two parts are timed in passes of their own (k launches each)."""
        torch = self.torch

        def timed(fn):
            ev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(k)]
            for s in range(k):
                self.flush.zero_()
                ev[s][0].record()
                fn()
                ev[s][1].record()
            torch.cuda.synchronize()
            return [e[0].elapsed_time(e[1]) for e in ev]
        att = lambda: self.attention(self.plan1 if single_boundary else None)
        if single_boundary:
            t = timed(att)
            return [(x, x, 0.0) for x in t]
        # the step as a caller issues it (the two calls back to back, no event between them: the second kernel's launch
        # overlaps the first one's tail); with parts=True each call on its own afterwards
        total = timed(lambda: (att(), self.verify()))
        if not parts:
            return [(x, 0.0, 0.0) for x in total]
        # the attention on its own after the flush; verify/select where it stands in the step -- behind the attention (untimed
        # here), not behind the flush, whose 256 MB of dirty lines would still be draining into HBM under its reads
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(k)]
        for s in range(k):
            self.flush.zero_()
            att()
            ev[s][0].record()
            self.verify()
            ev[s][1].record()
        torch.cuda.synchronize()
        return list(zip(total, timed(att), [e[0].elapsed_time(e[1]) for e in ev]))

    # end to end: host (pinned) buffers in, results back on the host, copies inside the timed region
    def setup_e2e(self):
        torch = self.torch
        self.pinned = {k: t.pin_memory() for k, t in self.host.items()}
        self.stage = {k: torch.empty_like(t, device="cuda") for k, t in self.host.items()}
        vp = self.vplan
        self.res_host = {k: torch.empty_like(getattr(vp, k), device="cpu").pin_memory()
                         for k in ("accept_len", "bonus", "gather_idx", "out_tokens", "selected")}
        self.h2d_bytes = sum(t.numel() * t.element_size() for t in self.pinned.values())
        self.d2h_bytes = sum(t.numel() * t.element_size() for t in self.res_host.values())

    def e2e_steps(self, k: int):
        torch = self.torch
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(k)]
        for s in range(k):
            self.flush.zero_()
            ev[s][0].record()
            for key, t in self.pinned.items():
                self.stage[key].copy_(t, non_blocking=True)
            self.attention(src=self.stage)
            self.verify(src=self.stage)
            for key, t in self.res_host.items():
                t.copy_(getattr(self.vplan, key), non_blocking=True)
            ev[s][1].record()
        torch.cuda.synchronize()
        return [e[0].elapsed_time(e[1]) for e in ev]


class LayerRunner:
    """The full-layer, long-context workload (cfg5): one draft call runs the whole backbone block around the
    all-boundary attention; greedy verify/select then gathers from the block's bf16 output."""

    def __init__(self, wl: W.Workload, seed: int):
        import torch
        import paper_2609_27396_b200 as dp
        self.torch = torch
        a, v, l = wl.attn, wl.verify, wl.layer
        ain = W.make_attn_inputs(a, seed, with_q=False, with_blk=False)
        lin = W.make_layer_inputs(l, a, seed)
        ver = W.make_verify_inputs(v, seed, reps=np.zeros((1,), np.uint16))
        bf = lambda bits: torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)
        self.attn, self.layer, self.ctx_offsets = a, l, [int(x) for x in ain.ctx_offsets]
        self.t = {k: bf(getattr(lin, k)) for k in ("x", "w_qkv", "w_o", "w_gate_up", "w_down", "rms1_w", "rms2_w", "qnorm_w", "knorm_w")}
        self.kv = {k: bf(getattr(ain, k)) for k in ("k_ctx", "v_ctx", "k_spine", "v_spine")}
        self.y = torch.zeros((a.batch, a.n_boundaries, a.block, l.hidden), dtype=torch.float32, device="cuda")
        self.y16 = torch.zeros((a.batch, a.n_boundaries, a.block, l.hidden), dtype=torch.bfloat16, device="cuda")
        lio = dp.make_layer_io(**self.t, rms_eps=l.rms_eps, rope_theta=l.rope_theta, use_rope=l.use_rope, y_f32=self.y, y_bf16=self.y16)
        self.plan = dp.DraftPlan(ctx_offsets=[int(x) for x in ain.ctx_offsets], n_boundaries=a.n_boundaries, block=a.block,
                                 n_q_heads=a.n_q_heads, n_kv_heads=a.n_kv_heads, head_dim=a.head_dim, prefix_base=a.prefix_base,
                                 n_spine=a.spine, layer=lio)
        self.vplan = dp.VerifyPlan(batch=v.batch, n_boundaries=v.n_boundaries, vocab=v.vocab, block=v.block, hidden=v.hidden, mode=0)
        self.target = torch.from_numpy(ver.target).cuda()
        self.tokens = torch.from_numpy(ver.draft_tokens).cuda()
        self.flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device="cuda")

    def step(self):
        self.plan(**self.kv)
        self.vplan(target=self.target, draft_tokens=self.tokens, reps=self.y16)

    def timed_steps(self, k: int):
        torch = self.torch
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(k)]
        for s in range(k):
            self.flush.zero_()
            ev[s][0].record()
            self.plan(**self.kv)
            ev[s][1].record()
            self.vplan(target=self.target, draft_tokens=self.tokens, reps=self.y16)
            ev[s][2].record()
        torch.cuda.synchronize()
        return [(e[0].elapsed_time(e[2]), e[0].elapsed_time(e[1]), e[1].elapsed_time(e[2])) for e in ev]


def _median_us(fn, k, flush):
    import torch
    ts = []
    for _ in range(3):
        fn()
    for _ in range(k):
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); fn(); e1.record()
        torch.cuda.synchronize()
        ts.append(e0.elapsed_time(e1) * 1e3)
    return statistics.median(ts)


def _layer_attention_only_us(self, k: int) -> float:
    """The all-boundary attention of the full-layer workload on its own (random q / block keys of the right shape)."""
    import torch
    import paper_2609_27396_b200 as dp
    a = self.attn
    g = torch.Generator(device="cuda").manual_seed(1)
    mk = lambda *sh: torch.randn(*sh, device="cuda", generator=g).to(torch.bfloat16)
    q, kb, vb = mk(a.batch, a.n_boundaries, a.block, a.n_q_heads, a.head_dim), mk(a.batch, a.n_boundaries, a.block, a.n_kv_heads, a.head_dim), mk(a.batch, a.n_boundaries, a.block, a.n_kv_heads, a.head_dim)
    out = torch.zeros_like(q)
    plan = dp.DraftPlan(ctx_offsets=self.ctx_offsets, n_boundaries=a.n_boundaries, block=a.block, n_q_heads=a.n_q_heads,
                        n_kv_heads=a.n_kv_heads, head_dim=a.head_dim, prefix_base=a.prefix_base, n_spine=a.spine)
    return _median_us(lambda: plan(q=q, **self.kv, k_blk=kb, v_blk=vb, out=out), k, self.flush)


def _graph_us(fn, flush, k: int = 10) -> float:
    """Device time of fn() per call: k x (L2 flush, fn) replayed from one CUDA graph, minus k x flush."""
    import torch

    def timed(body):
        s = torch.cuda.Stream()
        with torch.cuda.stream(s):
            for _ in range(2):
                body()
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=s):
                for _ in range(k):
                    flush.zero_(); body()
            ts = []
            for _ in range(5):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(s); g.replay(); e1.record(s)
                torch.cuda.synchronize()
                ts.append(e0.elapsed_time(e1) * 1e3 / k)
        return statistics.median(ts)
    return timed(fn) - timed(lambda: None)


def _layer_gemm_legs(self, peaks, k: int, only=None):
    """Each projection of the block on its own (dpara_gemm_bf16 at the block's shapes, buffers allocated up front, calls
    replayed from a CUDA graph so that no host time is in the figure)."""
    import ctypes as C
    import torch
    import paper_2609_27396_b200 as dp
    a, l = self.attn, self.layer
    M = a.batch * a.n_boundaries * a.block
    qd, kd = a.n_q_heads * a.head_dim, a.n_kv_heads * a.head_dim
    g = torch.Generator(device="cuda").manual_seed(2)
    act = lambda K: torch.randn(M, K, device="cuda", generator=g).to(torch.bfloat16)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    res = {}
    for name, w, K, N, epi in (("qkv", self.t["w_qkv"], l.hidden, qd + 2 * kd, 0), ("o", self.t["w_o"], qd, l.hidden, 1),
                               ("gate_up", self.t["w_gate_up"], l.hidden, l.intermediate, 2), ("down", self.t["w_down"], l.intermediate, l.hidden, 1)):
        if only is not None and name != only:
            continue
        x = act(K)
        resid = torch.zeros(M, N, dtype=torch.bfloat16 if name == "o" else torch.float32, device="cuda") if epi == 1 else None
        out = torch.empty(M, N, dtype=torch.float32 if epi == 1 else torch.bfloat16, device="cuda")
        io = dp.GemmIO(x.data_ptr(), w.data_ptr(), M, N, K, epi, resid.data_ptr() if resid is not None else None,
                       dp.BF16 if name == "o" else dp.F32, out.data_ptr(), None)

        def call():
            rc = dp.lib.dpara_gemm_bf16(C.byref(io), status.data_ptr(), torch.cuda.current_stream().cuda_stream)
            assert rc == 0
        us = _graph_us(call, self.flush, k)
        fl = 2.0 * M * K * N * (2 if epi == 2 else 1)
        res[name] = {"M": M, "N": N, "K": K, "us": us, "tflops": fl / (us * 1e-6) / 1e12, "frac_of_measured_burst": fl / (us * 1e-6) / 1e12 / peaks["bf16_tflops"]}
    return res


LayerRunner.attention_only_us = _layer_attention_only_us
LayerRunner.gemm_legs = _layer_gemm_legs


def backbone_leg(w5: W.Workload, peaks, k: int):
    """Two stacked blocks with the spine tokens as query rows (dpara_draft_backbone) at the full-layer workload's shapes:
    M = b * (J * Bq + S) rows per block, each block with its own 32 K-token context cache."""
    import torch
    import paper_2609_27396_b200 as dp
    a, l = w5.attn, w5.layer
    n_layers = 2
    R = a.n_boundaries * a.block + a.spine
    g = torch.Generator(device="cuda").manual_seed(3)
    mk = lambda sig, *sh: (torch.randn(*sh, device="cuda", generator=g) * sig).to(torch.bfloat16)
    off = [0]
    for L in a.ctx_lens:
        off.append(off[-1] + L)
    x = mk(1.0, a.batch, R, l.hidden)
    y = torch.zeros(a.batch, R, l.hidden, dtype=torch.float32, device="cuda")
    y16 = torch.zeros(a.batch, R, l.hidden, dtype=torch.bfloat16, device="cuda")
    qd, kd = a.n_q_heads * a.head_dim, a.n_kv_heads * a.head_dim
    layers, keep, kc, vc = [], [], [], []
    for _ in range(n_layers):
        t = dict(w_qkv=mk(l.weight_sigma, qd + 2 * kd, l.hidden), w_o=mk(l.weight_sigma, l.hidden, qd),
                 w_gate_up=mk(l.weight_sigma, 2 * l.intermediate, l.hidden), w_down=mk(l.weight_sigma, l.hidden, l.intermediate),
                 rms1_w=torch.ones(l.hidden, dtype=torch.bfloat16, device="cuda"), rms2_w=torch.ones(l.hidden, dtype=torch.bfloat16, device="cuda"),
                 qnorm_w=torch.ones(a.head_dim, dtype=torch.bfloat16, device="cuda"), knorm_w=torch.ones(a.head_dim, dtype=torch.bfloat16, device="cuda"))
        keep.append(t)
        layers.append(dp.make_layer_io(x=x, **t, rms_eps=l.rms_eps, rope_theta=l.rope_theta, use_rope=True, y_f32=y, y_bf16=y16))
        kc.append(mk(1.0, off[-1], a.n_kv_heads, a.head_dim)); vc.append(mk(1.0, off[-1], a.n_kv_heads, a.head_dim))
    plan = dp.BackbonePlan(ctx_offsets=off, n_boundaries=a.n_boundaries, block=a.block, n_q_heads=a.n_q_heads, n_kv_heads=a.n_kv_heads,
                           head_dim=a.head_dim, layers=layers, k_ctx=kc, v_ctx=vc, prefix_base=a.prefix_base, n_spine=a.spine)
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device="cuda")
    us = _median_us(lambda: plan(), k, flush)
    M = a.batch * R
    rows_fl = 0.0
    for L in a.ctx_lens:
        for j in range(a.n_boundaries):
            rows_fl += 4.0 * a.head_dim * a.block * a.n_q_heads * (L + min(j + a.prefix_base, a.spine) + a.block)
        for s_ in range(a.spine):
            rows_fl += 4.0 * a.head_dim * a.n_q_heads * (L + s_ + 1)
    fl = n_layers * (rows_fl + 2.0 * M * (l.hidden * (qd + 2 * kd) + qd * l.hidden + 3 * l.hidden * l.intermediate))
    return {"workload": f"{n_layers} blocks, spine tokens as query rows, {w5.name} shapes: M = {M} rows per block", "us": us, "us_per_block": us / n_layers,
            "flops": fl, "tflops": fl / (us * 1e-6) / 1e12, "tensor_frac_of_measured_burst": fl / (us * 1e-6) / 1e12 / peaks["bf16_tflops"]}


def graph_timed_b1(r: "StepRunner", k: int = 20):
    """The b = 1 step replayed from ONE CUDA graph (k x (L2 flush, attention, verify/select) minus k x flush): what the
    device spends when the launches come from a captured graph, as the paper's single-GPU deployment does, instead of
    from Python.  Both calls capture as they are (fixed addresses, no allocation)."""
    import torch

    def timed(fn):
        s = torch.cuda.Stream()
        with torch.cuda.stream(s):
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=s):
                for _ in range(k):
                    r.flush.zero_(); fn()
            ts = []
            for _ in range(5):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(s); g.replay(); e1.record(s)
                torch.cuda.synchronize()
                ts.append(e0.elapsed_time(e1) * 1e3 / k)
        return statistics.median(ts)
    base = timed(lambda: None)
    return {"graph_replay": {"step_us": timed(r.step) - base, "early_start_step_us": timed(r.step_early) - base, "attention_us": timed(r.attention) - base,
                             "verify_select_us": timed(r.verify) - base, "single_boundary_attention_us": timed(lambda: r.attention(r.plan1)) - base,
                             "note": "k x (flush, calls) replayed from one CUDA graph, minus k x flush"}}


def small_step_leg(index: int, k: int):
    w = W.workload(index)
    r = StepRunner(w, w.seed)
    for _ in range(5):
        r.step()
    p = r.timed_steps(k)
    return {"workload": w.name, "step_us": statistics.median(x[0] for x in p) * 1e3, "attention_us": statistics.median(x[1] for x in p) * 1e3,
            "verify_select_us": statistics.median(x[2] for x in p) * 1e3}


def sampling_select_leg(peaks, k: int):
    """Rejection-sampling verify/select (cfg4).  Algorithmic bytes: the 2 * gamma scalars of the accept tests plus rows p_r
    and q_r of each request and the gathered branch (read + write) -- not the whole probability tensors."""
    import torch
    import paper_2609_27396_b200 as dp
    w = W.workload(4)
    v = w.verify
    ver = W.make_verify_inputs(v, w.seed)
    bf = lambda bits: torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)
    t = dict(target=torch.from_numpy(ver.target).cuda(), draft_tokens=torch.from_numpy(ver.draft_tokens).cuda(), reps=bf(ver.reps),
             draft_probs=torch.from_numpy(ver.draft_probs).cuda(), uniforms=torch.from_numpy(ver.uniforms).cuda())
    plan = dp.VerifyPlan(batch=v.batch, n_boundaries=v.n_boundaries, vocab=v.vocab, block=v.block, hidden=v.hidden, mode=1)
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device="cuda")
    us = _median_us(lambda: plan(**t), k, flush)
    by = v.batch * (2 * v.vocab * 4 + 2 * v.block * v.hidden * 2)
    return {"workload": w.name, "us": us, "algorithmic_bytes": by, "gbs": by / (us * 1e-6) / 1e9, "frac_of_measured_hbm": by / (us * 1e-6) / 1e9 / peaks["hbm_gbs"],
            "bound": "latency (9.7 MB)"}


def cache_append_leg(wl: W.Workload, peaks, k: int, n_layers: int = 5):
    """Feature-cache append (dpara_cache_append) at the main workload's shapes: b requests x J candidate rows of `hidden`
    features into the caches of n_layers drafter layers.  Algorithmic bytes: each layer's [keys | values] projection once."""
    import torch
    import paper_2609_27396_b200 as dp
    a, v = wl.attn, wl.verify
    J, F, Hkv, D = a.n_boundaries, v.hidden, a.n_kv_heads, a.head_dim
    g = torch.Generator(device="cuda").manual_seed(4)
    mk = lambda sig, *sh: (torch.randn(*sh, device="cuda", generator=g) * sig).to(torch.bfloat16)
    cap = [L + 4 * J for L in a.ctx_lens]
    start = [0]
    for c in cap[:-1]:
        start.append(start[-1] + c)
    rows = sum(cap)
    kc = [torch.zeros(rows, Hkv, D, dtype=torch.bfloat16, device="cuda") for _ in range(n_layers)]
    vc = [torch.zeros(rows, Hkv, D, dtype=torch.bfloat16, device="cuda") for _ in range(n_layers)]
    lens0 = torch.tensor(list(a.ctx_lens), dtype=torch.int64, device="cuda")
    lens = lens0.clone()
    plan = dp.CachePlan(batch=a.batch, n_rows=J, w_kv=[mk(0.02, 2 * Hkv * D, F) for _ in range(n_layers)], k_ctx=kc, v_ctx=vc,
                        row_start=torch.tensor(start, dtype=torch.int64, device="cuda"), capacity=torch.tensor(cap, dtype=torch.int64, device="cuda"),
                        ctx_len=lens, norm_w=[torch.ones(F, dtype=torch.bfloat16, device="cuda")] * n_layers,
                        knorm_w=[torch.ones(D, dtype=torch.bfloat16, device="cuda") for _ in range(n_layers)])
    feats = mk(1.0, a.batch, J, F)
    acc = torch.randint(0, J, (a.batch,), device="cuda", generator=g).to(torch.int32)
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device="cuda")

    def call():
        lens.copy_(lens0)             # (a device-to-device copy of b lengths: keeps every timed call at the same fill level)
        plan.run(feats, acc)
    us = _median_us(call, k, flush)
    by = n_layers * 2 * Hkv * D * F * 2 + a.batch * J * F * 2
    return {"workload": f"{wl.name} shapes: b={a.batch}, {J} candidate rows x {F} features, {n_layers} layers, Hkv={Hkv}, D={D}", "us": us,
            "us_per_layer": us / n_layers, "algorithmic_bytes": by, "gbs": by / (us * 1e-6) / 1e9,
            "frac_of_measured_hbm": by / (us * 1e-6) / 1e9 / peaks["hbm_gbs"]}


def colocation_leg(peaks, n_layers: int = 2, standin_gb: float = 3.0):
    """One round on ONE GPU the way the paper's single-GPU deployment runs it (Sec. 3.3: T_step ~ max(T_verify, T_precompute) +
    T_Head; App. D, single-GPU paragraph: verification and backbone precomputation on two streams, everything captured in one CUDA
    graph).  Stream A: a STAND-IN for the target's verification forward (there is no target model here): a chain of library matmuls
    of the verified rows against `standin_gb` GB of bf16 weights, i.e. a weight-streaming load like a decoder forward.  Stream B: the
    all-boundary backbone pass (dpara_draft_backbone, spine tokens as query rows, the paper's main draft length d = 7).  After the
    join: verify/select, cache append, LM head + head loop.  Reported: each part alone, both together, and how much of the
    precompute the overlap hides."""
    import torch
    import paper_2609_27396_b200 as dp
    w3 = W.workload(3)
    a = W.AttnShape(w3.attn.ctx_lens, 40, 8, 128, 8, 8)           # b = 16 ragged contexts, d = 7: 8 boundaries x 8 slots
    hidden, inter, V = 5120, 17408, w3.verify.vocab
    b, J, Bq, S = a.batch, a.n_boundaries, a.block, a.spine
    R = J * Bq + S
    g = torch.Generator(device="cuda").manual_seed(5)
    mk = lambda sig, *sh: (torch.randn(*sh, device="cuda", generator=g) * sig).to(torch.bfloat16)
    ones = lambda n: torch.ones(n, dtype=torch.bfloat16, device="cuda")
    # caches with slack, one per layer
    cap = [L + 4 * J for L in a.ctx_lens]
    start = [0]
    for c in cap:
        start.append(start[-1] + c)
    kc = [mk(1.0, start[-1], a.n_kv_heads, a.head_dim) for _ in range(n_layers)]
    vc = [mk(1.0, start[-1], a.n_kv_heads, a.head_dim) for _ in range(n_layers)]
    lens = torch.tensor(list(a.ctx_lens), dtype=torch.int64, device="cuda")
    lens0 = lens.clone()
    qd, kd = a.n_q_heads * a.head_dim, a.n_kv_heads * a.head_dim
    x = mk(1.0, b, R, hidden)
    y = torch.zeros(b, R, hidden, dtype=torch.float32, device="cuda")
    y16 = torch.zeros(b, R, hidden, dtype=torch.bfloat16, device="cuda")
    keep, layers = [], []
    for _ in range(n_layers):
        t = dict(w_qkv=mk(0.02, qd + 2 * kd, hidden), w_o=mk(0.02, hidden, qd), w_gate_up=mk(0.02, 2 * inter, hidden), w_down=mk(0.02, hidden, inter),
                 rms1_w=ones(hidden), rms2_w=ones(hidden), qnorm_w=ones(a.head_dim), knorm_w=ones(a.head_dim))
        keep.append(t)
        layers.append(dp.make_layer_io(x=x, **t, y_f32=y, y_bf16=y16))
    bplan = dp.BackbonePlan(ctx_offsets=start, n_boundaries=J, block=Bq, n_q_heads=a.n_q_heads, n_kv_heads=a.n_kv_heads, head_dim=a.head_dim,
                            layers=layers, k_ctx=kc, v_ctx=vc, n_spine=S, ctx_lens=list(a.ctx_lens))
    # verification side: stand-in forward, then the real select / append / head calls
    n_mats = max(1, int(standin_gb * 1e9 / (8192 * 8192 * 2)))
    wt = [mk(0.01, 8192, 8192) for _ in range(n_mats)]
    xt = mk(1.0, b * J, 8192)
    ver = W.make_verify_inputs(W.VerifyShape(b, J, V, Bq, hidden, "greedy", 0.75, 2.0), w3.seed, reps=np.zeros((1,), np.uint16))
    target, tokens = torch.from_numpy(ver.target).cuda(), torch.from_numpy(ver.draft_tokens).cuda()
    vplan = dp.VerifyPlan(batch=b, n_boundaries=J, vocab=V, block=Bq, hidden=hidden, mode=0, rep_req_rows=R)
    cplan = dp.CachePlan(batch=b, n_rows=J, w_kv=[mk(0.02, 2 * kd, hidden) for _ in range(n_layers)], k_ctx=kc, v_ctx=vc,
                         row_start=torch.tensor(start[:-1], dtype=torch.int64, device="cuda"), capacity=torch.tensor(cap, dtype=torch.int64, device="cuda"),
                         ctx_len=lens, norm_w=[ones(hidden)] * n_layers, knorm_w=[ones(a.head_dim) for _ in range(n_layers)])
    feats = mk(1.0, b, J, hidden)
    hplan = dp.HeadPlan(b, Bq, hidden, V, 256)
    w_lm, ar_w, ar_e = mk(0.02, V, hidden), mk(1.0, V, 256), mk(0.05, V, 256)

    def standin():
        h = xt
        for wm in wt:
            h = torch.mm(h, wm)
        return h

    def tail():
        vplan(target=target, draft_tokens=tokens, reps=y16)
        lens.copy_(lens0)
        cplan.run(feats, vplan.accept_len)
        hplan.run(vplan.selected, w_lm, ar_w, ar_e, vplan.bonus)

    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device="cuda")
    s_main, s_b = torch.cuda.Stream(), torch.cuda.Stream()

    def graph_us(body, k=3):
        with torch.cuda.stream(s_main):
            body(); body()
            torch.cuda.synchronize()
            gr = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gr, stream=s_main):
                for _ in range(k):
                    flush.zero_(); body()
            ts = []
            for _ in range(5):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(s_main); gr.replay(); e1.record(s_main)
                torch.cuda.synchronize()
                ts.append(e0.elapsed_time(e1) * 1e3 / k)
        return statistics.median(ts)

    def both():
        s_b.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(s_b):
            bplan()
        standin()
        torch.cuda.current_stream().wait_stream(s_b)

    base = graph_us(lambda: None)
    t_v, t_p, t_both = graph_us(standin) - base, graph_us(lambda: bplan()) - base, graph_us(both) - base
    t_tail = graph_us(tail) - base
    t_round = graph_us(lambda: (both(), tail())) - base
    return {"workload": f"one round on one GPU: b={b} ragged contexts (sum {sum(a.ctx_lens)}), d=7 ({J} boundaries x {Bq} slots + {S} spine rows = {b * R} rows), "
                        f"{n_layers} backbone blocks (hidden {hidden}, inter {inter}); verification = STAND-IN: {n_mats} library matmuls of {b * J} rows against {n_mats * 0.134:.1f} GB of bf16 weights",
            "verify_standin_us": t_v, "precompute_us": t_p, "both_streams_us": t_both, "serial_us": t_v + t_p,
            "precompute_hidden_frac": (t_v + t_p - t_both) / t_p if t_p > 0 else None,
            "select_append_head_us": t_tail, "round_us": t_round, "round_serial_us": t_v + t_p + t_tail,
            "note": "CUDA graph replay, L2 flushed before every round; T_step ~ max(T_verify, T_precompute) + T_Head of Sec. 3.3 is both_streams_us + select_append_head_us"}


def parity_spot_check(run: "StepRunner", n_rows: int = 64):
    """max |delta| of the timed attention output against the oracle on a few seeded rows of the bench workload (the
    GPU tests check 4096 rows; this ties the timed configuration to the oracle inside the bench run itself)."""
    from oracle import attention as OA
    a = run.wl.attn
    rng = np.random.default_rng(7)
    rows = [(int(rng.integers(a.batch)), int(rng.integers(a.n_boundaries)), int(rng.integers(a.block)), int(rng.integers(a.n_q_heads)))
            for _ in range(n_rows)]
    i = run.inp
    ref = OA.draft_rows(i.q, i.k_ctx, i.v_ctx, i.ctx_offsets, i.k_spine, i.v_spine, i.k_blk, i.v_blk, rows, prefix_base=a.prefix_base)
    run.attention()
    run.torch.cuda.synchronize()
    o = run.out.float().cpu().numpy()
    got = np.stack([o[n, j, s_, h] for (n, j, s_, h) in rows]).astype(np.float64)
    return {"rows": n_rows, "attention_max_abs_delta": float(np.abs(got - ref).max()), "bound": 1e-2}


class HeadRunner:
    """The critical-path remainder T_Head at the main workload's shape: LM head on the selected branches
    (b * d rows against the [vocab][hidden] weight) + the autoregressive head loop (d dependent steps)."""

    def __init__(self, wl: W.Workload, seed: int, rank: int = 256):
        import torch
        import paper_2609_27396_b200 as dp
        self.torch, self.dp = torch, dp
        self.shape = W.head_shape(wl, rank)
        inp = W.make_head_inputs(self.shape, seed)
        bf = lambda bits: torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)
        self.t = [bf(x) for x in (inp.sel_reps, inp.w_lm, inp.ar_w, inp.ar_e)]
        self.bonus = torch.from_numpy(inp.bonus).cuda()
        sh = self.shape
        self.plan = dp.HeadPlan(sh.batch, sh.block, sh.hidden, sh.vocab, sh.rank)
        self.flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device="cuda")

    def step(self, sampling: bool = False):
        if sampling and not hasattr(self, "uniforms"):
            g = self.torch.Generator(device="cuda").manual_seed(11)
            sh = self.shape
            self.uniforms = (self.torch.randint(0, 1 << 24, (sh.batch, sh.block), generator=g, device="cuda").float() * 2.0 ** -24)
        self.plan.run(*self.t, self.bonus, uniforms=self.uniforms if sampling else None)

    def lm_head_only(self):
        sh = self.shape
        return self.dp.gemm_bf16(self.t[0].view(sh.batch * sh.block, sh.hidden), self.t[1], epilogue=3, status=self.plan.status)

    def timed(self, k: int, lm_only: bool = False, sampling: bool = False):
        torch = self.torch
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(k)]
        for s in range(k):
            self.flush.zero_()
            ev[s][0].record()
            if lm_only:
                self.lm_head_only()
            else:
                self.step(sampling)
            ev[s][1].record()
        torch.cuda.synchronize()
        return [e[0].elapsed_time(e[1]) for e in ev]


def head_bytes(sh: W.HeadShape):
    """Algorithmic HBM bytes of T_Head: LM head = weight once + hidden rows + fp32 logits written; head loop = the
    logits read back once (each step reads its own rows) + W once (it is re-read every step, from L2) + E rows."""
    lm = sh.vocab * sh.hidden * 2 + sh.batch * sh.block * sh.hidden * 2 + sh.batch * sh.block * sh.vocab * 4
    ar = sh.batch * sh.block * sh.vocab * 4 + sh.vocab * sh.rank * 2 + sh.batch * sh.block * sh.rank * 2
    return lm, ar


def layer_gemm_flops(a: W.AttnShape, l: W.LayerShape) -> float:
    M = a.batch * a.n_boundaries * a.block
    qd, kd = a.n_q_heads * a.head_dim, a.n_kv_heads * a.head_dim
    return 2.0 * M * (l.hidden * (qd + 2 * kd) + qd * l.hidden + 3 * l.hidden * l.intermediate)


# ----------------------------------------------------------------------------- the oracle arm (host cores)
def oracle_sample(wl: W.Workload, seed: int, n_pairs: int, n_verify_req: int, inp=None, ver=None):
    """Times the oracle, as it stands, on a bounded sample of the step: `n_pairs` (request, boundary)
    attentions (all slots, all heads) and greedy verify/select of `n_verify_req` requests.  Returns
    (seconds, estimated seconds for the full step, description)."""
    from oracle import attention as OA
    from oracle import verify as OV
    a, v = wl.attn, wl.verify
    inp = inp or W.make_attn_inputs(a, seed)
    ver = ver or W.make_verify_inputs(v, seed)
    rng = np.random.default_rng(seed)
    budget_s = 15.0 if n_pairs <= 0 else None          # n_pairs <= 0: as many pairs as fit in ~15 s (at most all)
    if n_pairs <= 0:
        n_pairs = a.batch * a.n_boundaries
    pairs = [(int(rng.integers(a.batch)), int(rng.integers(a.n_boundaries))) for _ in range(n_pairs)]
    t0 = time.perf_counter()
    flops = 0.0
    done = 0
    for (n, j) in pairs:
        if budget_s is not None and done >= 4 and time.perf_counter() - t0 > budget_s:
            break
        done += 1
        lo = int(inp.ctx_offsets[n]); hi = int(inp.ctx_offsets[n + 1])
        sub_off = np.array([0, hi - lo], dtype=np.int64)
        OA.draft_all_boundaries(inp.q[n:n + 1], inp.k_ctx[lo:hi], inp.v_ctx[lo:hi], sub_off, inp.k_spine[n:n + 1],
                                inp.v_spine[n:n + 1], inp.k_blk[n:n + 1], inp.v_blk[n:n + 1], prefix_base=a.prefix_base,
                                boundary_lo=j, boundary_hi=j + 1)
        flops += 4.0 * a.head_dim * a.block * a.n_q_heads * ((hi - lo) + min(j + a.prefix_base, a.spine) + a.block)
    t_att = time.perf_counter() - t0
    nv = min(n_verify_req, v.batch)
    t0 = time.perf_counter()
    OV.verify_greedy(ver.target[:nv], ver.draft_tokens[:nv], ver.reps[:nv] if ver.reps.ndim == 4 else None)
    t_ver = time.perf_counter() - t0
    est = t_att * attention_flops(a) / max(flops, 1.0) + t_ver * v.batch / nv
    desc = (f"{done} seeded (request, boundary) attentions of {a.batch * a.n_boundaries} + greedy verify of "
            f"{nv}/{v.batch} requests; full-step time extrapolated by flops / requests")
    return t_att + t_ver, est, desc


def oracle_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return int(max(n))
    except Exception:
        pass
    return len(os.sched_getaffinity(0))


# ----------------------------------------------------------------------------- single targets for a profiler
ONLY_TARGETS = {"colocation", "attention_cfg2", "attention_cfg3", "attention_cfg5", "verify_cfg2", "verify_cfg3", "verify_cfg4", "layer_cfg5", "gemm_qkv", "gemm_o",
                "gemm_gate_up", "gemm_down", "head", "head_sampling", "cache_append", "backbone_cfg5"}


def run_only(target: str, reps: int):
    """Runs the kernels of one leg `reps` times on cuda:0 (inputs as in the timed legs) and returns."""
    import torch
    torch.cuda.set_device(0)
    peaks = measured_peaks()
    if target.startswith("attention_cfg") and target != "attention_cfg5":
        w = W.workload(int(target[-1]))
        r = StepRunner(w, w.seed)
        fn = r.attention
    elif target.startswith("verify_cfg") and target != "verify_cfg4":
        w = W.workload(int(target[-1]))
        r = StepRunner(w, w.seed)
        fn = r.verify
    elif target == "verify_cfg4":
        sampling_select_leg(peaks, reps)
        return
    elif target in ("attention_cfg5", "layer_cfg5") or target.startswith("gemm_"):
        w5 = W.workload(5)
        r = LayerRunner(w5, w5.seed)
        if target == "layer_cfg5":
            fn = lambda: r.plan(**r.kv)
        elif target == "attention_cfg5":
            r.attention_only_us(reps)
            return
        else:
            r.gemm_legs(peaks, 2, only=target[5:])
            return
    elif target == "head":
        w = W.workload(3)
        r = HeadRunner(w, w.seed)
        fn = r.step
    elif target == "head_sampling":
        w = W.workload(3)
        r = HeadRunner(w, w.seed)
        fn = lambda: r.step(sampling=True)
    elif target == "cache_append":
        cache_append_leg(W.workload(3), peaks, reps)
        return
    elif target == "colocation":
        print(json.dumps(colocation_leg(peaks)))
        return
    else:
        backbone_leg(W.workload(5), peaks, reps)
        return
    for _ in range(reps):
        fn()
    torch.cuda.synchronize()


# ----------------------------------------------------------------------------- main
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg3", choices=["cfg2", "cfg3"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-layer", action="store_true", help="skip the full-layer (cfg5) leg")
    ap.add_argument("--no-head", action="store_true", help="skip the LM head + autoregressive head loop (T_Head) leg")
    ap.add_argument("--only", default=None, choices=sorted(ONLY_TARGETS), help="run ONE kernel family a few times and exit (no timing, "
                    "no JSON line): the small command a profiler is pointed at")
    ap.add_argument("--only-reps", type=int, default=3)
    args = ap.parse_args()
    if args.only:
        run_only(args.only, args.only_reps)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours":
        # started without a launcher: become one -- N ranks of this script, one per GPU; rank 0 prints the line
        from paper_2609_27396_b200.dist_util import launch_ranks
        sys.exit(launch_ranks([os.path.abspath(__file__)] + sys.argv[1:], args.gpus))
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    wl = W.workload({"cfg2": 2, "cfg3": 3}[args.workload])
    cfg = {"workload": f"{wl.name}: b={wl.attn.batch}, ctx={'ragged U[512,4096] sum=' + str(sum(wl.attn.ctx_lens)) if wl.index == 3 else wl.attn.ctx_lens[0]}, "
                       f"Hq/Hkv={wl.attn.n_q_heads}/{wl.attn.n_kv_heads}, D={wl.attn.head_dim}, boundaries={wl.attn.n_boundaries}, "
                       f"block={wl.attn.block}, vocab={wl.verify.vocab}, hidden={wl.verify.hidden}; step = all-boundary attention + greedy verify/select",
           "l2": f"{L2_FLUSH_BYTES >> 20} MiB flush write between timed steps", "parallelism": f"batch-sharded x{world} (no collective)"}

    if args.impl == "reference":
        if rank != 0:
            return
        steps = max(1, min(args.steps, 3))
        times, est = [], []
        inp, ver = W.make_attn_inputs(wl.attn, wl.seed), W.make_verify_inputs(wl.verify, wl.seed)
        for s in range(args.warmup and 1):
            oracle_sample(wl, wl.seed, 1, 1, inp, ver)
        for s in range(steps):
            t, e, desc = oracle_sample(wl, wl.seed + s, 6, 2, inp, ver)
            times.append(t); est.append(e)
        us = statistics.mean(est) * 1e6
        cores = oracle_threads()
        print(json.dumps({"impl": "reference", "metric": METRIC, "value": us, "unit": "us", "n_gpus": args.gpus, "steps": steps,
                          "warmup": 1 if args.warmup else 0, "ms_per_step": us / 1e3, "higher_is_better": False, "scaling": "weak",
                          "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": cfg,
                          "cpu_baseline": {"value": us, "unit": "us", "cores": cores, "kind": "oracle", "sample": desc},
                          "e2e": {"value": us, "unit": "us", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))
        return

    import torch
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    import paper_2609_27396_b200 as dp

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    from paper_2609_27396_b200.dist_util import max_over_ranks as _mor, rank_seed

    def max_over_ranks(x: float) -> float:
        return _mor(x, device="cuda")

    run = StepRunner(wl, rank_seed(wl.seed, rank))
    for _ in range(max(args.warmup, 3)):
        run.step()
    barrier()
    launches0 = dp.lib.dpara_kernel_launches()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    per = run.timed_steps(args.steps, parts=False)
    barrier()
    launches = dp.lib.dpara_kernel_launches() - launches0
    parts = run.timed_steps(args.steps)
    # keep the GPU busy a little longer so that the 100 ms sampler sees clocks under this load
    t_end = time.time() + 0.6
    while rank == 0 and time.time() < t_end:
        run.step()
    torch.cuda.synchronize()
    clocks = sampler.stop() if rank == 0 else None
    total_ms = max_over_ranks(sum(p[0] for p in per))
    att_ms = statistics.mean(p[1] for p in parts)
    ver_ms = statistics.mean(p[2] for p in parts)
    step_us = total_ms / args.steps * 1e3

    # end to end through the public call with host buffers
    run.setup_e2e()
    run.e2e_steps(2)
    barrier()
    e2e = run.e2e_steps(max(3, min(args.steps, 10)))
    barrier()
    e2e_us = max_over_ranks(statistics.mean(e2e)) * 1e3

    peaks = measured_peaks()
    fl = attention_flops(wl.attn)
    by = attention_bytes(wl.attn)
    ach_tf = fl / (att_ms * 1e-3) / 1e12
    ach_gb = by / (att_ms * 1e-3) / 1e9
    traffic = ncu_dram_traffic(args.workload)
    roofline = {"kernel": "all-boundary attention", "bound": "tensor", "achieved": ach_tf, "peak": peaks["bf16_tflops"],
                "unit": "TFLOP/s", "frac": ach_tf / peaks["bf16_tflops"], "traffic": traffic, "peak_source": peaks["source"] + " (burst)",
                "hbm": {"achieved": ach_gb, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": ach_gb / peaks["hbm_gbs"],
                        "note": "same launch against the HBM roofline (algorithmic bytes)"},
                "algorithmic": {"flops": fl, "bytes": by, "us": att_ms * 1e3},
                "verify_select": {"bound": "hbm", "achieved": verify_bytes(wl.verify) / (ver_ms * 1e-3) / 1e9, "peak": peaks["hbm_gbs"],
                                  "unit": "GB/s", "frac": verify_bytes(wl.verify) / (ver_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                  "us": ver_ms * 1e3, "bytes": verify_bytes(wl.verify)}}

    te16, same16 = run.timed_early_steps(args.steps)
    early16 = {"step_us": statistics.median(te16) * 1e3, "same_selection_as_plain_call": same16}
    out = {"metric": METRIC, "value": step_us, "unit": "us", "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
           "ms_per_step": step_us / 1e3, "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
           "data": "synthetic", "config": cfg, "clocks": clocks, "gpu_launches": int(launches),
           "e2e": {"value": e2e_us, "unit": "us", "h2d_bytes_per_step": run.h2d_bytes, "d2h_bytes_per_step": run.d2h_bytes},
           "roofline": roofline, "steps_per_s_all_gpus": world * 1e6 / step_us,
           "early_start_verify": early16}

    if rank == 0 and world == 1:
        # the b = 1 step (cfg2) and the single-boundary (conventional) draft step beside it
        w2 = W.workload(2)
        r2 = StepRunner(w2, w2.seed)
        for _ in range(5):
            r2.step(); r2.attention(r2.plan1)
        p2 = r2.timed_steps(max(args.steps, 20))
        s2 = r2.timed_steps(max(args.steps, 20), single_boundary=True)
        a2 = statistics.median(p[1] for p in p2) * 1e3
        out["b1"] = {"workload": w2.name, "step_us": statistics.median(p[0] for p in p2) * 1e3, "attention_us": a2,
                     "verify_select_us": statistics.median(p[2] for p in p2) * 1e3,
                     "single_boundary_attention_us": statistics.median(p[1] for p in s2) * 1e3,
                     "all_over_single": a2 / (statistics.median(p[1] for p in s2) * 1e3), "allowance": w2.attn.n_boundaries,
                     "attention_gbs": attention_bytes(w2.attn) / (a2 * 1e-6) / 1e9, "attention_tflops": attention_flops(w2.attn) / (a2 * 1e-6) / 1e12}
        te, same = r2.timed_early_steps(max(args.steps, 20))
        out["b1"]["early_start"] = {"step_us": statistics.median(te) * 1e3, "same_selection_as_plain_call": same,
                                    "note": "verify/select with DPARA_VERIFY_EARLY_START: it reads the (already resident) target logits while the "
                                            "attention kernel before it is still running and waits for it only before the branch gather"}
        out["b1"].update(graph_timed_b1(r2))
        del r2
        if not args.no_layer:
            w5 = W.workload(5)
            r5 = LayerRunner(w5, w5.seed)
            for _ in range(3):
                r5.step()
            p5 = r5.timed_steps(max(5, min(args.steps, 10)))
            d5 = statistics.median(p[1] for p in p5) * 1e3
            fl5 = attention_flops(w5.attn) + layer_gemm_flops(w5.attn, w5.layer)
            out["layer_cfg5"] = {"workload": w5.name, "step_us": statistics.median(p[0] for p in p5) * 1e3, "draft_layer_us": d5,
                                 "verify_select_us": statistics.median(p[2] for p in p5) * 1e3,
                                 "flops": fl5, "tflops": fl5 / (d5 * 1e-6) / 1e12,
                                 "tensor_frac_of_measured_burst": fl5 / (d5 * 1e-6) / 1e12 / peaks["bf16_tflops"],
                                 "tensor_frac_of_measured_sustained": fl5 / (d5 * 1e-6) / 1e12 / (peaks["bf16_tflops_sustained"] or peaks["bf16_tflops"]),
                                 "attention_us": r5.attention_only_us(max(5, min(args.steps, 10))),
                                 "attention_flops": attention_flops(w5.attn),
                                 "gemms": r5.gemm_legs(peaks, max(5, min(args.steps, 10)))}
            out["layer_cfg5"]["attention_tflops"] = attention_flops(w5.attn) / (out["layer_cfg5"]["attention_us"] * 1e-6) / 1e12
            del r5
            out["backbone_cfg5"] = backbone_leg(w5, peaks, max(3, min(args.steps, 5)))
        if not args.no_head:
            rh = HeadRunner(wl, wl.seed)
            for _ in range(3):
                rh.step()
            th = statistics.median(rh.timed(max(5, min(args.steps, 10)))) * 1e3
            tl = statistics.median(rh.timed(max(5, min(args.steps, 10)), lm_only=True)) * 1e3
            rh.step(sampling=True)
            ts = statistics.median(rh.timed(max(5, min(args.steps, 10)), sampling=True)) * 1e3
            lmb, arb = head_bytes(rh.shape)
            sh = rh.shape
            out["head"] = {"workload": "T_Head at %s: b=%d, d=%d, hidden=%d, vocab=%d, head rank=%d (greedy)" % (wl.name, sh.batch, sh.block, sh.hidden, sh.vocab, sh.rank),
                           "head_us": th, "lm_head_us": tl, "ar_loop_us": th - tl, "ar_step_us": (th - tl) / sh.block,
                           "sampling": {"head_us": ts, "ar_loop_us": ts - tl, "ar_step_us": (ts - tl) / sh.block,
                                        "note": "y_i ~ softmax(z_i) from supplied uniforms (temperature 1): per step one GEMM that writes z_i and one inverse-CDF kernel"},
                           "lm_head": {"bound": "hbm", "achieved": lmb / (tl * 1e-6) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                       "frac": lmb / (tl * 1e-6) / 1e9 / peaks["hbm_gbs"], "bytes": lmb,
                                       "tflops": 2.0 * sh.batch * sh.block * sh.hidden * sh.vocab / (tl * 1e-6) / 1e12},
                           "ar_loop": {"w_bytes_per_step": sh.vocab * sh.rank * 2, "hbm_bytes": arb,
                                       "w_read_gbs": sh.vocab * sh.rank * 2 * sh.block / ((th - tl) * 1e-6) / 1e9}}
            del rh
        out["cfg1"] = small_step_leg(1, max(args.steps, 20))
        out["cfg4_sampling_select"] = sampling_select_leg(peaks, max(args.steps, 20))
        out["cache_append"] = cache_append_leg(wl, peaks, max(args.steps, 20))
        out["parity_spot_check"] = parity_spot_check(run)
        if not args.no_layer and not args.no_head:
            out["colocation"] = colocation_leg(peaks)
        if not args.no_cpu_baseline:
            t, est, desc = oracle_sample(wl, wl.seed, 0, wl.verify.batch, run.inp, run.ver)
            out["cpu_baseline"] = {"value": est * 1e6, "unit": "us", "cores": oracle_threads(), "kind": "oracle", "sample": desc,
                                   "sample_seconds": t}
    if rank == 0:
        print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
