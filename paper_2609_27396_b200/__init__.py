"""Python binding of libdpara.so (B200 / sm_100a all-boundary draft step).

Argument marshalling only: every step of the path runs in the CUDA kernels behind the C ABI declared
in include/dpara.h.  PyTorch supplies device memory and streams.  There is no CPU fallback: if the
shared library is missing, importing this package raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdpara.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2609_27396_b200.build` "
        "(nvcc, sm_100a). This package has no CPU fallback.")

lib = C.CDLL(LIB_PATH)

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT, ERR_STATIC_LIMIT = 0, -1, -2, -3, -4, -5, -6
VERIFY_STATIC_SCRATCH_BYTES = 256 * 1024
STATUS_BAD_TOKEN, STATUS_TIMEOUT, STATUS_CACHE_FULL = 1, 2, 4
BF16, F32 = 0, 1


class Shape(C.Structure):
    _fields_ = [("batch", C.c_int32), ("n_boundaries", C.c_int32), ("block", C.c_int32), ("n_q_heads", C.c_int32),
                ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("prefix_base", C.c_int32), ("n_spine", C.c_int32),
                ("boundary_lo", C.c_int32), ("boundary_hi", C.c_int32), ("softmax_scale", C.c_float),
                ("spine_queries", C.c_int32)]


class AttnIO(C.Structure):
    _fields_ = [("q", C.c_void_p), ("k_ctx", C.c_void_p), ("v_ctx", C.c_void_p), ("ctx_offsets", C.c_void_p),
                ("host_ctx_offsets", C.c_void_p), ("k_spine", C.c_void_p), ("v_spine", C.c_void_p),
                ("k_blk", C.c_void_p), ("v_blk", C.c_void_p), ("out", C.c_void_p), ("out_dtype", C.c_int32),
                ("out_lse", C.c_void_p), ("ctx_lens", C.c_void_p), ("host_ctx_lens", C.c_void_p)]


class LayerIO(C.Structure):
    _fields_ = [("x", C.c_void_p), ("w_qkv", C.c_void_p), ("w_o", C.c_void_p), ("w_gate_up", C.c_void_p),
                ("w_down", C.c_void_p), ("rms1_w", C.c_void_p), ("rms2_w", C.c_void_p), ("qnorm_w", C.c_void_p),
                ("knorm_w", C.c_void_p), ("rms_eps", C.c_float), ("rope_theta", C.c_float), ("use_rope", C.c_int32),
                ("hidden", C.c_int32), ("intermediate", C.c_int32), ("y_f32", C.c_void_p), ("y_bf16", C.c_void_p)]


class VerifyIO(C.Structure):
    _fields_ = [("batch", C.c_int32), ("n_boundaries", C.c_int32), ("vocab", C.c_int32), ("block", C.c_int32),
                ("hidden", C.c_int32), ("mode", C.c_int32), ("target", C.c_void_p), ("draft_probs", C.c_void_p),
                ("draft_tokens", C.c_void_p), ("uniforms", C.c_void_p), ("reps", C.c_void_p), ("accept_len", C.c_void_p),
                ("bonus", C.c_void_p), ("gather_idx", C.c_void_p), ("out_tokens", C.c_void_p), ("selected", C.c_void_p),
                ("rep_req_rows", C.c_int32), ("flags", C.c_int32)]


lib.dpara_draft_workspace_bytes.restype = C.c_size_t
lib.dpara_draft_workspace_bytes.argtypes = [C.POINTER(Shape), C.c_void_p, C.POINTER(LayerIO), C.c_int]
lib.dpara_draft_all_boundaries.restype = C.c_int
lib.dpara_draft_all_boundaries.argtypes = [C.POINTER(Shape), C.POINTER(AttnIO), C.POINTER(LayerIO), C.c_void_p,
                                           C.c_size_t, C.c_void_p, C.c_void_p]
lib.dpara_verify_workspace_bytes.restype = C.c_size_t
lib.dpara_verify_workspace_bytes.argtypes = [C.POINTER(VerifyIO)]
lib.dpara_verify_select.restype = C.c_int
lib.dpara_verify_select.argtypes = [C.POINTER(VerifyIO), C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
lib.dpara_verify_select_static.restype = C.c_int
lib.dpara_verify_select_static.argtypes = [C.POINTER(VerifyIO), C.c_void_p, C.c_void_p]
lib.dpara_status_string.restype = C.c_char_p
lib.dpara_status_string.argtypes = [C.c_int]
lib.dpara_version.restype = C.c_int32
lib.dpara_kernel_launches.restype = C.c_int64

lib.dpara_layer_workspace_layout.restype = C.c_int
lib.dpara_layer_workspace_layout.argtypes = [C.POINTER(Shape), C.c_void_p, C.POINTER(LayerIO), C.POINTER(C.c_size_t)]

EXPORTED = ["dpara_layer_workspace_layout", "dpara_draft_workspace_bytes", "dpara_draft_all_boundaries", "dpara_verify_workspace_bytes",
            "dpara_verify_select", "dpara_verify_select_static", "dpara_status_string", "dpara_version", "dpara_kernel_launches"]


class GemmIO(C.Structure):
    _fields_ = [("a", C.c_void_p), ("w", C.c_void_p), ("M", C.c_int32), ("N", C.c_int32), ("K", C.c_int32),
                ("epilogue", C.c_int32), ("resid", C.c_void_p), ("resid_dtype", C.c_int32), ("out", C.c_void_p),
                ("out_bf16", C.c_void_p)]


lib.dpara_gemm_bf16.restype = C.c_int
lib.dpara_gemm_bf16.argtypes = [C.POINTER(GemmIO), C.c_void_p, C.c_void_p]
EXPORTED.append("dpara_gemm_bf16")


def gemm_bf16(a, w, *, epilogue: int = 0, resid=None, want_bf16_copy: bool = False, status=None, stream=None):
    """dpara_gemm_bf16: out = epilogue(a @ w.T); a [M][K], w [N][K] (epilogue 2: [2N][K]) bf16 CUDA tensors."""
    M, K = a.shape
    N = w.shape[0] // 2 if epilogue == 2 else w.shape[0]
    out = torch.empty((M, N), dtype=torch.float32 if epilogue in (1, 3) else torch.bfloat16, device=a.device)
    out16 = torch.empty((M, N), dtype=torch.bfloat16, device=a.device) if (want_bf16_copy and epilogue == 1) else None
    st = status if status is not None else torch.zeros(1, dtype=torch.int32, device=a.device)
    io = GemmIO(_ptr(a), _ptr(w), M, N, K, epilogue, _ptr(resid),
                BF16 if (resid is not None and resid.dtype == torch.bfloat16) else F32, _ptr(out), _ptr(out16))
    rc = lib.dpara_gemm_bf16(C.byref(io), st.data_ptr(), _stream_ptr(stream))
    if rc != OK:
        raise DparaError(rc)
    return (out, out16, st) if out16 is not None else (out, st)


lib.dpara_selftest_bounded_wait.restype = C.c_int
lib.dpara_selftest_bounded_wait.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p]
EXPORTED.append("dpara_selftest_bounded_wait")


def selftest_bounded_wait(limit_us: int = 1000, stream=None):
    """dpara_selftest_bounded_wait: returns (status_word, waited_ns) after the stream has drained."""
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    waited = torch.zeros(1, dtype=torch.int64, device="cuda")
    rc = lib.dpara_selftest_bounded_wait(st.data_ptr(), limit_us, waited.data_ptr(), _stream_ptr(stream))
    if rc != OK:
        raise DparaError(rc)
    torch.cuda.synchronize()
    return int(st.item()), int(waited.item())


class DparaError(RuntimeError):
    def __init__(self, code: int):
        self.code = code
        super().__init__(f"dpara: {lib.dpara_status_string(code).decode()} ({code})")


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    if not t.is_contiguous():
        raise ValueError("dpara: tensors must be contiguous")
    return t.data_ptr()


def _stream_ptr(stream) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream


def _host_offsets(ctx_offsets: Sequence[int]):
    arr = (C.c_int64 * len(ctx_offsets))(*[int(x) for x in ctx_offsets])
    return arr


class DraftPlan:
    """Fixed-address buffers for repeated draft calls on one shape (shape struct, host and device copies
    of the context offsets, workspace, status word).  Building the plan allocates; calling it does not."""

    def __init__(self, *, ctx_offsets: Sequence[int], n_boundaries: int, block: int, n_q_heads: int, n_kv_heads: int,
                 head_dim: int, prefix_base: int = 1, n_spine: Optional[int] = None, boundary_lo: int = 0,
                 boundary_hi: Optional[int] = None, softmax_scale: float = 0.0, layer: Optional[LayerIO] = None,
                 ctx_lens: Optional[Sequence[int]] = None, spine_queries: bool = False, device="cuda"):
        """ctx_lens: for caches kept with slack (dpara_cache_append) -- request n's context is the first ctx_lens[n] of
        its rows ctx_offsets[n]..ctx_offsets[n+1]; update it between calls with set_ctx_lens()."""
        b = len(ctx_offsets) - 1
        self.shape = Shape(b, n_boundaries, block, n_q_heads, n_kv_heads, head_dim, prefix_base,
                           n_boundaries if n_spine is None else n_spine, boundary_lo,
                           n_boundaries if boundary_hi is None else boundary_hi, softmax_scale, 1 if spine_queries else 0)
        self.host_off = _host_offsets(ctx_offsets)
        self.dev_off = torch.tensor([int(x) for x in ctx_offsets], dtype=torch.int64, device=device)
        self.layer = layer
        need = lib.dpara_draft_workspace_bytes(C.byref(self.shape), C.cast(self.host_off, C.c_void_p),
                                               C.byref(layer) if layer is not None else None, 1 if layer is not None else 0)
        self.workspace_bytes = int(need)
        self.workspace = torch.empty(max(need, 16), dtype=torch.uint8, device=device)
        self.status = torch.zeros(1, dtype=torch.int32, device=device)
        self.host_lens = self.dev_lens = None
        if ctx_lens is not None:
            self.host_lens = (C.c_int64 * b)(*[int(x) for x in ctx_lens])
            self.dev_lens = torch.tensor([int(x) for x in ctx_lens], dtype=torch.int64, device=device)

    def set_ctx_lens(self, ctx_lens: Sequence[int], dev_lens: Optional[torch.Tensor] = None) -> None:
        """New context lengths (host values; `dev_lens`: a device tensor that already holds them, e.g. the one
        dpara_cache_append updated, else they are copied to the device here)."""
        for n, x in enumerate(ctx_lens):
            self.host_lens[n] = int(x)
        if dev_lens is not None:
            self.dev_lens = dev_lens
        else:
            self.dev_lens.copy_(torch.tensor([int(x) for x in ctx_lens], dtype=torch.int64))

    def __call__(self, *, q=None, k_ctx=None, v_ctx=None, k_spine=None, v_spine=None, k_blk=None, v_blk=None,
                 out=None, out_lse=None, stream=None) -> None:
        io = AttnIO(_ptr(q), _ptr(k_ctx), _ptr(v_ctx), self.dev_off.data_ptr(), C.cast(self.host_off, C.c_void_p).value,
                    _ptr(k_spine), _ptr(v_spine), _ptr(k_blk), _ptr(v_blk), _ptr(out),
                    F32 if (out is not None and out.dtype == torch.float32) else BF16, _ptr(out_lse),
                    _ptr(self.dev_lens), C.cast(self.host_lens, C.c_void_p).value if self.host_lens is not None else None)
        rc = lib.dpara_draft_all_boundaries(C.byref(self.shape), C.byref(io),
                                            C.byref(self.layer) if self.layer is not None else None,
                                            self.workspace.data_ptr(), self.workspace.numel(), self.status.data_ptr(),
                                            _stream_ptr(stream))
        if rc != OK:
            raise DparaError(rc)


LAYER_STAGES = ("xn", "qkv", "q", "k", "v", "a", "h1", "hn", "act")


def layer_intermediates(plan: "DraftPlan") -> dict:
    """dpara_layer_workspace_layout: views of the block's intermediates that the last full-layer call of `plan`
    left in its workspace, keyed by LAYER_STAGES, each [M][width] (h1 fp32, the rest bf16)."""
    off = (C.c_size_t * 9)()
    rc = lib.dpara_layer_workspace_layout(C.byref(plan.shape), C.cast(plan.host_off, C.c_void_p), C.byref(plan.layer), off)
    if rc != OK:
        raise DparaError(rc)
    sh, L = plan.shape, plan.layer
    M = sh.batch * (sh.n_boundaries * sh.block + (sh.n_spine if sh.spine_queries else 0))
    QD, KD = sh.n_q_heads * sh.head_dim, sh.n_kv_heads * sh.head_dim
    width = dict(xn=L.hidden, qkv=QD + 2 * KD, q=QD, k=KD, v=KD, a=QD, h1=L.hidden, hn=L.hidden, act=L.intermediate)
    res = {}
    for name, o in zip(LAYER_STAGES, off):
        dt = torch.float32 if name == "h1" else torch.bfloat16
        nbytes = M * width[name] * (4 if name == "h1" else 2)
        res[name] = plan.workspace[o:o + nbytes].view(dt).view(M, width[name])
    return res


def make_layer_io(*, x, w_qkv, w_o, w_gate_up, w_down, rms1_w=None, rms2_w=None, qnorm_w=None, knorm_w=None,
                  rms_eps=1e-6, rope_theta=1e6, use_rope=True, y_f32=None, y_bf16=None) -> LayerIO:
    hidden = x.shape[-1]
    inter = w_down.shape[-1]
    return LayerIO(_ptr(x), _ptr(w_qkv), _ptr(w_o), _ptr(w_gate_up), _ptr(w_down), _ptr(rms1_w), _ptr(rms2_w),
                   _ptr(qnorm_w), _ptr(knorm_w), rms_eps, rope_theta, 1 if use_rope else 0, hidden, inter,
                   _ptr(y_f32), _ptr(y_bf16))


def draft_all_boundaries(q, k_ctx, v_ctx, ctx_offsets: Sequence[int], k_spine, v_spine, k_blk=None, v_blk=None, *,
                         prefix_base: int = 1, boundary_lo: int = 0, boundary_hi: Optional[int] = None,
                         softmax_scale: float = 0.0, out_dtype=torch.bfloat16, want_lse: bool = False, stream=None):
    """All-boundary attention (dpara_draft_all_boundaries, attention-only mode).
    q [b][J][Bq][Hq][D] bf16 CUDA tensor; returns out (same shape, out_dtype) and optionally lse."""
    b, J, Bq, Hq, D = q.shape
    Hkv = k_spine.shape[2]
    plan = DraftPlan(ctx_offsets=ctx_offsets, n_boundaries=J, block=Bq, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D,
                     prefix_base=prefix_base, n_spine=k_spine.shape[1], boundary_lo=boundary_lo, boundary_hi=boundary_hi,
                     softmax_scale=softmax_scale, device=q.device)
    out = torch.zeros(q.shape, dtype=out_dtype, device=q.device)
    lse = torch.full((b, J, Bq, Hq), float("-inf"), dtype=torch.float32, device=q.device) if want_lse else None
    plan(q=q, k_ctx=k_ctx, v_ctx=v_ctx, k_spine=k_spine, v_spine=v_spine, k_blk=k_blk, v_blk=v_blk, out=out, out_lse=lse,
         stream=stream)
    return (out, lse, plan.status) if want_lse else (out, plan.status)


def draft_with_spine_queries(q_rows, n_boundaries: int, block: int, k_ctx, v_ctx, ctx_offsets: Sequence[int], k_spine, v_spine,
                             k_blk=None, v_blk=None, *, prefix_base: int = 1, softmax_scale: float = 0.0,
                             out_dtype=torch.bfloat16, want_lse: bool = False, stream=None):
    """dpara_draft_all_boundaries with spine_queries = 1 (attention only): q_rows [b][J*Bq + S][Hq][D] holds each request's
    mask-slot rows in (boundary, slot) order followed by its S spine rows; out (and lse) come back in the same row order."""
    b, R, Hq, D = q_rows.shape
    S, Hkv = k_spine.shape[1], k_spine.shape[2]
    assert R == n_boundaries * block + S
    plan = DraftPlan(ctx_offsets=ctx_offsets, n_boundaries=n_boundaries, block=block, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D,
                     prefix_base=prefix_base, n_spine=S, softmax_scale=softmax_scale, spine_queries=True, device=q_rows.device)
    out = torch.zeros(q_rows.shape, dtype=out_dtype, device=q_rows.device)
    lse = torch.full((b, R, Hq), float("-inf"), dtype=torch.float32, device=q_rows.device) if want_lse else None
    plan(q=q_rows, k_ctx=k_ctx, v_ctx=v_ctx, k_spine=k_spine, v_spine=v_spine, k_blk=k_blk, v_blk=v_blk, out=out, out_lse=lse,
         stream=stream)
    return (out, lse, plan.status) if want_lse else (out, plan.status)


VERIFY_EARLY_START = 1


class VerifyPlan:
    """Fixed-address outputs and workspace for repeated verify/select calls on one shape."""

    def __init__(self, *, batch: int, n_boundaries: int, vocab: int, block: int, hidden: int, mode: int, rep_req_rows: int = 0,
                 early_start: bool = False, device="cuda"):
        """early_start: DPARA_VERIFY_EARLY_START -- the call may begin while the work enqueued right before it is still
        running and waits for it only before it reads `reps` (the caller promises that work writes none of the other
        inputs and touches neither the workspace nor the outputs)."""
        self.io = VerifyIO(batch, n_boundaries, vocab, block, hidden, mode)
        self.io.rep_req_rows = rep_req_rows
        self.io.flags = VERIFY_EARLY_START if early_start else 0
        self.accept_len = torch.zeros(batch, dtype=torch.int32, device=device)
        self.bonus = torch.zeros(batch, dtype=torch.int32, device=device)
        self.gather_idx = torch.zeros(batch, dtype=torch.int32, device=device)
        self.out_tokens = torch.zeros(batch, n_boundaries, dtype=torch.int32, device=device)
        self.selected = torch.zeros(batch, block, hidden, dtype=torch.bfloat16, device=device)
        self.status = torch.zeros(1, dtype=torch.int32, device=device)
        self.io.accept_len, self.io.bonus = self.accept_len.data_ptr(), self.bonus.data_ptr()
        self.io.gather_idx, self.io.out_tokens = self.gather_idx.data_ptr(), self.out_tokens.data_ptr()
        self.io.selected = self.selected.data_ptr()
        need = lib.dpara_verify_workspace_bytes(C.byref(self.io))
        self.workspace_bytes = int(need)
        # zero-filled once; every call leaves it zero-filled again
        self.workspace = torch.zeros(max(need, 16), dtype=torch.uint8, device=device)

    def __call__(self, *, target, draft_tokens, reps=None, draft_probs=None, uniforms=None, stream=None) -> None:
        io = self.io
        io.target, io.draft_tokens = _ptr(target), _ptr(draft_tokens)
        io.draft_probs, io.uniforms, io.reps = _ptr(draft_probs), _ptr(uniforms), _ptr(reps)
        rc = lib.dpara_verify_select(C.byref(io), self.workspace.data_ptr(), self.workspace.numel(),
                                     self.status.data_ptr(), _stream_ptr(stream))
        if rc != OK:
            raise DparaError(rc)


def verify_select_static(plan: "VerifyPlan", *, target, draft_tokens, reps=None, draft_probs=None, uniforms=None,
                         stream=None) -> None:
    """dpara_verify_select_static: the same verify/select, for callers that cannot allocate device memory
    (their own pool owns all of it, or an allocation would stall the decode loop).  Uses the library's
    fixed scratch array instead of a caller workspace; `plan` only supplies the output tensors.  The first
    call on a device does a one-time address lookup: make it at start-up, before any stream capture.
    Calls that overlap on one GPU race on the shared scratch."""
    io = plan.io
    io.target, io.draft_tokens = _ptr(target), _ptr(draft_tokens)
    io.draft_probs, io.uniforms, io.reps = _ptr(draft_probs), _ptr(uniforms), _ptr(reps)
    rc = lib.dpara_verify_select_static(C.byref(io), plan.status.data_ptr(), _stream_ptr(stream))
    if rc != OK:
        raise DparaError(rc)


def verify_select(target, draft_tokens, reps=None, *, mode: int = 0, draft_probs=None, uniforms=None, stream=None):
    """Accepted length, bonus token, selected branch (dpara_verify_select).  Returns a dict of CUDA tensors."""
    b, J, V = target.shape
    block, hidden = (reps.shape[2], reps.shape[3]) if reps is not None else (1, 8)
    plan = VerifyPlan(batch=b, n_boundaries=J, vocab=V, block=block, hidden=hidden, mode=mode, device=target.device)
    plan(target=target, draft_tokens=draft_tokens, reps=reps, draft_probs=draft_probs, uniforms=uniforms, stream=stream)
    return dict(accept_len=plan.accept_len, bonus=plan.bonus, gather_idx=plan.gather_idx, out_tokens=plan.out_tokens,
                selected=plan.selected if reps is not None else None, status=plan.status)


# ----------------------------------------------------------------------------- critical-path remainder: LM head + AR head loop
class HeadIO(C.Structure):
    _fields_ = [("sel_reps", C.c_void_p), ("w_lm", C.c_void_p), ("ar_w", C.c_void_p), ("ar_e", C.c_void_p),
                ("bonus", C.c_void_p), ("next_tokens", C.c_void_p), ("b", C.c_int32), ("block", C.c_int32),
                ("hidden", C.c_int32), ("vocab", C.c_int32), ("rank", C.c_int32), ("uniforms", C.c_void_p)]


lib.dpara_head_workspace_bytes.restype = C.c_size_t
lib.dpara_head_workspace_bytes.argtypes = [C.c_int32, C.c_int32, C.c_int32]
lib.dpara_draft_head.restype = C.c_int
lib.dpara_draft_head.argtypes = [C.POINTER(HeadIO), C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
EXPORTED += ["dpara_head_workspace_bytes", "dpara_draft_head"]


class HeadPlan:
    """Buffers of dpara_draft_head for fixed shapes (allocated once; a call allocates nothing)."""

    def __init__(self, b: int, block: int, hidden: int, vocab: int, rank: int, device="cuda"):
        self.b, self.block, self.hidden, self.vocab, self.rank = b, block, hidden, vocab, rank
        self.workspace_bytes = int(lib.dpara_head_workspace_bytes(b, block, vocab))
        self.workspace = torch.empty(self.workspace_bytes, dtype=torch.uint8, device=device)
        self.next_tokens = torch.full((b, block), -1, dtype=torch.int32, device=device)
        self.status = torch.zeros(1, dtype=torch.int32, device=device)

    def base_logits(self) -> torch.Tensor:
        """The fp32 base logits the last call left in the workspace (stored step-major [block][b][vocab]), as
        [b * block][vocab] in request-major row order."""
        n = self.b * self.block * self.vocab
        return self.workspace[: n * 4].view(torch.float32).view(self.block, self.b, self.vocab).permute(1, 0, 2).reshape(
            self.b * self.block, self.vocab)

    def run(self, sel_reps, w_lm, ar_w, ar_e, bonus, uniforms=None, stream=None):
        """uniforms [b][block] fp32 (each m * 2^-24): sample y_i from softmax(z_i); None: greedy."""
        io = HeadIO(_ptr(sel_reps), _ptr(w_lm), _ptr(ar_w), _ptr(ar_e), _ptr(bonus), _ptr(self.next_tokens),
                    self.b, self.block, self.hidden, self.vocab, self.rank, _ptr(uniforms))
        rc = lib.dpara_draft_head(C.byref(io), self.workspace.data_ptr(), self.workspace_bytes, self.status.data_ptr(),
                                  _stream_ptr(stream))
        if rc != OK:
            raise DparaError(rc)
        return self.next_tokens


def draft_head(sel_reps, w_lm, ar_w, ar_e, bonus, uniforms=None, stream=None):
    """dpara_draft_head: sel_reps [b][block][hidden], w_lm [vocab][hidden], ar_w / ar_e [vocab][rank] (bf16 CUDA
    tensors), bonus [b] int32.  Returns (next_tokens [b][block] int32, plan)."""
    b, block, hidden = sel_reps.shape
    plan = HeadPlan(b, block, hidden, w_lm.shape[0], ar_w.shape[1], sel_reps.device)
    plan.run(sel_reps, w_lm, ar_w, ar_e, bonus, uniforms, stream)
    return plan.next_tokens, plan


# ----------------------------------------------------------------------------- feature-cache append
class CacheIO(C.Structure):
    _fields_ = [("batch", C.c_int32), ("n_rows", C.c_int32), ("feat_dim", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("n_layers", C.c_int32), ("features", C.c_void_p), ("accept_len", C.c_void_p),
                ("host_w_kv", C.c_void_p), ("host_norm_w", C.c_void_p), ("host_knorm_w", C.c_void_p),
                ("host_k_ctx", C.c_void_p), ("host_v_ctx", C.c_void_p), ("row_start", C.c_void_p), ("capacity", C.c_void_p),
                ("ctx_len", C.c_void_p), ("rms_eps", C.c_float), ("rope_theta", C.c_float), ("use_rope", C.c_int32)]


lib.dpara_cache_append_workspace_bytes.restype = C.c_size_t
lib.dpara_cache_append_workspace_bytes.argtypes = [C.POINTER(CacheIO)]
lib.dpara_cache_append.restype = C.c_int
lib.dpara_cache_append.argtypes = [C.POINTER(CacheIO), C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
EXPORTED += ["dpara_cache_append_workspace_bytes", "dpara_cache_append"]


class CachePlan:
    """dpara_cache_append for fixed shapes and fixed per-layer tensors (weights, caches): pointer tables, workspace and
    status word are set up once; run() allocates nothing."""

    def __init__(self, *, batch: int, n_rows: int, w_kv: Sequence[torch.Tensor], k_ctx: Sequence[torch.Tensor],
                 v_ctx: Sequence[torch.Tensor], row_start: torch.Tensor, capacity: torch.Tensor, ctx_len: torch.Tensor,
                 norm_w: Optional[Sequence[torch.Tensor]] = None, knorm_w: Optional[Sequence[torch.Tensor]] = None,
                 rms_eps: float = 1e-6, rope_theta: float = 1e6, use_rope: bool = True):
        n_layers = len(w_kv)
        Hkv, D = k_ctx[0].shape[1], k_ctx[0].shape[2]
        self._keep = (list(w_kv), list(k_ctx), list(v_ctx), row_start, capacity, ctx_len, norm_w, knorm_w)
        table = lambda ts: (C.c_void_p * n_layers)(*[_ptr(t) for t in ts]) if ts is not None else None
        self._tabs = [table(w_kv), table(norm_w), table(knorm_w), table(k_ctx), table(v_ctx)]
        cast = lambda t: C.cast(t, C.c_void_p).value if t is not None else None
        self.io = CacheIO(batch, n_rows, w_kv[0].shape[1], Hkv, D, n_layers, None, None, *[cast(t) for t in self._tabs],
                          _ptr(row_start), _ptr(capacity), _ptr(ctx_len), rms_eps, rope_theta, 1 if use_rope else 0)
        self.workspace_bytes = int(lib.dpara_cache_append_workspace_bytes(C.byref(self.io)))
        self.workspace = torch.empty(max(self.workspace_bytes, 16), dtype=torch.uint8, device=ctx_len.device)
        self.status = torch.zeros(1, dtype=torch.int32, device=ctx_len.device)
        self.ctx_len = ctx_len

    def run(self, features: torch.Tensor, accept_len: torch.Tensor, stream=None) -> None:
        self.io.features, self.io.accept_len = _ptr(features), _ptr(accept_len)
        rc = lib.dpara_cache_append(C.byref(self.io), self.workspace.data_ptr(), self.workspace.numel(), self.status.data_ptr(),
                                    _stream_ptr(stream))
        if rc != OK:
            raise DparaError(rc)


# ----------------------------------------------------------------------------- stack of backbone blocks
class BackboneIO(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("host_layers", C.c_void_p), ("host_k_ctx", C.c_void_p), ("host_v_ctx", C.c_void_p)]


lib.dpara_backbone_workspace_bytes.restype = C.c_size_t
lib.dpara_backbone_workspace_bytes.argtypes = [C.POINTER(Shape), C.c_void_p, C.POINTER(BackboneIO)]
lib.dpara_draft_backbone.restype = C.c_int
lib.dpara_draft_backbone.argtypes = [C.POINTER(Shape), C.POINTER(AttnIO), C.POINTER(BackboneIO), C.c_void_p, C.c_size_t, C.c_void_p,
                                     C.c_void_p]
EXPORTED += ["dpara_backbone_workspace_bytes", "dpara_draft_backbone"]


class BackbonePlan:
    """dpara_draft_backbone for fixed shapes, weights and caches: a stack of blocks with the spine tokens as query rows.
    layers: LayerIO per block (make_layer_io; x of the first and y_f32 / y_bf16 of the last are the call's input and
    outputs, [b][J*Bq + S][hidden]); k_ctx / v_ctx: one cache tensor per block."""

    def __init__(self, *, ctx_offsets: Sequence[int], n_boundaries: int, block: int, n_q_heads: int, n_kv_heads: int, head_dim: int,
                 layers: Sequence[LayerIO], k_ctx: Sequence[torch.Tensor], v_ctx: Sequence[torch.Tensor], prefix_base: int = 1,
                 n_spine: Optional[int] = None, ctx_lens: Optional[Sequence[int]] = None, spine_queries: bool = True, device="cuda"):
        b = len(ctx_offsets) - 1
        nl = len(layers)
        self.shape = Shape(b, n_boundaries, block, n_q_heads, n_kv_heads, head_dim, prefix_base,
                           n_boundaries if n_spine is None else n_spine, 0, n_boundaries, 0.0, 1 if spine_queries else 0)
        self.host_off = _host_offsets(ctx_offsets)
        self.dev_off = torch.tensor([int(x) for x in ctx_offsets], dtype=torch.int64, device=device)
        self.host_lens = self.dev_lens = None
        if ctx_lens is not None:
            self.host_lens = (C.c_int64 * b)(*[int(x) for x in ctx_lens])
            self.dev_lens = torch.tensor([int(x) for x in ctx_lens], dtype=torch.int64, device=device)
        self._keep = (list(k_ctx), list(v_ctx))
        self.layers = (LayerIO * nl)(*layers)
        self.kc = (C.c_void_p * nl)(*[_ptr(t) for t in k_ctx])
        self.vc = (C.c_void_p * nl)(*[_ptr(t) for t in v_ctx])
        self.bb = BackboneIO(nl, C.cast(self.layers, C.c_void_p).value, C.cast(self.kc, C.c_void_p).value, C.cast(self.vc, C.c_void_p).value)
        self.workspace_bytes = int(lib.dpara_backbone_workspace_bytes(C.byref(self.shape), C.cast(self.host_off, C.c_void_p), C.byref(self.bb)))
        self.workspace = torch.empty(max(self.workspace_bytes, 16), dtype=torch.uint8, device=device)
        self.status = torch.zeros(1, dtype=torch.int32, device=device)

    def __call__(self, *, k_spine=None, v_spine=None, stream=None) -> None:
        io = AttnIO(None, None, None, self.dev_off.data_ptr(), C.cast(self.host_off, C.c_void_p).value, _ptr(k_spine), _ptr(v_spine),
                    None, None, None, BF16, None, _ptr(self.dev_lens),
                    C.cast(self.host_lens, C.c_void_p).value if self.host_lens is not None else None)
        rc = lib.dpara_draft_backbone(C.byref(self.shape), C.byref(io), C.byref(self.bb), self.workspace.data_ptr(),
                                      self.workspace.numel(), self.status.data_ptr(), _stream_ptr(stream))
        if rc != OK:
            raise DparaError(rc)
