"""Helpers shared by the GPU parity tests: move generated inputs to the device, call through the C ABI."""
import numpy as np
import torch

import paper_2609_27396_b200 as dp


def dev_bf16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def host_bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def run_attention(inp, *, out_dtype=torch.float32, want_lse=True, with_blk=True, **kw):
    sh = inp.shape
    args = [dev_bf16(x) for x in (inp.q, inp.k_ctx, inp.v_ctx)]
    ks, vs = dev_bf16(inp.k_spine), dev_bf16(inp.v_spine)
    kb, vb = (dev_bf16(inp.k_blk), dev_bf16(inp.v_blk)) if with_blk else (None, None)
    res = dp.draft_all_boundaries(args[0], args[1], args[2], [int(x) for x in inp.ctx_offsets], ks, vs, kb, vb,
                                  prefix_base=sh.prefix_base, out_dtype=out_dtype, want_lse=want_lse, **kw)
    torch.cuda.synchronize()
    return res


def run_verify(v, mode):
    kw = {}
    if mode == 1:
        kw = dict(draft_probs=torch.from_numpy(v.draft_probs).cuda(), uniforms=torch.from_numpy(v.uniforms).cuda())
    res = dp.verify_select(torch.from_numpy(v.target).cuda(), torch.from_numpy(v.draft_tokens).cuda(),
                           dev_bf16(v.reps) if v.reps is not None else None, mode=mode, **kw)
    torch.cuda.synchronize()
    return res


def check_verify(res, ref):
    for k in ("accept_len", "bonus", "gather_idx", "out_tokens"):
        assert np.array_equal(res[k].cpu().numpy(), ref[k]), k
    if ref["selected"] is not None:
        assert np.array_equal(host_bits(res["selected"]), ref["selected"])
    assert int(res["status"].item()) == ref["status"]
