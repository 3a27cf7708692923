"""GPU parity of the tensor-core projection GEMM (dpara_gemm_bf16) against the oracle's plain float64
products.  Tolerance: fp32 accumulation of K bf16 x bf16 products, |terms| <= |a||w|: error <~ K * 2^-24
relative to the row's absolute sum, far below the bf16 output rounding (2^-9 relative) that dominates."""
import numpy as np
import pytest
import torch

import workloads as W
from oracle import attention as OA
from oracle import layer as OL

pytestmark = pytest.mark.gpu


def _bits(rng, shape, sigma):
    return W.f32_to_bf16_bits((rng.standard_normal(shape) * sigma).astype(np.float32))


def _dev(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


@pytest.mark.parametrize("M,N,K", [(128, 256, 64), (128, 256, 256), (256, 512, 512), (200, 264, 192), (1024, 768, 1024), (40, 8, 64),
                                   (1024, 6144, 256),     # 192-column tiles, exact multiple (the QKV shape's tiling)
                                   (300, 1000, 128)])     # ragged rows and a part-filled last 192-column tile
def test_gemm_bf16_store(M, N, K):
    import paper_2609_27396_b200 as dp
    rng = np.random.default_rng(M + N + K)
    a, w = _bits(rng, (M, K), 1.0), _bits(rng, (N, K), 0.05)
    out, st = dp.gemm_bf16(_dev(a), _dev(w), epilogue=0)
    torch.cuda.synchronize()
    ref = OL.linear(OA.bf16_bits_to_f64(a), OA.bf16_bits_to_f64(w))
    got = out.float().cpu().numpy().astype(np.float64)
    tol = 2 ** -8 * np.abs(ref) + 1e-3
    assert int(st.item()) == 0
    assert np.all(np.abs(got - ref) <= tol), float(np.abs(got - ref).max())


@pytest.mark.parametrize("resid_bf16", [True, False])
def test_gemm_residual_fp32(resid_bf16):
    import paper_2609_27396_b200 as dp
    M, N, K = 384, 512, 320
    rng = np.random.default_rng(5)
    a, w = _bits(rng, (M, K), 1.0), _bits(rng, (N, K), 0.05)
    if resid_bf16:
        rb = _bits(rng, (M, N), 1.0)
        resid, r64 = _dev(rb), OA.bf16_bits_to_f64(rb)
    else:
        r32 = rng.standard_normal((M, N)).astype(np.float32)
        resid, r64 = torch.from_numpy(r32).cuda(), r32.astype(np.float64)
    out, out16, st = dp.gemm_bf16(_dev(a), _dev(w), epilogue=1, resid=resid, want_bf16_copy=True)
    torch.cuda.synchronize()
    ref = r64 + OL.linear(OA.bf16_bits_to_f64(a), OA.bf16_bits_to_f64(w))
    assert np.abs(out.cpu().numpy().astype(np.float64) - ref).max() < 1e-4
    assert np.abs(out16.float().cpu().numpy().astype(np.float64) - ref).max() < 2e-2
    assert int(st.item()) == 0


def test_gemm_swiglu():
    import paper_2609_27396_b200 as dp
    M, I, K = 256, 384, 256
    rng = np.random.default_rng(6)
    a, w = _bits(rng, (M, K), 1.0), _bits(rng, (2 * I, K), 0.08)
    out, st = dp.gemm_bf16(_dev(a), _dev(w), epilogue=2)
    torch.cuda.synchronize()
    ref = OL.swiglu_linear(OA.bf16_bits_to_f64(a), OA.bf16_bits_to_f64(w))
    got = out.float().cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got - ref) <= 2 ** -7 * np.abs(ref) + 1e-3), float(np.abs(got - ref).max())
    assert int(st.item()) == 0


def test_gemm_rejects_bad_k():
    import paper_2609_27396_b200 as dp
    a = torch.zeros(128, 72, dtype=torch.bfloat16, device="cuda")
    w = torch.zeros(256, 72, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(dp.DparaError) as e:
        dp.gemm_bf16(a, w)
    assert e.value.code == dp.ERR_UNSUPPORTED
