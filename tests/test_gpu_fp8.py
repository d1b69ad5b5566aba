"""GPU: FP8 (E4M3) row quantiser and tensor-core GEMM against the FP8 oracle.

Codes and scales are integer / exactly defined fp32 results and must match bit for bit; the GEMM
accumulates exact products in fp32, so it is compared with the oracle's float64 value of the SAME
codes within the bf16 rounding of the stored output."""
import numpy as np
import pytest

import pd_inputs as gen
from gpu_util import to_dev, from_dev, empty_bf16
from oracle import fp8

pytestmark = pytest.mark.gpu


def _quantize_dev(pdlib, x_np):
    import torch
    rows, k = x_np.shape
    dx = to_dev(x_np)
    codes = torch.zeros((rows, k), dtype=torch.uint8, device="cuda")
    scales = torch.zeros(rows, dtype=torch.float32, device="cuda")
    pdlib.pd_quantize_fp8_rows(dx, rows, k, codes, scales)
    torch.cuda.synchronize()
    return codes, scales


@pytest.mark.parametrize("rows,k,std", [(1, 16, 1.0), (5, 512, 1.0), (130, 4096, 0.02), (33, 14336, 3.0), (7, 1536, 1e-3)])
def test_quantize_rows_bit_exact(pdlib, rows, k, std):
    x = gen.normal_bf16(11, 50, (rows, k), std, sub=rows)
    if rows >= 5:
        x[2] = 0.0                       # all-zero row -> scale 1, codes 0
        x[3, 1:] = 0.0                   # single non-zero element -> +-448
        x[4, :8] = [448.0, -448.0, 1e-30, -1e-30, 0.5, -0.0, 3e38, -3e38]   # extremes of the bf16 range
        x = gen.bf16_round(x)
    q_ref, s_ref = fp8.quantize_rows(x)
    codes, scales = _quantize_dev(pdlib, x)
    assert np.array_equal(scales.cpu().numpy().view(np.uint32), s_ref.view(np.uint32))
    assert np.array_equal(codes.cpu().numpy(), q_ref)


def test_quantize_every_code_and_midpoint(pdlib):
    # one row holding every finite E4M3 magnitude, the midpoints between neighbours (ties) and 448 as the
    # row maximum, so that scale = 1 and the quotient is the element itself
    vals = fp8.e4m3_decode(np.arange(0, 127))
    mids = (vals[:-1] + vals[1:]) / 2      # 4 significant bits: exact in bf16
    row = np.concatenate([vals, -vals, mids, -mids, [448.0]]).astype(np.float32)
    row = np.concatenate([row, np.zeros((-len(row)) % 16, np.float32)])
    assert np.array_equal(gen.bf16_round(row), row)
    q_ref, s_ref = fp8.quantize_rows(row[None, :])
    assert s_ref[0] == 1.0
    codes, scales = _quantize_dev(pdlib, row[None, :])
    assert scales.cpu().numpy()[0] == 1.0
    assert np.array_equal(codes.cpu().numpy(), q_ref)


@pytest.mark.parametrize("m,n,k", [
    (128, 256, 128), (1, 768, 512), (37, 1536, 512), (200, 768, 1536), (129, 512, 512),
    (300, 3072, 512), (1000, 6144, 4096), (333, 4096, 14336), (2048, 28672, 4096), (16, 4096, 4096),
    (512, 6144, 128), (300, 6144, 256), (512, 4096, 1024), (384, 4096, 512),
])
def test_gemm_fp8_matches_oracle(pdlib, m, n, k):
    import torch
    a = gen.normal_bf16(2, 40, (m, k), 1.0, sub=m)
    b = gen.normal_bf16(2, 41, (n, k), 0.02, sub=n)
    qa, sa = _quantize_dev(pdlib, a)
    qb, sb = _quantize_dev(pdlib, b)
    qa_ref, sa_ref = fp8.quantize_rows(a)
    qb_ref, sb_ref = fp8.quantize_rows(b)
    assert np.array_equal(qa.cpu().numpy(), qa_ref) and np.array_equal(qb.cpu().numpy(), qb_ref)
    dc = empty_bf16(m, n)
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    pdlib.pd_gemm_fp8(qa, sa, qb, sb, dc, m, n, k, err_word=err)
    torch.cuda.synchronize()
    assert int(err.item()) == 0, "device-side wait timed out"
    got = from_dev(dc).astype(np.float64)
    if m * n * k <= 2 ** 33:
        ref = fp8.gemm_fp8(qa_ref, sa_ref, qb_ref, sb_ref)
    else:   # large: float32 BLAS on the decoded codes (exact inputs, ~1e-6 relative), scales applied in float64
        acc = fp8.e4m3_decode(qa_ref).astype(np.float32) @ fp8.e4m3_decode(qb_ref).astype(np.float32).T
        ref = acc.astype(np.float64) * sa_ref.astype(np.float64)[:, None] * sb_ref.astype(np.float64)[None, :]
    # fp32 accumulation of exact products, one bf16 rounding of the result: 2^-9 relative plus an absolute
    # term for cancelling sums (sqrt(k) terms of size |a||b|)
    bound = 2.0 ** -8 * np.abs(ref) + 1e-5 * np.sqrt(k) * 0.02
    assert np.all(np.abs(got - ref) <= bound), float(np.abs(got - ref).max())


def test_gemm_fp8_rejects_bad_shapes(pdlib):
    import torch
    q = torch.zeros((128, 192), dtype=torch.uint8, device="cuda")
    s = torch.ones(128, dtype=torch.float32, device="cuda")
    c = empty_bf16(128, 128)
    with pytest.raises(pdlib.PdError) as e:
        pdlib.pd_gemm_fp8(q, s, q, s, c, 128, 128, 192)      # K not a multiple of 128
    assert e.value.status == pdlib.PD_ERR_UNSUPPORTED_SHAPE
    with pytest.raises(pdlib.PdError) as e:
        pdlib.pd_gemm_fp8(q, None, q, s, c, 128, 128, 128)   # missing scales
    assert e.value.status == pdlib.PD_ERR_INVALID_ARG
