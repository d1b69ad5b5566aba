"""GPU: block-wise FP8 (one scale per 128 x 128 weight block and per token and 128 channels) against the oracle.

Codes and scales are integer / exactly defined fp32 results and must match bit for bit.  The GEMM sums exact
products of one K block in fp32 on the tensor cores and adds the scaled partial sums in fp32; it is compared with
the oracle's float64 value of the SAME codes and scales within one bf16 rounding of the result plus the fp32
rounding of k / 128 scaled additions."""
import numpy as np
import pytest

import pd_inputs as gen
from gpu_util import to_dev, from_dev, empty_bf16
from oracle import fp8

pytestmark = pytest.mark.gpu


def _groups_dev(pdlib, x_np):
    import torch
    rows, k = x_np.shape
    codes = torch.zeros((rows, k), dtype=torch.uint8, device="cuda")
    scales = torch.zeros((rows, k // 128), dtype=torch.float32, device="cuda")
    pdlib.pd_quantize_fp8_groups(to_dev(x_np), rows, k, codes, scales)
    torch.cuda.synchronize()
    return codes, scales


def _blocks_dev(pdlib, w_np):
    import torch
    n, k = w_np.shape
    codes = torch.zeros((n, k), dtype=torch.uint8, device="cuda")
    scales = torch.zeros(((n + 127) // 128, k // 128), dtype=torch.float32, device="cuda")
    pdlib.pd_quantize_fp8_blocks(to_dev(w_np), n, k, codes, scales)
    torch.cuda.synchronize()
    return codes, scales


@pytest.mark.parametrize("rows,k,std", [(1, 128, 1.0), (5, 512, 1.0), (130, 4096, 0.02), (33, 14336, 3.0), (7, 1536, 1e-3)])
def test_quantize_groups_bit_exact(pdlib, rows, k, std):
    x = gen.normal_bf16(12, 50, (rows, k), std, sub=rows)
    if rows >= 5:
        x[2, 128:256] = 0.0                 # an all-zero group -> scale 1, codes 0
        x[3, 1:128] = 0.0                   # single non-zero element in a group -> +-448
        x[4, :8] = [448.0, -448.0, 1e-30, -1e-30, 0.5, -0.0, 3e38, -3e38]   # extremes of the bf16 range
        x = gen.bf16_round(x)
    q_ref, s_ref = fp8.quantize_groups(x)
    codes, scales = _groups_dev(pdlib, x)
    assert np.array_equal(scales.cpu().numpy().view(np.uint32), s_ref.view(np.uint32))
    assert np.array_equal(codes.cpu().numpy(), q_ref)


@pytest.mark.parametrize("n,k,std", [(128, 128, 0.02), (256, 512, 0.02), (200, 384, 1.0), (16, 1536, 0.5), (4096, 1024, 0.02)])
def test_quantize_blocks_bit_exact(pdlib, n, k, std):
    w = gen.normal_bf16(13, 51, (n, k), std, sub=n)
    if n >= 128 and k >= 256:
        w[0:128, 128:256] = 0.0             # an all-zero block
        w[5, 7] = 3.0                       # an outlier: only its block's scale moves
        w = gen.bf16_round(w)
    q_ref, s_ref = fp8.quantize_blocks(w)
    codes, scales = _blocks_dev(pdlib, w)
    assert np.array_equal(scales.cpu().numpy().view(np.uint32), s_ref.view(np.uint32))
    assert np.array_equal(codes.cpu().numpy(), q_ref)


@pytest.mark.parametrize("m,n,k", [
    (128, 128, 128), (1, 768, 512), (37, 1536, 512), (200, 784, 1536), (129, 512, 512),
    (300, 3072, 512), (1000, 6144, 4096), (333, 4096, 14336), (16, 4096, 4096), (512, 6144, 128), (4096, 4096, 4096),
])
def test_gemm_fp8_blockwise_matches_oracle(pdlib, m, n, k):
    import torch
    a = gen.normal_bf16(3, 40, (m, k), 1.0, sub=m)
    b = gen.normal_bf16(3, 41, (n, k), 0.02, sub=n)
    # block structure that a per-row scheme could not follow: blocks and groups of very different magnitude
    a[:, : min(k, 128)] *= 8.0
    if n > 128 and k > 128:
        b[128:256, 128:256] *= 16.0
    a, b = gen.bf16_round(a), gen.bf16_round(b)
    qa, sa = _groups_dev(pdlib, a)
    qb, sb = _blocks_dev(pdlib, b)
    qa_ref, sa_ref = fp8.quantize_groups(a)
    qb_ref, sb_ref = fp8.quantize_blocks(b)
    assert np.array_equal(qa.cpu().numpy(), qa_ref) and np.array_equal(qb.cpu().numpy(), qb_ref)
    assert np.array_equal(sa.cpu().numpy(), sa_ref) and np.array_equal(sb.cpu().numpy(), sb_ref)
    dc = empty_bf16(m, n)
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    pdlib.pd_gemm_fp8_blockwise(qa, sa, qb, sb, dc, m, n, k, err_word=err)
    torch.cuda.synchronize()
    assert int(err.item()) == 0, "device-side wait timed out"
    got = from_dev(dc).astype(np.float64)
    if m * n * k <= 2 ** 33:
        ref = fp8.gemm_fp8_blockwise(qa_ref, sa_ref, qb_ref, sb_ref)
    else:   # large: float32 BLAS per K block on the decoded codes (exact inputs), scales applied in float64
        da, db = fp8.e4m3_decode(qa_ref).astype(np.float32), fp8.e4m3_decode(qb_ref).astype(np.float32)
        ref = np.zeros((m, n))
        rb = np.arange(n) // 128
        for j in range(k // 128):
            part = (da[:, j * 128:(j + 1) * 128] @ db[:, j * 128:(j + 1) * 128].T).astype(np.float64)
            ref += part * sa_ref[:, j].astype(np.float64)[:, None] * sb_ref[rb, j].astype(np.float64)[None, :]
    # one bf16 rounding of the result (2^-9) plus fp32 rounding of the scale product and of k / 128 additions, and an
    # absolute term for cancelling sums (sqrt(k) terms of the size of the scaled operands)
    bound = 2.0 ** -8 * np.abs(ref) + 1e-5 * np.sqrt(k) * 0.02 * 8 * 16
    assert np.all(np.abs(got - ref) <= bound), float(np.abs(got - ref).max())
    # and the scheme does what it is for: close to the unquantised product although one block is 16 times larger
    if m * n * k <= 2 ** 31:
        exact = a.astype(np.float64) @ b.astype(np.float64).T
        rel = np.linalg.norm(got - exact) / np.linalg.norm(exact)
        assert rel < 0.06, rel


def test_blockwise_rejects_bad_shapes(pdlib):
    import torch
    q = torch.zeros((128, 192), dtype=torch.uint8, device="cuda")
    s = torch.ones((128, 2), dtype=torch.float32, device="cuda")
    c = empty_bf16(128, 128)
    x = empty_bf16(128, 192)
    with pytest.raises(pdlib.PdError) as e:
        pdlib.pd_gemm_fp8_blockwise(q, s, q, s, c, 128, 128, 192)      # K not a multiple of 128
    assert e.value.status == pdlib.PD_ERR_UNSUPPORTED_SHAPE
    with pytest.raises(pdlib.PdError) as e:
        pdlib.pd_gemm_fp8_blockwise(q, None, q, s, c, 128, 128, 128)   # missing scales
    assert e.value.status == pdlib.PD_ERR_INVALID_ARG
    with pytest.raises(pdlib.PdError) as e:
        pdlib.pd_quantize_fp8_groups(x, 128, 192, q, s)                # K not a multiple of 128
    assert e.value.status == pdlib.PD_ERR_UNSUPPORTED_SHAPE
    with pytest.raises(pdlib.PdError) as e:
        pdlib.pd_quantize_fp8_blocks(x, 128, 192, q, s)
    assert e.value.status == pdlib.PD_ERR_UNSUPPORTED_SHAPE
    pdlib.pd_gemm_fp8_blockwise(q, s, q, s, c, 0, 128, 128)            # nothing to do
