"""GPU: the tensor-core GEMM against a float64 matmul of the same bf16 inputs."""
import numpy as np
import pytest

import pd_inputs as gen
from gpu_util import to_dev, from_dev, empty_bf16

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("m,n,k", [
    (128, 256, 64), (128, 64, 128), (1, 768, 512), (37, 1536, 512), (200, 768, 512), (129, 512, 1536),
    (300, 3072, 512), (1000, 6144, 4096), (333, 4096, 14336), (2048, 28672, 4096), (16, 4096, 4096),
    (512, 6144, 64), (300, 6144, 128), (2000, 4096, 8192),   # CTA-pair kernel: one K block; odd row tiles; tail halves
    (512, 4096, 1024), (384, 4096, 512), (130, 2048, 256),   # short batches against N = d_model: one wave of narrow tiles
])
def test_gemm_matches_float64(pdlib, m, n, k):
    import torch
    a = gen.normal_bf16(1, 40, (m, k), 1.0, sub=m)
    b = gen.normal_bf16(1, 41, (n, k), 0.05, sub=n)
    da, db, dc = to_dev(a), to_dev(b), empty_bf16(m, n)
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    pdlib.pd_gemm_bf16(da, db, dc, m, n, k, err_word=err)
    torch.cuda.synchronize()
    assert int(err.item()) == 0, "device-side wait timed out"
    got = from_dev(dc).astype(np.float64)
    if m * n * k <= 2 ** 33:
        ref = a.astype(np.float64) @ b.astype(np.float64).T
    else:                       # large: float32 BLAS on exact bf16 inputs, error ~1e-6 relative
        ref = (a @ b.T).astype(np.float64)
    scale = np.sqrt(k) * 0.05
    err_abs = np.abs(got - ref)
    assert np.all(err_abs <= 1e-2 * scale + 8e-3 * np.abs(ref)), (float(err_abs.max()), scale)


@pytest.mark.parametrize("m,n,k", [
    (512, 4096, 14336), (384, 4096, 8192), (300, 4096, 14336), (200, 2048, 8192),   # every tile cut along K on CTA pairs
    (512, 4096, 4096), (384, 4096, 2048),      # short K: narrow single-CTA tiles as without the workspace
    (512, 6144, 4096), (1024, 4096, 4096),     # too many tiles for that: whole tiles, half-width tail
    (2000, 4096, 8192), (4096, 4096, 14336),   # long K: as before
])
def test_gemm_with_k_split_workspace_matches_float64(pdlib, m, n, k):
    """The projections' launch path (pd_gemm_bf16_ws): tiles cut in two along K hand their fp32 partials over
    through the workspace.  Run twice on one workspace: the flags must be back at zero after a launch."""
    import torch
    a = gen.normal_bf16(3, 40, (m, k), 1.0, sub=m)
    b = gen.normal_bf16(3, 41, (n, k), 0.05, sub=n)
    da, db = to_dev(a), to_dev(b)
    ws_bytes = pdlib.pd_gemm_workspace_bytes()
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    ref = (a @ b.T).astype(np.float64)
    scale = np.sqrt(k) * 0.05
    for _ in range(2):
        dc = empty_bf16(m, n)
        pdlib.pd_gemm_bf16_ws(da, db, dc, m, n, k, ws, ws_bytes, err_word=err)
        torch.cuda.synchronize()
        assert int(err.item()) == 0, "device-side wait timed out"
        assert not torch.any(ws[:74 * 16].view(torch.int32) != 0), "a hand-over flag was left raised"
        got = from_dev(dc).astype(np.float64)
        assert np.all(np.abs(got - ref) <= 1e-2 * scale + 8e-3 * np.abs(ref)), float(np.abs(got - ref).max())


def test_gemm_rejects_bad_shapes(pdlib):
    a, b, c = empty_bf16(128, 96), empty_bf16(128, 96), empty_bf16(128, 128)
    with pytest.raises(pdlib.PdError) as e:
        pdlib.pd_gemm_bf16(a, b, c, 128, 128, 96)      # K not a multiple of 64
    assert e.value.status == pdlib.PD_ERR_UNSUPPORTED_SHAPE
