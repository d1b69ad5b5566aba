"""GPU: a bounded device-side wait that runs out.

pd_test_inject_wait_timeout arms one event: the next launch of the named kernel runs with a wait bound of
2 ms (instead of 4 s) and its producer leaves out one operand tile load.  A wait inside the kernel then gives
up: the block must raise its abort flag, free its tensor memory, pass the cluster barrier of a CTA pair and
return; the error word must read PD_ERR_DEVICE_TIMEOUT; and the next ordinary launch must be correct again.
Nothing faults and no wait is unbounded."""
import numpy as np
import pytest

import pd_inputs as gen
from oracle import decoder_layer as L
from gpu_util import DeviceLayer, assert_close, from_dev, i32_dev, to_dev, empty_bf16

pytestmark = pytest.mark.gpu

LIMIT_NS = 2_000_000


def _gemm(pd, m, n, k, seed):
    import torch
    a = gen.normal_bf16(seed, 40, (m, k), 1.0, sub=m)
    b = gen.normal_bf16(seed, 41, (n, k), 0.05, sub=n)
    dc = empty_bf16(m, n)
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    pd.pd_gemm_bf16(to_dev(a), to_dev(b), dc, m, n, k, err_word=err)
    torch.cuda.synchronize()
    return a, b, from_dev(dc).astype(np.float64), int(err.item())


@pytest.mark.parametrize("kind,shape", [("single", (128, 512, 512)), ("pair", (512, 6144, 512))])
def test_gemm_wait_runs_out_and_the_next_launch_is_correct(pdlib, kind, shape):
    m, n, k = shape            # (one row tile -> single-CTA kernel; several row tiles, N % 256 == 0 -> CTA pairs)
    pdlib.pd_test_inject_wait_timeout(pdlib.INJECT_GEMM if kind == "single" else pdlib.INJECT_GEMM_PAIR, LIMIT_NS)
    _, _, _, err = _gemm(pdlib, m, n, k, seed=60)
    assert err == 1, "the injected timeout was not reported"
    a, b, got, err = _gemm(pdlib, m, n, k, seed=60)
    assert err == 0
    ref = a.astype(np.float64) @ b.astype(np.float64).T
    assert np.all(np.abs(got - ref) <= 1e-2 * np.sqrt(k) * 0.05 + 8e-3 * np.abs(ref))
    pdlib.pd_test_inject_wait_timeout(pdlib.INJECT_NONE, 0)


def test_blockwise_fp8_gemm_wait_runs_out_and_the_next_launch_is_correct(pdlib):
    import torch
    from oracle import fp8
    m, n, k = 300, 512, 512
    a = gen.normal_bf16(62, 40, (m, k), 1.0, sub=m)
    b = gen.normal_bf16(62, 41, (n, k), 0.05, sub=n)
    qa = torch.zeros((m, k), dtype=torch.uint8, device="cuda"); sa = torch.zeros((m, k // 128), dtype=torch.float32, device="cuda")
    qb = torch.zeros((n, k), dtype=torch.uint8, device="cuda"); sb = torch.zeros((n // 128, k // 128), dtype=torch.float32, device="cuda")
    pdlib.pd_quantize_fp8_groups(to_dev(a), m, k, qa, sa)
    pdlib.pd_quantize_fp8_blocks(to_dev(b), n, k, qb, sb)
    dc = empty_bf16(m, n)
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    pdlib.pd_test_inject_wait_timeout(pdlib.INJECT_GEMM_FP8_BLOCKWISE, LIMIT_NS)
    pdlib.pd_gemm_fp8_blockwise(qa, sa, qb, sb, dc, m, n, k, err_word=err)
    torch.cuda.synchronize()
    assert int(err.item()) == 1, "the injected timeout was not reported"
    err.zero_()
    pdlib.pd_gemm_fp8_blockwise(qa, sa, qb, sb, dc, m, n, k, err_word=err)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    ref = fp8.gemm_fp8_blockwise(qa.cpu().numpy(), sa.cpu().numpy(), qb.cpu().numpy(), sb.cpu().numpy())
    got = from_dev(dc).astype(np.float64)
    assert np.all(np.abs(got - ref) <= 2.0 ** -8 * np.abs(ref) + 1e-5 * np.sqrt(k) * 0.05)
    pdlib.pd_test_inject_wait_timeout(pdlib.INJECT_NONE, 0)


def test_prefill_attention_wait_runs_out_and_layer_check_reports_it(pdlib):
    import torch
    shape = dict(d_model=512, n_q_heads=8, n_kv_heads=2, head_dim=64, d_ff=1536)
    w = gen.layer_weights(**shape, seed=61)
    ocfg, ow = L.LayerConfig(**shape), L.LayerWeights(**w)
    dl = DeviceLayer(pdlib, pdlib.LayerConfig(**shape, max_pos=512), w, 400, 0, 0)
    cu = [0, 400]
    x = gen.activations(61, 400, 512)
    k, v, cache = dl.make_cache(1, 400)
    dx, dout = to_dev(x), empty_bf16(400, 512)
    pdlib.pd_test_inject_wait_timeout(pdlib.INJECT_ATTN_PREFILL, LIMIT_NS)
    pdlib.pd_prefill_layer(dl.layer, dx, dout, i32_dev(cu), cu, cache, dl.ws, dl.ws_bytes)
    with pytest.raises(pdlib.PdError) as e:
        pdlib.pd_layer_check(dl.layer)
    assert e.value.status == pdlib.PD_ERR_DEVICE_TIMEOUT
    pdlib.pd_layer_check(dl.layer)                       # the error word was cleared
    pdlib.pd_prefill_layer(dl.layer, dx, dout, i32_dev(cu), cu, cache, dl.ws, dl.ws_bytes)
    pdlib.pd_layer_check(dl.layer)
    torch.cuda.synchronize()
    ref, _, _ = L.prefill_layer(ocfg, ow, x, cu)
    assert_close(from_dev(dout), ref, "prefill after the injected timeout")
