"""GPU: the allocation-free decode attention against the ordinary entry point and against the oracle.

pd_decode_attention_noalloc serves callers that cannot cudaMalloc a workspace (a process
whose memory pool owns the device, code under stream capture, a loop that must avoid the
allocator); its scratch is a fixed array inside the library that every call reuses.  Two
calls in a row with different shapes check that the leftovers of the first call do not leak
into the second.  This file sorts last on purpose, so a run that stops at the first failure
has already been through every other test.
"""
import numpy as np
import pytest

import pd_inputs as gen
from oracle import decoder_layer as L
from gpu_util import assert_close, from_dev, i32_dev, to_dev, empty_bf16

pytestmark = pytest.mark.gpu


def _both(pd, cfg, q, kv_len, cache, cap):
    import torch
    b = len(kv_len)
    width = cfg.n_q_heads * cfg.head_dim
    dq, dlen = to_dev(q), i32_dev(kv_len)
    ws_bytes = pd.pd_decode_attention_workspace_bytes(cfg, b, cap)
    ws = torch.zeros(max(ws_bytes, 256), dtype=torch.uint8, device="cuda")
    ref, got = empty_bf16(b, width), empty_bf16(b, width)
    pd.pd_decode_attention(cfg, dq, width, ref, dlen, b, cap, cache, ws, ws_bytes)
    pd.pd_decode_attention_noalloc(cfg, dq, width, got, dlen, b, cap, cache)
    torch.cuda.synchronize()
    return from_dev(got), from_dev(ref)


def _oracle(hq, hkv, hd, q, k0, v0, kv_len):
    """The oracle's attention core on each sequence: entries 0 .. kv_len[b] of cache slot b."""
    ocfg = L.LayerConfig(d_model=hq * hd, n_q_heads=hq, n_kv_heads=hkv, head_dim=hd, d_ff=64)
    out = np.empty((len(kv_len), hq * hd))
    for b, n in enumerate(kv_len):
        keys = k0[b, :, :n + 1].transpose(1, 0, 2).astype(np.float64)
        vals = v0[b, :, :n + 1].transpose(1, 0, 2).astype(np.float64)
        qb = q[b].reshape(1, hq, hd).astype(np.float64)
        out[b] = L._attend(qb, keys, vals, np.array([n]), np.arange(n + 1), ocfg, None)[0]
    return out


def test_noalloc_matches_workspace_version_twice(pdlib):
    hq, hkv, hd, cap = 32, 8, 128, 2304
    cfg = pdlib.LayerConfig(hq * hd, hq, hkv, hd, 64)
    k0, v0 = gen.kv_cache(21, 4, hkv, cap, hd)
    dk, dv = to_dev(k0), to_dev(v0)
    cache = pdlib.kv_cache_struct(dk, dv, 4, cap)
    # first call: 4 sequences, the KV range is split 4 ways -> the scratch is written
    q1 = gen.normal_bf16(21, gen.S_X, (4, hq * hd), 1.0, sub=1)
    got1, ref1 = _both(pdlib, cfg, q1, [2303, 1500, 700, 5], cache, cap)
    assert_close(got1, ref1, "first call")
    assert_close(got1, _oracle(hq, hkv, hd, q1, k0, v0, [2303, 1500, 700, 5]), "first call against the oracle")
    # second call straight after: other inputs, fewer sequences, a different split count
    q2 = gen.normal_bf16(21, gen.S_X, (2, hq * hd), 1.0, sub=2)
    got2, ref2 = _both(pdlib, cfg, q2, [900, 1023], cache, 1024)
    assert_close(got2, ref2, "second call")
    assert_close(got2, _oracle(hq, hkv, hd, q2, k0, v0, [900, 1023]), "second call against the oracle")
    assert np.abs(ref2).max() > 0.01


def test_noalloc_rejects_oversized_problem(pdlib):
    # 130 sequences of up to 8192 keys get 4 splits each: 130 x 64 heads x 4 x 130 floats = 17.3 MB > the 8 MiB array
    hq, hkv, hd, b, cap = 64, 8, 128, 130, 8192
    cfg = pdlib.LayerConfig(hq * hd, hq, hkv, hd, 64)
    need = pdlib.pd_decode_attention_workspace_bytes(cfg, b, cap)
    assert need > pdlib.NOALLOC_SCRATCH_BYTES
    k = empty_bf16(b, hkv, cap, hd)
    cache = pdlib.kv_cache_struct(k, k, b, cap)
    q, out = empty_bf16(b, hq * hd), empty_bf16(b, hq * hd)
    with pytest.raises(pdlib.PdError) as e:
        pdlib.pd_decode_attention_noalloc(cfg, q, hq * hd, out, i32_dev([cap - 1] * b), b, cap, cache)
    assert e.value.status == pdlib.PD_ERR_WORKSPACE_TOO_SMALL
