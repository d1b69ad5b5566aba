"""GPU: the decode-attention kernel alone against the oracle's attention core."""
import numpy as np
import pytest

import pd_inputs as gen
from oracle import decoder_layer as L
from gpu_util import assert_close, from_dev, i32_dev, to_dev, empty_bf16

pytestmark = pytest.mark.gpu


def oracle_attention(ocfg, q, k0, v0, kv_len):
    out = np.empty((len(kv_len), ocfg.n_q_heads * ocfg.head_dim))
    for b, n in enumerate(kv_len):
        keys = k0[b, :, :n + 1].transpose(1, 0, 2).astype(np.float64)
        vals = v0[b, :, :n + 1].transpose(1, 0, 2).astype(np.float64)
        qb = q[b].reshape(1, ocfg.n_q_heads, ocfg.head_dim).astype(np.float64)
        out[b] = L._attend(qb, keys, vals, np.array([n]), np.arange(n + 1), ocfg, None)[0]
    return out


@pytest.mark.parametrize("hq,hkv,hd,kv_len", [
    (8, 2, 64, [0, 1, 15, 16, 17, 63, 64, 143]),                 # tiny shape: every tail of the 16-key warp tile
    (32, 8, 128, [2047, 1000, 1, 0, 2300, 63, 64, 255, 256, 257]),  # group of 4, ragged, several splits
    (64, 8, 128, [4351, 17, 4100]),                              # group of 8
    (16, 1, 128, [700, 300]),                                    # group of 16: both halves of the MMA rows
])
def test_decode_attention_matches_oracle(pdlib, hq, hkv, hd, kv_len):
    import torch
    b, cap = len(kv_len), max(kv_len) + 1
    ocfg = L.LayerConfig(d_model=hq * hd, n_q_heads=hq, n_kv_heads=hkv, head_dim=hd, d_ff=64)
    cfg = pdlib.LayerConfig(hq * hd, hq, hkv, hd, 64)
    k0, v0 = gen.kv_cache(9, b, hkv, cap, hd)
    q = gen.normal_bf16(9, gen.S_X, (b, hq * hd), 1.0, sub=hd)
    dk, dv = to_dev(k0), to_dev(v0)
    cache = pdlib.kv_cache_struct(dk, dv, b, cap)
    ws_bytes = pdlib.pd_decode_attention_workspace_bytes(cfg, b, cap)
    ws = torch.zeros(max(ws_bytes, 256), dtype=torch.uint8, device="cuda")
    out = empty_bf16(b, hq * hd)
    pdlib.pd_decode_attention(cfg, to_dev(q), hq * hd, out, i32_dev(kv_len), b, cap, cache, ws, ws_bytes)
    torch.cuda.synchronize()
    assert_close(from_dev(out), oracle_attention(ocfg, q, k0, v0, kv_len), "decode attention")


def test_decode_attention_full_size_batch(pdlib):
    """B = 256 over KV length 2149 (the benchmark's launch shape): sampled sequences, run twice for determinism."""
    import torch
    hq, hkv, hd, b, cap = 32, 8, 128, 256, 2304
    ocfg = L.LayerConfig(d_model=hq * hd, n_q_heads=hq, n_kv_heads=hkv, head_dim=hd, d_ff=64)
    cfg = pdlib.LayerConfig(hq * hd, hq, hkv, hd, 64)
    k0, v0 = gen.kv_cache(10, b, hkv, cap, hd)
    q = gen.normal_bf16(10, gen.S_X, (b, hq * hd), 1.0)
    kv_len = [2148] * b
    dk, dv = to_dev(k0), to_dev(v0)
    cache = pdlib.kv_cache_struct(dk, dv, b, cap)
    ws_bytes = pdlib.pd_decode_attention_workspace_bytes(cfg, b, cap)
    ws = torch.zeros(max(ws_bytes, 256), dtype=torch.uint8, device="cuda")
    outs = []
    for _ in range(2):
        out = empty_bf16(b, hq * hd)
        pdlib.pd_decode_attention(cfg, to_dev(q), hq * hd, out, i32_dev(kv_len), b, 2149, cache, ws, ws_bytes)
        torch.cuda.synchronize()
        outs.append(from_dev(out))
    np.testing.assert_array_equal(outs[0], outs[1])
    sel = [0, 1, 100, 255]
    ref = oracle_attention(ocfg, q[sel], k0[sel], v0[sel], [2148] * len(sel))
    assert_close(outs[0][sel], ref, "decode attention B=256")
