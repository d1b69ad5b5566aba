"""GPU: the prefill-attention kernel alone (pd_prefill_attention) against the oracle's attention core,
on request lengths and cached prefixes around every tile boundary of the kernel (128-key tiles, 256-row
blocks).  Cache rows beyond a request's keys hold NaN: they must never reach the output."""
import numpy as np
import pytest

import pd_inputs as gen
from oracle import decoder_layer as L
from gpu_util import assert_close, from_dev, i32_dev, to_dev, empty_bf16

pytestmark = pytest.mark.gpu


def run_case(pd, hq, hkv, hd, lens, prefixes, seed, slots=None):
    import torch
    n_req = len(lens)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    total = int(cu[-1])
    cap = max(p + l for p, l in zip(prefixes, lens)) + 3
    batch_cap = n_req if slots is None else max(slots) + 1
    ocfg = L.LayerConfig(d_model=hq * hd, n_q_heads=hq, n_kv_heads=hkv, head_dim=hd, d_ff=64)
    cfg = pd.LayerConfig(hq * hd, hq, hkv, hd, 64)
    k0, v0 = gen.kv_cache(seed, batch_cap, hkv, cap, hd)
    for r in range(n_req):                       # everything past a request's keys is poison
        s = r if slots is None else slots[r]
        k0[s, :, prefixes[r] + lens[r]:] = np.nan
        v0[s, :, prefixes[r] + lens[r]:] = np.nan
    q = gen.normal_bf16(seed, gen.S_X, (max(total, 1), hq * hd), 1.0, sub=hd)[:total]
    dk, dv = to_dev(k0), to_dev(v0)
    cache = pd.kv_cache_struct(dk, dv, batch_cap, cap)
    out = empty_bf16(max(total, 1), hq * hd)
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    dq = to_dev(q) if total else empty_bf16(1, hq * hd)
    pd.pd_prefill_attention(cfg, dq, hq * hd, out, i32_dev(cu), list(cu), cache,
                            prefix_dev=i32_dev(prefixes), prefix_host=list(prefixes),
                            slots_dev=None if slots is None else i32_dev(slots), err_word=err)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    got = from_dev(out)[:total]
    for r in range(n_req):
        lo, hi, pre = int(cu[r]), int(cu[r + 1]), prefixes[r]
        if hi == lo:
            continue
        s = r if slots is None else slots[r]
        keys = k0[s, :, :pre + hi - lo].transpose(1, 0, 2).astype(np.float64)
        vals = v0[s, :, :pre + hi - lo].transpose(1, 0, 2).astype(np.float64)
        qr = q[lo:hi].reshape(hi - lo, hq, hd).astype(np.float64)
        ref = L._attend(qr, keys, vals, pre + np.arange(hi - lo), np.arange(pre + hi - lo), ocfg, None)
        assert_close(got[lo:hi], ref, f"request {r} (len {hi - lo}, prefix {pre})")


@pytest.mark.parametrize("prefix", [0, 17, 128])
def test_tile_boundary_lengths_tiny_heads(pdlib, prefix):
    lens = [1, 127, 128, 129, 255, 257, 1000]
    run_case(pdlib, 8, 2, 64, lens, [prefix] * len(lens), seed=40 + prefix)


def test_head_dim_128_group_of_four_mixed_prefixes_and_slots(pdlib):
    lens = [1, 129, 0, 257, 1000, 128]
    run_case(pdlib, 32, 8, 128, lens, [128, 0, 5, 17, 300, 127], seed=44, slots=[3, 0, 5, 1, 2, 4])


def test_group_of_eight_long_request(pdlib):
    run_case(pdlib, 64, 8, 128, [2500], [0], seed=45)


def test_argument_errors(pdlib):
    cfg = pdlib.LayerConfig(512, 8, 2, 64, 64)
    k = empty_bf16(1, 2, 16, 64)
    cache = pdlib.kv_cache_struct(k, k, 1, 16)
    q = empty_bf16(16, 512)
    with pytest.raises(pdlib.PdError) as e:       # prefix + length beyond the cache
        pdlib.pd_prefill_attention(cfg, q, 512, q, i32_dev([0, 10]), [0, 10], cache, prefix_dev=i32_dev([7]), prefix_host=[7])
    assert e.value.status == pdlib.PD_ERR_INVALID_ARG
    with pytest.raises(pdlib.PdError) as e:       # row pitch narrower than the heads
        pdlib.pd_prefill_attention(cfg, q, 256, q, i32_dev([0, 10]), [0, 10], cache)
    assert e.value.status == pdlib.PD_ERR_INVALID_ARG
