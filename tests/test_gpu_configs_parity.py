"""GPU parity at the sizes and through the code paths the benchmark configurations run: long requests of the
long-input configuration (8192 and 32768 tokens), decode batches above 256 of the decode-heavy configuration
(ragged KV lengths 512-2560), the 70B-shaped layer at L_in 4096 and at batch 128 over the mixed workload's ragged
KV lengths, and the two stack calls (the path the benchmark times) over two 8B-shaped layers.  Sampled rows /
sequences against the oracle, as in test_gpu_layer.py; the unit-scale intermediates q and attention output are
held to the literal bound as well."""
import numpy as np
import pytest

import pd_inputs as gen
from oracle import decoder_layer as L
from gpu_util import (DeviceLayer, assert_close, assert_parity, assert_stages, big_cache, from_dev, i32_dev,
                      literal_outliers, read_ws_rows, store_bf16, to_dev, empty_bf16)

pytestmark = pytest.mark.gpu

M8B = dict(d_model=4096, n_q_heads=32, n_kv_heads=8, head_dim=128, d_ff=14336)
M70B = dict(d_model=8192, n_q_heads=64, n_kv_heads=8, head_dim=128, d_ff=28672)


def _layer(pd, shape, max_pos, max_tokens, max_batch, max_kv_len, seed, layer=0):
    w = gen.layer_weights(**shape, seed=seed, layer=layer)
    dl = DeviceLayer(pd, pd.LayerConfig(**shape, max_pos=max_pos), w, max_tokens, max_batch, max_kv_len)
    return L.LayerConfig(**shape), L.LayerWeights(**w), dl


def _prefill_sampled(pd, shape, ocfg, ow, dl, x, cu, rows, what, cache_samples):
    """pd_prefill_layer on (x, cu); sampled rows against the exact and the storage-rounded oracle, q and the
    attention output against the exact oracle, and cache entries at `cache_samples` = [(request, positions)]."""
    import torch
    n_req, total = len(cu) - 1, int(cu[-1])
    len_cap = int(np.max(np.diff(cu)))
    k, v, cache = dl.make_cache(n_req, len_cap)
    dout = empty_bf16(total, shape["d_model"])
    pd.pd_prefill_layer(dl.layer, to_dev(x), dout, i32_dev(cu), [int(c) for c in cu], cache, dl.ws, dl.ws_bytes)
    pd.pd_layer_check(dl.layer)
    torch.cuda.synchronize()
    rows_t = torch.as_tensor(rows, device="cuda")
    out = from_dev(dout[rows_t].contiguous())
    stages, stages_s = {}, {}
    ref, kr, vr = L.prefill_layer(ocfg, ow, x, cu, rows=rows, stages=stages)
    ref_s, _, _ = L.prefill_layer(ocfg, ow, x, cu, rows=rows, store=store_bf16, stages=stages_s)
    assert_parity(out, ref, ref_s, what)
    hq_w = shape["n_q_heads"] * shape["head_dim"]
    assert_stages(pd, dl, total, rows, stages, stages_s, hq_w, ocfg.n_qkv, what)
    for r, positions in cache_samples:
        pos = np.asarray(positions)
        idx = torch.as_tensor(pos, device="cuda")
        kd = from_dev(k[r][:, idx].contiguous()).transpose(1, 0, 2)
        vd = from_dev(v[r][:, idx].contiguous()).transpose(1, 0, 2)
        assert_close(kd, kr[int(cu[r]) + pos], f"{what}: K cache of request {r}")
        assert_close(vd, vr[int(cu[r]) + pos], f"{what}: V cache of request {r}")
    n_out, n_all = literal_outliers(out, ref)
    print(f"{what}: {n_out} of {n_all} output elements outside the literal bound against the exact oracle")


# ------------------------------------------------------------- configuration 3: long inputs
def test_8b_long_requests_8192_and_32768(pdlib):
    lens = [8192, 32768]
    cu = np.array([0, 8192, 8192 + 32768], dtype=np.int32)
    total = int(cu[-1])
    ocfg, ow, dl = _layer(pdlib, M8B, 33024, total, 0, 0, seed=50)
    x = gen.activations(50, total, 4096)
    near = lambda c: [c - 129, c - 1, c, c + 1, c + 127]
    picks = [0, 1, 8190, 8191] + [8192 + p for p in [0, 1] + near(4096) + near(16384) + [32766, 32767]]
    rnd = [int(r) for r in gen.uniform_lengths(50, 16, 0, total - 1, sub=9)]
    rows = np.array(sorted(set(picks) | set(rnd)), dtype=np.int64)
    _prefill_sampled(pdlib, M8B, ocfg, ow, dl, x, cu, rows, "8B L_in 8192 + 32768",
                     [(0, [0, 4095, 4096, 8191]), (1, [0, 4095, 4096, 4097, 16383, 16384, 32766, 32767])])


# ------------------------------------------------------ configuration 4: decode batches above 256
@pytest.mark.parametrize("b", [384, 512])
def test_8b_decode_wide_batch_ragged_kv(pdlib, b):
    import torch
    cap = 2561
    sel = [0, 100, 255, 256, 257, b - 1]
    ocfg, ow, dl = _layer(pdlib, M8B, 2561, 0, b, cap, seed=51, layer=b)
    kv_len = [int(v) for v in gen.uniform_lengths(51, b, 512, 2559, sub=b)]
    kv_len[0], kv_len[b - 1] = 2559, 512
    k, v, k_sel, v_sel = big_cache(51 + b, b, 8, cap, 128, sel)
    cache = pdlib.kv_cache_struct(k, v, b, cap)
    x = gen.activations(51, b, 4096, sub=b)
    dout = empty_bf16(b, 4096)
    pdlib.pd_decode_layer(dl.layer, to_dev(x), dout, i32_dev(kv_len), b, max(kv_len) + 1, cache, dl.ws, dl.ws_bytes)
    pdlib.pd_layer_check(dl.layer)
    torch.cuda.synchronize()
    got = from_dev(dout)
    assert np.all(np.isfinite(got))
    lens_sel = [kv_len[s] for s in sel]
    stages, stages_s = {}, {}
    ok, ov = k_sel.astype(np.float64), v_sel.astype(np.float64)
    ref = L.decode_layer(ocfg, ow, x[sel], lens_sel, ok, ov, stages=stages)
    ref_s = L.decode_layer(ocfg, ow, x[sel], lens_sel, k_sel.astype(np.float64), v_sel.astype(np.float64), store=store_bf16,
                           stages=stages_s)
    assert_parity(got[sel], ref, ref_s, f"8B decode B={b}")
    assert_stages(pdlib, dl, b, sel, stages, stages_s, 4096, ocfg.n_qkv, f"8B decode B={b}")
    for j, s in enumerate(sel):                      # the appended entries
        n = kv_len[s]
        assert_close(from_dev(k[s, :, n].contiguous()), ok[j, :, n], "appended K")
        assert_close(from_dev(v[s, :, n].contiguous()), ov[j, :, n], "appended V")
        np.testing.assert_array_equal(from_dev(k[s, :, :n].contiguous()), k_sel[j, :, :n])


# ----------------------------------------------------------------- configuration 5: 70B shape
def test_70b_prefill_4096_and_decode_128_ragged_mix(pdlib):
    import torch
    # the mixed workload's stationary decode batch: L_in ~ U[1024, 8192] plus a uniform share of L_out ~ U[128, 1024]
    l_in = gen.uniform_lengths(3, 512, 1024, 8192, sub=0)
    l_out = gen.uniform_lengths(3, 512, 128, 1024, sub=1)
    prog = gen.uniform_lengths(3, 512, 0, 10**6, sub=2) / 1e6
    b = 128
    kv_len = [int(t) for t in (l_in + np.floor(prog * l_out)).astype(np.int32)[:b]]
    cap = 9216 + 16
    ocfg, ow, dl = _layer(pdlib, M70B, cap, 4096, b, cap, seed=52)
    # prefill, one request of 4096 tokens
    cu = np.array([0, 4096], dtype=np.int32)
    x = gen.activations(52, 4096, 8192)
    rows = gen.sample_rows(52, cu, n_random=10)
    rows = np.array(sorted(set([0, 1, 127, 128, 129, 2047, 2048, 4094, 4095]) | set(int(r) for r in rows[::3])), dtype=np.int64)
    _prefill_sampled(pdlib, M70B, ocfg, ow, dl, x, cu, rows, "70B L_in 4096", [(0, [0, 127, 128, 2048, 4095])])
    # decode, B = 128 over the ragged mix
    longest, shortest = int(np.argmax(kv_len)), int(np.argmin(kv_len))
    sel = sorted({0, 63, 64, 127, longest, shortest})
    k, v, k_sel, v_sel = big_cache(53, b, 8, cap, 128, sel)
    cache = pdlib.kv_cache_struct(k, v, b, cap)
    xs = gen.activations(52, b, 8192, sub=1)
    dout = empty_bf16(b, 8192)
    pdlib.pd_decode_layer(dl.layer, to_dev(xs), dout, i32_dev(kv_len), b, max(kv_len) + 1, cache, dl.ws, dl.ws_bytes)
    pdlib.pd_layer_check(dl.layer)
    torch.cuda.synchronize()
    got = from_dev(dout)
    assert np.all(np.isfinite(got))
    lens_sel = [kv_len[s] for s in sel]
    stages, stages_s = {}, {}
    ref = L.decode_layer(ocfg, ow, xs[sel], lens_sel, k_sel.astype(np.float64), v_sel.astype(np.float64), stages=stages)
    ref_s = L.decode_layer(ocfg, ow, xs[sel], lens_sel, k_sel.astype(np.float64), v_sel.astype(np.float64), store=store_bf16,
                           stages=stages_s)
    assert_parity(got[sel], ref, ref_s, "70B decode B=128 ragged")
    assert_stages(pdlib, dl, b, sel, stages, stages_s, 8192, ocfg.n_qkv, "70B decode B=128 ragged")


# ------------------------------------------------ the stack calls at the benchmark's launch shapes
def test_8b_prefill_stack_two_layers_4096(pdlib):
    """pd_prefill_stack (what the benchmark times): layer 0 alone, then layers 0 + 1; each layer against the oracle
    on the input the GPU gave it."""
    import torch
    cu = [0, 4096]
    ocfg, ow0, dl0 = _layer(pdlib, M8B, 4096, 4096, 0, 0, seed=54, layer=0)
    _, ow1, dl1 = _layer(pdlib, M8B, 4096, 4096, 0, 0, seed=54, layer=1)
    x = gen.activations(54, 4096, 4096)
    caches = [dl0.make_cache(1, 4096), dl1.make_cache(1, 4096)]
    cs = [c[2] for c in caches]
    dx = to_dev(x)
    out1, out2 = empty_bf16(4096, 4096), empty_bf16(4096, 4096)
    pdlib.pd_prefill_stack([dl0.layer], cs[:1], dx, out1, False, i32_dev(cu), cu, dl0.ws, dl0.ws_bytes)
    pdlib.pd_prefill_stack([dl0.layer, dl1.layer], cs, dx, out2, False, i32_dev(cu), cu, dl0.ws, dl0.ws_bytes)
    pdlib.pd_layer_check(dl0.layer); pdlib.pd_layer_check(dl1.layer)
    torch.cuda.synchronize()
    mid, fin = from_dev(out1), from_dev(out2)
    rows = gen.sample_rows(54, cu, n_random=24)
    for name, ow, xin, got in (("layer 0", ow0, x, mid), ("layer 1", ow1, mid, fin)):
        ref, _, _ = L.prefill_layer(ocfg, ow, xin, cu, rows=rows)
        ref_s, _, _ = L.prefill_layer(ocfg, ow, xin, cu, rows=rows, store=store_bf16)
        assert_parity(got[rows], ref, ref_s, f"8B prefill stack, {name}")


def test_8b_decode_stack_two_layers_batch_256(pdlib):
    """pd_decode_stack at B = 256 (the next layer's first RMSNorm fused into the previous layer's last kernel):
    layer 0 alone, then layers 0 + 1; each layer against the oracle on the input the GPU gave it."""
    import torch
    b, cap, t = 256, 2304, 77
    sel = [0, 1, 127, 128, 200, 255]
    ocfg, ow0, dl0 = _layer(pdlib, M8B, 4096, 0, b, cap, seed=55, layer=0)
    _, ow1, dl1 = _layer(pdlib, M8B, 4096, 0, b, cap, seed=55, layer=1)
    kv_len = [2048 + t] * b
    k0, v0, k0s, v0s = big_cache(56, b, 8, cap, 128, sel)
    k1, v1, k1s, v1s = big_cache(57, b, 8, cap, 128, sel)
    cs = [pdlib.kv_cache_struct(k0, v0, b, cap), pdlib.kv_cache_struct(k1, v1, b, cap)]
    x = gen.activations(55, b, 4096)
    dx, dkv = to_dev(x), i32_dev(kv_len)
    out1, out2 = empty_bf16(b, 4096), empty_bf16(b, 4096)
    pdlib.pd_decode_stack([dl0.layer], cs[:1], dx, out1, False, dkv, b, 2048 + t + 1, dl0.ws, dl0.ws_bytes)
    pdlib.pd_decode_stack([dl0.layer, dl1.layer], cs, dx, out2, False, dkv, b, 2048 + t + 1, dl0.ws, dl0.ws_bytes)
    pdlib.pd_layer_check(dl0.layer); pdlib.pd_layer_check(dl1.layer)
    torch.cuda.synchronize()
    mid, fin = from_dev(out1), from_dev(out2)
    lens_sel = [kv_len[s] for s in sel]
    for name, ow, xin, got, ks, vs in (("layer 0", ow0, x, mid, k0s, v0s), ("layer 1", ow1, mid, fin, k1s, v1s)):
        ref = L.decode_layer(ocfg, ow, xin[sel], lens_sel, ks.astype(np.float64), vs.astype(np.float64))
        ref_s = L.decode_layer(ocfg, ow, xin[sel], lens_sel, ks.astype(np.float64), vs.astype(np.float64), store=store_bf16)
        assert_parity(got[sel], ref, ref_s, f"8B decode stack B=256, {name}")
    # host-I/O variant of the same call: identical up to the order of the K-split reductions
    xh = torch.from_numpy(gen.to_bf16_bits(x).view(np.int16)).pin_memory()
    oh = torch.zeros_like(xh).pin_memory()
    kvh = np.asarray(kv_len, dtype=np.int32)
    pdlib.pd_decode_stack([dl0.layer, dl1.layer], cs, xh, oh, True, kvh, b, 2048 + t + 1, dl0.ws, dl0.ws_bytes)
    host = gen.from_bf16_bits(oh.numpy().view(np.uint16))
    assert np.all(np.abs(host - fin) <= 2e-2 * 3 + 2e-2 * np.abs(fin))
