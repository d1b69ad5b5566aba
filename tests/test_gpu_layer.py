"""GPU parity: the CUDA layer (through the C ABI) against the CPU oracle on the same
seeded inputs, element by element, within |gpu - ref| <= 2e-2 + 2e-2 |ref|."""
import numpy as np
import pytest

import pd_inputs as gen
from oracle import decoder_layer as L
from gpu_util import DeviceLayer, assert_close, assert_parity, from_dev, i32_dev, store_bf16, to_dev, empty_bf16

pytestmark = pytest.mark.gpu

TINY = dict(d_model=512, n_q_heads=8, n_kv_heads=2, head_dim=64, d_ff=1536)
M8B = dict(d_model=4096, n_q_heads=32, n_kv_heads=8, head_dim=128, d_ff=14336)
M70B = dict(d_model=8192, n_q_heads=64, n_kv_heads=8, head_dim=128, d_ff=28672)


def setup(pd, shape, max_pos, max_tokens, max_batch, max_kv_len, seed=0, layer=0):
    w = gen.layer_weights(**shape, seed=seed, layer=layer)
    ocfg = L.LayerConfig(**shape)
    cfg = pd.LayerConfig(**shape, max_pos=max_pos)
    dl = DeviceLayer(pd, cfg, w, max_tokens, max_batch, max_kv_len)
    return ocfg, L.LayerWeights(**w), dl


def run_prefill(pd, dl, x, cu, slots=None, batch_cap=None, len_cap=None):
    import torch
    n_req = len(cu) - 1
    batch_cap = batch_cap or max(n_req, 1)
    len_cap = len_cap or max(int(np.max(np.diff(cu))), 1)
    k, v, cache = dl.make_cache(batch_cap, len_cap)
    dx, dout = to_dev(x), empty_bf16(*x.shape)
    pd.pd_prefill_layer(dl.layer, dx, dout, i32_dev(cu), list(cu), cache, dl.ws, dl.ws_bytes,
                        slots_dev=None if slots is None else i32_dev(slots))
    pd.pd_layer_check(dl.layer)
    torch.cuda.synchronize()
    return from_dev(dout), from_dev(k), from_dev(v)


def check_cache(k_dev, v_dev, k_ref, v_ref, cu, slots=None):
    """Device cache [slot, Hkv, pos, hd] against oracle k, v [T, Hkv, hd]."""
    for r in range(len(cu) - 1):
        lo, hi = int(cu[r]), int(cu[r + 1])
        s = r if slots is None else int(slots[r])
        assert_close(k_dev[s, :, :hi - lo].transpose(1, 0, 2), k_ref[lo:hi], f"K cache of request {r}")
        assert_close(v_dev[s, :, :hi - lo].transpose(1, 0, 2), v_ref[lo:hi], f"V cache of request {r}")


# ------------------------------------------------------------------ tiny config
def test_tiny_prefill_all_rows(pdlib):
    ocfg, ow, dl = setup(pdlib, TINY, 256, 128, 4, 144)
    x = gen.activations(0, 128, 512)
    cu = [0, 128]
    out, k, v = run_prefill(pdlib, dl, x, cu)
    ref, kr, vr = L.prefill_layer(ocfg, ow, x, cu)
    assert_close(out, ref, "tiny prefill")
    check_cache(k, v, kr, vr, cu)


def test_tiny_ragged_packed_batch_with_slots(pdlib):
    lens = [37, 128, 1, 200, 0, 129]
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    slots = [5, 0, 3, 1, 2, 4]
    ocfg, ow, dl = setup(pdlib, TINY, 256, int(cu[-1]), 0, 0)
    x = gen.activations(1, int(cu[-1]), 512)
    out, k, v = run_prefill(pdlib, dl, x, cu, slots=slots, batch_cap=6, len_cap=203)
    ref, kr, vr = L.prefill_layer(ocfg, ow, x, cu)
    assert_close(out, ref, "ragged prefill")
    check_cache(k, v, kr, vr, cu, slots)


def test_tiny_prefill_then_16_decode_steps(pdlib):
    """Config 1: four requests of 128 tokens fill the cache, then 16 decode steps at batch 4."""
    import torch
    b, l0, steps = 4, 128, 16
    ocfg, ow, dl = setup(pdlib, TINY, 256, b * l0, b, l0 + steps)
    cu = [i * l0 for i in range(b + 1)]
    x = gen.activations(0, b * l0, 512)
    k, v, cache = dl.make_cache(b, l0 + steps)
    dout = empty_bf16(b * l0, 512)
    pdlib.pd_prefill_layer(dl.layer, to_dev(x), dout, i32_dev(cu), cu, cache, dl.ws, dl.ws_bytes)
    ref, kr, vr = L.prefill_layer(ocfg, ow, x, cu)
    assert_close(from_dev(dout), ref, "prefill of the decode test")
    ok = np.zeros((b, 2, l0 + steps, 64))
    ov = np.zeros_like(ok)
    for r in range(b):
        ok[r, :, :l0] = kr[r * l0:(r + 1) * l0].transpose(1, 0, 2)
        ov[r, :, :l0] = vr[r * l0:(r + 1) * l0].transpose(1, 0, 2)
    dstep = empty_bf16(b, 512)
    for t in range(steps):
        xs = gen.activations(0, b, 512, sub=t, stream=gen.S_XSTEP)
        kv_len = [l0 + t] * b
        pdlib.pd_decode_layer(dl.layer, to_dev(xs), dstep, i32_dev(kv_len), b, l0 + t + 1, cache, dl.ws, dl.ws_bytes)
        pdlib.pd_layer_check(dl.layer)
        ref_t = L.decode_layer(ocfg, ow, xs, kv_len, ok, ov)
        assert_close(from_dev(dstep), ref_t, f"decode step {t}")
    torch.cuda.synchronize()
    assert_close(from_dev(k), ok, "K cache after decode")
    assert_close(from_dev(v), ov, "V cache after decode")


def test_tiny_decode_equals_prefill_row_on_gpu(pdlib):
    ocfg, ow, dl = setup(pdlib, TINY, 256, 96, 1, 96)
    ln = 96
    x = gen.activations(2, ln, 512)
    out, k, v = run_prefill(pdlib, dl, x, [0, ln])
    for t in (0, 1, 47, 95):
        kc, vc, cache = dl.make_cache(1, ln, k_np=k, v_np=v)      # prefix of the prefill's own cache
        dstep = empty_bf16(1, 512)
        pdlib.pd_decode_layer(dl.layer, to_dev(x[t:t + 1]), dstep, i32_dev([t]), 1, t + 1, cache, dl.ws, dl.ws_bytes)
        got = from_dev(dstep)[0]
        # both are bf16 results of the same math in a different order: a few bf16 ulps apart
        assert np.all(np.abs(got - out[t]) <= 2e-2 + 2e-2 * np.abs(out[t]))


@pytest.mark.parametrize("b", [17, 100, 300])
def test_tiny_decode_batch_sizes_span_every_skinny_tile(pdlib, b):
    """Decode batches that fall into the 32-, 128- and (two) 256-wide batch tiles of the projection kernel."""
    cap = 48
    ocfg, ow, dl = setup(pdlib, TINY, 64, 0, b, cap)
    k0, v0 = gen.kv_cache(11, b, 2, cap, 64)
    k, v, cache = dl.make_cache(b, cap, k0, v0)
    x = gen.activations(11, b, 512, sub=b)
    kv_len = [int(v_) for v_ in gen.uniform_lengths(11, b, 0, cap - 1, sub=b)]
    dout = empty_bf16(b, 512)
    pdlib.pd_decode_layer(dl.layer, to_dev(x), dout, i32_dev(kv_len), b, max(kv_len) + 1, cache, dl.ws, dl.ws_bytes)
    pdlib.pd_layer_check(dl.layer)
    ref = L.decode_layer(ocfg, ow, x, kv_len, k0.astype(np.float64), v0.astype(np.float64))
    assert_close(from_dev(dout), ref, f"tiny decode B={b}")


def _run_chunks(pd, dl, ocfg, ow, x, lens, bounds, cap, what, parity=None):
    """Feeds every request in chunks (bounds[r] = chunk boundaries) through pd_prefill_chunk_layer and the
    oracle's extend_layer, comparing chunk by chunk; returns the GPU output assembled in request order."""
    import torch
    cu = np.concatenate([[0], np.cumsum(lens)])
    n_req = len(lens)
    k, v, cache = dl.make_cache(n_req, cap)
    hkv, hd = ocfg.n_kv_heads, ocfg.head_dim
    ok = np.zeros((n_req, hkv, cap, hd)); ov = np.zeros_like(ok)
    oks, ovs = ok.copy(), ov.copy()
    out = np.zeros((int(cu[-1]), ocfg.d_model), dtype=np.float32)
    for step in range(max(len(b) for b in bounds) - 1):
        rows, cu_c, pre = [], [0], []
        for r in range(n_req):
            b = bounds[r]
            lo, hi = (b[step], b[step + 1]) if step + 1 < len(b) else (b[-1], b[-1])
            rows += list(range(int(cu[r]) + lo, int(cu[r]) + hi))
            cu_c.append(cu_c[-1] + hi - lo)
            pre.append(lo)
        if not rows:
            continue
        xc = x[rows]
        dout = empty_bf16(len(rows), ocfg.d_model)
        pd.pd_prefill_chunk_layer(dl.layer, to_dev(xc), dout, i32_dev(cu_c), cu_c, i32_dev(pre), pre, cache, dl.ws,
                                  dl.ws_bytes)
        pd.pd_layer_check(dl.layer)
        got = from_dev(dout)
        ref = L.extend_layer(ocfg, ow, xc, cu_c, pre, ok, ov)
        if parity is None:
            assert_close(got, ref, f"{what} chunk step {step}")
        else:
            ref_s = L.extend_layer(ocfg, ow, xc, cu_c, pre, oks, ovs, store=store_bf16)
            assert_parity(got, ref, ref_s, f"{what} chunk step {step}")
        out[rows] = got
    torch.cuda.synchronize()
    return out, from_dev(k), from_dev(v), ok, ov


def test_tiny_chunked_prefill_matches_oracle_and_full_prefill(pdlib):
    lens = [300, 129, 40]
    bounds = [[0, 17, 128, 200, 300], [0, 128, 129], [0, 40]]      # ragged chunks, prefixes off the 128-key tiles
    ocfg, ow, dl = setup(pdlib, TINY, 512, sum(lens), 0, 0)
    x = gen.activations(12, sum(lens), 512)
    out, k, v, ok, ov = _run_chunks(pdlib, dl, ocfg, ow, x, lens, bounds, 320, "tiny")
    for r, ln in enumerate(lens):
        assert_close(k[r, :, :ln], ok[r, :, :ln], "K cache after chunks")
        assert_close(v[r, :, :ln], ov[r, :, :ln], "V cache after chunks")
    # the whole requests in one go give the same rows (bf16 results of the same math in another order)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    full, _, _ = run_prefill(pdlib, dl, x, cu, batch_cap=3, len_cap=320)
    assert np.all(np.abs(out - full) <= 2e-2 + 2e-2 * np.abs(full))


def test_8b_chunked_prefill_two_chunks(pdlib):
    lens = [700]
    ocfg, ow, dl = setup(pdlib, M8B, 1024, 700, 0, 0, layer=3)
    x = gen.activations(13, 700, 4096)
    _run_chunks(pdlib, dl, ocfg, ow, x, lens, [[0, 300, 700]], 768, "8B", parity=True)


def test_two_layer_stack_matches_chained_oracle(pdlib):
    import torch
    ocfg, ow0, dl0 = setup(pdlib, TINY, 256, 160, 0, 0, layer=0)
    _, ow1, dl1 = setup(pdlib, TINY, 256, 160, 0, 0, layer=1)
    cu = [0, 100, 160]
    x = gen.activations(3, 160, 512)
    caches = [dl0.make_cache(2, 100), dl1.make_cache(2, 100)]
    dout = empty_bf16(160, 512)
    pdlib.pd_prefill_stack([dl0.layer, dl1.layer], [c[2] for c in caches], to_dev(x), dout, False, i32_dev(cu), cu,
                           dl0.ws, dl0.ws_bytes)
    torch.cuda.synchronize()
    r0, _, _ = L.prefill_layer(ocfg, ow0, x, cu)
    r1, _, _ = L.prefill_layer(ocfg, ow1, r0, cu)
    assert_close(from_dev(dout), r1, "two-layer stack")
    # host-I/O variant: same result through pinned host buffers
    xh = torch.from_numpy(gen.to_bf16_bits(x).view(np.int16)).pin_memory()
    oh = torch.zeros_like(xh).pin_memory()
    pdlib.pd_prefill_stack([dl0.layer, dl1.layer], [c[2] for c in caches], xh, oh, True, None, cu, dl0.ws, dl0.ws_bytes)
    np.testing.assert_array_equal(oh.numpy(), dout.cpu().numpy())


@pytest.mark.parametrize("fp8_mode", [False, True])
@pytest.mark.parametrize("b", [5, 70])
def test_three_layer_decode_stack_matches_chained_oracle(pdlib, b, fp8_mode):
    """pd_decode_stack over three layers (the first RMSNorm of layers 1 and 2 runs inside the previous layer's
    last row-wise kernel) against the oracle's layers chained, and against three pd_decode_layer calls."""
    import torch
    from oracle import fp8 as ofp8
    cap = 40
    ws_, ocfgs, ows, dls, pjs = [], [], [], [], []
    for i in range(3):
        w = gen.layer_weights(**TINY, seed=4, layer=i)
        cfg = pdlib.LayerConfig(**TINY, max_pos=64, fp8_projections=fp8_mode)
        dls.append(DeviceLayer(pdlib, cfg, w, 0, b, cap))
        ows.append(L.LayerWeights(**w))
        pjs.append(ofp8.Fp8Projector(ows[-1]) if fp8_mode else None)
    ocfg = L.LayerConfig(**TINY)
    kv_len = [int(v_) for v_ in gen.uniform_lengths(31, b, 0, cap - 1, sub=b)]
    x = gen.activations(31, b, 512, sub=b)
    k0s, v0s, caches_a, caches_b, keep = [], [], [], [], []
    for i in range(3):
        k0, v0 = gen.kv_cache(31 + i, b, 2, cap, 64)
        k0s.append(k0); v0s.append(v0)
        for lst in (caches_a, caches_b):
            k, v, c = dls[i].make_cache(b, cap, k0, v0)
            keep += [k, v]; lst.append(c)
    dout = empty_bf16(b, 512)
    pdlib.pd_decode_stack([d.layer for d in dls], caches_a, to_dev(x), dout, False, i32_dev(kv_len), b,
                          max(kv_len) + 1, dls[0].ws, dls[0].ws_bytes)
    for d in dls:
        pdlib.pd_layer_check(d.layer)
    torch.cuda.synchronize()
    got = from_dev(dout)
    # layer by layer through pd_decode_layer, each layer checked against the oracle on the input the GPU gave it
    # (with FP8 projections an end-to-end bar over several layers is not meaningful: one flipped code in layer 0
    # is a different input for layer 1)
    cur_np, cur = x, to_dev(x)
    chained = x
    for i in range(3):
        nxt = empty_bf16(b, 512)
        pdlib.pd_decode_layer(dls[i].layer, cur, nxt, i32_dev(kv_len), b, max(kv_len) + 1, caches_b[i], dls[i].ws,
                              dls[i].ws_bytes)
        torch.cuda.synchronize()
        kw = dict(store=store_bf16, proj=pjs[i]) if fp8_mode else {}
        ref_i = L.decode_layer(ocfg, ows[i], cur_np, kv_len, k0s[i].astype(np.float64), v0s[i].astype(np.float64), **kw)
        assert_close(from_dev(nxt), ref_i, f"layer {i} of the chain")
        if not fp8_mode:
            chained = L.decode_layer(ocfg, ows[i], chained, kv_len, k0s[i].astype(np.float64),
                                     v0s[i].astype(np.float64))
        cur, cur_np = nxt, from_dev(nxt)
    one_by_one = cur_np
    # the stack call computes the same values up to the order of the sum of squares in the fused RMSNorm
    assert_close(got, one_by_one, "three-layer decode stack against the layer-by-layer calls", atol=3e-2)
    if not fp8_mode:
        assert_close(got, chained, "three-layer decode stack against the chained oracle")
    # the appended K/V rows of the last layer agree as well
    for s_ in (0, b - 1):
        np.testing.assert_allclose(from_dev(keep[4 * 2])[s_, :, kv_len[s_]], from_dev(keep[4 * 2 + 2])[s_, :, kv_len[s_]],
                                   rtol=2e-2, atol=2e-2)


def test_argument_errors(pdlib):
    ocfg, ow, dl = setup(pdlib, TINY, 64, 64, 2, 64)
    k, v, cache = dl.make_cache(2, 64)
    x = empty_bf16(64, 512)
    with pytest.raises(pdlib.PdError) as e:        # non-monotone cu_seqlens
        pdlib.pd_prefill_layer(dl.layer, x, x, i32_dev([0, 40, 30]), [0, 40, 30], cache, dl.ws, dl.ws_bytes)
    assert e.value.status == pdlib.PD_ERR_INVALID_ARG
    with pytest.raises(pdlib.PdError) as e:        # request longer than the cache
        pdlib.pd_prefill_layer(dl.layer, x, x, i32_dev([0, 65]), [0, 65], cache, dl.ws, dl.ws_bytes)
    assert e.value.status == pdlib.PD_ERR_INVALID_ARG
    with pytest.raises(pdlib.PdError) as e:        # workspace too small
        pdlib.pd_prefill_layer(dl.layer, x, x, i32_dev([0, 64]), [0, 64], cache, dl.ws, 1024)
    assert e.value.status == pdlib.PD_ERR_WORKSPACE_TOO_SMALL
    with pytest.raises(pdlib.PdError) as e:        # batch beyond the cache
        pdlib.pd_decode_layer(dl.layer, x, x, i32_dev([0, 0, 0]), 3, 1, cache, dl.ws, dl.ws_bytes)
    assert e.value.status == pdlib.PD_ERR_INVALID_ARG
    # a stack whose layers differ in shape is refused before anything is launched
    wide = dict(TINY, d_ff=3072)
    _, _, dl_wide = setup(pdlib, wide, 64, 64, 2, 64)
    for call in (lambda: pdlib.pd_prefill_stack([dl.layer, dl_wide.layer], [cache], x, x, False, i32_dev([0, 64]), [0, 64],
                                                dl.ws, dl.ws_bytes),
                 lambda: pdlib.pd_decode_stack([dl.layer, dl_wide.layer], [cache], x, x, False, i32_dev([3, 3]), 2, 4,
                                               dl.ws, dl.ws_bytes)):
        with pytest.raises(pdlib.PdError) as e:
            call()
        assert e.value.status == pdlib.PD_ERR_INVALID_ARG
    # empty inputs are accepted
    pdlib.pd_prefill_layer(dl.layer, x, x, i32_dev([0, 0]), [0, 0], cache, dl.ws, dl.ws_bytes)
    pdlib.pd_decode_layer(dl.layer, x, x, i32_dev([0]), 0, 1, cache, dl.ws, dl.ws_bytes)
    # a kv_len beyond the cache is caught by the kernel and reported, not written
    pdlib.pd_decode_layer(dl.layer, x, x, i32_dev([64, 3]), 2, 64, cache, dl.ws, dl.ws_bytes)
    with pytest.raises(pdlib.PdError) as e:
        pdlib.pd_layer_check(dl.layer)
    assert e.value.status == pdlib.PD_ERR_INVALID_ARG
    pdlib.pd_layer_check(dl.layer)                 # the error word was cleared


# ------------------------------------------------------------ 8B-shaped layer
def test_8b_prefill_ragged_sampled_rows(pdlib):
    lens = [1000, 333]
    cu = [0, 1000, 1333]
    ocfg, ow, dl = setup(pdlib, M8B, 4096, 1333, 0, 0)
    x = gen.activations(4, 1333, 4096)
    out, k, v = run_prefill(pdlib, dl, x, cu)
    rows = gen.sample_rows(4, cu, n_random=40)
    ref, kr, vr = L.prefill_layer(ocfg, ow, x, cu, rows=rows)
    ref_s, _, _ = L.prefill_layer(ocfg, ow, x, cu, rows=rows, store=store_bf16)
    assert_parity(out[rows], ref, ref_s, "8B prefill sampled rows")
    check_cache(k, v, kr, vr, cu)


def test_8b_decode_ragged_kv_lengths(pdlib):
    import torch
    kv_len = [2047, 1000, 1, 0, 2300, 63, 64]
    b, cap = len(kv_len), 2304
    ocfg, ow, dl = setup(pdlib, M8B, 4096, 0, b, cap)
    k0, v0 = gen.kv_cache(5, b, 8, cap, 128)
    k, v, cache = dl.make_cache(b, cap, k0, v0)
    x = gen.activations(5, b, 4096)
    dout = empty_bf16(b, 4096)
    pdlib.pd_decode_layer(dl.layer, to_dev(x), dout, i32_dev(kv_len), b, max(kv_len) + 1, cache, dl.ws, dl.ws_bytes)
    pdlib.pd_layer_check(dl.layer)
    ok, ov = k0.astype(np.float64), v0.astype(np.float64)
    ref = L.decode_layer(ocfg, ow, x, kv_len, ok, ov)
    ref_s = L.decode_layer(ocfg, ow, x, kv_len, k0.astype(np.float64), v0.astype(np.float64), store=store_bf16)
    assert_parity(from_dev(dout), ref, ref_s, "8B decode")
    kd, vd = from_dev(k), from_dev(v)
    for i, n in enumerate(kv_len):                 # appended entries, and nothing else, changed
        assert_close(kd[i, :, n], ok[i, :, n], "appended K")
        assert_close(vd[i, :, n], ov[i, :, n], "appended V")
        np.testing.assert_array_equal(kd[i, :, :n], k0[i, :, :n])
        np.testing.assert_array_equal(kd[i, :, n + 1:], k0[i, :, n + 1:])


def test_8b_full_size_prefill_4096_sampled(pdlib):
    """The benchmark's prefill launch configuration (one request of 4096 tokens), sampled rows."""
    cu = [0, 4096]
    ocfg, ow, dl = setup(pdlib, M8B, 4096, 4096, 0, 0, layer=1)
    x = gen.activations(6, 4096, 4096)
    out, k, v = run_prefill(pdlib, dl, x, cu)
    rows = gen.sample_rows(6, cu, n_random=32)
    ref, kr, vr = L.prefill_layer(ocfg, ow, x, cu, rows=rows)
    ref_s, _, _ = L.prefill_layer(ocfg, ow, x, cu, rows=rows, store=store_bf16)
    assert_parity(out[rows], ref, ref_s, "8B L_in 4096 sampled rows")
    sel = np.arange(0, 4096, 97)
    assert_close(k[0][:, sel].transpose(1, 0, 2), kr[sel], "K cache sample")
    assert_close(v[0][:, sel].transpose(1, 0, 2), vr[sel], "V cache sample")


def test_8b_full_size_decode_batch_256_sampled(pdlib):
    """The benchmark's decode launch configuration (B = 256, KV length 2048 + t), sampled sequences."""
    import torch
    b, cap, t = 256, 2304, 100
    ocfg, ow, dl = setup(pdlib, M8B, 4096, 0, b, cap, layer=2)
    k0, v0 = gen.kv_cache(7, b, 8, cap, 128)
    k, v, cache = dl.make_cache(b, cap, k0, v0)
    x = gen.activations(7, b, 4096)
    kv_len = [2048 + t] * b
    dout = empty_bf16(b, 4096)
    pdlib.pd_decode_layer(dl.layer, to_dev(x), dout, i32_dev(kv_len), b, 2048 + t + 1, cache, dl.ws, dl.ws_bytes)
    pdlib.pd_layer_check(dl.layer)
    got = from_dev(dout)
    sel = [0, 1, 127, 128, 200, 255]
    ref = L.decode_layer(ocfg, ow, x[sel], [2048 + t] * len(sel), k0[sel].astype(np.float64), v0[sel].astype(np.float64))
    ref_s = L.decode_layer(ocfg, ow, x[sel], [2048 + t] * len(sel), k0[sel].astype(np.float64),
                           v0[sel].astype(np.float64), store=store_bf16)
    assert_parity(got[sel], ref, ref_s, "8B decode B=256 sampled sequences")
    assert np.all(np.isfinite(got))


# ----------------------------------------------------------- 70B-shaped layer
def test_70b_prefill_and_decode(pdlib):
    cu = [0, 300]
    kv_len = [4100, 17, 4351]
    ocfg, ow, dl = setup(pdlib, M70B, 8192, 300, 3, 4352)
    x = gen.activations(8, 300, 8192)
    out, k, v = run_prefill(pdlib, dl, x, cu)
    rows = gen.sample_rows(8, cu, n_random=16)
    ref, kr, vr = L.prefill_layer(ocfg, ow, x, cu, rows=rows)
    ref_s, _, _ = L.prefill_layer(ocfg, ow, x, cu, rows=rows, store=store_bf16)
    assert_parity(out[rows], ref, ref_s, "70B prefill sampled rows")
    k0, v0 = gen.kv_cache(8, 3, 8, 4352, 128)
    kc, vc, cache = dl.make_cache(3, 4352, k0, v0)
    xs = gen.activations(8, 3, 8192, sub=1)
    dout = empty_bf16(3, 8192)
    pdlib.pd_decode_layer(dl.layer, to_dev(xs), dout, i32_dev(kv_len), 3, 4352, cache, dl.ws, dl.ws_bytes)
    pdlib.pd_layer_check(dl.layer)
    ref = L.decode_layer(ocfg, ow, xs, kv_len, k0.astype(np.float64), v0.astype(np.float64))
    ref_s = L.decode_layer(ocfg, ow, xs, kv_len, k0.astype(np.float64), v0.astype(np.float64), store=store_bf16)
    assert_parity(from_dev(dout), ref, ref_s, "70B decode")
