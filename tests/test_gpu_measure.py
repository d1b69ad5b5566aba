"""GPU: the measurement harness (pd_measure), the trace calls and the allocation pipeline
fed with measured numbers."""
import numpy as np
import pytest

from oracle import allocation as A

pytestmark = pytest.mark.gpu

TINY = dict(d_model=512, n_q_heads=8, n_kv_heads=2, head_dim=64, d_ff=1536)


def test_measure_tiny_config_and_allocate(pdlib):
    """Config 1: prefill 1 x 128, decode B = 4 for 16 steps on KV length 128, then pd_allocate with
    TP_total 1e4 tok/s, L_in 128, L_out 16, TTFT 1 s, TPOT 50 ms; integers must equal the oracle's
    when both are fed the same measured numbers."""
    cfg = pdlib.LayerConfig(**TINY, max_pos=256)
    m = pdlib.pd_measure(cfg, n_layers_run=1, n_layers_model=1, warmup=2, reps=5, seed=0, l_in=[128],
                         batch_sizes=[1, 2, 4], kv_len_start=128, n_steps=16, step_stride=5,
                         peak_bf16_flops=1.4e15, peak_hbm_bytes_s=6.4e12)
    assert m["prefill_tok_s"] > 0 and m["prefill_time_s"] > 0
    assert m["prefill_flops"] == pytest.approx(2 * 128 * 3.0147e6 + 4 * 8 * 64 * 128 * 129 / 2, rel=1e-3)
    assert m["batch"] == [1, 2, 4] and all(t > 0 for t in m["tpot_s"])
    assert m["gpu_launches"] > 0
    # 4 sequences of 144 tokens fit L2 many times over: the attention-only time is flagged, not reported as an HBM rate
    assert m["attn_l2_resident"] == [1, 1, 1] and m["attn_frac_hbm_peak"] == [0.0, 0.0, 0.0]
    assert all(t > 0 for t in m["attn_time_s"]) and m["decode_kv_ring"] == [1, 1, 1] and m["prefill_kv_ring"] == 1
    args = (1e4, 128.0, 16.0, 1.0, 0.05, m["prefill_tok_s"], m["batch"], m["tpot_s"])
    got = pdlib.pd_allocate(*args)
    ref = A.allocate(*args)
    assert got["status"] == 0 and ref.status == "ok"
    assert (got["feasible_batch"], got["n_prefill"], got["n_decode"], got["n_prefill_ceil"], got["n_decode_ceil"]) == \
           (ref.feasible_batch, ref.n_prefill, ref.n_decode, ref.n_prefill_ceil, ref.n_decode_ceil)
    assert got["tp_decode_eff"] == ref.tp_decode_eff and got["tp_prefill_eff"] == ref.tp_prefill_eff


def test_measure_tiny_fp8_projections(pdlib):
    """The harness with FP8 projections: it builds quantised layers from its own seeded weights and reports
    the same quantities; the FP8 layer must not be slower than a generous multiple of the bf16 one."""
    out = {}
    for fp8 in (False, True):
        cfg = pdlib.LayerConfig(**TINY, max_pos=256, fp8_projections=fp8)
        out[fp8] = pdlib.pd_measure(cfg, n_layers_run=2, n_layers_model=2, warmup=2, reps=5, seed=0, l_in=[128, 100],
                                    batch_sizes=[1, 4], kv_len_start=128, n_steps=8, step_stride=4,
                                    peak_bf16_flops=1.4e15, peak_hbm_bytes_s=6.4e12)
    assert out[True]["prefill_tok_s"] > 0 and all(t > 0 for t in out[True]["tpot_s"])
    assert out[True]["prefill_flops"] == out[False]["prefill_flops"]
    assert out[True]["gpu_launches"] > out[False]["gpu_launches"]          # the quantiser launches
    assert out[True]["prefill_time_s"] < 5 * out[False]["prefill_time_s"]


def test_measure_8b_shape_two_layers_scaled(pdlib):
    """Two 8B-shaped layers scaled to 32: ragged prefill batch, decode sweep with ragged KV lengths;
    TPOT must not decrease with the batch size beyond timing noise."""
    shape = dict(d_model=4096, n_q_heads=32, n_kv_heads=8, head_dim=128, d_ff=14336)
    cfg = pdlib.LayerConfig(**shape, max_pos=4096)
    mix = [2048 - 37 * i for i in range(32)]
    m = pdlib.pd_measure(cfg, n_layers_run=2, n_layers_model=32, warmup=2, reps=5, seed=1, l_in=[1024, 333, 2048],
                         batch_sizes=[1, 8, 32], kv_len_start=2048, n_steps=64, step_stride=32, kv_len_mix=mix,
                         peak_bf16_flops=1.4e15, peak_hbm_bytes_s=6.4e12)
    assert 1e4 < m["prefill_tok_s"] < 5e5
    assert 0.05 < m["prefill_frac_bf16_peak"] < 1.2
    t = m["tpot_s"]
    assert t[2] > 0.9 * t[0]
    assert all(0 < f < 1.3 for f in m["decode_frac_hbm_peak"])
    assert m["decode_bytes"][2] > m["decode_bytes"][0]
    # B = 1 over 2 layers is 2 x 17 MB of K/V (L2-resident: flagged); B = 32 is 2 x 0.5 GB (an HBM figure)
    assert m["attn_l2_resident"] == [1, 1, 0] and 0 < m["attn_frac_hbm_peak"][2] < 1.3


def test_measure_whole_model_step_adds_the_head(pdlib):
    """vocab > 0: the prefill time and every TPOT contain the embedding + final norm + LM head + sampling
    time, which is also reported on its own; the LM head alone must stream the table at a plausible rate."""
    shape = dict(d_model=4096, n_q_heads=32, n_kv_heads=8, head_dim=128, d_ff=14336)
    cfg = pdlib.LayerConfig(**shape, max_pos=1024)
    vocab = 128256
    m = pdlib.pd_measure(cfg, n_layers_run=1, n_layers_model=32, warmup=2, reps=5, seed=2, l_in=[512, 100],
                         batch_sizes=[1, 64], kv_len_start=256, n_steps=2, step_stride=1,
                         peak_bf16_flops=1.4e15, peak_hbm_bytes_s=6.4e12, vocab=vocab)
    table_bytes = vocab * 4096 * 2
    assert 0 < m["prefill_head_s"] < m["prefill_time_s"]
    for tpot, head in zip(m["tpot_s"], m["decode_head_s"]):
        assert 0 < head < tpot
        assert 0.3e12 < table_bytes / head < 8e12          # between 5 % of and just above the HBM rate
    plain = pdlib.pd_measure(cfg, n_layers_run=1, n_layers_model=32, warmup=2, reps=5, seed=2, l_in=[512, 100],
                             batch_sizes=[1, 64], kv_len_start=256, n_steps=2, step_stride=1)
    assert plain["prefill_head_s"] == 0.0 and plain["decode_head_s"] == [0.0, 0.0]
    assert m["prefill_flops"] > plain["prefill_flops"]


def test_trace_reports_every_kernel_class(pdlib):
    import torch
    import pd_inputs as gen
    from gpu_util import DeviceLayer, to_dev, i32_dev, empty_bf16
    cfg = pdlib.LayerConfig(**TINY, max_pos=256)
    dl = DeviceLayer(pdlib, cfg, gen.layer_weights(**TINY, seed=0), 128, 4, 144)
    k, v, cache = dl.make_cache(4, 144)
    x = to_dev(gen.activations(0, 128, 512))
    out = empty_bf16(128, 512)
    n0 = pdlib.pd_launch_count()
    pdlib.pd_trace_begin()
    pdlib.pd_prefill_layer(dl.layer, x, out, i32_dev([0, 128]), [0, 128], cache, dl.ws, dl.ws_bytes)
    pdlib.pd_decode_layer(dl.layer, x, out, i32_dev([128, 100, 3, 0]), 4, 129, cache, dl.ws, dl.ws_bytes)
    rep = pdlib.pd_trace_end()
    torch.cuda.synchronize()
    assert pdlib.pd_launch_count() - n0 >= 12
    for name in ("gemm_qkv", "gemm_o", "gemm_gate_up", "gemm_down", "attn_prefill", "attn_decode", "rmsnorm"):
        secs, launches = rep[name]
        assert launches >= 1 and 0 < secs < 0.1, name
    pdlib.pd_trace_begin()
    assert all(v == (0.0, 0) for v in pdlib.pd_trace_end().values())
