"""Benchmark of the prefill/decode measurement hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Workload (the 8B-shaped configuration): 32 distinct layers, d_model 4096, 32 query / 8 KV
heads, head_dim 128, d_ff 14336, bf16 synthetic weights ~N(0, 0.02).  One step is one pass
of the whole hot path:
  1. prefill of one 4096-token request through the 32 layers (maximum prefill throughput),
  2. `--decode-steps` decode steps at the TPOT-feasible batch over KV length 2048 + t,
  3. the allocation model and the TTFT queue replay on the numbers just measured (host).
Before the timed steps the TPOT-versus-batch curve is measured once over B in {1..256}
and the feasible batch is taken from it.  `value` is prefill tokens/s of the 32-layer
stack; decode tokens/s, TPOT, the feasible batch and the P/D counts ride along in the
same JSON line.  With N > 1 (torchrun) every rank runs an independent replica.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

SHAPE = dict(d_model=4096, n_q_heads=32, n_kv_heads=8, head_dim=128, d_ff=14336)
N_LAYERS = 32
L_IN = 4096
KV_START = 2048
L_OUT = 256
SWEEP = [1, 2, 4, 8, 16, 32, 64, 128, 256]
TTFT_SLO, TPOT_SLO, TP_TOTAL = 2.0, 0.050, 2e5
# DRAM traffic per launch from ncu (dram__bytes_read.sum + dram__bytes_write.sum), captured on the same shapes with
# one layer (profiles/gemm_tc_prefill_8b_ncu_full.md, profiles/prefill_attn_tc_and_decode_kernels_ncu_full.md).
# Set an entry to None whenever the kernel changes after the capture.
NCU_TRAFFIC = {
    "gemm_tc_kernel": {"bytes_per_launch": 317.4e6, "algorithmic_bytes_per_launch": 238.8e6,
                       "note": "gemm_tc_pair_kernel, mean over the four prefill projections of a layer (1269.8 MB / 4)"},
    "decode_attn_kernel": {"bytes_per_launch": 2.1562e9, "algorithmic_bytes_per_launch": 2.1485e9,
                           "note": "B = 256 at KV length 2049; grows in proportion to the KV length"},
}
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# Datasheet figures of the part (dense bf16 without 2:4 sparsity; HBM3e of the HGX board), quoted beside the measured peaks.
NOMINAL = {"bf16_tflops": 2250.0, "hbm_gbs": 7700.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["source"] = "fallback"
    return p


def layer_params():
    d, f = SHAPE["d_model"], SHAPE["d_ff"]
    nqkv = (SHAPE["n_q_heads"] + 2 * SHAPE["n_kv_heads"]) * SHAPE["head_dim"]
    return d * nqkv + SHAPE["n_q_heads"] * SHAPE["head_dim"] * d + 3 * d * f


def prefill_flops(l_in, n_layers):
    gemm = 2.0 * l_in * layer_params()
    attn = 4.0 * SHAPE["n_q_heads"] * SHAPE["head_dim"] * (l_in * (l_in + 1) / 2.0)
    return (gemm + attn) * n_layers, gemm * n_layers, attn * n_layers


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons every 200 ms while running."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0]))
                mx = float(parts[1])
            except ValueError:
                continue
            for name, val in zip(names, parts[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


def oracle_prefill_sample(l_in):
    """Times the CPU oracle on one 8B-shaped layer with l_in tokens; returns (seconds, threads)."""
    import numpy as np
    import pd_inputs as gen
    from oracle import decoder_layer as L
    cfg = L.LayerConfig(**SHAPE)
    w = L.LayerWeights(**gen.layer_weights(**SHAPE, seed=0))
    x = gen.activations(0, l_in, SHAPE["d_model"])
    t0 = time.perf_counter()
    L.prefill_layer(cfg, w, x, [0, l_in])
    dt = time.perf_counter() - t0
    threads = os.cpu_count() or 1
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] or [threads])
    except Exception:
        pass
    return dt, threads


def run_reference(args, rank):
    """The reference arm: the CPU oracle as it stands, on a bounded sample of the workload."""
    if rank != 0:
        return
    sample_l = 512
    times = []
    threads = 1
    for i in range(args.warmup + args.steps):
        dt, threads = oracle_prefill_sample(sample_l)
        if i >= args.warmup:
            times.append(dt)
    per_layer = statistics.mean(times)
    value = sample_l / (per_layer * N_LAYERS)
    sample = f"prefill of {sample_l} tokens through 1 of {N_LAYERS} layers per step, scaled to {N_LAYERS} layers"
    print(json.dumps({
        "impl": "reference", "metric": "prefill tok/s (% bf16 peak); decode tok/s at TPOT-feasible batch (% HBM BW)",
        "value": value, "unit": "tok/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": per_layer * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "8B-shaped dense layers (configs[1]), CPU oracle sample", "l_in": sample_l},
        "cpu_baseline": {"value": value, "unit": "tok/s", "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tok/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--decode-steps", type=int, default=8, help="decode steps per benchmark step")
    ap.add_argument("--layers", type=int, default=N_LAYERS, help="layers actually run (times are scaled to 32)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--skip-sweep", action="store_true",
                    help="profiling aid: skip the TPOT(B) sweep and decode at the largest batch")
    ap.add_argument("--no-graphs", action="store_true", help="launch the layer stacks eagerly instead of replaying CUDA graphs")
    ap.add_argument("--no-fp8", action="store_true", help="skip the FP8-projection section")
    ap.add_argument("--decode-batch", type=int, default=0,
                    help="profiling aid: decode at this batch instead of the TPOT-feasible one")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        run_reference(args, rank)
        return

    import numpy as np
    import torch
    import paper_2603_04716_b200 as pd
    from paper_2603_04716_b200.replicas import max_over_ranks

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist_mod.init_process_group("nccl", device_id=dev)
        dist = dist_mod
    peaks = load_peaks()
    n_layers = args.layers
    scale = N_LAYERS / n_layers
    cfg = pd.LayerConfig(**SHAPE, max_pos=max(L_IN, KV_START + L_OUT))
    d = SHAPE["d_model"]
    kv_row = SHAPE["n_kv_heads"] * SHAPE["head_dim"]

    # ---- synthetic layers (torch is the allocator and the random source; values are inputs)
    gen_t = torch.Generator(device=dev)
    gen_t.manual_seed(1234 + rank)

    def randn_bf16(*shape, std=1.0, mean=0.0):
        t = torch.randn(*shape, generator=gen_t, device=dev, dtype=torch.float32) * std + mean
        return t.to(torch.bfloat16)

    nqkv = cfg.n_qkv
    layers = []
    for _ in range(n_layers):
        w = {"w_qkv": randn_bf16(nqkv, d, std=0.02), "w_o": randn_bf16(d, SHAPE["n_q_heads"] * SHAPE["head_dim"], std=0.02),
             "w_gate": randn_bf16(SHAPE["d_ff"], d, std=0.02), "w_up": randn_bf16(SHAPE["d_ff"], d, std=0.02),
             "w_down": randn_bf16(d, SHAPE["d_ff"], std=0.02), "g_attn": randn_bf16(d, std=0.02, mean=1.0),
             "g_mlp": randn_bf16(d, std=0.02, mean=1.0)}
        layers.append(pd.Layer(cfg, w))
        torch.cuda.synchronize()
        del w
    b_max = max(SWEEP)
    cap = KV_START + L_OUT
    pre_caches, dec_caches, keep = [], [], []
    for _ in range(n_layers):
        k = torch.empty((1, SHAPE["n_kv_heads"], L_IN, SHAPE["head_dim"]), dtype=torch.bfloat16, device=dev)
        v = torch.empty_like(k)
        keep += [k, v]
        pre_caches.append(pd.kv_cache_struct(k, v, 1, L_IN))
        k = randn_bf16(b_max, SHAPE["n_kv_heads"], cap, SHAPE["head_dim"])
        v = randn_bf16(b_max, SHAPE["n_kv_heads"], cap, SHAPE["head_dim"])
        keep += [k, v]
        dec_caches.append(pd.kv_cache_struct(k, v, b_max, cap))
    ws_bytes = pd.pd_workspace_bytes(cfg, L_IN, b_max, cap)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
    x_pre = randn_bf16(L_IN, d)
    y_pre = torch.empty_like(x_pre)
    cu_host = [0, L_IN]
    cu_dev = torch.tensor(cu_host, dtype=torch.int32, device=dev)
    x_dec = randn_bf16(b_max, d)
    y_dec = torch.empty_like(x_dec)
    kv_lens = {t: torch.full((b_max,), KV_START + t, dtype=torch.int32, device=dev) for t in range(L_OUT)}
    torch.cuda.synchronize()

    def ev():
        return torch.cuda.Event(enable_timing=True)

    def prefill_pass():
        pd.pd_prefill_stack(layers, pre_caches, x_pre, y_pre, False, cu_dev, cu_host, ws, ws_bytes)

    def decode_pass(batch, t):
        pd.pd_decode_stack(layers, dec_caches, x_dec, y_dec, False, kv_lens[t], batch, KV_START + t + 1, ws, ws_bytes)

    # The layer stacks only enqueue kernels (no allocation, no synchronisation), so each pass is captured
    # once into a CUDA graph and replayed: this removes most of the launch gaps between the ~13 small
    # kernels of a decode layer.
    graphs = {}

    def runner(key, fn):
        """Callable that replays `fn` (captured on first use) and the number of kernels it launches."""
        if key not in graphs:
            fn()
            torch.cuda.synchronize()
            n0 = pd.pd_launch_count()
            if args.no_graphs:
                fn()
                graphs[key] = (fn, pd.pd_launch_count() - n0)
            else:
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g):
                    fn()
                graphs[key] = (g.replay, pd.pd_launch_count() - n0)
            torch.cuda.synchronize()
        return graphs[key]

    def run_prefill():
        runner("prefill", prefill_pass)[0]()

    def run_decode(batch, t):
        runner(("decode", batch, t), lambda: decode_pass(batch, t))[0]()

    # ---- TPOT(B) curve, measured once (not part of the timed steps)
    sweep_t = [0, L_OUT // 2, L_OUT - 1]
    curve = {}
    for b in ([] if args.skip_sweep else SWEEP):
        per_t = []
        for t in sweep_t:
            run_decode(b, t)
            reps = []
            for _ in range(3):
                e0, e1 = ev(), ev()
                e0.record()
                run_decode(b, t)
                e1.record()
                e1.synchronize()
                reps.append(e0.elapsed_time(e1) * 1e-3)
            per_t.append(statistics.median(reps))
        curve[b] = statistics.mean(per_t) * scale
    pd.pd_layer_check(layers[0])

    # prefill probe for the allocation inputs
    run_prefill()
    e0, e1 = ev(), ev()
    e0.record()
    run_prefill()
    e1.record()
    e1.synchronize()
    tp_max_probe = L_IN / (e0.elapsed_time(e1) * 1e-3 * scale)
    if args.skip_sweep:
        curve = {b_max: TPOT_SLO}
    alloc = pd.pd_allocate(TP_TOTAL, L_IN, L_OUT, TTFT_SLO, TPOT_SLO, tp_max_probe, list(curve), list(curve.values()))
    b_star = alloc["feasible_batch"] or SWEEP[0]
    if args.decode_batch:
        b_star = min(b_max, args.decode_batch)
    dec_ts = [int(round(i * (L_OUT - 1) / max(1, args.decode_steps - 1))) for i in range(args.decode_steps)]

    rng = np.random.Generator(np.random.Philox(key=99))
    replay_n = 100_000

    def host_part(tp_max, curve_now):
        a = pd.pd_allocate(TP_TOTAL, L_IN, L_OUT, TTFT_SLO, TPOT_SLO, tp_max, list(curve_now), list(curve_now.values()))
        soj = None
        if a["status"] == 0:
            gaps = rng.exponential(1.0 / a["lam"], size=replay_n)
            soj, _ = pd.pd_queue_replay(gaps, np.full(replay_n, L_IN / tp_max))
        return a, soj

    def step(timing=None):
        e0, e1, e2 = ev(), ev(), ev()
        e0.record()
        run_prefill()
        e1.record()
        for t in dec_ts:
            run_decode(b_star, t)
        e2.record()
        if timing is not None:
            timing.append((e0, e1, e2))

    def barrier():
        if dist:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(3, args.warmup)):
        step()
    barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    launches_per_step = runner("prefill", prefill_pass)[1] + sum(
        runner(("decode", b_star, t), lambda t=t: decode_pass(b_star, t))[1] for t in dec_ts)
    timing = []
    t_wall0 = time.perf_counter()
    g0, g1 = ev(), ev()
    g0.record()
    for _ in range(args.steps):
        step(timing)
    g1.record()
    barrier()
    t_wall = time.perf_counter() - t_wall0
    launches = launches_per_step * args.steps
    clocks = sampler.stop()
    pd.pd_layer_check(layers[0])
    total_s = g0.elapsed_time(g1) * 1e-3
    pre_s = sum(a.elapsed_time(b) for a, b, _ in timing) * 1e-3
    dec_s = sum(b.elapsed_time(c) for _, b, c in timing) * 1e-3
    total_s, pre_s, dec_s = max_over_ranks([total_s, pre_s, dec_s], dist, dev)
    pre_model_s = pre_s / args.steps * scale                       # one prefill pass, 32 layers
    tpot_s = dec_s / (args.steps * len(dec_ts)) * scale            # one decode step, 32 layers
    prefill_tok_s = world * L_IN / pre_model_s
    decode_tok_s = world * b_star / tpot_s
    curve_now = dict(curve)
    curve_now[b_star] = tpot_s
    alloc, sojourn = host_part(L_IN / pre_model_s, curve_now)

    # ---- per-kernel attribution: one traced pass of the same step
    pd.pd_trace_begin()
    prefill_pass()
    tr_pre = pd.pd_trace_end()
    pd.pd_trace_begin()
    for t in dec_ts:
        decode_pass(b_star, t)
    tr_dec = pd.pd_trace_end()
    flops_all, flops_gemm, flops_attn = prefill_flops(L_IN, n_layers)
    gemm_s = sum(tr_pre[k][0] for k in ("gemm_qkv", "gemm_o", "gemm_gate_up", "gemm_down"))
    gemm_n = sum(tr_pre[k][1] for k in ("gemm_qkv", "gemm_o", "gemm_gate_up", "gemm_down"))
    peak_tf = peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])
    gemm_tf = flops_gemm / gemm_s / 1e12
    attn_dec_s, attn_dec_n = tr_dec["attn_decode"]
    kv_bytes = sum(b_star * (KV_START + t + 1) * 2 * kv_row * 2 for t in dec_ts) * n_layers
    attn_gbs = kv_bytes / attn_dec_s / 1e9
    dec_bytes_step = n_layers * (2 * layer_params() + 2 * kv_row * 2 * b_star) + kv_bytes / len(dec_ts)

    # ---- end to end: host buffers in and out through the stack calls
    xh = x_pre.cpu().pin_memory()
    yh = torch.empty_like(xh).pin_memory()
    xdh = x_dec[:b_star].cpu().pin_memory()
    ydh = torch.empty_like(xdh).pin_memory()
    kvh = {t: [KV_START + t] * b_star for t in dec_ts}
    import ctypes
    kv_host = {t: (ctypes.c_int32 * b_star)(*kvh[t]) for t in dec_ts}
    pd.pd_prefill_stack(layers, pre_caches, xh, yh, True, None, cu_host, ws, ws_bytes)
    barrier()
    e2e_pre, e2e_dec = [], []
    for _ in range(args.steps):
        t0 = time.perf_counter()
        pd.pd_prefill_stack(layers, pre_caches, xh, yh, True, None, cu_host, ws, ws_bytes)
        t1 = time.perf_counter()
        for t in dec_ts:
            pd.pd_decode_stack(layers, dec_caches, xdh, ydh, True, ctypes.addressof(kv_host[t]), b_star,
                               KV_START + t + 1, ws, ws_bytes)
        t2 = time.perf_counter()
        e2e_pre.append(t1 - t0)
        e2e_dec.append((t2 - t1) / len(dec_ts))
    e2e_pre_s = statistics.mean(e2e_pre)
    (e2e_pre_s,) = max_over_ranks([e2e_pre_s], dist, dev)
    e2e_value = world * L_IN / (e2e_pre_s * scale)

    # ---- whole-model step over the same layers: token ids in, greedy token out (embedding, final norm,
    # LM head over a 128256-entry vocabulary and the sampler added to the stack)
    vocab = 128256
    model = pd.Model(layers, vocab, randn_bf16(vocab, d), randn_bf16(d, std=0.02, mean=1.0),
                     randn_bf16(vocab, d, std=0.02))
    mws_bytes = pd.pd_model_workspace_bytes(model, L_IN, 1, b_max, cap)
    mws = torch.empty(mws_bytes, dtype=torch.uint8, device=dev)
    tok_pre = torch.randint(0, vocab, (L_IN,), dtype=torch.int32, device=dev, generator=gen_t)
    tok_dec = torch.randint(0, vocab, (b_max,), dtype=torch.int32, device=dev, generator=gen_t)
    next_pre = torch.zeros(1, dtype=torch.int32, device=dev)
    next_dec = torch.zeros(b_max, dtype=torch.int32, device=dev)
    t_mid = dec_ts[len(dec_ts) // 2]

    def timed(fn, reps=3):
        fn()
        out_s = []
        for _ in range(reps):
            a, b = ev(), ev()
            a.record()
            fn()
            b.record()
            b.synchronize()
            out_s.append(a.elapsed_time(b) * 1e-3)
        return statistics.median(out_s)

    def model_prefill():
        pd.pd_model_prefill(model, tok_pre, cu_dev, cu_host, pre_caches, next_pre, mws, mws_bytes)

    def model_decode():
        pd.pd_model_decode_step(model, tok_dec, kv_lens[t_mid], b_star, KV_START + t_mid + 1, dec_caches, next_dec,
                                mws, mws_bytes)

    wm_pre = timed(runner("model_prefill", model_prefill)[0])
    wm_dec = timed(runner("model_decode", model_decode)[0])
    pd.pd_model_check(model)

    def head_time(fn):
        """Embedding + LM head + sampler kernels of one traced (eager) pass, by their CUDA events."""
        pd.pd_trace_begin()
        fn()
        tr = pd.pd_trace_end()
        return sum(tr[k][0] for k in ("embed", "lm_head", "sample"))

    head_pre, head_dec = head_time(model_prefill), head_time(model_decode)
    # whole-model time at 32 layers: the measured pass with its layer-stack part scaled up
    wm_pre_s, wm_dec_s = (wm_pre - head_pre) * scale + head_pre, (wm_dec - head_dec) * scale + head_dec
    wm_pre_s, wm_dec_s = max_over_ranks([wm_pre_s, wm_dec_s], dist, dev)
    whole_model = {"vocab": vocab, "ttft_compute_ms": wm_pre_s * 1e3, "prefill_tok_s": world * L_IN / wm_pre_s,
                   "tpot_ms": wm_dec_s * 1e3, "decode_tok_s": world * b_star / wm_dec_s,
                   "head_ms_prefill": head_pre * 1e3, "head_ms_decode": head_dec * 1e3,
                   "lm_head_gbs_decode": vocab * d * 2 / head_dec / 1e9 if head_dec > 0 else None,
                   "first_token": int(next_pre.item()),
                   "note": "graph replay of pd_model_prefill / pd_model_decode_step; head = embedding + LM head + "
                           "sampler kernels by CUDA events in a traced pass"}

    # ---- the same stack with FP8 (E4M3) projections: a separate precision, reported beside the bf16 headline
    fp8_out = None
    if not args.no_fp8:
        del model, mws
        cfg8 = pd.LayerConfig(**SHAPE, max_pos=max(L_IN, KV_START + L_OUT), fp8_projections=True)
        layers8 = []
        for _ in range(n_layers):
            w = {"w_qkv": randn_bf16(nqkv, d, std=0.02), "w_o": randn_bf16(d, SHAPE["n_q_heads"] * SHAPE["head_dim"], std=0.02),
                 "w_gate": randn_bf16(SHAPE["d_ff"], d, std=0.02), "w_up": randn_bf16(SHAPE["d_ff"], d, std=0.02),
                 "w_down": randn_bf16(d, SHAPE["d_ff"], std=0.02), "g_attn": randn_bf16(d, std=0.02, mean=1.0),
                 "g_mlp": randn_bf16(d, std=0.02, mean=1.0)}
            layers8.append(pd.Layer(cfg8, w))
            torch.cuda.synchronize()
            del w
        ws8_bytes = pd.pd_workspace_bytes(cfg8, L_IN, b_max, cap)
        ws8 = torch.empty(ws8_bytes, dtype=torch.uint8, device=dev)

        def prefill8():
            pd.pd_prefill_stack(layers8, pre_caches, x_pre, y_pre, False, cu_dev, cu_host, ws8, ws8_bytes)

        def decode8(batch):
            pd.pd_decode_stack(layers8, dec_caches, x_dec, y_dec, False, kv_lens[t_mid], batch, KV_START + t_mid + 1,
                               ws8, ws8_bytes)

        pre8_s = timed(runner("prefill_fp8", prefill8)[0], reps=5) * scale
        dec8 = {}
        for b in sorted({1, 64, b_star}):
            dec8[b] = timed(runner(("decode_fp8", b), lambda b=b: decode8(b))[0], reps=5) * scale
        pd.pd_layer_check(layers8[0])
        pd.pd_trace_begin()
        prefill8()
        tr8 = pd.pd_trace_end()
        gemm8_s = sum(tr8[k][0] for k in ("gemm_qkv", "gemm_o", "gemm_gate_up", "gemm_down"))
        (pre8_s,) = max_over_ranks([pre8_s], dist, dev)
        peak8 = 2.0 * peaks["bf16_tflops"]      # dense FP8 runs at twice the bf16 rate (nominal ratio x measured bf16 burst)
        fp8_out = {"prefill_tok_s": world * L_IN / pre8_s, "prefill_ms_per_pass": pre8_s * 1e3,
                   "prefill_tflops": flops_all * scale / pre8_s / 1e12,
                   "gemm_tflops_incl_quantisers": flops_gemm / gemm8_s / 1e12,
                   "gemm_frac_of_fp8_peak": flops_gemm / gemm8_s / 1e12 / peak8, "fp8_peak_tflops": peak8,
                   "peak_source": "2 x measured bf16 burst (nominal FP8 : bf16 ratio)",
                   "tpot_ms": {str(b): v * 1e3 for b, v in dec8.items()},
                   "decode_tok_s": world * b_star / dec8[b_star],
                   "kernel_time_ms_prefill": {k: v[0] * 1e3 for k, v in tr8.items() if v[1]},
                   "note": "E4M3 weights per output channel, activations per token; attention, norms, residual stream "
                           "and KV cache stay bf16; not part of `value`"}
        # block-wise scales (one per 128 x 128 weight block and per token and 128 channels): the stand-alone GEMM on
        # the down-projection shape of this workload, timed launch by launch (L2 flushed by the previous launches'
        # operands: three weight matrices of 59 MB of codes take turns)
        bw_m, bw_n, bw_k = L_IN, SHAPE["d_model"], SHAPE["d_ff"]
        bw_a = torch.randn(bw_m, bw_k, device=dev).to(torch.bfloat16)
        bw_qa = torch.empty((bw_m, bw_k), dtype=torch.uint8, device=dev)
        bw_sa = torch.empty((bw_m, bw_k // 128), dtype=torch.float32, device=dev)
        bw_c = torch.empty((bw_m, bw_n), dtype=torch.bfloat16, device=dev)
        bw_w = []
        for _ in range(3):
            w_ = (torch.randn(bw_n, bw_k, device=dev) * 0.02).to(torch.bfloat16)
            q_ = torch.empty((bw_n, bw_k), dtype=torch.uint8, device=dev)
            s_ = torch.empty(((bw_n + 127) // 128, bw_k // 128), dtype=torch.float32, device=dev)
            pd.pd_quantize_fp8_blocks(w_, bw_n, bw_k, q_, s_)
            bw_w.append((q_, s_))
            del w_
        pd.pd_quantize_fp8_groups(bw_a, bw_m, bw_k, bw_qa, bw_sa)
        bw_i = [0]

        def bw_step():
            q_, s_ = bw_w[bw_i[0] % 3]
            bw_i[0] += 1
            pd.pd_gemm_fp8_blockwise(bw_qa, bw_sa, q_, s_, bw_c, bw_m, bw_n, bw_k)
        bw_s = timed(bw_step, reps=9)
        bwq_s = timed(lambda: pd.pd_quantize_fp8_groups(bw_a, bw_m, bw_k, bw_qa, bw_sa), reps=5)
        fp8_out["blockwise_gemm"] = {"shape_mnk": [bw_m, bw_n, bw_k], "ms": bw_s * 1e3,
                                     "tflops": 2.0 * bw_m * bw_n * bw_k / bw_s / 1e12,
                                     "frac_of_fp8_peak": 2.0 * bw_m * bw_n * bw_k / bw_s / 1e12 / peak8,
                                     "activation_quantiser_ms": bwq_s * 1e3,
                                     "note": "pd_gemm_fp8_blockwise: 128 x 128 tiles on single CTAs, scaled accumulation in "
                                             "registers per K block; not used by the layer passes above"}
        del bw_w, bw_a, bw_qa, bw_sa, bw_c
        del layers8, ws8

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        sample_l = L_IN
        dt, threads = oracle_prefill_sample(sample_l)
        cpu = {"value": sample_l / (dt * N_LAYERS), "unit": "tok/s", "cores": threads, "kind": "oracle",
               "sample": f"prefill of {sample_l} tokens through 1 layer ({dt:.1f} s), scaled to {N_LAYERS} layers"}

    if rank == 0:
        out = {
            "metric": "prefill tok/s (% bf16 peak); decode tok/s at TPOT-feasible batch (% HBM BW)",
            "value": prefill_tok_s, "unit": "tok/s", "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": total_s / args.steps * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "8B-shaped dense model (configs[1]): 32 layers, prefill 1 x 4096 tokens; "
                                   f"decode B={b_star} over KV 2048+t, L_out 256",
                       "layers_run": n_layers, "l_in": L_IN, "decode_batch": b_star, "decode_steps_per_step": len(dec_ts),
                       "l2": "inputs larger than L2: every layer has its own weights (436 MB) and KV buffers",
                       "multi_gpu": "replicas only",
                       "launch": "eager" if args.no_graphs else "CUDA graph replay of each layer-stack pass"},
            "prefill": {"tok_s": prefill_tok_s, "ms_per_pass": pre_model_s * 1e3,
                        "tflops": flops_all * scale / pre_model_s / 1e12 * 1.0,
                        "frac_bf16_sustained": flops_all * scale / pre_model_s / 1e12 / peak_tf,
                        "frac_bf16_burst": flops_all * scale / pre_model_s / 1e12 / peaks["bf16_tflops"],
                        "frac_bf16_nominal": flops_all * scale / pre_model_s / 1e12 / NOMINAL["bf16_tflops"]},
            "decode": {"tok_s": decode_tok_s, "tpot_ms": tpot_s * 1e3, "feasible_batch": b_star,
                       "sweep_capped": bool(alloc["sweep_capped"]), "tpot_curve_ms": {str(k): v * 1e3 for k, v in curve.items()},
                       "frac_hbm": dec_bytes_step * scale / tpot_s / 1e9 / peaks["hbm_gbs"],
                       "frac_hbm_nominal": dec_bytes_step * scale / tpot_s / 1e9 / NOMINAL["hbm_gbs"]},
            "allocation": {"status": alloc["status"], "tp_prefill_eff": alloc["tp_prefill_eff"],
                           "tp_decode_eff": alloc["tp_decode_eff"], "n_prefill": alloc["n_prefill"],
                           "n_decode": alloc["n_decode"], "ratio_pd": alloc["ratio_pd"], "rho": alloc["rho"],
                           "mm1_sojourn_s": None if alloc["status"] else 1.0 / (alloc["mu"] - alloc["lam"]),
                           "replayed_sojourn_s_deterministic_service": sojourn},
            # The launches are timed one by one with CUDA events (a traced pass), i.e. in isolation: the burst peak is
            # the denominator; the sustained and the datasheet figure ride along.
            "roofline": {"kernel": "gemm_tc_pair_kernel (QKV, O, gate/up, down projections of the prefill pass)",
                         "bound": "tensor", "achieved": gemm_tf, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                         "frac": gemm_tf / peaks["bf16_tflops"], "frac_of_sustained_peak": gemm_tf / peak_tf,
                         "frac_of_nominal_peak": gemm_tf / NOMINAL["bf16_tflops"], "nominal_peak": NOMINAL["bf16_tflops"],
                         "peak_source": peaks["source"] + " (burst bf16, torch.matmul 8192^3)", "launches": gemm_n,
                         "avg_launch_ms": gemm_s / max(1, gemm_n) * 1e3,
                         "traffic": NCU_TRAFFIC["gemm_tc_kernel"]["bytes_per_launch"], "traffic_unit": "DRAM bytes per launch (ncu)",
                         "traffic_detail": NCU_TRAFFIC["gemm_tc_kernel"],
                         "timing": "CUDA events around each launch in a separate traced pass of the same step"},
            "roofline_decode_attention": {"kernel": "decode_attn_kernel", "bound": "hbm", "achieved": attn_gbs,
                                          "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": attn_gbs / peaks["hbm_gbs"],
                                          "frac_of_nominal_peak": attn_gbs / NOMINAL["hbm_gbs"], "nominal_peak": NOMINAL["hbm_gbs"],
                                          "peak_source": peaks["source"] + " (device copy: read + write bytes; a pure read stream "
                                                         "can exceed it slightly)",
                                          "launches": attn_dec_n, "avg_launch_ms": attn_dec_s / max(1, attn_dec_n) * 1e3,
                                          "traffic": NCU_TRAFFIC["decode_attn_kernel"]["bytes_per_launch"],
                                          "traffic_unit": "DRAM bytes per launch (ncu)",
                                          "traffic_detail": NCU_TRAFFIC["decode_attn_kernel"]},
            "kernel_time_ms": {"prefill": {k: v[0] * 1e3 for k, v in tr_pre.items() if v[1]},
                               "decode": {k: v[0] * 1e3 / len(dec_ts) for k, v in tr_dec.items() if v[1]}},
            "e2e": {"value": e2e_value, "unit": "tok/s", "h2d_bytes_per_step": xh.numel() * 2 + 8,
                    "d2h_bytes_per_step": yh.numel() * 2,
                    "decode_tok_s": world * b_star / (statistics.mean(e2e_dec) * scale)},
            "whole_model": whole_model,
            "fp8_projections": fp8_out,
            "gpu_launches": launches, "clocks": clocks, "wall_s_timed_region": t_wall,
        }
        if cpu:
            out["cpu_baseline"] = cpu
        print(json.dumps(out))
    if dist:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
