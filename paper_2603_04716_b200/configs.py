"""The five benchmark configurations, and the chunked-prefill sweep, as runnable drivers.

    python -m paper_2603_04716_b200.configs <tiny|8b|long_input|decode_heavy|70b|chunked> [--quick] [--out FILE]

Each driver measures what the allocation method needs on the current GPU (maximum prefill
throughput and the TPOT-versus-batch curve, both through pd_measure), feeds the numbers to
pd_allocate (Eq. 5-7, 13) and, for the long-input configuration, replays a seeded Poisson
arrival stream through a FIFO server whose service times are the measured prefill times, to
compare the M/M/1 prediction of Eq. 12 with what a queue of real prefill passes does.
Inputs are synthetic: shapes, length distributions and SLOs are those of the configurations.
`--quick` shrinks grids and repetitions for smoke runs.

This module holds loops and I/O only: every number comes from a call into the library (pd_measure,
pd_allocate, pd_mixture_throughput, pd_interp_service_times, pd_mm1_sojourn, pd_mg1_sojourn,
pd_refine_next_batch, pd_queue_replay).  Every allocation result is stored together with the exact
inputs it was computed from ("inputs"), so that the result file can be re-checked later, on a machine
without a GPU, against an independent implementation of the allocation equations.
"""
from __future__ import annotations

import argparse
import json
import sys

import numpy as np

import paper_2603_04716_b200 as pd
import pd_inputs as gen

SHAPE_TINY = dict(d_model=512, n_q_heads=8, n_kv_heads=2, head_dim=64, d_ff=1536)
SHAPE_8B = dict(d_model=4096, n_q_heads=32, n_kv_heads=8, head_dim=128, d_ff=14336)
SHAPE_70B = dict(d_model=8192, n_q_heads=64, n_kv_heads=8, head_dim=128, d_ff=28672)


def _peaks():
    import os
    path = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return p.get("bf16_tflops_sustained", p["bf16_tflops"]) * 1e12, p["hbm_gbs"] * 1e9, "measured"
    return 1.4e15, 6.65e12, "fallback"


ALLOC_KEYS = ("status", "tp_prefill_eff", "tp_decode_eff", "mu", "lam", "rho", "feasible_batch", "sweep_capped",
              "n_prefill_frac", "n_decode_frac", "ratio_pd", "n_prefill", "n_decode", "n_prefill_ceil", "n_decode_ceil",
              "achieved_total_tok_s")


def _alloc(tp_total, l_in, l_out, ttft, tpot, tp_max, batch, tpot_s, t_overhead=0.0):
    """pd_allocate, with the inputs recorded beside the result."""
    a = pd.pd_allocate(tp_total, l_in, l_out, ttft, tpot, tp_max, batch, tpot_s, t_overhead)
    out = {k: a[k] for k in ALLOC_KEYS}
    out["inputs"] = {"tp_total_tok_s": float(tp_total), "l_in": float(l_in), "l_out": float(l_out),
                     "ttft_slo_s": float(ttft), "tpot_slo_s": float(tpot), "prefill_max_tok_s": float(tp_max),
                     "batch": [int(b) for b in batch], "tpot_s": [float(t) for t in tpot_s],
                     "t_overhead_s": float(t_overhead)}
    return out


def _prefill_time_grid(cfg, lengths, n_layers_run, n_layers_model, reps, peaks):
    """Measured prefill time of one request of each length (seconds, whole model): one pd_measure call, one
    layer stack, every length timed on its own."""
    m = pd.pd_measure(cfg, n_layers_run=n_layers_run, n_layers_model=n_layers_model, warmup=1, reps=reps, seed=0,
                      l_in_grid=[int(l) for l in lengths], peak_bf16_flops=peaks[0], peak_hbm_bytes_s=peaks[1])
    return {"l": m["grid_l"], "time_s": m["grid_time_s"]}


def refine_feasible_batch(measure_tpot, batch, tpot_s, tpot_slo_s, max_probes=8):
    """Integer refinement of the TPOT-feasible batch (paper, "Acquire decode throughput ...": determine the batch
    size that satisfies the target TPOT): pd_refine_next_batch names the next batch size to measure until the
    largest feasible integer is bracketed.  `measure_tpot(b)` returns the measured TPOT of batch b in seconds.
    Returns the extended point lists (batch, tpot_s) and the probes made."""
    batch, tpot_s, probes = list(batch), list(tpot_s), []
    while len(probes) < max_probes:
        nxt = pd.pd_refine_next_batch(batch, tpot_s, tpot_slo_s)
        if nxt == 0:
            break
        t = measure_tpot(nxt)
        batch.append(nxt)
        tpot_s.append(t)
        probes.append((nxt, t))
    return batch, tpot_s, probes


def run_tiny(quick=False):
    peaks = _peaks()
    cfg = pd.LayerConfig(**SHAPE_TINY, max_pos=256)
    m = pd.pd_measure(cfg, n_layers_run=1, n_layers_model=1, warmup=3, reps=10, seed=0, l_in=[128], batch_sizes=[1, 2, 4],
                      kv_len_start=128, n_steps=16, step_stride=1, peak_bf16_flops=peaks[0], peak_hbm_bytes_s=peaks[1])
    return {"config": "tiny", "measure": m,
            "allocation": _alloc(1e4, 128, 16, 1.0, 0.050, m["prefill_tok_s"], m["batch"], m["tpot_s"])}


def run_8b(quick=False, fp8=False):
    peaks = _peaks()
    cfg = pd.LayerConfig(**SHAPE_8B, max_pos=4096, fp8_projections=fp8)
    nl = 8 if quick else 32
    grid = {}
    for l_in in ([4096] if quick else [1024, 2048, 4096]):
        for n_req in ([1] if quick else [1, 2, 4, 8]):
            m = pd.pd_measure(cfg, n_layers_run=nl, n_layers_model=32, warmup=2, reps=3 if quick else 7, seed=0,
                              l_in=[l_in] * n_req, peak_bf16_flops=peaks[0], peak_hbm_bytes_s=peaks[1])
            grid[f"{l_in}x{n_req}"] = {"tok_s": m["prefill_tok_s"], "time_s": m["prefill_time_s"],
                                       "frac_bf16_peak": m["prefill_frac_bf16_peak"]}
    sweep = [1, 8, 64, 256] if quick else [1, 2, 4, 8, 16, 32, 64, 128, 256]
    d = pd.pd_measure(cfg, n_layers_run=nl, n_layers_model=32, warmup=1, reps=3, seed=0, batch_sizes=sweep,
                      kv_len_start=2048, n_steps=256, step_stride=128 if quick else 32,
                      peak_bf16_flops=peaks[0], peak_hbm_bytes_s=peaks[1])
    alloc = {}
    for l_in in ([4096] if quick else [1024, 2048, 4096]):
        # sequential requests (n_req = 1) are what the M/M/1 model assumes; batched ones are reported above
        alloc[str(l_in)] = _alloc(2e5, l_in, 256, 2.0, 0.050, grid[f"{l_in}x1"]["tok_s"], d["batch"], d["tpot_s"])
    return {"config": "8b", "fp8_projections": fp8, "layers_run": nl, "prefill_grid": grid, "decode": d, "allocation": alloc}


def run_long_input(quick=False):
    peaks = _peaks()
    cfg = pd.LayerConfig(**SHAPE_8B, max_pos=32768 + 256)
    nl = 4 if quick else 8
    lengths = gen.lognormal_lengths(1, 4096, 8192.0, 0.5, 2048, 32768)
    # the kernels work in tiles of 256 rows: on a grid of 256-multiples, with lengths rounded up to the next one,
    # the measured times are exact for every request length (no interpolation between tile counts)
    quantum = 1 if quick else 256
    grid_l = [2048, 8192, 20480, 32768] if quick else list(range(2048, 32768 + 1, 256))
    # interpolation check on seeded off-grid lengths, timed in the same pd_measure call as the grid (same clocks: under
    # the power cap two calls differ by more than the interpolation does)
    off = sorted(int(v) for v in gen.uniform_lengths(2, 2 if quick else 7, 2100, 32000, sub=7))
    both = _prefill_time_grid(cfg, grid_l + off, nl, 32, 2 if quick else 3, peaks)
    grid = {"l": both["l"][:len(grid_l)], "time_s": both["time_s"][:len(grid_l)]}
    off_meas = {"l": both["l"][len(grid_l):], "time_s": both["time_s"][len(grid_l):]}
    off_interp = pd.pd_interp_service_times(grid["l"], grid["time_s"], off, quantum)
    off_linear = pd.pd_interp_service_times(grid["l"], grid["time_s"], off, 1)
    interp_check = [{"l": l, "measured_s": tm, "interpolated_s": float(ti), "linear_s": float(tl)}
                    for l, tm, ti, tl in zip(off_meas["l"], off_meas["time_s"], off_interp, off_linear)]
    service = pd.pd_interp_service_times(grid["l"], grid["time_s"], lengths, quantum)
    tp_max, mean_l = pd.pd_mixture_throughput(lengths, service)     # total tokens over total time; mean length
    sweep = [1, 64] if quick else [1, 2, 4, 8, 16, 32, 64, 128, 256]
    d = pd.pd_measure(cfg, n_layers_run=nl, n_layers_model=32, warmup=1, reps=3, seed=0, batch_sizes=sweep,
                      kv_len_start=int(round(mean_l)), n_steps=256, step_stride=128,
                      peak_bf16_flops=peaks[0], peak_hbm_bytes_s=peaks[1])
    alloc = _alloc(2e5, mean_l, 256, 4.0, 0.050, tp_max, d["batch"], d["tpot_s"])
    mu = alloc["mu"]                                                 # Eq. 9 with the mean input length
    n_arr = 20_000 if quick else 200_000
    svc = service[np.arange(n_arr) % len(lengths)]
    replay = []
    for rho in ([0.5, 0.9] if quick else [0.1, 0.2, 0.3, 0.4, 0.5, 0.6, 0.7, 0.8, 0.9, 0.95]):
        lam = rho * mu
        gaps = gen.exponential_gaps(2, n_arr, lam)
        soj, wait = pd.pd_queue_replay(gaps, svc)
        replay.append({"rho": rho, "lambda": lam, "mm1_sojourn_s": pd.pd_mm1_sojourn(mu, lam), "replayed_sojourn_s": soj,
                       "pollaczek_khinchine_s": pd.pd_mg1_sojourn(service, lam)})
    return {"config": "long_input", "layers_run": nl, "sigma": 0.5, "tile_quantum": quantum, "mean_l_in": mean_l, "prefill_max_tok_s": tp_max,
            "prefill_time_grid": grid, "interpolation_check": interp_check, "queue": replay, "decode": d,
            "lengths": {"generator": "pd_inputs.lognormal_lengths(1, 4096, 8192.0, 0.5, 2048, 32768)"},
            "allocation": alloc}


def run_decode_heavy(quick=False):
    peaks = _peaks()
    cfg = pd.LayerConfig(**SHAPE_8B, max_pos=512 + 2048)
    nl = 4 if quick else 32
    p = pd.pd_measure(cfg, n_layers_run=nl, n_layers_model=32, warmup=2, reps=5, seed=0, l_in=[512],
                      peak_bf16_flops=peaks[0], peak_hbm_bytes_s=peaks[1])
    sweep = [1, 64, 512] if quick else [1, 2, 4, 8, 16, 32, 64, 128, 256, 384, 512]
    d = pd.pd_measure(cfg, n_layers_run=nl, n_layers_model=32, warmup=1, reps=3, seed=0, batch_sizes=sweep,
                      kv_len_start=512, n_steps=2048, step_stride=1024 if quick else 256,
                      peak_bf16_flops=peaks[0], peak_hbm_bytes_s=peaks[1])
    def tpot_at(b):
        m = pd.pd_measure(cfg, n_layers_run=nl, n_layers_model=32, warmup=1, reps=3, seed=0, batch_sizes=[int(b)],
                          kv_len_start=512, n_steps=2048, step_stride=1024 if quick else 256,
                          peak_bf16_flops=peaks[0], peak_hbm_bytes_s=peaks[1])
        return m["tpot_s"][0]

    per_slo = {}
    for slo_ms in (20, 35, 50, 75, 100):
        a = _alloc(5e5, 512, 2048, 2.0, slo_ms * 1e-3, p["prefill_tok_s"], d["batch"], d["tpot_s"])
        if a["status"] == 0 and not a["sweep_capped"]:
            # the SLO binds between two sweep points: bracket the largest feasible integer batch by measurement
            b_all, t_all, probes = refine_feasible_batch(tpot_at, d["batch"], d["tpot_s"], slo_ms * 1e-3,
                                                         max_probes=3 if quick else 8)
            a["refined"] = _alloc(5e5, 512, 2048, 2.0, slo_ms * 1e-3, p["prefill_tok_s"], b_all, t_all)
            a["refined"]["probes"] = probes
        per_slo[str(slo_ms)] = a
    return {"config": "decode_heavy", "layers_run": nl, "ttft_slo_s": 2.0, "prefill": p, "decode": d,
            "allocation_per_tpot_slo_ms": per_slo}


def run_70b(quick=False):
    peaks = _peaks()
    cfg = pd.LayerConfig(**SHAPE_70B, max_pos=8192 + 1024 + 16)
    nl = 2 if quick else 8
    p = pd.pd_measure(cfg, n_layers_run=nl, n_layers_model=80, warmup=2, reps=5, seed=0, l_in=[4096],
                      peak_bf16_flops=peaks[0], peak_hbm_bytes_s=peaks[1])
    sweep = [1, 32, 128] if quick else [1, 2, 4, 8, 16, 32, 64, 128]
    d = pd.pd_measure(cfg, n_layers_run=nl, n_layers_model=80, warmup=1, reps=3, seed=0, batch_sizes=sweep,
                      kv_len_start=4096, n_steps=256, step_stride=128, peak_bf16_flops=peaks[0],
                      peak_hbm_bytes_s=peaks[1])
    # mixed workload: L_in ~ U[1024, 8192], L_out ~ U[128, 1024]
    l_in = gen.uniform_lengths(3, 512, 1024, 8192, sub=0)
    l_out = gen.uniform_lengths(3, 512, 128, 1024, sub=1)
    quantum = 1 if quick else 256
    grid_l = [1024, 4096, 8192] if quick else list(range(1024, 8192 + 1, 256))
    grid = _prefill_time_grid(cfg, grid_l, nl, 80, 2, peaks)
    tp_max_mix, mean_l_in = pd.pd_mixture_throughput(l_in, pd.pd_interp_service_times(grid["l"], grid["time_s"], l_in, quantum))
    # stationary decode batch: sequence i sits at a uniformly random point of its output
    prog = gen.uniform_lengths(3, 512, 0, 10**6, sub=2) / 1e6
    mix = (l_in + np.floor(prog * l_out)).astype(np.int32)
    dm = pd.pd_measure(cfg, n_layers_run=nl, n_layers_model=80, warmup=1, reps=3, seed=0, batch_sizes=sweep,
                       kv_len_start=0, n_steps=8, step_stride=4, kv_len_mix=[int(v) for v in mix[:max(sweep)]],
                       peak_bf16_flops=peaks[0], peak_hbm_bytes_s=peaks[1])
    return {"config": "70b", "layers_run": nl, "layers_model": 80, "prefill": p, "decode": d,
            "allocation": _alloc(2e5, 4096, 256, 3.0, 0.060, p["prefill_tok_s"], d["batch"], d["tpot_s"]),
            "mixed": {"mean_l_in": mean_l_in, "mean_l_out": float(l_out.mean()), "tile_quantum": quantum,
                      "prefill_max_tok_s": tp_max_mix, "prefill_time_grid": grid, "decode": dm,
                      "allocation": _alloc(2e5, mean_l_in, float(l_out.mean()), 3.0, 0.060, tp_max_mix,
                                           dm["batch"], dm["tpot_s"])}}


def run_chunked(quick=False):
    """Maximum prefill throughput versus chunked-prefill size (paper, "Acquire prefill throughput ...": a larger
    chunk raises the peak prefill throughput until saturation).  One request of L_in tokens goes through the
    layer stack chunk by chunk inside pd_measure (graph-captured like every other measured pass); each chunk
    attends to the cached prefix."""
    peaks = _peaks()
    l_in = 4096 if quick else 8192
    nl = 2 if quick else 8
    cfg = pd.LayerConfig(**SHAPE_8B, max_pos=l_in)
    out = {}
    for chunk in ([1024, 4096] if quick else [256, 512, 1024, 2048, 4096, 8192]):
        m = pd.pd_measure(cfg, n_layers_run=nl, n_layers_model=32, warmup=1, reps=3 if quick else 5, seed=0,
                          l_in=[l_in], chunk_tokens=chunk, peak_bf16_flops=peaks[0], peak_hbm_bytes_s=peaks[1])
        out[str(chunk)] = {"time_s": m["prefill_time_s"], "prefill_max_tok_s": m["prefill_tok_s"],
                           "chunks": m["prefill_chunks"], "frac_bf16_peak": m["prefill_frac_bf16_peak"]}
    return {"config": "chunked", "l_in": l_in, "layers_run": nl, "chunk_sweep": out}


RUNNERS = {"chunked": run_chunked, "tiny": run_tiny, "8b": run_8b, "long_input": run_long_input, "decode_heavy": run_decode_heavy,
           "70b": run_70b}


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("config", choices=sorted(RUNNERS))
    ap.add_argument("--quick", action="store_true")
    ap.add_argument("--out", default="")
    ap.add_argument("--fp8", action="store_true", help="8b only: run the projections in FP8 (E4M3)")
    args = ap.parse_args(argv)
    if args.fp8 and args.config != "8b":
        ap.error("--fp8 is implemented for the 8b configuration")
    res = run_8b(args.quick, fp8=True) if args.fp8 else RUNNERS[args.config](args.quick)
    res["peaks"] = _peaks()[2]
    text = json.dumps(res, indent=1)
    if args.out:
        with open(args.out, "w") as f:
            f.write(text)
    print(text)


if __name__ == "__main__":
    sys.exit(main())
