"""CPU-only checks of the product's host side: the library loads and exports the
symbols the header declares; pd_allocate and pd_queue_replay agree with the oracle
(integers and doubles bit for bit, both being IEEE double in the same order)."""
import ctypes
import math
import os
import random
import re

import numpy as np
import pytest

from oracle import allocation as A

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol(pdlib):
    header = open(os.path.join(ROOT, "include", "pd.h")).read()
    declared = set(re.findall(r"\b(pd_[a-z0-9_]+)\s*\(", header))
    assert declared == set(pdlib.EXPORTS)
    lib = ctypes.CDLL(pdlib.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), name
    assert pdlib.pd_version() >= 1


def test_struct_sizes_match_c_layout(pdlib):
    # natural C layout: checked against hand-computed sizes of include/pd.h
    assert ctypes.sizeof(pdlib.pd_layer_cfg) == 40
    assert ctypes.sizeof(pdlib.pd_workspace_layout) == 8 + 5 * 8
    assert ctypes.sizeof(pdlib.pd_layer_weights) == 8 + 7 * 8
    assert ctypes.sizeof(pdlib.pd_kv_cache) == 32
    assert ctypes.sizeof(pdlib.pd_alloc_in) == 8 + 7 * 8 + 8 + 16
    assert ctypes.sizeof(pdlib.pd_alloc_out) == 8 + 5 * 8 + 8 + 3 * 8 + 16 + 8
    assert ctypes.sizeof(pdlib.pd_measurement) == (8 + 4 * 8 + 8 + 32 * 4 + 5 * 32 * 8 + 8 + 8 + 32 * 8
                                                   + 8 + 2 * 32 * 4 + 8 + 128 * 4 + 128 * 8)
    # 5 x 4 (+4 pad) | seed 8 | l_in 8 | n_req 4 (+4) | batch_sizes 8 | 4 x 4 | kv_len_mix 8 | 2 x 4 | l_in_grid 8 | n_grid 4 (+4)
    assert ctypes.sizeof(pdlib.pd_measure_cfg) == 24 + 8 + 8 + 8 + 8 + 16 + 8 + 8 + 8 + 8


def _same(a, b):
    return (math.isnan(a) and math.isnan(b)) or a == b


def test_allocate_matches_oracle_bit_for_bit(pdlib):
    rnd = random.Random(11)
    status_names = {0: "ok", pdlib.PD_ERR_INFEASIBLE_TTFT: "infeasible_ttft", pdlib.PD_ERR_INFEASIBLE_TPOT: "infeasible_tpot"}
    seen = set()
    for trial in range(2000):
        n = rnd.randint(1, 16)
        batch = rnd.sample(range(1, 1024), n)
        tpot = [rnd.uniform(0.002, 0.12) for _ in range(n)]
        if trial % 3:
            order = sorted(range(n), key=lambda i: batch[i])
            srt = sorted(tpot)
            for rank, i in enumerate(order):
                tpot[i] = srt[rank]
        args = dict(tp_total=rnd.uniform(1e3, 1e6), l_in=float(rnd.randint(16, 32768)), l_out=float(rnd.randint(1, 4096)),
                    ttft=rnd.uniform(0.05, 8.0), tpot_slo=rnd.uniform(0.001, 0.13), tp_max=rnd.uniform(5e3, 2e5),
                    t_over=rnd.choice([0.0, 0.1, rnd.uniform(0, 0.3)]))
        o = A.allocate(args["tp_total"], args["l_in"], args["l_out"], args["ttft"], args["tpot_slo"], args["tp_max"],
                       batch, tpot, args["t_over"])
        p = pdlib.pd_allocate(args["tp_total"], args["l_in"], args["l_out"], args["ttft"], args["tpot_slo"],
                              args["tp_max"], batch, tpot, args["t_over"])
        assert status_names[p["status"]] == o.status
        seen.add(o.status)
        assert p["feasible_batch"] == o.feasible_batch and bool(p["sweep_capped"]) == o.sweep_capped
        assert (p["n_prefill"], p["n_decode"], p["n_prefill_ceil"], p["n_decode_ceil"]) == \
               (o.n_prefill, o.n_decode, o.n_prefill_ceil, o.n_decode_ceil)
        for mine, theirs in (("tp_prefill_eff", o.tp_prefill_eff), ("tp_decode_eff", o.tp_decode_eff), ("mu", o.mu),
                             ("lam", o.lam), ("rho", o.rho), ("n_prefill_frac", o.n_prefill_frac),
                             ("n_decode_frac", o.n_decode_frac), ("ratio_pd", o.ratio_pd),
                             ("achieved_total_tok_s", o.achieved_total_tok_s)):
            assert _same(p[mine], theirs), (mine, p[mine], theirs)
    assert seen == {"ok", "infeasible_ttft", "infeasible_tpot"}


def test_allocate_ext_matches_oracle_bit_for_bit(pdlib):
    """Prefix-cache hit fraction and data-parallel prefill groups: every field against the oracle."""
    rnd = random.Random(23)
    status_names = {0: "ok", pdlib.PD_ERR_INFEASIBLE_TTFT: "infeasible_ttft", pdlib.PD_ERR_INFEASIBLE_TPOT: "infeasible_tpot"}
    seen = set()
    for trial in range(1500):
        n = rnd.randint(1, 8)
        batch = sorted(rnd.sample(range(1, 1024), n))
        tpot = sorted(rnd.uniform(0.002, 0.12) for _ in range(n))
        hit = rnd.choice([0.0, 0.5, rnd.uniform(0.0, 0.95)])
        groups = rnd.choice([1, 1, 2, 4, 8, 16])
        args = (rnd.uniform(1e3, 1e6), float(rnd.randint(16, 32768)), float(rnd.randint(1, 4096)), rnd.uniform(0.05, 8.0),
                rnd.uniform(0.001, 0.13), rnd.uniform(5e3, 2e5), batch, tpot, rnd.choice([0.0, 0.1]))
        o = A.allocate_ext(*args, prefix_hit_frac=hit, dp_groups=groups)
        p = pdlib.pd_allocate_ext(*args, prefix_hit_frac=hit, dp_groups=groups)
        assert status_names[p["status"]] == o.status
        seen.add(o.status)
        assert (p["feasible_batch"], p["n_prefill"], p["n_decode"], p["n_prefill_ceil"], p["n_decode_ceil"]) == \
               (o.feasible_batch, o.n_prefill, o.n_decode, o.n_prefill_ceil, o.n_decode_ceil)
        for mine, theirs in (("tp_prefill_eff", o.tp_prefill_eff), ("tp_decode_eff", o.tp_decode_eff), ("mu", o.mu),
                             ("lam", o.lam), ("rho", o.rho), ("n_prefill_frac", o.n_prefill_frac),
                             ("n_decode_frac", o.n_decode_frac), ("ratio_pd", o.ratio_pd),
                             ("achieved_total_tok_s", o.achieved_total_tok_s)):
            assert _same(p[mine], theirs), (mine, p[mine], theirs)
        if hit == 0.0 and groups == 1:
            q = pdlib.pd_allocate(*args)
            assert all(_same(q[k], p[k]) if isinstance(q[k], float) else q[k] == p[k] for k in q)
    assert seen == {"ok", "infeasible_ttft", "infeasible_tpot"}
    for bad in (dict(prefix_hit_frac=1.0), dict(prefix_hit_frac=-0.1), dict(dp_groups=0)):
        with pytest.raises(pdlib.PdError):
            pdlib.pd_allocate_ext(1e4, 10, 10, 1, 0.05, 1e4, [1], [0.01], **bad)


def test_allocate_worked_example(pdlib, worked_example):
    g = worked_example
    b = 34
    p = pdlib.pd_allocate(g["tp_total_tokens_per_min"] / 60.0, g["l_in"], g["l_out"], g["ttft_slo_s"], g["tpot_slo_s"],
                          g["prefill_max_tok_s"], [b], [b / g["tp_decode_eff"]], g["t_overhead_s"])
    assert p["status"] == 0
    assert (p["n_prefill"], p["n_decode"]) == (int(g["n_prefill"]), int(g["n_decode"]))
    assert abs(p["tp_prefill_eff"] - g["tp_prefill_eff_approx"]) <= g["tp_prefill_eff_tol"]
    assert abs(p["ratio_pd"] - g["ratio_pd_printed"]) <= g["ratio_pd_tol"]


def test_allocate_rejects_bad_arguments(pdlib):
    with pytest.raises(pdlib.PdError):
        pdlib.pd_allocate(-1.0, 10, 10, 1, 0.05, 1e4, [1], [0.01])
    with pytest.raises(pdlib.PdError):
        pdlib.pd_allocate(1e4, 10, 10, 1, 0.05, 1e4, [0], [0.01])
    with pytest.raises(pdlib.PdError):
        pdlib.pd_allocate(1e4, 10, 10, 1, 0.05, 1e4, [1], [float("nan")])


def test_queue_replay_matches_oracle(pdlib):
    rng = np.random.Generator(np.random.Philox(key=3))
    for n in (1, 2, 1000, 50_000):
        gaps = rng.exponential(0.3, size=n)
        svc = rng.exponential(0.25, size=n)
        soj, wait = pdlib.pd_queue_replay(gaps, svc)
        o_soj, o_wait = A.queue_replay(gaps.tolist(), svc.tolist())
        assert soj == o_soj and wait == o_wait
    with pytest.raises(pdlib.PdError):
        pdlib.pd_queue_replay(np.array([-1.0]), np.array([1.0]))


def test_workspace_bytes_and_config_validation(pdlib):
    cfg = pdlib.LayerConfig(512, 8, 2, 64, 1536, max_pos=256)
    small = pdlib.pd_workspace_bytes(cfg, 128, 4, 144)
    big = pdlib.pd_workspace_bytes(cfg, 1024, 4, 144)
    assert 0 < small < big and small % 256 == 0
    for bad in (pdlib.LayerConfig(512, 8, 3, 64, 1536), pdlib.LayerConfig(512, 8, 2, 96, 1536),
                pdlib.LayerConfig(500, 8, 2, 64, 1536)):
        with pytest.raises(pdlib.PdError) as e:
            pdlib.pd_workspace_bytes(bad, 128, 4, 144)
        assert e.value.status == pdlib.PD_ERR_UNSUPPORTED_SHAPE


def test_decode_attention_split_rule_through_the_workspace_size(pdlib):
    """pd_decode_attention_workspace_bytes is host arithmetic: B * n_q_heads * splits * (head_dim + 2) floats.  It
    pins the split rule the header documents: few blocks -> split up to about 112 blocks, never under 512 keys per
    split, and a block's key range capped near 2048 keys."""
    cfg = pdlib.LayerConfig(4096, 32, 8, 128, 64)

    def splits(b, kv):
        n = pdlib.pd_decode_attention_workspace_bytes(cfg, b, kv)
        per = b * 32 * 130 * 4
        assert n >= per and n < per * 65
        return round(n / per) if n % per == 0 else -(-n // per)   # the size is rounded up to 256 bytes

    assert splits(256, 2304) == 1          # the benchmark's decode shape: one block per (sequence, KV head)
    assert splits(256, 3071) == 1 and splits(256, 3072) == 2
    assert splits(16, 2304) == 1 and splits(16, 9216) == 5
    assert splits(64, 8192) == 4 and splits(128, 8192) == 4
    assert splits(1, 2304) == 4            # 8 blocks: split, but not below 512 keys
    assert splits(1, 511) == 1 and splits(4, 100000) == 49 and splits(1, 100000) == 49
    assert splits(1, 200000) == 64         # upper limit


def test_workload_statistics_match_oracle_bit_for_bit(pdlib):
    rnd = random.Random(21)
    rng = np.random.Generator(np.random.Philox(key=21))
    for trial in range(200):
        n = rnd.randint(1, 3000)
        ls = rng.integers(16, 40000, size=n).astype(np.int32)
        grid_l = sorted(rnd.sample(range(16, 40000), rnd.randint(1, 40)))
        grid_t = sorted(rnd.uniform(1e-3, 3.0) for _ in grid_l)
        quantum = rnd.choice([1, 1, 64, 256])
        svc = pdlib.pd_interp_service_times(grid_l, grid_t, ls, quantum)
        o_svc = A.interp_service_times(grid_l, grid_t, ls.tolist(), quantum)
        assert svc.tolist() == o_svc
        tp, mean_l = pdlib.pd_mixture_throughput(ls, svc)
        assert (tp, mean_l) == A.mixture_throughput(ls.tolist(), o_svc)
        mu = tp / mean_l
        lam = rnd.uniform(0.05, 0.97) * mu
        assert pdlib.pd_mm1_sojourn(mu, lam) == A.mm1_sojourn(mu, lam)
        if lam * (sum(o_svc) / n) < 0.999:
            assert pdlib.pd_mg1_sojourn(svc, lam) == A.mg1_sojourn(o_svc, lam)
    with pytest.raises(pdlib.PdError) as e:
        pdlib.pd_mm1_sojourn(1.0, 1.0)
    assert e.value.status == pdlib.PD_ERR_INFEASIBLE_TTFT
    with pytest.raises(pdlib.PdError) as e:
        pdlib.pd_mg1_sojourn([1.0, 1.0], 1.0)
    assert e.value.status == pdlib.PD_ERR_INFEASIBLE_TTFT
    with pytest.raises(pdlib.PdError):
        pdlib.pd_interp_service_times([10, 10], [1.0, 2.0], [5])
    with pytest.raises(pdlib.PdError):
        pdlib.pd_mixture_throughput([0], [1.0])


def test_refine_next_batch_matches_oracle(pdlib):
    rnd = random.Random(22)
    for trial in range(2000):
        n = rnd.randint(0, 14)
        batch = rnd.sample(range(1, 600), n)
        tpot = [rnd.uniform(0.002, 0.12) for _ in range(n)]
        if trial % 2:
            order = sorted(range(n), key=lambda i: batch[i])     # a monotone curve every other trial
            srt = sorted(tpot)
            for rank, i in enumerate(order):
                tpot[i] = srt[rank]
        slo = rnd.uniform(0.001, 0.13)
        assert pdlib.pd_refine_next_batch(batch, tpot, slo) == A.refine_next_batch(batch, tpot, slo)


def test_binding_constants_match_the_header(pdlib):
    """Status codes and wait-injection kinds of the Python binding are the header's enumerators."""
    import os
    import re
    hdr = open(os.path.join(os.path.dirname(__file__), "..", "include", "pd.h")).read()
    enums = dict((m.group(1), int(m.group(2))) for m in re.finditer(r"\b(PD_[A-Z0-9_]+)\s*=\s*(-?\d+)", hdr))
    for name in ("PD_OK", "PD_ERR_INVALID_ARG", "PD_ERR_UNSUPPORTED_SHAPE", "PD_ERR_DEVICE_TIMEOUT"):
        assert getattr(pdlib, name) == enums[name], name
    for name in ("NONE", "ATTN_PREFILL", "GEMM", "GEMM_PAIR", "GEMM_FP8_BLOCKWISE"):
        assert getattr(pdlib, "INJECT_" + name) == enums["PD_INJECT_" + name], name
    # an injection kind outside the enumeration is refused (no GPU needed: the check precedes any device call)
    with pytest.raises(pdlib.PdError) as e:
        pdlib.pd_test_inject_wait_timeout(max(v for k, v in enums.items() if k.startswith("PD_INJECT_")) + 1, 1_000_000)
    assert e.value.status == pdlib.PD_ERR_INVALID_ARG
    pdlib.pd_test_inject_wait_timeout(pdlib.INJECT_NONE, 0)
