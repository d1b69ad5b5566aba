"""Re-checks a result file of the configuration drivers against the allocation oracle.

Every allocation the drivers store carries the exact inputs it was computed from (the measured
maximum prefill throughput and the measured TPOT curve among them).  Feeding those inputs to
oracle.allocation must reproduce the stored result: integers bit for bit, doubles equal.  The
check needs no GPU, so the same file can be verified on the machine that measured it and later
on one without a device.
"""
import math

import pd_inputs as gen
from oracle import allocation as A

STATUS = {0: "ok", -6: "infeasible_ttft", -7: "infeasible_tpot"}
INT_KEYS = ("feasible_batch", "n_prefill", "n_decode", "n_prefill_ceil", "n_decode_ceil")
DBL_KEYS = ("tp_prefill_eff", "tp_decode_eff", "mu", "rho", "n_prefill_frac", "n_decode_frac", "ratio_pd",
            "achieved_total_tok_s")


def _same(a, b):
    return (isinstance(a, float) and isinstance(b, float) and math.isnan(a) and math.isnan(b)) or a == b


def check_allocation(node, where, pd=None):
    i = node["inputs"]
    args = (i["tp_total_tok_s"], i["l_in"], i["l_out"], i["ttft_slo_s"], i["tpot_slo_s"], i["prefill_max_tok_s"],
            i["batch"], i["tpot_s"], i["t_overhead_s"])
    ref = A.allocate(*args)
    sources = [("stored", node)]
    if pd is not None:
        sources.append(("pd_allocate", pd.pd_allocate(*args)))
    for name, got in sources:
        assert STATUS[got["status"]] == ref.status, (where, name)
        for k in INT_KEYS:
            assert int(got[k]) == getattr(ref, k), (where, name, k, got[k], getattr(ref, k))
        assert bool(got["sweep_capped"]) == ref.sweep_capped, (where, name)
        for k in DBL_KEYS:
            assert _same(float(got[k]), float(getattr(ref, k))), (where, name, k, got[k], getattr(ref, k))
        assert _same(float(got["lam"]), float(ref.lam)), (where, name, "lam")


def walk_allocations(node, where=""):
    if isinstance(node, dict):
        if "inputs" in node and "feasible_batch" in node:
            yield where, node
        for k, v in node.items():
            yield from walk_allocations(v, f"{where}/{k}")
    elif isinstance(node, list):
        for j, v in enumerate(node):
            yield from walk_allocations(v, f"{where}[{j}]")


def check_result(res, pd=None):
    """Returns the number of allocations checked."""
    n = 0
    for where, node in walk_allocations(res):
        check_allocation(node, where, pd)
        n += 1
        if "refined" in node:
            # the refinement stopped because the bracket closed (or it ran out of probes): the refined batch is
            # feasible, at least the sweep's, and the oracle's step rule agrees with the stored probe sequence
            r, i = node["refined"], node["refined"]["inputs"]
            assert r["feasible_batch"] >= node["feasible_batch"]
            pts_b, pts_t = list(node["inputs"]["batch"]), list(node["inputs"]["tpot_s"])
            for b, t in r["probes"]:
                assert A.refine_next_batch(pts_b, pts_t, i["tpot_slo_s"]) == b, where
                pts_b.append(b); pts_t.append(t)
            assert pts_b == i["batch"] and pts_t == i["tpot_s"]
    if res.get("config") == "long_input":
        lengths = gen.lognormal_lengths(1, 4096, 8192.0, 0.5, 2048, 32768)
        g = res["prefill_time_grid"]
        quantum = res.get("tile_quantum", 1)
        svc = A.interp_service_times(g["l"], g["time_s"], lengths.tolist(), quantum)
        tp, mean_l = A.mixture_throughput(lengths.tolist(), svc)
        assert tp == res["prefill_max_tok_s"] and mean_l == res["mean_l_in"]
        mu = A.service_rate(tp, mean_l)
        assert mu == res["allocation"]["mu"]
        for q in res["queue"]:
            assert q["mm1_sojourn_s"] == A.mm1_sojourn(mu, q["lambda"])
            assert q["pollaczek_khinchine_s"] == A.mg1_sojourn(svc, q["lambda"])
            # the replay of the measured (far from exponential) service times sits at the M/G/1 mean; Eq. 12 is
            # the pessimistic side for a service distribution with coefficient of variation below one
            if q["rho"] <= 0.9:
                assert abs(q["replayed_sojourn_s"] / q["pollaczek_khinchine_s"] - 1.0) < 0.15
            es, es2 = A.service_moments(svc)
            if es2 <= 2.0 * es * es:
                assert q["pollaczek_khinchine_s"] <= q["mm1_sojourn_s"] * (1 + 1e-12)
        for c in res["interpolation_check"]:
            assert c["interpolated_s"] == A.interp_service_times(g["l"], g["time_s"], [c["l"]], quantum)[0]
    if res.get("config") == "70b":
        m = res["mixed"]
        l_in = gen.uniform_lengths(3, 512, 1024, 8192, sub=0)
        g = m["prefill_time_grid"]
        tp, mean_l = A.mixture_throughput(l_in.tolist(), A.interp_service_times(g["l"], g["time_s"], l_in.tolist(),
                                                                                m.get("tile_quantum", 1)))
        assert tp == m["prefill_max_tok_s"] and mean_l == m["mean_l_in"]
    return n
