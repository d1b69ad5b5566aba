"""Pins for the allocation oracle: the paper's worked example, the algebraic
identities between Eq. 1-7 and Eq. 9-13, monotonicity, queueing closed forms and
brute force.  None of these re-type the oracle's own formulas as the expectation."""
import math
import random

import numpy as np
import pytest

from oracle import allocation as A


def test_worked_example_matches_paper(worked_example):
    g = worked_example
    tp_total = g["tp_total_tokens_per_min"] / 60.0
    tp_p = A.effective_prefill_throughput(g["prefill_max_tok_s"], g["l_in"], g["ttft_slo_s"], g["t_overhead_s"])
    assert abs(tp_p - g["tp_prefill_eff_approx"]) <= g["tp_prefill_eff_tol"]
    # one-point "curve": the paper reads ~1700 tok/s at the TPOT-feasible batch off Fig. 2
    b = 34
    alloc = A.allocate(tp_total, g["l_in"], g["l_out"], g["ttft_slo_s"], g["tpot_slo_s"],
                       g["prefill_max_tok_s"], [b], [b / g["tp_decode_eff"]], g["t_overhead_s"])
    assert alloc.status == "ok"
    assert alloc.tp_decode_eff == pytest.approx(g["tp_decode_eff"], rel=1e-12)
    assert (alloc.n_prefill, alloc.n_decode) == (int(g["n_prefill"]), int(g["n_decode"]))
    assert abs(alloc.ratio_pd - g["ratio_pd_printed"]) <= g["ratio_pd_tol"]
    # The paper rounds TP_prefill to 25000 before Eq. 7: that reproduces its printed ratio
    r_rounded = (g["l_in"] * g["tp_decode_eff"]) / (g["l_out"] * g["tp_prefill_eff_approx"])
    assert round(r_rounded, 2) == g["ratio_pd_printed"]
    # model-predicted sustained throughput is on the same side of the target as the measurement
    mtpm_34 = alloc.achieved_total_tok_s * 60 / 1e6
    mtpm_33 = A.achieved_total_throughput(3, 3, alloc.tp_prefill_eff, alloc.tp_decode_eff, g["l_in"], g["l_out"]) * 60 / 1e6
    assert 4.5 < mtpm_34 < 5.0 and abs(mtpm_34 - g["measured_3p4d_mtpm"]) < 0.3
    assert mtpm_33 < mtpm_34 and abs(mtpm_33 - g["measured_3p3d_mtpm"]) < 0.5
    # 3P3D is decode (TPOT) bound, as the paper observes
    side_p = 3 * alloc.tp_prefill_eff * (g["l_in"] + g["l_out"]) / g["l_in"]
    side_d = 3 * alloc.tp_decode_eff * (g["l_in"] + g["l_out"]) / g["l_out"]
    assert side_d < side_p


def test_eq13_is_eq12_solved_for_throughput():
    rnd = random.Random(1)
    for _ in range(200):
        tp_max = rnd.uniform(1e3, 1e5)
        l_in = rnd.uniform(16, 32768)
        t_over = rnd.uniform(0, 0.5)
        mu = A.service_rate(tp_max, l_in)
        ttft = t_over + (1.0 / mu) * rnd.uniform(1.05, 50)
        tp = A.effective_prefill_throughput(tp_max, l_in, ttft, t_over)
        lam = tp / l_in                       # Eq. 10-11: TP = TP_max * lambda / mu
        assert A.mm1_sojourn(mu, lam) == pytest.approx(ttft - t_over, rel=1e-9)
        assert tp == pytest.approx(tp_max * (lam / mu), rel=1e-12)


def test_counts_balance_the_pipeline_and_recover_eq1():
    rnd = random.Random(2)
    for _ in range(200):
        tp_total = rnd.uniform(1e3, 1e6)
        l_in, l_out = rnd.uniform(16, 32768), rnd.uniform(1, 4096)
        tp_p, tp_d = rnd.uniform(1e3, 1e5), rnd.uniform(1e2, 1e4)
        b = 8
        al = A.allocate(tp_total, l_in, l_out, 1e9, 1.0, tp_p, [b], [b / tp_d], 0.0)
        n_req = rnd.uniform(1, 1e6)
        t_p, t_d = A.phase_times(n_req, l_in, l_out, al.tp_prefill_eff, al.tp_decode_eff,
                                 al.n_prefill_frac, al.n_decode_frac)
        assert t_p == pytest.approx(t_d, rel=1e-9)                                    # Eq. 4
        assert A.total_throughput(n_req, l_in, l_out, t_p) == pytest.approx(tp_total, rel=1e-9)   # Eq. 1
        assert al.n_prefill_frac / al.n_decode_frac == pytest.approx(al.ratio_pd, rel=1e-9)     # Eq. 7
        # with fractional counts the deployment sustains exactly the target
        assert A.achieved_total_throughput(al.n_prefill_frac, al.n_decode_frac, al.tp_prefill_eff,
                                           al.tp_decode_eff, l_in, l_out) == pytest.approx(tp_total, rel=1e-9)


def test_insights_after_eq13():
    # lower TTFT -> lower effective throughput; higher max throughput -> higher utilisation
    tps = [A.effective_prefill_throughput(28300, 6144, t, 0.1) for t in (0.5, 1, 2, 4, 8)]
    assert all(a < b for a, b in zip(tps, tps[1:]))
    rhos = []
    for tp_max in (1e4, 2e4, 4e4, 8e4):
        al = A.allocate(1e5, 6144, 512, 2.0, 1.0, tp_max, [1], [0.01], 0.1)
        rhos.append(al.rho)
    assert all(a < b for a, b in zip(rhos, rhos[1:]))


def test_infeasible_cases():
    al = A.allocate(1e5, 6144, 512, 0.1, 0.02, 28300, [1, 2], [0.01, 0.03], 0.1)
    assert al.status == "infeasible_ttft"
    al = A.allocate(1e5, 6144, 512, 0.3, 0.02, 28300, [1, 2], [0.01, 0.03], 0.0)   # 6144/0.3 > 28300? no: 20480 < 28300
    assert al.status == "ok"
    al = A.allocate(1e5, 6144, 512, 0.2, 0.02, 28300, [1, 2], [0.01, 0.03], 0.0)   # 30720 > 28300
    assert al.status == "infeasible_ttft" and al.feasible_batch == 1
    al = A.allocate(1e5, 6144, 512, 2.0, 0.005, 28300, [1, 2], [0.01, 0.03], 0.0)
    assert al.status == "infeasible_tpot" and al.feasible_batch == 0


def test_feasible_batch_brute_force():
    rnd = random.Random(3)
    for trial in range(300):
        n = rnd.randint(1, 12)
        batch = sorted(rnd.sample(range(1, 600), n))
        if trial % 2 == 0:
            tpot = sorted(rnd.uniform(0.001, 0.1) for _ in range(n))
        else:
            tpot = [rnd.uniform(0.001, 0.1) for _ in range(n)]
        perm = list(range(n))
        rnd.shuffle(perm)
        slo = rnd.uniform(0.0, 0.11)
        # brute force over every candidate: all points with B' <= B feasible
        expect = 0
        for i in range(n):
            if all(tpot[j] <= slo for j in range(n) if batch[j] <= batch[i]):
                expect = max(expect, batch[i])
        idx, b_star, capped = A.feasible_batch([batch[p] for p in perm], [tpot[p] for p in perm], slo)
        assert b_star == expect
        assert capped == (expect == batch[-1])
        if trial % 2 == 0 and expect:       # monotone curve: equals plain "largest feasible"
            assert expect == max(b for b, t in zip(batch, tpot) if t <= slo)


def test_rounding_rule():
    assert [A.round_count(v) for v in (0.01, 0.49, 0.5, 1.49, 1.5, 3.07, 3.77)] == [1, 1, 1, 1, 2, 3, 4]
    assert [A.ceil_count(v) for v in (0.01, 1.0, 1.0001, 3.07, 3.77)] == [1, 1, 2, 4, 4]


def test_queue_replay_mm1_and_md1_closed_forms():
    n = 400_000
    mu = 4.0
    rng = np.random.Generator(np.random.Philox(key=7))
    for rho in (0.3, 0.7):
        lam = rho * mu
        gaps = rng.exponential(1.0 / lam, size=n)
        svc = rng.exponential(1.0 / mu, size=n)
        soj, wait = A.queue_replay(gaps.tolist(), svc.tolist())
        # M/M/1 sojourn variance is 1/(mu-lam)^2; correlated samples -> generous 5% band
        assert soj == pytest.approx(A.mm1_sojourn(mu, lam), rel=0.05)
        soj_d, _ = A.queue_replay(gaps.tolist(), [1.0 / mu] * n)
        assert soj_d == pytest.approx(A.md1_sojourn(mu, lam), rel=0.03)
        assert soj_d < soj
        assert A.pollaczek_khinchine_sojourn(lam, 1 / mu, 1 / mu ** 2) == pytest.approx(A.md1_sojourn(mu, lam), rel=1e-12)
        assert A.pollaczek_khinchine_sojourn(lam, 1 / mu, 2 / mu ** 2) == pytest.approx(A.mm1_sojourn(mu, lam), rel=1e-12)


def test_queue_replay_hand_case():
    # arrivals at t=0,1,2 ; services 3,1,1 -> waits 0,2,2 ; sojourns 3,3,3
    soj, wait = A.queue_replay([0.0, 1.0, 1.0], [3.0, 1.0, 1.0])
    assert soj == pytest.approx(3.0) and wait == pytest.approx(4.0 / 3.0)
    # idle server: no waiting
    soj, wait = A.queue_replay([0.0, 10.0, 10.0], [3.0, 1.0, 2.0])
    assert wait == 0.0 and soj == pytest.approx(2.0)


# ------------------------------------------------ prefix cache and data-parallel prefill groups
def test_allocate_ext_defaults_equal_the_paper_case_bit_for_bit():
    rnd = random.Random(5)
    for _ in range(200):
        args = (rnd.uniform(1e3, 1e6), rnd.uniform(16, 30000), rnd.uniform(1, 4000), rnd.uniform(0.2, 8.0),
                rnd.uniform(0.005, 0.2), rnd.uniform(1e3, 2e5), [1, 2, 4, 8], [rnd.uniform(0.004, 0.3) for _ in range(4)])
        a, b = A.allocate(*args), A.allocate_ext(*args)
        for f in a.__dataclass_fields__:
            x, y = getattr(a, f), getattr(b, f)
            assert x == y or (isinstance(x, float) and math.isnan(x) and math.isnan(y)), f


def test_dp_groups_are_independent_mm1_queues():
    """G groups, each with 1/G of the instance's maximum throughput and 1/G of its arrivals: every group's
    M/M/1 sojourn time is the TTFT budget, and a replay of ONE group's queue (exponential gaps at lam,
    exponential service at mu) reproduces it."""
    tp_max, l_in, ttft, over = 80_000.0, 2048.0, 1.5, 0.1
    one = A.allocate_ext(2e5, l_in, 256.0, ttft, 0.05, tp_max, [8], [0.02], over)
    rng = np.random.Generator(np.random.Philox(key=11))
    for g in (1, 2, 4, 8):
        a = A.allocate_ext(2e5, l_in, 256.0, ttft, 0.05, tp_max, [8], [0.02], over, dp_groups=g)
        assert a.status == "ok"
        assert 1.0 / (a.mu - a.lam) == pytest.approx(ttft - over, rel=1e-12)          # Eq. 12 per group
        assert a.mu == pytest.approx(tp_max / g / l_in, rel=1e-15)
        # the instance loses the same L_in / budget per group: linear in G
        assert tp_max - a.tp_prefill_eff == pytest.approx(g * (tp_max - one.tp_prefill_eff), rel=1e-12)
        assert a.n_prefill_frac >= one.n_prefill_frac
        n = 300_000
        soj, _ = A.queue_replay(rng.exponential(1.0 / a.lam, size=n).tolist(), rng.exponential(1.0 / a.mu, size=n).tolist())
        assert soj == pytest.approx(ttft - over, rel=0.06)
    # so many groups that a lone request already misses the budget
    assert A.allocate_ext(2e5, l_in, 256.0, ttft, 0.05, tp_max, [8], [0.02], over, dp_groups=64).status == "infeasible_ttft"


def test_prefix_cache_hits_shorten_the_effective_input():
    base = dict(tp_total=2e5, l_in=4096.0, l_out=256.0, ttft_slo=2.0, tpot_slo=0.05, prefill_max_tok_s=8e4,
                batch=[64, 128], tpot=[0.03, 0.045])
    prev = None
    for hit in (0.0, 0.25, 0.5, 0.9):
        a = A.allocate_ext(**base, prefix_hit_frac=hit)
        # the service rate of Eq. 9 rises as 1 / (1 - hit): only the missed tokens are computed
        assert a.mu * (1.0 - hit) == pytest.approx(8e4 / 4096.0, rel=1e-12)
        # with hit fraction h the method sees a workload of input length L_in (1 - h)
        b = A.allocate(2e5, 4096.0 * (1.0 - hit), 256.0, 2.0, 0.05, 8e4, [64, 128], [0.03, 0.045])
        assert (a.n_prefill, a.n_decode, a.feasible_batch) == (b.n_prefill, b.n_decode, b.feasible_batch)
        if prev is not None:
            assert a.tp_prefill_eff > prev.tp_prefill_eff          # Eq. 13: a shorter input costs less queueing
            assert a.ratio_pd < prev.ratio_pd                      # Eq. 7: fewer prefill instances per decode instance
        prev = a
    with pytest.raises(ValueError):
        A.allocate_ext(**base, prefix_hit_frac=1.0)
    with pytest.raises(ValueError):
        A.allocate_ext(**base, dp_groups=0)


def test_mixture_throughput_special_cases():
    # equal requests: the mix runs at L / t; mean length L
    tp, mean_l = A.mixture_throughput([4096] * 7, [0.05] * 7)
    assert tp == pytest.approx(4096 / 0.05, rel=1e-12) and mean_l == 4096
    # hand case: 1000 tokens in 1 s and 3000 tokens in 1 s -> 2000 tok/s, mean 2000
    assert A.mixture_throughput([1000, 3000], [1.0, 1.0]) == (2000.0, 2000.0)
    # a server that replays the mix back to back is busy sum(t) and emits sum(L): Eq. 9's mu = tp / mean_l
    rnd = random.Random(4)
    ls = [rnd.randint(100, 9000) for _ in range(500)]
    ts = [1e-5 * l + 1e-9 * l * l for l in ls]
    tp, mean_l = A.mixture_throughput(ls, ts)
    assert A.service_rate(tp, mean_l) == pytest.approx(len(ls) / sum(ts), rel=1e-12)   # requests per busy second
    with pytest.raises(ValueError):
        A.mixture_throughput([1, 2], [1.0])


def test_mg1_sojourn_reduces_to_md1_and_mm1_and_matches_a_replay():
    mu = 5.0
    assert A.mg1_sojourn([1 / mu] * 100, 3.0) == pytest.approx(A.md1_sojourn(mu, 3.0), rel=1e-12)
    rng = np.random.Generator(np.random.Philox(key=17))
    svc = rng.exponential(1 / mu, size=400_000)
    # exponential samples: E[S^2] ~ 2 / mu^2, so the M/G/1 mean approaches Eq. 12
    assert A.mg1_sojourn(svc.tolist(), 3.0) == pytest.approx(A.mm1_sojourn(mu, 3.0), rel=0.02)
    # a two-point service distribution replayed through the queue agrees with the formula
    two = np.where(rng.random(400_000) < 0.8, 0.05, 0.6)
    lam = 0.7 / two.mean()
    soj, _ = A.queue_replay(rng.exponential(1 / lam, size=two.size).tolist(), two.tolist())
    assert soj == pytest.approx(A.mg1_sojourn(two.tolist(), lam), rel=0.05)
    with pytest.raises(ValueError):
        A.mg1_sojourn([1.0, 1.0], 1.0)


def test_interp_service_times_against_numpy():
    rnd = random.Random(6)
    grid_l = sorted(rnd.sample(range(100, 40000), 9))
    grid_t = sorted(rnd.uniform(0.01, 2.0) for _ in grid_l)
    ls = [rnd.randint(50, 41000) for _ in range(300)] + grid_l
    got = A.interp_service_times(grid_l, grid_t, ls)
    np.testing.assert_allclose(got, np.interp(ls, grid_l, grid_t), rtol=1e-12)
    # exact at the grid points and on a straight line
    assert A.interp_service_times([10, 20], [1.0, 2.0], [10, 15, 20, 5, 30]) == [1.0, 1.5, 2.0, 1.0, 2.0]
    # tile quantum: a length counts as the next multiple of the quantum (a step function on a grid of multiples)
    assert A.interp_service_times([8, 16, 24], [1.0, 2.0, 4.0], [1, 8, 9, 16, 17, 24], quantum=8) == [1.0, 1.0, 2.0, 2.0, 4.0, 4.0]
    assert A.interp_service_times([8, 24], [1.0, 3.0], [9, 13], quantum=4) == [1.5, 2.0]


def test_refine_next_batch_brackets_the_largest_feasible_integer():
    rnd = random.Random(5)
    for _ in range(300):
        a, b0 = rnd.uniform(1e-5, 2e-4), rnd.uniform(1e-3, 5e-3)
        curve = lambda b: b0 + a * b                     # TPOT grows with the batch
        batch = [1, 2, 4, 8, 16, 32, 64, 128, 256, 512]
        tpot = [curve(b) for b in batch]
        slo = rnd.uniform(b0 + a, b0 + 600 * a)
        probes = 0
        while True:
            nxt = A.refine_next_batch(batch, tpot, slo)
            if nxt == 0:
                break
            assert nxt not in batch
            batch.append(nxt); tpot.append(curve(nxt)); probes += 1
        feas = [b for b in range(1, 513) if curve(b) <= slo]       # brute force over every integer
        _, b_star, capped = A.feasible_batch(batch, tpot, slo)
        assert b_star == (max(feas) if feas else 0)
        assert probes <= 8 and capped == (b_star == 512)
    assert A.refine_next_batch([4, 8], [0.1, 0.2], 0.05) == 0       # nothing feasible
    assert A.refine_next_batch([4, 8], [0.01, 0.02], 0.05) == 0     # nothing infeasible: capped by the sweep
    assert A.refine_next_batch([8, 4, 5], [0.2, 0.01, 0.3], 0.05) == 0   # neighbours
