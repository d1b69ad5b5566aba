"""CPU oracle for the P/D allocation model (Eq. 1-13) and the TTFT queue replay.

TEST INFRASTRUCTURE ONLY: shares no code with the GPU library's host-side
`pd_allocate` / `pd_queue_replay` and is never imported by the product path.

Every function is the paper's closed form written out in IEEE double (Python
floats), in the parenthesisation given in its docstring, so that integer
results can be compared bit-exactly with an independent implementation.

Readings where the paper is silent:
  * instance counts are rounded to nearest (half up, at least 1): the only simple
    rule that reproduces the Evaluation section's 3P4D from 3.07 and 3.77; the
    ceiling is returned alongside as the SLO-safe count;
  * the TPOT-feasible batch is the largest sweep point such that every sweep point
    up to and including it meets the SLO (no interpolation);
  * T_overhead is an explicit input;
  * a workload of mixed input lengths ("Preliminaries" takes L_in and L_out as averages): the
    maximum prefill throughput of the mix is its total tokens over its total service time,
    and L_in in Eq. 5-13 is the mean length;
  * the integer between two sweep points of the TPOT curve is found by measuring at the
    midpoint of the bracket [largest feasible, smallest infeasible] until they are neighbours;
  * prefix caching ("Acquire prefill throughput under TTFT constraints", closing remark): the
    input length is replaced, everywhere it occurs in Eq. 1-13, by the length that misses
    the cache, L_in (1 - hit fraction); throughputs then count computed tokens;
  * prefill data parallelism (same section): each of the G groups of an instance is its own
    M/M/1 queue with 1/G of the instance's maximum throughput, so Eq. 13 becomes
    TP_prefill = TP_max - G L_in / (TTFT - T_overhead); G = 1 is the paper's case.
"""
from __future__ import annotations

import math
from dataclasses import dataclass


def total_throughput(n_req: float, l_in: float, l_out: float, t_total: float) -> float:
    """Eq. 1: TP_total = N_req (L_in + L_out) / T_total."""
    return n_req * (l_in + l_out) / t_total


def phase_times(n_req, l_in, l_out, tp_prefill, tp_decode, n_prefill, n_decode):
    """Eq. 2-3: (T_prefill, T_decode)."""
    return (n_req * l_in / (tp_prefill * n_prefill),
            n_req * l_out / (tp_decode * n_decode))


def service_rate(tp_prefill_max: float, l_in: float) -> float:
    """Eq. 9: mu = max prefill throughput / L_in."""
    return tp_prefill_max / l_in


def mm1_sojourn(mu: float, lam: float) -> float:
    """Eq. 12: T_s = 1 / (mu - lambda), lambda < mu."""
    if not lam < mu:
        raise ValueError("arrival rate must be below the service rate")
    return 1.0 / (mu - lam)


def effective_prefill_throughput(tp_prefill_max, l_in, ttft, t_overhead=0.0) -> float:
    """Eq. 13: TP_prefill = TP_max - L_in / (TTFT - T_overhead)."""
    budget = ttft - t_overhead
    if not budget > 0.0:
        raise ValueError("TTFT budget is not positive")
    return tp_prefill_max - l_in / budget


def feasible_batch(batch, tpot, tpot_slo):
    """Section "Acquire decode throughput under TPOT constraints".

    Sweep points sorted by batch size; returns (index, B*, capped) of the largest
    point whose whole prefix satisfies tpot <= slo, or (-1, 0, False) if none.
    """
    order = sorted(range(len(batch)), key=lambda i: batch[i])
    best = -1
    for i in order:
        if tpot[i] <= tpot_slo:
            best = i
        else:
            break
    if best < 0:
        return -1, 0, False
    return best, int(batch[best]), best == order[-1]


def round_count(n: float) -> int:
    return max(1, int(math.floor(n + 0.5)))


def ceil_count(n: float) -> int:
    return max(1, int(math.ceil(n)))


def achieved_total_throughput(n_prefill, n_decode, tp_prefill, tp_decode, l_in, l_out) -> float:
    """Total tokens/s an mPnD deployment sustains: Eq. 1 with T_total = max of Eq. 2-3."""
    side_p = n_prefill * tp_prefill * (l_in + l_out) / l_in
    side_d = n_decode * tp_decode * (l_in + l_out) / l_out
    return min(side_p, side_d)


@dataclass
class Allocation:
    status: str               # "ok" | "infeasible_ttft" | "infeasible_tpot"
    tp_prefill_eff: float = math.nan
    tp_decode_eff: float = math.nan
    mu: float = math.nan
    lam: float = math.nan
    rho: float = math.nan
    feasible_batch: int = 0
    sweep_capped: bool = False
    n_prefill_frac: float = math.nan
    n_decode_frac: float = math.nan
    ratio_pd: float = math.nan
    n_prefill: int = 0
    n_decode: int = 0
    n_prefill_ceil: int = 0
    n_decode_ceil: int = 0
    achieved_total_tok_s: float = math.nan


def allocate(tp_total, l_in, l_out, ttft_slo, tpot_slo, prefill_max_tok_s,
             batch, tpot, t_overhead=0.0) -> Allocation:
    """Full pipeline: Eq. 13 -> feasible batch -> Eq. 5, 6, 7 -> integer counts."""
    a = Allocation(status="ok")
    a.mu = prefill_max_tok_s / l_in                                   # Eq. 9
    budget = ttft_slo - t_overhead                                     # Eq. 12
    if budget > 0.0:
        a.tp_prefill_eff = prefill_max_tok_s - l_in / budget           # Eq. 13
    if not (budget > 0.0 and a.tp_prefill_eff > 0.0):
        a.status = "infeasible_ttft"
    else:
        a.lam = a.tp_prefill_eff / l_in                                # Eq. 10-11
        a.rho = a.lam / a.mu                                           # Eq. 10

    idx, b_star, capped = feasible_batch(batch, tpot, tpot_slo)
    if idx < 0:
        if a.status == "ok":
            a.status = "infeasible_tpot"
    else:
        a.feasible_batch = b_star
        a.sweep_capped = capped
        a.tp_decode_eff = b_star / tpot[idx]

    if a.status != "ok":
        return a
    a.n_prefill_frac = (tp_total * l_in) / ((l_in + l_out) * a.tp_prefill_eff)   # Eq. 5
    a.n_decode_frac = (tp_total * l_out) / ((l_in + l_out) * a.tp_decode_eff)    # Eq. 6
    a.ratio_pd = (l_in * a.tp_decode_eff) / (l_out * a.tp_prefill_eff)           # Eq. 7
    a.n_prefill = round_count(a.n_prefill_frac)
    a.n_decode = round_count(a.n_decode_frac)
    a.n_prefill_ceil = ceil_count(a.n_prefill_frac)
    a.n_decode_ceil = ceil_count(a.n_decode_frac)
    a.achieved_total_tok_s = achieved_total_throughput(
        a.n_prefill, a.n_decode, a.tp_prefill_eff, a.tp_decode_eff, l_in, l_out)
    return a


def allocate_ext(tp_total, l_in, l_out, ttft_slo, tpot_slo, prefill_max_tok_s, batch, tpot,
                 t_overhead=0.0, prefix_hit_frac=0.0, dp_groups=1) -> Allocation:
    """`allocate` with a prefix-cache hit fraction and G data-parallel prefill groups.

    mu, lam, rho describe ONE group: mu = (TP_max / G) / L, lam = (TP_prefill / G) / L with
    L the non-cached input length; everything else is per instance.
    """
    if not (0.0 <= prefix_hit_frac < 1.0) or dp_groups < 1:
        raise ValueError("hit fraction in [0, 1), at least one group")
    l_eff = l_in * (1.0 - prefix_hit_frac)
    g = float(dp_groups)
    a = Allocation(status="ok")
    a.mu = (prefill_max_tok_s / g) / l_eff                             # Eq. 9 for one group
    budget = ttft_slo - t_overhead
    if budget > 0.0:
        a.tp_prefill_eff = prefill_max_tok_s - (g * l_eff) / budget    # Eq. 13, G queues
    if not (budget > 0.0 and a.tp_prefill_eff > 0.0):
        a.status = "infeasible_ttft"
    else:
        a.lam = (a.tp_prefill_eff / g) / l_eff
        a.rho = a.lam / a.mu
    idx, b_star, capped = feasible_batch(batch, tpot, tpot_slo)
    if idx < 0:
        if a.status == "ok":
            a.status = "infeasible_tpot"
    else:
        a.feasible_batch = b_star
        a.sweep_capped = capped
        a.tp_decode_eff = b_star / tpot[idx]
    if a.status != "ok":
        return a
    a.n_prefill_frac = (tp_total * l_eff) / ((l_eff + l_out) * a.tp_prefill_eff)
    a.n_decode_frac = (tp_total * l_out) / ((l_eff + l_out) * a.tp_decode_eff)
    a.ratio_pd = (l_eff * a.tp_decode_eff) / (l_out * a.tp_prefill_eff)
    a.n_prefill = round_count(a.n_prefill_frac)
    a.n_decode = round_count(a.n_decode_frac)
    a.n_prefill_ceil = ceil_count(a.n_prefill_frac)
    a.n_decode_ceil = ceil_count(a.n_decode_frac)
    a.achieved_total_tok_s = achieved_total_throughput(
        a.n_prefill, a.n_decode, a.tp_prefill_eff, a.tp_decode_eff, l_eff, l_out)
    return a


def queue_replay(arrival_gaps, service_times):
    """FIFO single-server replay (Lindley recursion).

    Request n arrives gaps[n] after request n-1 (request 0 at time gaps[0]) and
    needs service_times[n].  Returns (mean sojourn, mean wait): sojourn = wait +
    service, the quantity Eq. 12 predicts as 1 / (mu - lambda).
    """
    wait = 0.0
    sum_wait = 0.0
    sum_soj = 0.0
    n = len(service_times)
    prev_service = 0.0
    for i in range(n):
        if i > 0:
            wait = max(0.0, wait + prev_service - arrival_gaps[i])
        sum_wait += wait
        sum_soj += wait + service_times[i]
        prev_service = service_times[i]
    return sum_soj / n, sum_wait / n


def md1_sojourn(mu: float, lam: float) -> float:
    """Textbook M/D/1 mean sojourn: 1/mu + rho / (2 mu (1 - rho))."""
    rho = lam / mu
    return 1.0 / mu + rho / (2.0 * mu * (1.0 - rho))


def pollaczek_khinchine_sojourn(lam: float, mean_s: float, mean_s2: float) -> float:
    """Textbook M/G/1 mean sojourn: E[S] + lambda E[S^2] / (2 (1 - rho))."""
    rho = lam * mean_s
    return mean_s + lam * mean_s2 / (2.0 * (1.0 - rho))


def _seq_sum(values) -> float:
    """Left-to-right IEEE double sum (the built-in sum() compensates, which another
    implementation need not do; the order is part of the definition here)."""
    acc = 0.0
    for v in values:
        acc += float(v)
    return acc


def mixture_throughput(l_in, service_times):
    """Maximum prefill throughput of a request mix served one request at a time.

    Request i has l_in[i] tokens and takes service_times[i] seconds alone on a saturated
    instance; the mix then runs at (sum of tokens) / (sum of times) tokens per second
    ("Acquire prefill throughput under TTFT constraints": the maximum throughput is what the
    instance sustains when continuously busy).  Returns (tp_max, mean input length).
    """
    n = len(l_in)
    if n == 0 or n != len(service_times):
        raise ValueError("need one service time per request")
    tokens = _seq_sum(l_in)
    busy = _seq_sum(service_times)
    return tokens / busy, tokens / n


def service_moments(service_times):
    """(E[S], E[S^2]) of the sampled service times, sums taken left to right."""
    n = len(service_times)
    return _seq_sum(service_times) / n, _seq_sum(float(s) * float(s) for s in service_times) / n


def mg1_sojourn(service_times, lam: float) -> float:
    """Mean sojourn of an M/G/1 queue whose service-time distribution is the sample's
    (Pollaczek-Khinchine); Eq. 12 is its special case for exponential service."""
    es, es2 = service_moments(service_times)
    if not lam * es < 1.0:
        raise ValueError("arrival rate must keep the server utilisation below one")
    return pollaczek_khinchine_sojourn(lam, es, es2)


def interp_service_times(grid_l, grid_t, lengths, quantum=1):
    """Service time of each length by linear interpolation between measured grid points
    (grid_l strictly increasing); lengths outside the grid take the end values.  A length is
    first rounded up to a multiple of `quantum` (a server that works in tiles of that many
    tokens takes as long for L tokens as for the next full tile)."""
    out = []
    n = len(grid_l)
    for l in lengths:
        l = -(-int(l) // quantum) * quantum
        if l <= grid_l[0]:
            out.append(float(grid_t[0]))
            continue
        if l >= grid_l[n - 1]:
            out.append(float(grid_t[n - 1]))
            continue
        i = 0
        while grid_l[i + 1] < l:
            i += 1
        w = (float(l) - float(grid_l[i])) / (float(grid_l[i + 1]) - float(grid_l[i]))
        out.append(grid_t[i] + (grid_t[i + 1] - grid_t[i]) * w)
    return out


def refine_next_batch(batch, tpot, tpot_slo) -> int:
    """Next batch size to measure when refining the TPOT-feasible batch to an integer
    ("Acquire decode throughput under TPOT constraints": determine the batch size that
    satisfies the target TPOT).  With the points measured so far sorted by batch size, lo is
    the largest one whose whole prefix meets the SLO and hi the first one that does not;
    the next measurement goes to floor((lo + hi) / 2).  Returns 0 when nothing is left to
    measure: no feasible point, no infeasible point, or lo and hi are neighbours."""
    order = sorted(range(len(batch)), key=lambda i: batch[i])
    lo = hi = 0
    for i in order:
        if tpot[i] <= tpot_slo:
            lo = int(batch[i])
        else:
            hi = int(batch[i])
            break
    if lo == 0 or hi == 0 or hi - lo <= 1:
        return 0
    return (lo + hi) // 2
