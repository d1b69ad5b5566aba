// Host-side scalar part of the library: the allocation model (Eq. 1-13) and the
// FIFO queue replay used to check the M/M/1 prediction of Eq. 12.
// Compiled with floating-point contraction off so that the integer results do not
// depend on whether the compiler fuses a multiply with an add.
#include <cmath>
#include <cstring>
#include <limits>
#include <vector>
#include <algorithm>

#include "pd.h"

namespace {

int32_t nearest_count(double n) {
  double r = std::floor(n + 0.5);
  if (!(r >= 1.0)) return 1;
  if (r > 2147483647.0) return 2147483647;
  return static_cast<int32_t>(r);
}

int32_t ceil_count(double n) {
  double r = std::ceil(n);
  if (!(r >= 1.0)) return 1;
  if (r > 2147483647.0) return 2147483647;
  return static_cast<int32_t>(r);
}

}  // namespace

extern "C" const char* pd_status_str(pd_status s) {
  switch (s) {
    case PD_OK: return "ok";
    case PD_ERR_INVALID_ARG: return "invalid argument";
    case PD_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
    case PD_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case PD_ERR_CUDA: return "CUDA error";
    case PD_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
    case PD_ERR_INFEASIBLE_TTFT: return "TTFT SLO infeasible";
    case PD_ERR_INFEASIBLE_TPOT: return "TPOT SLO infeasible";
    case PD_ERR_ARCH: return "device is not sm_100";
  }
  return "unknown status";
}

extern "C" int pd_version(void) { return 1; }

namespace {
pd_status allocate_impl(const pd_alloc_in* in, double prefix_hit_frac, int32_t dp_groups, pd_alloc_out* out);
}

extern "C" pd_status pd_allocate(const pd_alloc_in* in, pd_alloc_out* out) {
  return allocate_impl(in, 0.0, 1, out);
}

extern "C" pd_status pd_allocate_ext(const pd_alloc_in* in, double prefix_hit_frac, int32_t dp_groups,
                                     pd_alloc_out* out) {
  if (!(prefix_hit_frac >= 0.0) || !(prefix_hit_frac < 1.0) || dp_groups < 1) return PD_ERR_INVALID_ARG;
  return allocate_impl(in, prefix_hit_frac, dp_groups, out);
}

namespace {
// L_in is the input length that misses the prefix cache; the G data-parallel groups of a prefill instance
// are G M/M/1 queues with 1/G of its maximum throughput each (hit fraction 0 and G = 1: the paper's case,
// where the two extra factors are exact no-ops in IEEE arithmetic).
pd_status allocate_impl(const pd_alloc_in* in, double prefix_hit_frac, int32_t dp_groups, pd_alloc_out* out) {
  if (!in || !out || in->struct_size != sizeof(pd_alloc_in)) return PD_ERR_INVALID_ARG;
  const double nan = std::numeric_limits<double>::quiet_NaN();
  std::memset(out, 0, sizeof(*out));
  out->struct_size = sizeof(pd_alloc_out);
  out->tp_prefill_eff = out->tp_decode_eff = out->mu = out->lambda = out->rho = nan;
  out->n_prefill_frac = out->n_decode_frac = out->ratio_pd = out->achieved_total_tok_s = nan;

  const double L_in = in->l_in * (1.0 - prefix_hit_frac), L_out = in->l_out;
  const double G = static_cast<double>(dp_groups);
  if (!(in->tp_total_tok_s > 0.0) || !(in->l_in > 0.0) || !(L_out > 0.0) || !(in->prefill_max_tok_s > 0.0) ||
      !(in->tpot_slo_s > 0.0) || !(in->t_overhead_s >= 0.0) || in->n_points < 0 ||
      (in->n_points > 0 && (!in->batch || !in->tpot_s)))
    return PD_ERR_INVALID_ARG;
  for (int i = 0; i < in->n_points; ++i)
    if (in->batch[i] <= 0 || !(in->tpot_s[i] > 0.0)) return PD_ERR_INVALID_ARG;

  pd_status status = PD_OK;

  // Prefill side: service rate (Eq. 9), TTFT budget (Eq. 8, 12), effective throughput (Eq. 13).
  out->mu = (in->prefill_max_tok_s / G) / L_in;  // one group
  const double budget = in->ttft_slo_s - in->t_overhead_s;
  bool prefill_ok = false;
  if (budget > 0.0) {
    out->tp_prefill_eff = in->prefill_max_tok_s - (G * L_in) / budget;
    prefill_ok = out->tp_prefill_eff > 0.0;
  }
  if (prefill_ok) {
    out->lambda = (out->tp_prefill_eff / G) / L_in;  // Eq. 11 solved for lambda with Eq. 10, one group
    out->rho = out->lambda / out->mu;           // Eq. 10
  } else {
    status = PD_ERR_INFEASIBLE_TTFT;
  }

  // Decode side: walk the curve in order of batch size; stop at the first point over the SLO.
  std::vector<int> order(in->n_points);
  for (int i = 0; i < in->n_points; ++i) order[i] = i;
  std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return in->batch[a] < in->batch[b]; });
  int best = -1;
  for (int idx : order) {
    if (in->tpot_s[idx] <= in->tpot_slo_s) best = idx; else break;
  }
  if (best < 0) {
    if (status == PD_OK) status = PD_ERR_INFEASIBLE_TPOT;
  } else {
    out->feasible_batch = in->batch[best];
    out->sweep_capped = (best == order.back()) ? 1 : 0;
    out->tp_decode_eff = static_cast<double>(in->batch[best]) / in->tpot_s[best];
  }
  if (status != PD_OK) return status;

  const double TP_total = in->tp_total_tok_s, TP_p = out->tp_prefill_eff, TP_d = out->tp_decode_eff;
  out->n_prefill_frac = (TP_total * L_in) / ((L_in + L_out) * TP_p);   // Eq. 5
  out->n_decode_frac = (TP_total * L_out) / ((L_in + L_out) * TP_d);   // Eq. 6
  out->ratio_pd = (L_in * TP_d) / (L_out * TP_p);                      // Eq. 7
  out->n_prefill = nearest_count(out->n_prefill_frac);
  out->n_decode = nearest_count(out->n_decode_frac);
  out->n_prefill_ceil = ceil_count(out->n_prefill_frac);
  out->n_decode_ceil = ceil_count(out->n_decode_frac);
  // Pipelined phases: the slower one sets the pace (Eq. 2-4), total tokens per request L_in + L_out (Eq. 1).
  const double side_p = out->n_prefill * TP_p * (L_in + L_out) / L_in;
  const double side_d = out->n_decode * TP_d * (L_in + L_out) / L_out;
  out->achieved_total_tok_s = side_p < side_d ? side_p : side_d;
  return PD_OK;
}
}  // namespace

extern "C" pd_status pd_queue_replay(const double* gaps, const double* service, int64_t n, double* mean_sojourn_s,
                                     double* mean_wait_s) {
  if (!gaps || !service || n <= 0 || !mean_sojourn_s || !mean_wait_s) return PD_ERR_INVALID_ARG;
  // Lindley recursion: W(i) = max(0, W(i-1) + S(i-1) - gap(i)).
  double wait = 0.0, sum_wait = 0.0, sum_soj = 0.0;
  for (int64_t i = 0; i < n; ++i) {
    if (!(service[i] >= 0.0) || !(gaps[i] >= 0.0)) return PD_ERR_INVALID_ARG;
    if (i > 0) {
      double w = wait + service[i - 1] - gaps[i];
      wait = w > 0.0 ? w : 0.0;
    }
    sum_wait += wait;
    sum_soj += wait + service[i];
  }
  *mean_sojourn_s = sum_soj / static_cast<double>(n);
  *mean_wait_s = sum_wait / static_cast<double>(n);
  return PD_OK;
}

// ----------------------------------------------------------------- workload statistics
// Everything below is sequential IEEE double arithmetic in a fixed order, so that an independent
// implementation that follows the same order agrees bit for bit.

extern "C" pd_status pd_mixture_throughput(const int32_t* l_in, const double* service_s, int64_t n,
                                           double* tp_max_tok_s, double* mean_l_in) {
  if (!l_in || !service_s || n <= 0 || !tp_max_tok_s || !mean_l_in) return PD_ERR_INVALID_ARG;
  double tokens = 0.0, busy = 0.0;
  for (int64_t i = 0; i < n; ++i) {
    if (l_in[i] <= 0 || !(service_s[i] > 0.0)) return PD_ERR_INVALID_ARG;
    tokens += static_cast<double>(l_in[i]);
  }
  for (int64_t i = 0; i < n; ++i) busy += service_s[i];
  *tp_max_tok_s = tokens / busy;
  *mean_l_in = tokens / static_cast<double>(n);
  return PD_OK;
}

extern "C" pd_status pd_interp_service_times(const int32_t* grid_l, const double* grid_time_s, int32_t n_grid,
                                             const int32_t* l_in, int64_t n, int32_t quantum, double* service_s) {
  if (!grid_l || !grid_time_s || n_grid <= 0 || !l_in || n < 0 || !service_s || quantum < 1) return PD_ERR_INVALID_ARG;
  for (int i = 0; i + 1 < n_grid; ++i)
    if (grid_l[i + 1] <= grid_l[i]) return PD_ERR_INVALID_ARG;
  for (int64_t r = 0; r < n; ++r) {
    if (l_in[r] < 0 || l_in[r] > 2147483647 - quantum) return PD_ERR_INVALID_ARG;
    const int32_t l = (l_in[r] + quantum - 1) / quantum * quantum;  // the next full tile
    if (l <= grid_l[0]) { service_s[r] = grid_time_s[0]; continue; }
    if (l >= grid_l[n_grid - 1]) { service_s[r] = grid_time_s[n_grid - 1]; continue; }
    int lo = 0, hi = n_grid - 1;  // grid_l[lo] < l <= grid_l[hi]
    while (hi - lo > 1) {
      const int mid = (lo + hi) / 2;
      if (grid_l[mid] < l) lo = mid; else hi = mid;
    }
    const double w = (static_cast<double>(l) - static_cast<double>(grid_l[lo])) /
                     (static_cast<double>(grid_l[hi]) - static_cast<double>(grid_l[lo]));
    service_s[r] = grid_time_s[lo] + (grid_time_s[hi] - grid_time_s[lo]) * w;
  }
  return PD_OK;
}

extern "C" pd_status pd_mm1_sojourn(double mu, double lambda, double* sojourn_s) {
  if (!sojourn_s || !(mu > 0.0) || !(lambda >= 0.0)) return PD_ERR_INVALID_ARG;
  if (!(lambda < mu)) return PD_ERR_INFEASIBLE_TTFT;  // the queue has no steady state
  *sojourn_s = 1.0 / (mu - lambda);                   // Eq. 12
  return PD_OK;
}

extern "C" pd_status pd_mg1_sojourn(const double* service_s, int64_t n, double lambda, double* sojourn_s) {
  if (!service_s || n <= 0 || !sojourn_s || !(lambda >= 0.0)) return PD_ERR_INVALID_ARG;
  double s1 = 0.0, s2 = 0.0;
  for (int64_t i = 0; i < n; ++i) {
    if (!(service_s[i] >= 0.0)) return PD_ERR_INVALID_ARG;
    s1 += service_s[i];
  }
  for (int64_t i = 0; i < n; ++i) s2 += service_s[i] * service_s[i];
  const double es = s1 / static_cast<double>(n), es2 = s2 / static_cast<double>(n);
  const double rho = lambda * es;
  if (!(rho < 1.0)) return PD_ERR_INFEASIBLE_TTFT;
  *sojourn_s = es + lambda * es2 / (2.0 * (1.0 - rho));  // Pollaczek-Khinchine
  return PD_OK;
}

extern "C" pd_status pd_refine_next_batch(const int32_t* batch, const double* tpot_s, int32_t n_points,
                                          double tpot_slo_s, int32_t* next_batch) {
  if (!next_batch || n_points < 0 || (n_points > 0 && (!batch || !tpot_s)) || !(tpot_slo_s > 0.0))
    return PD_ERR_INVALID_ARG;
  for (int i = 0; i < n_points; ++i)
    if (batch[i] <= 0 || !(tpot_s[i] > 0.0)) return PD_ERR_INVALID_ARG;
  std::vector<int> order(n_points);
  for (int i = 0; i < n_points; ++i) order[i] = i;
  std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return batch[a] < batch[b]; });
  int32_t lo = 0, hi = 0;
  for (int idx : order) {
    if (tpot_s[idx] <= tpot_slo_s) lo = batch[idx];
    else { hi = batch[idx]; break; }
  }
  *next_batch = (lo == 0 || hi == 0 || hi - lo <= 1) ? 0 : lo + (hi - lo) / 2;
  return PD_OK;
}
