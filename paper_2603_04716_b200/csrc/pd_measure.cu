// Measurement harness: the empirical benchmarking the allocation method feeds on.
// Builds a stack of distinct synthetic layers on the current device, times the prefill
// pass (maximum prefill throughput) and decode steps over a batch sweep (TPOT versus
// batch) with CUDA events, and reports algorithmic work against the given peaks.
#include <algorithm>
#include <cstring>
#include <vector>

#include "pd_common.cuh"

using pd::bf16;

namespace {

struct DevBuf {
  void* p = nullptr;
  ~DevBuf() { if (p) cudaFree(p); }
  cudaError_t alloc(size_t bytes) { return cudaMalloc(&p, bytes ? bytes : 16); }
};

struct Stack {
  std::vector<pd_layer*> layers;
  ~Stack() { for (pd_layer* l : layers) pd_layer_destroy(l); }
};

struct ModelGuard {
  pd_model* m = nullptr;
  ~ModelGuard() { pd_model_destroy(m); }
};

struct Events {
  cudaEvent_t a = nullptr, b = nullptr;
  ~Events() { if (a) cudaEventDestroy(a); if (b) cudaEventDestroy(b); }
};

// Times work that `enqueue` puts on stream `st` (no allocation, no synchronisation inside).  After one
// eager run the work is captured into a CUDA graph and the graph is replayed for the warm-up and timed
// repetitions, which removes most of the per-kernel launch gaps of the ~13 small kernels per decode
// layer; if capture is not possible the repetitions are launched eagerly.  `launches` receives the number
// of kernels of one run.
template <class F>
pd_status time_enqueued(F&& enqueue, cudaStream_t st, Events& ev, int warmup, int reps, std::vector<double>* times,
                        long long* launches) {
  const long long l0 = pd::g_launch_count;
  PD_TRY(enqueue());
  *launches = pd::g_launch_count - l0;
  PD_CUDA_TRY(cudaStreamSynchronize(st));
  cudaGraph_t graph = nullptr;
  cudaGraphExec_t exec = nullptr;
  if (cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal) == cudaSuccess) {
    const pd_status s = enqueue();
    const cudaError_t e = cudaStreamEndCapture(st, &graph);
    if (s != PD_OK || e != cudaSuccess || cudaGraphInstantiate(&exec, graph, 0) != cudaSuccess) exec = nullptr;
  }
  (void)cudaGetLastError();  // a failed capture leaves a sticky-free error behind
  pd_status result = PD_OK;
  for (int it = 0; it < warmup + reps && result == PD_OK; ++it) {
    cudaError_t e = cudaEventRecord(ev.a, st);
    if (e == cudaSuccess) {
      if (exec) e = cudaGraphLaunch(exec, st);
      else result = enqueue();
    }
    if (e == cudaSuccess) e = cudaEventRecord(ev.b, st);
    if (e == cudaSuccess) e = cudaEventSynchronize(ev.b);
    float ms = 0.f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, ev.a, ev.b);
    if (e != cudaSuccess) result = pd::cuda_fail(e);
    else if (it >= warmup) times->push_back(ms * 1e-3);
  }
  if (exec) cudaGraphExecDestroy(exec);
  if (graph) cudaGraphDestroy(graph);
  return result;
}

double median(std::vector<double> v) {
  std::sort(v.begin(), v.end());
  const size_t n = v.size();
  return n % 2 ? v[n / 2] : 0.5 * (v[n / 2 - 1] + v[n / 2]);
}

size_t layer_param_count(const pd_layer_cfg& c) {
  const size_t d = c.d_model, nqkv = static_cast<size_t>(c.n_q_heads + 2 * c.n_kv_heads) * c.head_dim;
  return d * nqkv + static_cast<size_t>(c.n_q_heads) * c.head_dim * d + 3 * d * static_cast<size_t>(c.d_ff);
}

pd_status build_stack(const pd_layer_cfg& cfg, int n_layers, uint64_t seed, cudaStream_t st, Stack* out) {
  const size_t d = cfg.d_model, f = cfg.d_ff, hq = static_cast<size_t>(cfg.n_q_heads) * cfg.head_dim;
  const size_t nqkv = static_cast<size_t>(cfg.n_q_heads + 2 * cfg.n_kv_heads) * cfg.head_dim;
  DevBuf wqkv, wo, wg, wu, wd, ga, gm;
  PD_CUDA_TRY(wqkv.alloc(nqkv * d * 2));
  PD_CUDA_TRY(wo.alloc(d * hq * 2));
  PD_CUDA_TRY(wg.alloc(f * d * 2));
  PD_CUDA_TRY(wu.alloc(f * d * 2));
  PD_CUDA_TRY(wd.alloc(d * f * 2));
  PD_CUDA_TRY(ga.alloc(d * 2));
  PD_CUDA_TRY(gm.alloc(d * 2));
  for (int l = 0; l < n_layers; ++l) {
    const uint64_t s0 = static_cast<uint64_t>(l) * 16;
    PD_TRY(pd::launch_fill_normal(static_cast<bf16*>(wqkv.p), nqkv * d, seed, s0 + 0, 0.f, 0.02f, st));
    PD_TRY(pd::launch_fill_normal(static_cast<bf16*>(wo.p), d * hq, seed, s0 + 1, 0.f, 0.02f, st));
    PD_TRY(pd::launch_fill_normal(static_cast<bf16*>(wg.p), f * d, seed, s0 + 2, 0.f, 0.02f, st));
    PD_TRY(pd::launch_fill_normal(static_cast<bf16*>(wu.p), f * d, seed, s0 + 3, 0.f, 0.02f, st));
    PD_TRY(pd::launch_fill_normal(static_cast<bf16*>(wd.p), d * f, seed, s0 + 4, 0.f, 0.02f, st));
    PD_TRY(pd::launch_fill_normal(static_cast<bf16*>(ga.p), d, seed, s0 + 5, 1.f, 0.02f, st));
    PD_TRY(pd::launch_fill_normal(static_cast<bf16*>(gm.p), d, seed, s0 + 6, 1.f, 0.02f, st));
    pd_layer_weights w{};
    w.struct_size = sizeof(w);
    w.w_qkv = wqkv.p; w.w_o = wo.p; w.w_gate = wg.p; w.w_up = wu.p; w.w_down = wd.p; w.g_attn = ga.p; w.g_mlp = gm.p;
    pd_layer* L = nullptr;
    PD_TRY(pd_layer_create(&cfg, &w, st, &L));
    out->layers.push_back(L);
    PD_CUDA_TRY(cudaStreamSynchronize(st));  // the temporaries are refilled for the next layer
  }
  return PD_OK;
}

// Synthetic embedding table, final gain and LM head over the stack's layers.
pd_status build_model(const pd_layer_cfg& cfg, Stack& stack, int vocab, uint64_t seed, cudaStream_t st, ModelGuard* out) {
  const size_t table = static_cast<size_t>(vocab) * cfg.d_model;
  DevBuf e, h, g;
  PD_CUDA_TRY(e.alloc(table * 2));
  PD_CUDA_TRY(h.alloc(table * 2));
  PD_CUDA_TRY(g.alloc(static_cast<size_t>(cfg.d_model) * 2));
  PD_TRY(pd::launch_fill_normal(static_cast<bf16*>(e.p), table, seed, 5000, 0.f, 1.f, st));
  PD_TRY(pd::launch_fill_normal(static_cast<bf16*>(h.p), table, seed, 5001, 0.f, 0.02f, st));
  PD_TRY(pd::launch_fill_normal(static_cast<bf16*>(g.p), cfg.d_model, seed, 5002, 1.f, 0.02f, st));
  pd_model_weights w{};
  w.struct_size = sizeof(w);
  w.vocab = vocab; w.embed = e.p; w.g_final = g.p; w.lm_head = h.p;
  PD_TRY(pd_model_create(stack.layers.data(), static_cast<int>(stack.layers.size()), &w, st, &out->m));
  PD_CUDA_TRY(cudaStreamSynchronize(st));  // the temporaries die here
  return PD_OK;
}

// Uniform token ids from a counter hash (host side; the values only steer which embedding rows are read).
std::vector<int32_t> synthetic_tokens(size_t n, int vocab, uint64_t seed) {
  std::vector<int32_t> t(n);
  for (size_t i = 0; i < n; ++i) {
    uint64_t z = seed * 0x9E3779B97F4A7C15ull + i + 0x7F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    z ^= z >> 31;
    t[i] = static_cast<int32_t>(z % static_cast<uint64_t>(vocab));
  }
  return t;
}

// Number of KV buffers to cycle through: one per layer if memory allows, otherwise as many as
// fit in 70 % of the free memory (still far larger than L2 in total).
int cache_ring(size_t bytes_per_cache, int n_layers) {
  size_t free_b = 0, total_b = 0;
  if (cudaMemGetInfo(&free_b, &total_b) != cudaSuccess) return 1;
  const size_t budget = static_cast<size_t>(0.7 * static_cast<double>(free_b));
  size_t fit = bytes_per_cache ? budget / bytes_per_cache : static_cast<size_t>(n_layers);
  if (fit < 1) fit = 1;
  return static_cast<int>(std::min<size_t>(fit, static_cast<size_t>(n_layers)));
}

}  // namespace

extern "C" pd_status pd_measure(const pd_layer_cfg* cfg_in, const pd_measure_cfg* m, double peak_bf16_flops,
                                double peak_hbm_bytes_s, pd_measurement* out) {
  if (!cfg_in || !m || !out || m->struct_size != sizeof(pd_measure_cfg) || cfg_in->struct_size != sizeof(pd_layer_cfg))
    return PD_ERR_INVALID_ARG;
  if (m->n_layers_run <= 0 || m->n_layers_model <= 0 || m->warmup < 0 || m->reps <= 0) return PD_ERR_INVALID_ARG;
  if (m->n_req < 0 || m->n_batch_sizes < 0 || m->n_batch_sizes > 32 || m->vocab < 0) return PD_ERR_INVALID_ARG;
  if ((m->n_req > 0 && !m->l_in) || (m->n_batch_sizes > 0 && (!m->batch_sizes || m->n_steps <= 0 || m->kv_len_start < 0)))
    return PD_ERR_INVALID_ARG;
  std::memset(out, 0, sizeof(*out));
  out->struct_size = sizeof(pd_measurement);
  pd_layer_cfg cfg = *cfg_in;
  const double scale_layers = static_cast<double>(m->n_layers_model) / m->n_layers_run;
  const int nl = m->n_layers_run;
  const size_t d = cfg.d_model;
  const size_t kv_row = static_cast<size_t>(cfg.n_kv_heads) * cfg.head_dim * 2;  // bytes of K (or V) per token

  cudaStream_t st = nullptr;
  PD_CUDA_TRY(cudaStreamCreateWithFlags(&st, cudaStreamNonBlocking));
  struct StreamGuard { cudaStream_t s; ~StreamGuard() { cudaStreamDestroy(s); } } sg{st};
  Events ev;
  PD_CUDA_TRY(cudaEventCreate(&ev.a));
  PD_CUDA_TRY(cudaEventCreate(&ev.b));

  Stack stack;
  PD_TRY(build_stack(cfg, nl, m->seed, st, &stack));
  ModelGuard model;
  if (m->vocab > 0) PD_TRY(build_model(cfg, stack, m->vocab, m->seed, st, &model));
  const long long launches_before = pd::g_launch_count;
  long long timed_launches = 0;

  // ------------------------------------------------------------------ prefill
  // Median time of one prefill pass of the batch `lens` through the nl layers of the stack (not yet scaled to the
  // model's layer count): in one piece, or, with chunk_tokens > 0, chunk after chunk, every chunk through all layers.
  DevBuf x_keep, y_keep, cu_keep;  // buffers of the main batch, reused by the whole-model head below
  auto measure_prefill = [&](const int32_t* lens, int n_req, bool keep, double* time_s, int* ring_out,
                             int* chunks_out) -> pd_status {
    std::vector<int32_t> cu(n_req + 1, 0);
    int max_len = 0;
    for (int r = 0; r < n_req; ++r) {
      if (lens[r] < 0 || lens[r] > cfg.max_pos) return PD_ERR_INVALID_ARG;
      cu[r + 1] = cu[r] + lens[r];
      max_len = std::max(max_len, lens[r]);
    }
    const int tokens = cu[n_req];
    *time_s = 0.0; *ring_out = 0; *chunks_out = 0;
    if (tokens == 0) return PD_OK;
    const size_t cache_bytes = static_cast<size_t>(n_req) * max_len * kv_row;
    const int ring = cache_ring(2 * cache_bytes, nl);
    std::vector<DevBuf> kbuf(ring), vbuf(ring);
    std::vector<pd_kv_cache> caches(ring);
    for (int i = 0; i < ring; ++i) {
      PD_CUDA_TRY(kbuf[i].alloc(cache_bytes));
      PD_CUDA_TRY(vbuf[i].alloc(cache_bytes));
      caches[i].struct_size = sizeof(pd_kv_cache);
      caches[i].k = kbuf[i].p; caches[i].v = vbuf[i].p;
      caches[i].batch_cap = n_req; caches[i].len_cap = max_len;
    }
    // chunk schedule: step s holds rows [s c, (s + 1) c) of every request that still has rows
    const int chunk = m->chunk_tokens > 0 ? m->chunk_tokens : max_len;
    const int n_steps = (max_len + chunk - 1) / chunk;
    std::vector<int32_t> meta(static_cast<size_t>(n_steps) * (2 * n_req + 1));  // per step: cu[n_req + 1], prefix[n_req]
    int max_chunk_tokens = 0;
    for (int sidx = 0; sidx < n_steps; ++sidx) {
      int32_t* cu_s = meta.data() + static_cast<size_t>(sidx) * (2 * n_req + 1);
      int32_t* pre_s = cu_s + n_req + 1;
      cu_s[0] = 0;
      for (int r = 0; r < n_req; ++r) {
        const int lo = std::min(lens[r], sidx * chunk), hi = std::min(lens[r], (sidx + 1) * chunk);
        cu_s[r + 1] = cu_s[r] + (hi - lo);
        pre_s[r] = lo;
      }
      max_chunk_tokens = std::max(max_chunk_tokens, cu_s[n_req]);
    }
    size_t ws_bytes = 0;
    PD_TRY(pd_workspace_bytes(&cfg, max_chunk_tokens, 0, 0, &ws_bytes));
    DevBuf ws, x_loc, y_loc, meta_dev;
    DevBuf& x = keep ? x_keep : x_loc;
    DevBuf& y = keep ? y_keep : y_loc;
    PD_CUDA_TRY(ws.alloc(ws_bytes));
    PD_CUDA_TRY(x.alloc(tokens * d * 2));
    PD_CUDA_TRY(y.alloc(tokens * d * 2));
    PD_CUDA_TRY(meta_dev.alloc(meta.size() * 4));
    PD_CUDA_TRY(cudaMemcpyAsync(meta_dev.p, meta.data(), meta.size() * 4, cudaMemcpyHostToDevice, st));
    if (keep) {
      PD_CUDA_TRY(cu_keep.alloc(cu.size() * 4));
      PD_CUDA_TRY(cudaMemcpyAsync(cu_keep.p, cu.data(), cu.size() * 4, cudaMemcpyHostToDevice, st));
    }
    PD_TRY(pd::launch_fill_normal(static_cast<bf16*>(x.p), tokens * d, m->seed, 1000, 0.f, 1.f, st));
    std::vector<double> times;
    long long per_run = 0;
    PD_TRY(time_enqueued(
        [&]() -> pd_status {
          for (int sidx = 0; sidx < n_steps; ++sidx) {
            const size_t off = static_cast<size_t>(sidx) * (2 * n_req + 1);
            const int32_t* cu_h = meta.data() + off;
            const int32_t* cu_d = static_cast<const int32_t*>(meta_dev.p) + off;
            if (m->chunk_tokens > 0)
              PD_TRY(pd_prefill_chunk_stack(stack.layers.data(), caches.data(), nl, ring, x.p, y.p, cu_d, cu_h, n_req,
                                            cu_d + n_req + 1, cu_h + n_req + 1, ws.p, ws_bytes, st));
            else
              PD_TRY(pd_prefill_stack(stack.layers.data(), caches.data(), nl, ring, x.p, y.p, 0, cu_d, cu_h, n_req,
                                      ws.p, ws_bytes, st));
          }
          return PD_OK;
        },
        st, ev, m->warmup, m->reps, &times, &per_run));
    timed_launches += per_run * m->reps;
    PD_TRY(pd_layer_check(stack.layers[0], st));
    *time_s = median(times);
    *ring_out = ring;
    *chunks_out = n_steps;
    return PD_OK;
  };

  if (m->n_grid < 0 || m->n_grid > PD_MEASURE_GRID_MAX || (m->n_grid > 0 && !m->l_in_grid) || m->chunk_tokens < 0)
    return PD_ERR_INVALID_ARG;
  for (int gi = 0; gi < m->n_grid; ++gi) {
    if (m->l_in_grid[gi] <= 0) return PD_ERR_INVALID_ARG;
    double t = 0.0;
    int ring = 0, chunks = 0;
    PD_TRY(measure_prefill(&m->l_in_grid[gi], 1, false, &t, &ring, &chunks));
    out->grid_l[gi] = m->l_in_grid[gi];
    out->grid_time_s[gi] = t * scale_layers;
    out->n_grid = gi + 1;
  }

  if (m->n_req > 0) {
    double attn_flops = 0.0;
    int tokens = 0;
    for (int r = 0; r < m->n_req; ++r) {
      const double l = m->l_in[r];
      attn_flops += 4.0 * cfg.n_q_heads * cfg.head_dim * (l * (l + 1.0) / 2.0);
      tokens += m->l_in[r] > 0 ? m->l_in[r] : 0;
    }
    double t_run = 0.0;
    PD_TRY(measure_prefill(m->l_in, m->n_req, true, &t_run, &out->prefill_kv_ring, &out->prefill_chunks));
    if (tokens > 0) {
      const double gemm_flops = 2.0 * tokens * static_cast<double>(layer_param_count(cfg));
      out->prefill_flops = (gemm_flops + attn_flops) * m->n_layers_model;
      out->prefill_time_s = t_run * scale_layers;
      DevBuf& x = x_keep;
      DevBuf& y = y_keep;
      DevBuf& cu_dev = cu_keep;
      if (model.m) {  // embedding in front, final norm + LM head + sampling behind: once per pass
        const std::vector<int32_t> tok = synthetic_tokens(tokens, m->vocab, m->seed);
        DevBuf tok_dev, sel, norm, logits, next;
        PD_CUDA_TRY(tok_dev.alloc(tok.size() * 4));
        PD_CUDA_TRY(sel.alloc(m->n_req * d * 2));
        PD_CUDA_TRY(norm.alloc(m->n_req * d * 2));
        PD_CUDA_TRY(logits.alloc(static_cast<size_t>(m->n_req) * m->vocab * 4));
        PD_CUDA_TRY(next.alloc(m->n_req * 4));
        PD_CUDA_TRY(cudaMemcpyAsync(tok_dev.p, tok.data(), tok.size() * 4, cudaMemcpyHostToDevice, st));
        std::vector<double> htimes;
        long long hrun = 0;
        PD_TRY(time_enqueued(
            [&] {
              PD_TRY(pd::model_embed(model.m, static_cast<const int32_t*>(tok_dev.p), tokens, static_cast<bf16*>(x.p), st));
              return pd::model_head(model.m, static_cast<const bf16*>(y.p), static_cast<const int32_t*>(cu_dev.p),
                                    m->n_req, static_cast<bf16*>(sel.p), static_cast<bf16*>(norm.p),
                                    static_cast<float*>(logits.p), static_cast<int32_t*>(next.p), st);
            },
            st, ev, m->warmup, m->reps, &htimes, &hrun));
        timed_launches += hrun * m->reps;
        PD_TRY(pd_model_check(model.m, st));
        out->prefill_head_s = median(htimes);
        out->prefill_time_s += out->prefill_head_s;
        out->prefill_flops += 2.0 * m->n_req * static_cast<double>(m->vocab) * d;
      }
      out->prefill_tok_s = tokens / out->prefill_time_s;
      if (peak_bf16_flops > 0) out->prefill_frac_bf16_peak = out->prefill_flops / out->prefill_time_s / peak_bf16_flops;
    }
  }

  // ------------------------------------------------------------------- decode
  if (m->n_batch_sizes > 0) {
    int max_b = 0;
    for (int i = 0; i < m->n_batch_sizes; ++i) {
      if (m->batch_sizes[i] <= 0 || m->batch_sizes[i] > 4096) return PD_ERR_INVALID_ARG;
      max_b = std::max(max_b, m->batch_sizes[i]);
    }
    int max_start = m->kv_len_start;
    if (m->kv_len_mix)
      for (int b = 0; b < max_b; ++b) {
        if (m->kv_len_mix[b] < 0) return PD_ERR_INVALID_ARG;
        max_start = std::max(max_start, m->kv_len_mix[b]);
      }
    const int len_cap = max_start + m->n_steps;
    if (len_cap > cfg.max_pos) return PD_ERR_INVALID_ARG;
    // steps sampled: 0, stride, 2*stride, ... and the last one
    std::vector<int> steps;
    const int stride = m->step_stride > 0 ? m->step_stride : 1;
    for (int t = 0; t < m->n_steps; t += stride) steps.push_back(t);
    if (steps.back() != m->n_steps - 1) steps.push_back(m->n_steps - 1);

    const size_t params_bytes = layer_param_count(cfg) * 2;
    for (int bi = 0; bi < m->n_batch_sizes; ++bi) {
      const int B = m->batch_sizes[bi];
      const size_t cache_bytes = static_cast<size_t>(B) * len_cap * kv_row;
      const int ring = cache_ring(2 * cache_bytes, nl);
      std::vector<DevBuf> kbuf(ring), vbuf(ring);
      std::vector<pd_kv_cache> caches(ring);
      for (int i = 0; i < ring; ++i) {
        PD_CUDA_TRY(kbuf[i].alloc(cache_bytes));
        PD_CUDA_TRY(vbuf[i].alloc(cache_bytes));
        PD_TRY(pd::launch_fill_normal(static_cast<bf16*>(kbuf[i].p), cache_bytes / 2, m->seed, 2000 + 2 * i, 0.f, 1.f, st));
        PD_TRY(pd::launch_fill_normal(static_cast<bf16*>(vbuf[i].p), cache_bytes / 2, m->seed, 2001 + 2 * i, 0.f, 1.f, st));
        caches[i].struct_size = sizeof(pd_kv_cache);
        caches[i].k = kbuf[i].p; caches[i].v = vbuf[i].p; caches[i].batch_cap = B; caches[i].len_cap = len_cap;
      }
      size_t ws_bytes = 0;
      PD_TRY(pd_workspace_bytes(&cfg, 0, B, len_cap, &ws_bytes));
      DevBuf ws, x, y, kv_dev;
      PD_CUDA_TRY(ws.alloc(ws_bytes));
      PD_CUDA_TRY(x.alloc(B * d * 2));
      PD_CUDA_TRY(y.alloc(B * d * 2));
      PD_CUDA_TRY(kv_dev.alloc(steps.size() * B * 4));
      std::vector<int32_t> kv_host(steps.size() * B);
      double kv_tokens_mean = 0.0;
      for (size_t si = 0; si < steps.size(); ++si)
        for (int b = 0; b < B; ++b) {
          const int start = m->kv_len_mix ? m->kv_len_mix[b] : m->kv_len_start;
          kv_host[si * B + b] = start + steps[si];
          kv_tokens_mean += start + steps[si] + 1;
        }
      kv_tokens_mean /= static_cast<double>(steps.size());  // sum over the batch, mean over steps
      PD_CUDA_TRY(cudaMemcpyAsync(kv_dev.p, kv_host.data(), kv_host.size() * 4, cudaMemcpyHostToDevice, st));
      PD_TRY(pd::launch_fill_normal(static_cast<bf16*>(x.p), B * d, m->seed, 3000 + bi, 0.f, 1.f, st));
      PD_CUDA_TRY(cudaStreamSynchronize(st));

      double step_time_sum = 0.0, attn_time_sum = 0.0;
      for (size_t si = 0; si < steps.size(); ++si) {
        const int32_t* kvp = static_cast<const int32_t*>(kv_dev.p) + si * B;
        int max_kv = 0;
        for (int b = 0; b < B; ++b) max_kv = std::max(max_kv, kv_host[si * B + b] + 1);
        std::vector<double> times;
        long long per_run = 0;
        PD_TRY(time_enqueued(
            [&] {
              return pd_decode_stack(stack.layers.data(), caches.data(), nl, ring, x.p, y.p, 0, kvp, B, max_kv, ws.p,
                                     ws_bytes, st);
            },
            st, ev, m->warmup, m->reps, &times, &per_run));
        timed_launches += per_run * m->reps;
        step_time_sum += median(times);

        // the attention kernel alone, over the same caches (q = whatever the last pass left in the workspace)
        pd::DecodeAttnArgs a{};
        // reuse the library's own carving by running one decode layer first would be circular: place q, o and the
        // partials at the start of the workspace instead (the kernel only needs valid, finite inputs)
        const size_t q_bytes = pd::align_up(static_cast<size_t>(B) * stack.layers[0]->n_qkv * 2, 256);
        const size_t o_bytes = pd::align_up(static_cast<size_t>(B) * cfg.n_q_heads * cfg.head_dim * 2, 256);
        uint8_t* wsb = static_cast<uint8_t*>(ws.p);
        a.q = reinterpret_cast<bf16*>(wsb); a.ldq = stack.layers[0]->n_qkv;
        a.o = reinterpret_cast<bf16*>(wsb + q_bytes);
        a.partial = reinterpret_cast<float*>(wsb + q_bytes + o_bytes);
        a.kv_len = kvp; a.batch = B; a.max_kv_len = max_kv;
        a.n_splits = pd::decode_attention_splits(B, cfg.n_kv_heads, max_kv);
        a.n_q_heads = cfg.n_q_heads; a.n_kv_heads = cfg.n_kv_heads; a.head_dim = cfg.head_dim; a.len_cap = len_cap;
        PD_TRY(pd::launch_fill_normal(const_cast<bf16*>(a.q), static_cast<size_t>(B) * a.ldq, m->seed, 4000, 0.f, 1.f, st));
        std::vector<double> atimes;
        for (int it = 0; it < m->warmup + m->reps; ++it) {
          PD_CUDA_TRY(cudaEventRecord(ev.a, st));
          for (int l = 0; l < nl; ++l) {
            a.k_cache = static_cast<bf16*>(caches[l % ring].k);
            a.v_cache = static_cast<bf16*>(caches[l % ring].v);
            PD_TRY(pd::launch_decode_attention(a, st));
          }
          PD_CUDA_TRY(cudaEventRecord(ev.b, st));
          PD_CUDA_TRY(cudaEventSynchronize(ev.b));
          float ms = 0.f;
          PD_CUDA_TRY(cudaEventElapsedTime(&ms, ev.a, ev.b));
          if (it >= m->warmup) atimes.push_back(ms * 1e-3 / nl);
        }
        attn_time_sum += median(atimes);
      }
      PD_TRY(pd_layer_check(stack.layers[0], st));
      double head_time = 0.0;
      if (model.m) {
        const std::vector<int32_t> tok = synthetic_tokens(B, m->vocab, m->seed + bi);
        DevBuf tok_dev, norm, logits, next;
        PD_CUDA_TRY(tok_dev.alloc(tok.size() * 4));
        PD_CUDA_TRY(norm.alloc(B * d * 2));
        PD_CUDA_TRY(logits.alloc(static_cast<size_t>(B) * m->vocab * 4));
        PD_CUDA_TRY(next.alloc(B * 4));
        PD_CUDA_TRY(cudaMemcpyAsync(tok_dev.p, tok.data(), tok.size() * 4, cudaMemcpyHostToDevice, st));
        std::vector<double> htimes;
        long long hrun = 0;
        PD_TRY(time_enqueued(
            [&] {
              PD_TRY(pd::model_embed(model.m, static_cast<const int32_t*>(tok_dev.p), B, static_cast<bf16*>(x.p), st));
              return pd::model_head(model.m, static_cast<const bf16*>(y.p), nullptr, B, nullptr,
                                    static_cast<bf16*>(norm.p), static_cast<float*>(logits.p),
                                    static_cast<int32_t*>(next.p), st);
            },
            st, ev, m->warmup, m->reps, &htimes, &hrun));
        timed_launches += hrun * m->reps;
        PD_TRY(pd_model_check(model.m, st));
        head_time = median(htimes);
      }
      const double step_time = step_time_sum / steps.size();  // n_layers_run layers
      const double attn_time = attn_time_sum / steps.size();  // one layer
      const double kv_bytes_layer = kv_tokens_mean * 2.0 * kv_row;
      const double bytes_layer = static_cast<double>(params_bytes) + kv_bytes_layer + B * 2.0 * kv_row + 2.0 * B * d * 2;
      const int pi = out->n_points++;
      out->batch[pi] = B;
      out->tpot_s[pi] = step_time * scale_layers + head_time;
      out->decode_head_s[pi] = head_time;
      out->decode_bytes[pi] = bytes_layer * m->n_layers_model;
      if (model.m)  // LM head once, embedding rows, logits written and read back by the sampler
        out->decode_bytes[pi] += static_cast<double>(m->vocab) * d * 2 + 2.0 * B * d * 2 + 2.0 * B * m->vocab * 4.0;
      out->attn_time_s[pi] = attn_time;
      out->decode_kv_ring[pi] = ring;
      // The attention-only pass walks `ring` distinct K/V buffers back to back.  When all of them together stay
      // below twice the L2 size, part of the "HBM" stream is served from L2 and the rate is not an HBM figure.
      {
        int dev = 0, l2 = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&l2, cudaDevAttrL2CacheSize, dev) != cudaSuccess)
          l2 = 128 << 20;
        out->attn_l2_resident[pi] = (kv_bytes_layer * ring < 2.0 * l2) ? 1 : 0;
      }
      if (peak_hbm_bytes_s > 0) {
        out->decode_frac_hbm_peak[pi] = out->decode_bytes[pi] / out->tpot_s[pi] / peak_hbm_bytes_s;
        if (!out->attn_l2_resident[pi]) out->attn_frac_hbm_peak[pi] = kv_bytes_layer / attn_time / peak_hbm_bytes_s;
      }
    }
  }
  (void)launches_before;
  out->gpu_launches = static_cast<int32_t>(std::min<long long>(timed_launches, 2147483647ll));
  return PD_OK;
}
