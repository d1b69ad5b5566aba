// Whole-model step around the layer stack: token embedding in front, final RMSNorm, LM-head
// projection and greedy sampling behind it, so that a prefill pass ends with the first output
// token (the event TTFT is measured to) and a decode step with the next token of every
// sequence (the event TPOT is measured between).
//
// The head reuses the decode-mode weight-streaming GEMM: only one row per request (prefill) or
// per sequence (decode) reaches it, so the LM head is read once per step and is HBM-bound like
// the other decode projections.  Logits stay in fp32; the sampled token is the lowest index
// among the largest logits.
#include <new>
#include <vector>

#include "pd_common.cuh"

using pd::bf16;

struct pd_model {
  std::vector<pd_layer*> layers;  // borrowed
  pd_layer_cfg cfg;
  int vocab;
  bf16* embed;    // [V, d]
  bf16* lm_head;  // [V, d]
  bf16* g_final;  // [d]
  int* err_word;
};

namespace {

// x[i, :] = E[tokens[i], :]; an id outside [0, V) zeroes the row and raises the error word.
__global__ void __launch_bounds__(128) embed_gather_kernel(const int32_t* __restrict__ tokens,
                                                           const bf16* __restrict__ embed, bf16* __restrict__ x, int d,
                                                           int vocab, int* err_word) {
  const int row = blockIdx.x;
  const int tok = tokens[row];
  uint4* dst = reinterpret_cast<uint4*>(x + static_cast<size_t>(row) * d);
  const int chunks = d / 8;
  if (tok < 0 || tok >= vocab) {
    if (threadIdx.x == 0 && err_word) atomicExch(err_word, 3);
    for (int c = threadIdx.x; c < chunks; c += blockDim.x) dst[c] = make_uint4(0u, 0u, 0u, 0u);
    return;
  }
  const uint4* src = reinterpret_cast<const uint4*>(embed + static_cast<size_t>(tok) * d);
  for (int c = threadIdx.x; c < chunks; c += blockDim.x) dst[c] = src[c];
}

// sel[r, :] = h[cu[r+1] - 1, :] (the last row of request r), zeros for an empty request.
__global__ void __launch_bounds__(128) select_last_rows_kernel(const bf16* __restrict__ h,
                                                               const int32_t* __restrict__ cu, bf16* __restrict__ sel,
                                                               int d) {
  const int r = blockIdx.x;
  const int lo = cu[r], hi = cu[r + 1];
  uint4* dst = reinterpret_cast<uint4*>(sel + static_cast<size_t>(r) * d);
  const int chunks = d / 8;
  if (hi <= lo) {
    for (int c = threadIdx.x; c < chunks; c += blockDim.x) dst[c] = make_uint4(0u, 0u, 0u, 0u);
    return;
  }
  const uint4* src = reinterpret_cast<const uint4*>(h + static_cast<size_t>(hi - 1) * d);
  for (int c = threadIdx.x; c < chunks; c += blockDim.x) dst[c] = src[c];
}

// next[r] = argmax_v logits[r, v], the lowest index among equal maxima; -1 for an empty request.
constexpr int ARG_THREADS = 512;
__device__ __forceinline__ void take(float v, int i, float& best, int& best_i) {
  if (v > best || (v == best && i < best_i)) {
    best = v;
    best_i = i;
  }
}
__global__ void __launch_bounds__(ARG_THREADS) argmax_rows_kernel(const float* __restrict__ logits,
                                                                  const int32_t* __restrict__ cu,
                                                                  int32_t* __restrict__ next, int vocab) {
  const int r = blockIdx.x;
  if (cu && cu[r + 1] <= cu[r]) {
    if (threadIdx.x == 0) next[r] = -1;
    return;
  }
  const float* row = logits + static_cast<size_t>(r) * vocab;
  float best = -INFINITY;
  int best_i = 0x7fffffff;
  const int quads = vocab / 4;  // vocab is a multiple of 4 (checked at creation): rows stay 16-byte aligned
  for (int q = threadIdx.x; q < quads; q += ARG_THREADS) {
    const float4 v = reinterpret_cast<const float4*>(row)[q];
    take(v.x, 4 * q, best, best_i);
    take(v.y, 4 * q + 1, best, best_i);
    take(v.z, 4 * q + 2, best, best_i);
    take(v.w, 4 * q + 3, best, best_i);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, best, o);
    const int oi = __shfl_xor_sync(0xffffffffu, best_i, o);
    take(ov, oi, best, best_i);
  }
  __shared__ float sv[ARG_THREADS / 32];
  __shared__ int si[ARG_THREADS / 32];
  if ((threadIdx.x & 31) == 0) {
    sv[threadIdx.x >> 5] = best;
    si[threadIdx.x >> 5] = best_i;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < ARG_THREADS / 32; ++w) take(sv[w], si[w], best, best_i);
    next[r] = best_i == 0x7fffffff ? 0 : best_i;  // a row of NaNs compares false everywhere
  }
}

__global__ void fill_i32_kernel(int32_t* p, int n, int32_t v) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) p[i] = v;
}

struct ModelWs {
  size_t x0, h, sel, norm, logits, stack, total;
};

// Head buffers first, then the layer stack's own workspace.
ModelWs carve_model(const pd_model* m, size_t tokens, size_t rows, size_t stack_bytes, bool own_logits) {
  const size_t d = m->cfg.d_model;
  ModelWs w{};
  size_t off = 0;
  auto take_b = [&](size_t bytes) {
    const size_t o = off;
    off += pd::align_up(bytes, 256);
    return o;
  };
  w.x0 = take_b(tokens * d * 2);
  w.h = take_b(tokens * d * 2);
  w.sel = take_b(rows * d * 2);
  w.norm = take_b(rows * d * 2);
  w.logits = take_b(own_logits ? rows * static_cast<size_t>(m->vocab) * 4 : 0);
  w.stack = off;
  w.total = off + stack_bytes;
  return w;
}

}  // namespace

namespace pd {

pd_status model_embed(pd_model* m, const int32_t* tokens_dev, int n, bf16* x, cudaStream_t st) {
  if (n == 0) return PD_OK;
  TraceScope ts(PD_K_EMBED, st);
  embed_gather_kernel<<<n, 128, 0, st>>>(tokens_dev, m->embed, x, m->cfg.d_model, m->vocab, m->err_word);
  count_launch();
  PD_CUDA_TRY(cudaGetLastError());
  return PD_OK;
}

// h -> next tokens.  cu_dev != NULL: prefill mode, row r of the head is the last row of request r.
pd_status model_head(pd_model* m, const bf16* h, const int32_t* cu_dev, int rows, bf16* sel, bf16* norm,
                     float* logits, int32_t* next_dev, cudaStream_t st) {
  if (rows == 0) return PD_OK;
  const int d = m->cfg.d_model;
  const bf16* src = h;
  if (cu_dev) {
    TraceScope ts(PD_K_RMSNORM, st);
    select_last_rows_kernel<<<rows, 128, 0, st>>>(h, cu_dev, sel, d);
    count_launch();
    PD_CUDA_TRY(cudaGetLastError());
    src = sel;
  }
  { TraceScope ts(PD_K_RMSNORM, st); PD_TRY(launch_rmsnorm(src, m->g_final, norm, rows, d, m->cfg.rms_eps, st)); }
  SkinnyGemmArgs g{};
  g.x = norm; g.w = m->lm_head; g.acc = logits; g.batch = rows; g.n = m->vocab; g.k = d; g.ldx = d;
  g.err_word = m->err_word; g.acc_zeroed = false;
  { TraceScope ts(PD_K_LM_HEAD, st); PD_TRY(gemm_skinny(g, st)); }
  {
    TraceScope ts(PD_K_SAMPLE, st);
    argmax_rows_kernel<<<rows, ARG_THREADS, 0, st>>>(logits, cu_dev, next_dev, m->vocab);
    count_launch();
    PD_CUDA_TRY(cudaGetLastError());
  }
  return PD_OK;
}

}  // namespace pd

extern "C" pd_status pd_model_create(pd_layer* const* layers, int32_t n_layers, const pd_model_weights* w,
                                     void* stream, pd_model** out) {
  if (!layers || n_layers <= 0 || !w || w->struct_size != sizeof(pd_model_weights) || !out) return PD_ERR_INVALID_ARG;
  if (!w->embed || !w->g_final || !w->lm_head || w->vocab <= 0) return PD_ERR_INVALID_ARG;
  if (w->vocab % 4 != 0) return PD_ERR_UNSUPPORTED_SHAPE;
  for (int i = 0; i < n_layers; ++i) {
    if (!layers[i]) return PD_ERR_INVALID_ARG;
    const pd_layer_cfg &a = layers[i]->cfg, &b = layers[0]->cfg;
    if (a.d_model != b.d_model || a.n_q_heads != b.n_q_heads || a.n_kv_heads != b.n_kv_heads ||
        a.head_dim != b.head_dim || a.d_ff != b.d_ff || a.fp8_projections != b.fp8_projections)
      return PD_ERR_INVALID_ARG;
  }
  pd_model* m = new (std::nothrow) pd_model();
  if (!m) return PD_ERR_INVALID_ARG;
  m->layers.assign(layers, layers + n_layers);
  m->cfg = layers[0]->cfg;
  m->vocab = w->vocab;
  m->embed = m->lm_head = m->g_final = nullptr;
  m->err_word = nullptr;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t d = m->cfg.d_model, table = static_cast<size_t>(w->vocab) * d * 2;
  auto fail = [&](cudaError_t e) {
    pd_model_destroy(m);
    return pd::cuda_fail(e);
  };
  cudaError_t e;
  if ((e = cudaMalloc(&m->embed, table)) != cudaSuccess) return fail(e);
  if ((e = cudaMalloc(&m->lm_head, table)) != cudaSuccess) return fail(e);
  if ((e = cudaMalloc(&m->g_final, d * 2)) != cudaSuccess) return fail(e);
  if ((e = cudaMalloc(&m->err_word, sizeof(int))) != cudaSuccess) return fail(e);
  const cudaMemcpyKind d2d = cudaMemcpyDeviceToDevice;
  if ((e = cudaMemcpyAsync(m->embed, w->embed, table, d2d, st)) != cudaSuccess) return fail(e);
  if ((e = cudaMemcpyAsync(m->lm_head, w->lm_head, table, d2d, st)) != cudaSuccess) return fail(e);
  if ((e = cudaMemcpyAsync(m->g_final, w->g_final, d * 2, d2d, st)) != cudaSuccess) return fail(e);
  if ((e = cudaMemsetAsync(m->err_word, 0, sizeof(int), st)) != cudaSuccess) return fail(e);
  *out = m;
  return PD_OK;
}

extern "C" pd_status pd_model_destroy(pd_model* m) {
  if (!m) return PD_OK;
  cudaFree(m->embed); cudaFree(m->lm_head); cudaFree(m->g_final); cudaFree(m->err_word);
  delete m;
  return PD_OK;
}

extern "C" pd_status pd_model_check(pd_model* m, void* stream) {
  if (!m) return PD_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  pd_status worst = PD_OK;
  for (pd_layer* l : m->layers) {
    const pd_status s = pd_layer_check(l, stream);
    if (s != PD_OK && worst == PD_OK) worst = s;
  }
  int word = 0;
  PD_CUDA_TRY(cudaMemcpyAsync(&word, m->err_word, sizeof(int), cudaMemcpyDeviceToHost, st));
  PD_CUDA_TRY(cudaStreamSynchronize(st));
  if (word != 0) {
    PD_CUDA_TRY(cudaMemsetAsync(m->err_word, 0, sizeof(int), st));
    if (worst == PD_OK) worst = word == 1 ? PD_ERR_DEVICE_TIMEOUT : PD_ERR_INVALID_ARG;
  }
  return worst;
}

extern "C" pd_status pd_model_workspace_bytes(const pd_model* m, int32_t max_tokens, int32_t max_requests,
                                              int32_t max_batch, int32_t max_kv_len, size_t* out_bytes) {
  if (!m || !out_bytes || max_tokens < 0 || max_requests < 0 || max_batch < 0 || max_kv_len < 0)
    return PD_ERR_INVALID_ARG;
  size_t stack = 0;
  PD_TRY(pd_workspace_bytes(&m->cfg, max_tokens, max_batch, max_kv_len, &stack));
  const size_t tokens = static_cast<size_t>(max_tokens > max_batch ? max_tokens : max_batch);
  const size_t rows = static_cast<size_t>(max_requests > max_batch ? max_requests : max_batch);
  *out_bytes = carve_model(m, tokens, rows, stack, true).total;
  return PD_OK;
}

extern "C" pd_status pd_model_prefill(pd_model* m, const int32_t* tokens_dev, const int32_t* cu_dev,
                                      const int32_t* cu_host, int32_t n_req, const pd_kv_cache* caches,
                                      int32_t n_caches, int32_t* next_dev, float* logits_dev, void* workspace,
                                      size_t workspace_bytes, void* stream) {
  if (!m || !cu_host || n_req < 0 || n_req > 4095 || !caches || n_caches <= 0) return PD_ERR_INVALID_ARG;
  if (n_req == 0) return PD_OK;
  if (cu_host[0] != 0 || cu_host[n_req] < 0) return PD_ERR_INVALID_ARG;
  if (!tokens_dev || !cu_dev || !next_dev || !workspace) return PD_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(workspace) & 255u) return PD_ERR_INVALID_ARG;
  if (logits_dev && (reinterpret_cast<uintptr_t>(logits_dev) & 15u)) return PD_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int tokens = cu_host[n_req];
  if (tokens == 0) {  // only empty requests: no token follows any of them
    fill_i32_kernel<<<(n_req + 255) / 256, 256, 0, st>>>(next_dev, n_req, -1);
    pd::count_launch();
    PD_CUDA_TRY(cudaGetLastError());
    if (logits_dev) PD_CUDA_TRY(cudaMemsetAsync(logits_dev, 0, static_cast<size_t>(n_req) * m->vocab * 4, st));
    return PD_OK;
  }
  size_t stack_bytes = 0;
  PD_TRY(pd_workspace_bytes(&m->cfg, tokens, 0, 0, &stack_bytes));
  const ModelWs w = carve_model(m, tokens, n_req, stack_bytes, logits_dev == nullptr);
  if (workspace_bytes < w.total) return PD_ERR_WORKSPACE_TOO_SMALL;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  bf16* x0 = reinterpret_cast<bf16*>(ws + w.x0);
  bf16* h = reinterpret_cast<bf16*>(ws + w.h);
  float* logits = logits_dev ? logits_dev : reinterpret_cast<float*>(ws + w.logits);
  PD_TRY(pd::model_embed(m, tokens_dev, tokens, x0, st));
  PD_TRY(pd_prefill_stack(m->layers.data(), caches, static_cast<int>(m->layers.size()), n_caches, x0, h, 0, cu_dev,
                          cu_host, n_req, ws + w.stack, workspace_bytes - w.stack, stream));
  return pd::model_head(m, h, cu_dev, n_req, reinterpret_cast<bf16*>(ws + w.sel), reinterpret_cast<bf16*>(ws + w.norm),
                        logits, next_dev, st);
}

extern "C" pd_status pd_model_decode_step(pd_model* m, const int32_t* tokens_dev, const int32_t* kv_len_dev,
                                          int32_t B, int32_t max_kv_len, const pd_kv_cache* caches, int32_t n_caches,
                                          int32_t* next_dev, float* logits_dev, void* workspace,
                                          size_t workspace_bytes, void* stream) {
  if (!m || B < 0 || B > 4096 || !caches || n_caches <= 0) return PD_ERR_INVALID_ARG;
  if (B == 0) return PD_OK;
  if (!tokens_dev || !kv_len_dev || !next_dev || !workspace || max_kv_len <= 0) return PD_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(workspace) & 255u) return PD_ERR_INVALID_ARG;
  if (logits_dev && (reinterpret_cast<uintptr_t>(logits_dev) & 15u)) return PD_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  size_t stack_bytes = 0;
  PD_TRY(pd_workspace_bytes(&m->cfg, 0, B, max_kv_len, &stack_bytes));
  const ModelWs w = carve_model(m, B, B, stack_bytes, logits_dev == nullptr);
  if (workspace_bytes < w.total) return PD_ERR_WORKSPACE_TOO_SMALL;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  bf16* x0 = reinterpret_cast<bf16*>(ws + w.x0);
  bf16* h = reinterpret_cast<bf16*>(ws + w.h);
  float* logits = logits_dev ? logits_dev : reinterpret_cast<float*>(ws + w.logits);
  PD_TRY(pd::model_embed(m, tokens_dev, B, x0, st));
  PD_TRY(pd_decode_stack(m->layers.data(), caches, static_cast<int>(m->layers.size()), n_caches, x0, h, 0, kv_len_dev,
                         B, max_kv_len, ws + w.stack, workspace_bytes - w.stack, stream));
  return pd::model_head(m, h, nullptr, B, nullptr, reinterpret_cast<bf16*>(ws + w.norm), logits, next_dev, st);
}
