// The layer object and the two layer passes (prefill, decode): argument validation on
// the host, workspace carving, and the kernel sequence.  Nothing here allocates or
// synchronises except pd_layer_create / pd_layer_destroy / pd_layer_check and the
// host-I/O variants of the stack calls.
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "pd_common.cuh"

using pd::bf16;

namespace {

// Batches beyond one 256-wide batch tile run the projections on the prefill GEMM (fused epilogues, tail
// tiles split): the weight-streaming kernel would read every weight once per batch tile (measured per
// 8B-shaped layer: 327 -> 242 us at B = 384, 352 -> 275 us at B = 512; at B = 256 the two paths tie).
constexpr int kWideDecodeBatchDefault = 257;
// (PD_WIDE_DECODE_BATCH in the environment overrides it, for A/B timing.)
int wide_decode_batch() {
  static const int v = [] {
    const char* e = std::getenv("PD_WIDE_DECODE_BATCH");
    const int n = e ? std::atoi(e) : kWideDecodeBatchDefault;
    return n > 0 ? n : kWideDecodeBatchDefault;
  }();
  return v;
}

// From this batch on the gate/up projection of a decode step runs on the prefill GEMM (CTA pairs, SwiGLU in the
// epilogue) instead of the weight-streaming kernel: with N = 2 d_ff it has enough 256-wide tiles to fill the pairs
// even at one or two row tiles, and the tensor pipe, not the weight stream, is what bounds it there (measured per
// 8B-shaped layer: gate/up 74.7 -> 66.0 us at B = 256, 68.6 -> 64.4 at 192, no gain at 129; the other three
// projections are faster on the weight-streaming kernel up to B = 256: the whole layer on the prefill GEMM takes 483
// against 455 us at B = 256).
// PD_GU_GEMM_BATCH in the environment overrides the threshold (for A/B timing; 0 = never).
int gate_up_gemm_batch() {
  static const int v = [] {
    const char* e = std::getenv("PD_GU_GEMM_BATCH");
    const int n = e ? std::atoi(e) : 192;
    return n > 0 ? n : 1 << 30;
  }();
  return v;
}

struct Workspace {
  // byte offsets into the caller's workspace
  size_t norm, qkv, attn_o, resid, acc_qkv, acc_o, acc_gu, acc_down, act, partial, stage_a, stage_b, meta, splitk;
  size_t q_act, s_act;  // FP8 mode: codes and per-row scales of the activation matrix a projection is about to read
  size_t total;
};

Workspace carve(const pd_layer_cfg& c, size_t tokens, size_t max_batch, int max_kv_len) {
  const size_t d = c.d_model, nqkv = static_cast<size_t>(c.n_q_heads + 2 * c.n_kv_heads) * c.head_dim;
  const size_t hq = static_cast<size_t>(c.n_q_heads) * c.head_dim, f = c.d_ff;
  Workspace w{};
  size_t off = 0;
  auto take = [&](size_t bytes) {
    const size_t o = off;
    off += pd::align_up(bytes, 256);
    return o;
  };
  w.norm = take(tokens * d * 2);
  w.qkv = take(tokens * nqkv * 2);
  w.attn_o = take(tokens * hq * 2);
  w.resid = take(tokens * d * 2);
  w.act = take(tokens * f * 2);
  {  // fp32 sums of the four decode-mode projections, one buffer each (a buffer is cleared by a row-wise kernel
     // earlier in the chain while another one is in use); batches beyond the weight-streaming path need none
    const size_t rows = max_batch < static_cast<size_t>(wide_decode_batch()) ? max_batch : 0;
    w.acc_qkv = take(rows * nqkv * 4);
    w.acc_o = take(rows * d * 4);
    w.acc_gu = take(rows * 2 * f * 4);
    w.acc_down = take(rows * d * 4);
  }
  const int splits = max_batch ? pd::decode_attention_splits(1, c.n_kv_heads, max_kv_len) : 1;  // worst case: B = 1
  w.partial = take(max_batch * c.n_kv_heads * static_cast<size_t>(splits) * (c.n_q_heads / c.n_kv_heads) *
                   (c.head_dim + 2) * 4);
  w.stage_a = take(tokens * d * 2);  // activations between layers of a stack / staged host input
  w.stage_b = take(tokens * d * 2);
  w.meta = take(4096 * 4);           // staged cu_seqlens / kv_len of the host-I/O stack calls
  w.splitk = take(tokens > 128 ? pd::kSplitScratchBytes : 0);  // fp32 partial tiles of K-split GEMM tiles
  const size_t widest = f > hq ? (f > d ? f : d) : (hq > d ? hq : d);
  w.q_act = take(c.fp8_projections ? tokens * widest : 0);
  w.s_act = take(c.fp8_projections ? tokens * 4 : 0);
  w.total = off;
  return w;
}

pd_status check_cfg(const pd_layer_cfg* c) {
  if (!c || c->struct_size != sizeof(pd_layer_cfg)) return PD_ERR_INVALID_ARG;
  if (c->d_model <= 0 || c->n_q_heads <= 0 || c->n_kv_heads <= 0 || c->d_ff <= 0 || c->max_pos <= 0 ||
      !(c->rms_eps > 0.f) || !(c->rope_theta > 0.f))
    return PD_ERR_INVALID_ARG;
  if (c->head_dim != 64 && c->head_dim != 128) return PD_ERR_UNSUPPORTED_SHAPE;
  if (c->n_q_heads % c->n_kv_heads != 0 || c->n_q_heads / c->n_kv_heads > 16) return PD_ERR_UNSUPPORTED_SHAPE;
  if (c->d_model % 64 != 0 || c->d_ff % 64 != 0 || c->d_model > 16384) return PD_ERR_UNSUPPORTED_SHAPE;
  if (c->fp8_projections != 0 && c->fp8_projections != 1) return PD_ERR_INVALID_ARG;
  if (c->fp8_projections && (c->d_model % 128 != 0 || c->d_ff % 128 != 0 || (c->n_q_heads * c->head_dim) % 128 != 0))
    return PD_ERR_UNSUPPORTED_SHAPE;
  return PD_OK;
}

// FP8 mode: quantises the rows of `a` (the matrix a projection is about to read) into the workspace and points
// the GEMM at the codes and scales of both operands.
// (`quantised`: the producer of `a` has already left its codes and scales there.)
pd_status use_fp8(pd_layer* L, pd::GemmArgs& g, const uint8_t* w_codes, const float* w_scales, uint8_t* ws,
                  const Workspace& w, cudaStream_t st, bool quantised = false) {
  uint8_t* q = ws + w.q_act;
  float* sc = reinterpret_cast<float*>(ws + w.s_act);
  if (!quantised) PD_TRY(pd::launch_quantize_rows_fp8(g.a, g.lda, g.m, g.k, q, g.k, sc, st));
  g.a = reinterpret_cast<const bf16*>(q);
  g.lda = g.k;
  g.b = reinterpret_cast<const bf16*>(w_codes);
  g.fp8 = 1; g.scale_a = sc; g.scale_b = w_scales;
  (void)L;
  return PD_OK;
}

// The stack calls carve one workspace and one pair of inter-layer buffers from the first layer's shape, so
// every layer of a stack must have that shape (the norm constants and the RoPE table length may differ).
bool same_shape(const pd_layer_cfg& a, const pd_layer_cfg& b) {
  return a.d_model == b.d_model && a.n_q_heads == b.n_q_heads && a.n_kv_heads == b.n_kv_heads &&
         a.head_dim == b.head_dim && a.d_ff == b.d_ff && a.fp8_projections == b.fp8_projections;
}

pd_status check_cache(const pd_layer* L, const pd_kv_cache* c) {
  (void)L;
  if (!c || c->struct_size != sizeof(pd_kv_cache) || !c->k || !c->v || c->batch_cap <= 0 || c->len_cap <= 0)
    return PD_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(c->k) & 15u) || (reinterpret_cast<uintptr_t>(c->v) & 15u)) return PD_ERR_INVALID_ARG;
  return PD_OK;
}

// Lets a prefill GEMM cut the tiles of its last partial wave in two along K.
void enable_tail_split(pd_layer* L, pd::GemmArgs& g, uint8_t* ws, const Workspace& w, size_t tokens) {
  if (tokens <= 128) return;
  g.split_scratch = reinterpret_cast<float*>(ws + w.splitk);
  g.split_scratch_bytes = pd::kSplitScratchBytes;
  g.split_flags = L->split_flags;
}

// MLP half shared by both modes: h (residual stream after attention) -> out.
pd_status mlp_half(pd_layer* L, const bf16* h, bf16* out, int tokens, uint8_t* ws, const Workspace& w,
                   cudaStream_t st) {
  const pd_layer_cfg& c = L->cfg;
  bf16* norm = reinterpret_cast<bf16*>(ws + w.norm);
  bf16* act = reinterpret_cast<bf16*>(ws + w.act);
  const bool f8 = c.fp8_projections != 0;  // the norm then also emits the codes and scales the projection reads
  {
    pd::TraceScope ts(PD_K_RMSNORM, st);
    PD_TRY(pd::launch_rmsnorm(h, L->g_mlp, norm, tokens, c.d_model, c.rms_eps, st, f8 ? ws + w.q_act : nullptr,
                              f8 ? reinterpret_cast<float*>(ws + w.s_act) : nullptr));
  }
  pd::GemmArgs g{};
  g.a = norm; g.b = L->w_gu; g.c = act; g.m = tokens; g.n = 2 * c.d_ff; g.k = c.d_model;
  g.lda = c.d_model; g.ldb = c.d_model; g.ldc = c.d_ff; g.epilogue = pd::EPI_SWIGLU; g.err_word = L->err_word;
  {
    pd::TraceScope ts(PD_K_GEMM_GATE_UP, st);
    if (f8) PD_TRY(use_fp8(L, g, L->q_gu, L->s_gu, ws, w, st, true));
    PD_TRY(pd::gemm(g, st));
  }
  pd::GemmArgs g2{};
  g2.a = act; g2.b = L->w_down; g2.c = out; g2.r = h; g2.m = tokens; g2.n = c.d_model; g2.k = c.d_ff;
  g2.lda = c.d_ff; g2.ldb = c.d_ff; g2.ldc = c.d_model; g2.ldr = c.d_model; g2.epilogue = pd::EPI_RESIDUAL;
  g2.err_word = L->err_word;
  enable_tail_split(L, g2, ws, w, tokens);
  {
    pd::TraceScope ts(PD_K_GEMM_DOWN, st);
    if (c.fp8_projections) PD_TRY(use_fp8(L, g2, L->q_down, L->s_down, ws, w, st));
    PD_TRY(pd::gemm(g2, st));
  }
  return PD_OK;
}

// Attention-input half shared by both modes: x -> qkv (q rotated in place, k/v written to the cache).
pd_status qkv_half(pd_layer* L, const bf16* x, int tokens, const pd::RopeEpilogue& rope, uint8_t* ws,
                   const Workspace& w, cudaStream_t st) {
  const pd_layer_cfg& c = L->cfg;
  bf16* norm = reinterpret_cast<bf16*>(ws + w.norm);
  bf16* qkv = reinterpret_cast<bf16*>(ws + w.qkv);
  const bool f8 = c.fp8_projections != 0;
  {
    pd::TraceScope ts(PD_K_RMSNORM, st);
    PD_TRY(pd::launch_rmsnorm(x, L->g_attn, norm, tokens, c.d_model, c.rms_eps, st, f8 ? ws + w.q_act : nullptr,
                              f8 ? reinterpret_cast<float*>(ws + w.s_act) : nullptr));
  }
  pd::GemmArgs g{};
  g.a = norm; g.b = L->w_qkv; g.c = qkv; g.m = tokens; g.n = L->n_qkv; g.k = c.d_model;
  g.lda = c.d_model; g.ldb = c.d_model; g.ldc = L->n_qkv; g.epilogue = pd::EPI_ROPE_KV; g.rope = &rope;
  g.err_word = L->err_word;
  enable_tail_split(L, g, ws, w, tokens);
  {
    pd::TraceScope ts(PD_K_GEMM_QKV, st);
    if (f8) PD_TRY(use_fp8(L, g, L->q_qkv, L->s_qkv, ws, w, st, true));
    PD_TRY(pd::gemm(g, st));
  }
  return PD_OK;
}

pd_status oproj(pd_layer* L, const bf16* x, int tokens, uint8_t* ws, const Workspace& w, cudaStream_t st) {
  const pd_layer_cfg& c = L->cfg;
  const int hq = c.n_q_heads * c.head_dim;
  pd::GemmArgs g{};
  g.a = reinterpret_cast<bf16*>(ws + w.attn_o); g.b = L->w_o; g.c = reinterpret_cast<bf16*>(ws + w.resid); g.r = x;
  g.m = tokens; g.n = c.d_model; g.k = hq; g.lda = hq; g.ldb = hq; g.ldc = c.d_model; g.ldr = c.d_model;
  g.epilogue = pd::EPI_RESIDUAL; g.err_word = L->err_word;
  enable_tail_split(L, g, ws, w, tokens);
  pd::TraceScope ts(PD_K_GEMM_O, st);
  if (c.fp8_projections) PD_TRY(use_fp8(L, g, L->q_o, L->s_o, ws, w, st));
  return pd::gemm(g, st);
}

pd_status validate_prefill(const pd_layer* L, const int32_t* cu_host, int n_req, const pd_kv_cache* cache,
                           bool default_slots, int* tokens, int* max_len, const int32_t* prefix_host = nullptr) {
  if (!L || !cu_host || n_req < 0 || n_req > 4095) return PD_ERR_INVALID_ARG;
  PD_TRY(check_cache(L, cache));
  if (cu_host[0] != 0) return PD_ERR_INVALID_ARG;
  int mx = 0;
  for (int r = 0; r < n_req; ++r) {
    const int len = cu_host[r + 1] - cu_host[r];
    if (len < 0) return PD_ERR_INVALID_ARG;
    const int pre = prefix_host ? prefix_host[r] : 0;
    if (pre < 0 || pre > cache->len_cap - len || pre + len > L->cfg.max_pos) return PD_ERR_INVALID_ARG;
    if (len > mx) mx = len;
  }
  if (default_slots && n_req > cache->batch_cap) return PD_ERR_INVALID_ARG;
  *tokens = cu_host[n_req];
  *max_len = mx;
  return PD_OK;
}

pd_status prefill_impl(pd_layer* L, const bf16* x, bf16* out, const int32_t* cu_dev, int n_req, int tokens,
                       int max_len, const int32_t* slots_dev, const pd_kv_cache* cache, uint8_t* ws,
                       const Workspace& w, cudaStream_t st, const int32_t* prefix_dev = nullptr) {
  const pd_layer_cfg& c = L->cfg;
  pd::RopeEpilogue r{};
  r.k_cache = static_cast<bf16*>(cache->k); r.v_cache = static_cast<bf16*>(cache->v); r.rope_tab = L->rope_tab;
  r.cu_seqlens = cu_dev; r.slots = slots_dev; r.prefix = prefix_dev; r.kv_len = nullptr; r.n_req = n_req;
  r.n_q_heads = c.n_q_heads; r.n_kv_heads = c.n_kv_heads; r.head_dim = c.head_dim; r.len_cap = cache->len_cap;
  r.max_pos = c.max_pos; r.batch_cap = cache->batch_cap;
  PD_TRY(qkv_half(L, x, tokens, r, ws, w, st));
  pd::PrefillAttnArgs a{};
  a.q = reinterpret_cast<bf16*>(ws + w.qkv); a.ldq = L->n_qkv;
  a.k_cache = static_cast<bf16*>(cache->k); a.v_cache = static_cast<bf16*>(cache->v);
  a.o = reinterpret_cast<bf16*>(ws + w.attn_o); a.cu_seqlens = cu_dev; a.slots = slots_dev; a.prefix = prefix_dev;
  a.n_req = n_req; a.n_tokens = tokens; a.max_len = max_len;
  a.n_q_heads = c.n_q_heads; a.n_kv_heads = c.n_kv_heads; a.head_dim = c.head_dim; a.len_cap = cache->len_cap;
  a.batch_cap = cache->batch_cap;
  a.sched = L->attn_sched;
  {
    pd::TraceScope ts(PD_K_ATTN_PREFILL, st);
    PD_TRY(pd::launch_prefill_attention_tc(a, L->err_word, st));
  }
  PD_TRY(oproj(L, x, tokens, ws, w, st));
  PD_TRY(mlp_half(L, reinterpret_cast<bf16*>(ws + w.resid), out, tokens, ws, w, st));
  return PD_OK;
}


pd_status decode_impl_wide(pd_layer* L, const bf16* x, bf16* out, const int32_t* kv_len_dev, int B, int max_kv_len,
                           const pd_kv_cache* cache, uint8_t* ws, const Workspace& w, cudaStream_t st) {
  const pd_layer_cfg& c = L->cfg;
  pd::RopeEpilogue r{};
  r.k_cache = static_cast<bf16*>(cache->k); r.v_cache = static_cast<bf16*>(cache->v); r.rope_tab = L->rope_tab;
  r.cu_seqlens = nullptr; r.slots = nullptr; r.prefix = nullptr; r.kv_len = kv_len_dev; r.n_req = B;
  r.n_q_heads = c.n_q_heads; r.n_kv_heads = c.n_kv_heads; r.head_dim = c.head_dim; r.len_cap = cache->len_cap;
  r.max_pos = c.max_pos; r.batch_cap = cache->batch_cap;
  PD_TRY(qkv_half(L, x, B, r, ws, w, st));
  pd::DecodeAttnArgs a{};
  a.q = reinterpret_cast<bf16*>(ws + w.qkv); a.ldq = L->n_qkv;
  a.k_cache = static_cast<bf16*>(cache->k); a.v_cache = static_cast<bf16*>(cache->v);
  a.o = reinterpret_cast<bf16*>(ws + w.attn_o); a.kv_len = kv_len_dev;
  a.partial = reinterpret_cast<float*>(ws + w.partial);
  a.batch = B; a.max_kv_len = max_kv_len; a.n_splits = pd::decode_attention_splits(B, c.n_kv_heads, max_kv_len);
  a.n_q_heads = c.n_q_heads; a.n_kv_heads = c.n_kv_heads; a.head_dim = c.head_dim; a.len_cap = cache->len_cap;
  { pd::TraceScope ts(PD_K_ATTN_DECODE, st); PD_TRY(pd::launch_decode_attention(a, st)); }
  PD_TRY(oproj(L, x, B, ws, w, st));
  PD_TRY(mlp_half(L, reinterpret_cast<bf16*>(ws + w.resid), out, B, ws, w, st));
  return PD_OK;
}

// How a decode layer is chained to its neighbours inside a stack call: the last row-wise kernel of a
// layer can also produce the next layer's first RMSNorm (its gain is next_gain), in which case that next
// layer is told that the normalised rows (and, with FP8 projections, their codes and scales) and the
// cleared QKV accumulator are already in the workspace.
struct DecodeLink {
  bool norm_ready = false;
  const bf16* next_gain = nullptr;
};

pd_status decode_impl(pd_layer* L, const bf16* x, bf16* out, const int32_t* kv_len_dev, int B, int max_kv_len,
                      const pd_kv_cache* cache, uint8_t* ws, const Workspace& w, cudaStream_t st,
                      const DecodeLink& link = DecodeLink{}) {
  if (B >= wide_decode_batch()) return decode_impl_wide(L, x, out, kv_len_dev, B, max_kv_len, cache, ws, w, st);
  const pd_layer_cfg& c = L->cfg;
  const int hq = c.n_q_heads * c.head_dim;
  bf16* norm = reinterpret_cast<bf16*>(ws + w.norm);
  bf16* qkv = reinterpret_cast<bf16*>(ws + w.qkv);
  bf16* attn_o = reinterpret_cast<bf16*>(ws + w.attn_o);
  bf16* resid = reinterpret_cast<bf16*>(ws + w.resid);
  bf16* act = reinterpret_cast<bf16*>(ws + w.act);
  float* acc_qkv = reinterpret_cast<float*>(ws + w.acc_qkv);
  float* acc_o = reinterpret_cast<float*>(ws + w.acc_o);
  float* acc_gu = reinterpret_cast<float*>(ws + w.acc_gu);
  float* acc_down = reinterpret_cast<float*>(ws + w.acc_down);
  pd::RopeEpilogue r{};
  r.k_cache = static_cast<bf16*>(cache->k); r.v_cache = static_cast<bf16*>(cache->v); r.rope_tab = L->rope_tab;
  r.cu_seqlens = nullptr; r.slots = nullptr; r.kv_len = kv_len_dev; r.n_req = B;
  r.n_q_heads = c.n_q_heads; r.n_kv_heads = c.n_kv_heads; r.head_dim = c.head_dim; r.len_cap = cache->len_cap;
  r.max_pos = c.max_pos; r.batch_cap = cache->batch_cap;

  // The whole chain is launched with programmatic serialization (each kernel waits for its predecessor
  // only where it first needs it).  A K-split projection adds into its fp32 buffer; that buffer is cleared
  // by a row-wise kernel two or more launches earlier, never by a memset between the kernels.
  const int n_gu = 2 * c.d_ff;
  const bool f8 = c.fp8_projections != 0;
  float* z_qkv = pd::gemm_skinny_splits(B, L->n_qkv, c.d_model, f8) > 1 ? acc_qkv : nullptr;
  float* z_o = pd::gemm_skinny_splits(B, c.d_model, hq, f8) > 1 ? acc_o : nullptr;
  float* z_gu = pd::gemm_skinny_splits(B, n_gu, c.d_model, f8) > 1 ? acc_gu : nullptr;
  float* z_down = pd::gemm_skinny_splits(B, c.d_model, c.d_ff, f8) > 1 ? acc_down : nullptr;
  // Gate/up is not split along K at these shapes: SwiGLU then runs in its epilogue (no fp32 round trip, one launch
  // fewer) and the buffer of the down projection is cleared one kernel earlier.
  const bool gu_gemm = B >= gate_up_gemm_batch() && B > 128;
  const bool fuse_swiglu = gu_gemm || pd::gemm_skinny_fuses_swiglu(B, n_gu, c.d_model, f8);
  // FP8 mode: a row-wise quantiser in front of every projection (same programmatic-serialization chain)
  uint8_t* q_act = ws + w.q_act;
  float* s_act = reinterpret_cast<float*>(ws + w.s_act);
  auto fp8_in = [&](pd::SkinnyGemmArgs& a, const uint8_t* w_codes, const float* w_scales, bool quantised) -> pd_status {
    if (!f8) return PD_OK;
    if (!quantised) PD_TRY(pd::launch_quantize_rows_fp8(a.x, a.ldx, B, a.k, q_act, a.k, s_act, st));
    a.x = reinterpret_cast<const bf16*>(q_act); a.ldx = a.k;
    a.w = reinterpret_cast<const bf16*>(w_codes);
    a.fp8 = 1; a.scale_x = s_act; a.scale_w = w_scales;
    return PD_OK;
  };

  if (!link.norm_ready) {
    pd::TraceScope ts(PD_K_RMSNORM, st);
    PD_TRY(pd::launch_rmsnorm_decode(x, L->g_attn, norm, B, c.d_model, c.rms_eps, z_qkv, L->n_qkv, st,
                                     f8 ? q_act : nullptr, f8 ? s_act : nullptr));
  }
  pd::SkinnyGemmArgs g{};
  g.batch = B; g.err_word = L->err_word; g.acc_zeroed = true;
  {
    pd::TraceScope ts(PD_K_GEMM_QKV, st);
    g.x = norm; g.w = L->w_qkv; g.acc = acc_qkv; g.n = L->n_qkv; g.k = c.d_model; g.ldx = c.d_model;
    PD_TRY(fp8_in(g, L->q_qkv, L->s_qkv, true));
    PD_TRY(pd::gemm_skinny(g, st));
    PD_TRY(pd::launch_skinny_rope_kv(acc_qkv, qkv, r, B, L->err_word, z_o, c.d_model, st));
  }
  pd::DecodeAttnArgs a{};
  a.q = qkv; a.ldq = L->n_qkv;
  a.k_cache = static_cast<bf16*>(cache->k); a.v_cache = static_cast<bf16*>(cache->v);
  a.o = attn_o; a.kv_len = kv_len_dev;
  a.partial = reinterpret_cast<float*>(ws + w.partial);
  a.batch = B; a.max_kv_len = max_kv_len; a.n_splits = pd::decode_attention_splits(B, c.n_kv_heads, max_kv_len);
  a.n_q_heads = c.n_q_heads; a.n_kv_heads = c.n_kv_heads; a.head_dim = c.head_dim; a.len_cap = cache->len_cap;
  { pd::TraceScope ts(PD_K_ATTN_DECODE, st); PD_TRY(pd::launch_decode_attention(a, st)); }
  {
    pd::TraceScope ts(PD_K_GEMM_O, st);  // h = x + o W_o^T and n2 = RMSNorm(h) in the same row-wise pass
    g.x = attn_o; g.w = L->w_o; g.acc = acc_o; g.n = c.d_model; g.k = hq; g.ldx = hq;
    PD_TRY(fp8_in(g, L->q_o, L->s_o, false));
    PD_TRY(pd::gemm_skinny(g, st));
    PD_TRY(pd::launch_skinny_residual(acc_o, x, resid, L->g_mlp, norm, B, c.d_model, c.rms_eps,
                                      fuse_swiglu ? z_down : z_gu, fuse_swiglu ? c.d_model : n_gu, st,
                                      f8 ? q_act : nullptr, f8 ? s_act : nullptr));
  }
  {
    pd::TraceScope ts(PD_K_GEMM_GATE_UP, st);
    if (gu_gemm) {
      pd::GemmArgs gg{};
      gg.a = norm; gg.b = L->w_gu; gg.c = act; gg.m = B; gg.n = n_gu; gg.k = c.d_model;
      gg.lda = c.d_model; gg.ldb = c.d_model; gg.ldc = c.d_ff; gg.epilogue = pd::EPI_SWIGLU; gg.err_word = L->err_word;
      if (f8) PD_TRY(use_fp8(L, gg, L->q_gu, L->s_gu, ws, w, st, true));  // (the codes of norm are already in place)
      PD_TRY(pd::gemm(gg, st));
    } else {
      g.x = norm; g.w = L->w_gu; g.acc = acc_gu; g.n = n_gu; g.k = c.d_model; g.ldx = c.d_model;
      PD_TRY(fp8_in(g, L->q_gu, L->s_gu, true));
      g.swiglu_out = fuse_swiglu ? act : nullptr;
      PD_TRY(pd::gemm_skinny(g, st));
      g.swiglu_out = nullptr;
      if (!fuse_swiglu) PD_TRY(pd::launch_skinny_swiglu(acc_gu, act, B, c.d_ff, z_down, c.d_model, st));
    }
  }
  {
    pd::TraceScope ts(PD_K_GEMM_DOWN, st);
    g.x = act; g.w = L->w_down; g.acc = acc_down; g.n = c.d_model; g.k = c.d_ff; g.ldx = c.d_ff;
    PD_TRY(fp8_in(g, L->q_down, L->s_down, false));
    PD_TRY(pd::gemm_skinny(g, st));
    if (link.next_gain)  // out = h + down, and the next layer's first RMSNorm of it in the same pass
      PD_TRY(pd::launch_skinny_residual(acc_down, resid, out, link.next_gain, norm, B, c.d_model, c.rms_eps, z_qkv,
                                        L->n_qkv, st, f8 ? q_act : nullptr, f8 ? s_act : nullptr));
    else
      PD_TRY(pd::launch_skinny_residual(acc_down, resid, out, nullptr, nullptr, B, c.d_model, c.rms_eps, nullptr, 0, st));
  }
  return PD_OK;
}

}  // namespace

extern "C" pd_status pd_workspace_bytes(const pd_layer_cfg* cfg, int32_t max_tokens, int32_t max_batch,
                                        int32_t max_kv_len, size_t* out_bytes) {
  PD_TRY(check_cfg(cfg));
  if (!out_bytes || max_tokens < 0 || max_batch < 0 || max_kv_len < 0) return PD_ERR_INVALID_ARG;
  const size_t tokens = static_cast<size_t>(max_tokens > max_batch ? max_tokens : max_batch);
  *out_bytes = carve(*cfg, tokens, static_cast<size_t>(max_batch), max_kv_len).total;
  return PD_OK;
}

extern "C" pd_status pd_workspace_offsets(const pd_layer_cfg* cfg, int32_t tokens, pd_workspace_layout* out) {
  PD_TRY(check_cfg(cfg));
  if (!out || out->struct_size != sizeof(pd_workspace_layout) || tokens < 0) return PD_ERR_INVALID_ARG;
  const Workspace w = carve(*cfg, static_cast<size_t>(tokens), 0, 0);  // these five do not depend on the decode sizes
  out->norm = w.norm; out->qkv = w.qkv; out->attn_o = w.attn_o; out->resid = w.resid; out->act = w.act;
  return PD_OK;
}

extern "C" pd_status pd_layer_create(const pd_layer_cfg* cfg, const pd_layer_weights* w, void* stream,
                                     pd_layer** out) {
  PD_TRY(check_cfg(cfg));
  if (!w || w->struct_size != sizeof(pd_layer_weights) || !out) return PD_ERR_INVALID_ARG;
  if (!w->w_qkv || !w->w_o || !w->w_gate || !w->w_up || !w->w_down || !w->g_attn || !w->g_mlp)
    return PD_ERR_INVALID_ARG;
  int dev = 0, major = 0;
  PD_CUDA_TRY(cudaGetDevice(&dev));
  PD_CUDA_TRY(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
  if (major != 10) return PD_ERR_ARCH;
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  pd_layer* L = new (std::nothrow) pd_layer();
  if (!L) return PD_ERR_INVALID_ARG;
  L->cfg = *cfg;
  L->n_qkv = (cfg->n_q_heads + 2 * cfg->n_kv_heads) * cfg->head_dim;
  const size_t d = cfg->d_model, f = cfg->d_ff, hq = static_cast<size_t>(cfg->n_q_heads) * cfg->head_dim;
  const size_t half = cfg->head_dim / 2;
  auto fail = [&](cudaError_t e) {
    pd_layer_destroy(L);
    return pd::cuda_fail(e);
  };
  cudaError_t e;
  if ((e = cudaMalloc(&L->w_qkv, L->n_qkv * d * 2)) != cudaSuccess) return fail(e);
  if ((e = cudaMalloc(&L->w_o, d * hq * 2)) != cudaSuccess) return fail(e);
  if ((e = cudaMalloc(&L->w_gu, 2 * f * d * 2)) != cudaSuccess) return fail(e);
  if ((e = cudaMalloc(&L->w_down, d * f * 2)) != cudaSuccess) return fail(e);
  if ((e = cudaMalloc(&L->g_attn, d * 2)) != cudaSuccess) return fail(e);
  if ((e = cudaMalloc(&L->g_mlp, d * 2)) != cudaSuccess) return fail(e);
  if ((e = cudaMalloc(&L->rope_tab, static_cast<size_t>(cfg->max_pos) * half * sizeof(float2))) != cudaSuccess)
    return fail(e);
  if ((e = cudaMalloc(&L->err_word, sizeof(int))) != cudaSuccess) return fail(e);
  if ((e = cudaMalloc(&L->split_flags, pd::kSplitMaxTiles * 4 * sizeof(int))) != cudaSuccess) return fail(e);
  if ((e = cudaMemsetAsync(L->split_flags, 0, pd::kSplitMaxTiles * 4 * sizeof(int), st)) != cudaSuccess) return fail(e);
  if ((e = cudaMalloc(&L->attn_sched, 2 * sizeof(int))) != cudaSuccess) return fail(e);
  if ((e = cudaMemsetAsync(L->attn_sched, 0, 2 * sizeof(int), st)) != cudaSuccess) return fail(e);
  const cudaMemcpyKind d2d = cudaMemcpyDeviceToDevice;
  if ((e = cudaMemcpyAsync(L->w_qkv, w->w_qkv, L->n_qkv * d * 2, d2d, st)) != cudaSuccess) return fail(e);
  if ((e = cudaMemcpyAsync(L->w_o, w->w_o, d * hq * 2, d2d, st)) != cudaSuccess) return fail(e);
  // 64 gate rows, the matching 64 up rows, and so on: a GEMM tile then holds both halves of its SwiGLU outputs
  if ((e = cudaMemcpy2DAsync(L->w_gu, 128 * d * 2, w->w_gate, 64 * d * 2, 64 * d * 2, f / 64, d2d, st)) != cudaSuccess)
    return fail(e);
  if ((e = cudaMemcpy2DAsync(L->w_gu + 64 * d, 128 * d * 2, w->w_up, 64 * d * 2, 64 * d * 2, f / 64, d2d, st)) != cudaSuccess)
    return fail(e);
  if ((e = cudaMemcpyAsync(L->w_down, w->w_down, d * f * 2, d2d, st)) != cudaSuccess) return fail(e);
  if ((e = cudaMemcpyAsync(L->g_attn, w->g_attn, d * 2, d2d, st)) != cudaSuccess) return fail(e);
  if ((e = cudaMemcpyAsync(L->g_mlp, w->g_mlp, d * 2, d2d, st)) != cudaSuccess) return fail(e);
  if ((e = cudaMemsetAsync(L->err_word, 0, sizeof(int), st)) != cudaSuccess) return fail(e);

  if (cfg->fp8_projections) {
    // per-output-channel E4M3 codes and scales of the four (repacked) matrices; the bf16 copies are then released
    struct Q { bf16** src; uint8_t** codes; float** scales; size_t rows, k; } qs[4] = {
        {&L->w_qkv, &L->q_qkv, &L->s_qkv, static_cast<size_t>(L->n_qkv), d}, {&L->w_o, &L->q_o, &L->s_o, d, hq},
        {&L->w_gu, &L->q_gu, &L->s_gu, 2 * f, d}, {&L->w_down, &L->q_down, &L->s_down, d, f}};
    for (auto& q : qs) {
      if ((e = cudaMalloc(q.codes, q.rows * q.k)) != cudaSuccess) return fail(e);
      if ((e = cudaMalloc(q.scales, q.rows * sizeof(float))) != cudaSuccess) return fail(e);
      const pd_status qs_st = pd::launch_quantize_rows_fp8(*q.src, static_cast<int>(q.k), static_cast<int>(q.rows),
                                                           static_cast<int>(q.k), *q.codes, static_cast<int>(q.k),
                                                           *q.scales, st);
      if (qs_st != PD_OK) { pd_layer_destroy(L); return qs_st; }
    }
    if ((e = cudaStreamSynchronize(st)) != cudaSuccess) return fail(e);
    for (auto& q : qs) { cudaFree(*q.src); *q.src = nullptr; }
  }

  // RoPE table in double on the host: (cos, sin)(pos * theta^(-2i/hd))
  std::vector<float2> tab(static_cast<size_t>(cfg->max_pos) * half);
  std::vector<double> inv_freq(half);
  for (size_t i = 0; i < half; ++i)
    inv_freq[i] = std::pow(static_cast<double>(cfg->rope_theta), -2.0 * static_cast<double>(i) / cfg->head_dim);
  for (int p = 0; p < cfg->max_pos; ++p)
    for (size_t i = 0; i < half; ++i) {
      const double ang = static_cast<double>(p) * inv_freq[i];
      tab[static_cast<size_t>(p) * half + i] = make_float2(static_cast<float>(std::cos(ang)), static_cast<float>(std::sin(ang)));
    }
  // the table is a stack temporary: copy synchronously with respect to the host
  if ((e = cudaMemcpy(L->rope_tab, tab.data(), tab.size() * sizeof(float2), cudaMemcpyHostToDevice)) != cudaSuccess)
    return fail(e);
  *out = L;
  return PD_OK;
}

extern "C" pd_status pd_layer_destroy(pd_layer* L) {
  if (!L) return PD_OK;
  cudaFree(L->w_qkv); cudaFree(L->w_o); cudaFree(L->w_gu); cudaFree(L->w_down);
  cudaFree(L->q_qkv); cudaFree(L->q_o); cudaFree(L->q_gu); cudaFree(L->q_down);
  cudaFree(L->s_qkv); cudaFree(L->s_o); cudaFree(L->s_gu); cudaFree(L->s_down);
  cudaFree(L->g_attn); cudaFree(L->g_mlp); cudaFree(L->rope_tab); cudaFree(L->err_word); cudaFree(L->split_flags);
  cudaFree(L->attn_sched);
  delete L;
  return PD_OK;
}

extern "C" pd_status pd_layer_check(pd_layer* L, void* stream) {
  if (!L) return PD_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int word = 0;
  PD_CUDA_TRY(cudaMemcpyAsync(&word, L->err_word, sizeof(int), cudaMemcpyDeviceToHost, st));
  PD_CUDA_TRY(cudaStreamSynchronize(st));
  if (word != 0) {
    PD_CUDA_TRY(cudaMemsetAsync(L->err_word, 0, sizeof(int), st));
    // an aborted K-split GEMM may have left a hand-over flag raised
    PD_CUDA_TRY(cudaMemsetAsync(L->split_flags, 0, pd::kSplitMaxTiles * 4 * sizeof(int), st));
    PD_CUDA_TRY(cudaMemsetAsync(L->attn_sched, 0, 2 * sizeof(int), st));
    return word == 2 ? PD_ERR_INVALID_ARG : PD_ERR_DEVICE_TIMEOUT;
  }
  return PD_OK;
}

extern "C" pd_status pd_prefill_layer(pd_layer* L, const void* x, void* out, const int32_t* cu_dev,
                                      const int32_t* cu_host, int32_t n_req, const int32_t* slots_dev,
                                      const pd_kv_cache* cache, void* workspace, size_t workspace_bytes,
                                      void* stream) {
  int tokens = 0, max_len = 0;
  PD_TRY(validate_prefill(L, cu_host, n_req, cache, slots_dev == nullptr, &tokens, &max_len));
  if (tokens == 0) return PD_OK;
  if (!x || !out || !cu_dev || !workspace) return PD_ERR_INVALID_ARG;
  const Workspace w = carve(L->cfg, tokens, 0, 0);
  if (workspace_bytes < w.total) return PD_ERR_WORKSPACE_TOO_SMALL;
  if (reinterpret_cast<uintptr_t>(workspace) & 255u) return PD_ERR_INVALID_ARG;
  return prefill_impl(L, static_cast<const bf16*>(x), static_cast<bf16*>(out), cu_dev, n_req, tokens, max_len,
                      slots_dev, cache, static_cast<uint8_t*>(workspace), w, static_cast<cudaStream_t>(stream));
}

extern "C" pd_status pd_prefill_chunk_layer(pd_layer* L, const void* x, void* out, const int32_t* cu_dev,
                                            const int32_t* cu_host, int32_t n_req, const int32_t* prefix_dev,
                                            const int32_t* prefix_host, const int32_t* slots_dev,
                                            const pd_kv_cache* cache, void* workspace, size_t workspace_bytes,
                                            void* stream) {
  if (!prefix_dev || !prefix_host) return PD_ERR_INVALID_ARG;
  int tokens = 0, max_len = 0;
  PD_TRY(validate_prefill(L, cu_host, n_req, cache, slots_dev == nullptr, &tokens, &max_len, prefix_host));
  if (tokens == 0) return PD_OK;
  if (!x || !out || !cu_dev || !workspace) return PD_ERR_INVALID_ARG;
  const Workspace w = carve(L->cfg, tokens, 0, 0);
  if (workspace_bytes < w.total) return PD_ERR_WORKSPACE_TOO_SMALL;
  if (reinterpret_cast<uintptr_t>(workspace) & 255u) return PD_ERR_INVALID_ARG;
  return prefill_impl(L, static_cast<const bf16*>(x), static_cast<bf16*>(out), cu_dev, n_req, tokens, max_len,
                      slots_dev, cache, static_cast<uint8_t*>(workspace), w, static_cast<cudaStream_t>(stream),
                      prefix_dev);
}

extern "C" pd_status pd_decode_layer(pd_layer* L, const void* x, void* out, const int32_t* kv_len_dev, int32_t B,
                                     int32_t max_kv_len, const pd_kv_cache* cache, void* workspace,
                                     size_t workspace_bytes, void* stream) {
  if (!L || B < 0) return PD_ERR_INVALID_ARG;
  if (B == 0) return PD_OK;
  PD_TRY(check_cache(L, cache));
  if (!x || !out || !kv_len_dev || !workspace) return PD_ERR_INVALID_ARG;
  if (B > cache->batch_cap || max_kv_len <= 0 || max_kv_len > cache->len_cap || max_kv_len > L->cfg.max_pos)
    return PD_ERR_INVALID_ARG;
  const Workspace w = carve(L->cfg, B, B, max_kv_len);
  if (workspace_bytes < w.total) return PD_ERR_WORKSPACE_TOO_SMALL;
  if (reinterpret_cast<uintptr_t>(workspace) & 255u) return PD_ERR_INVALID_ARG;
  return decode_impl(L, static_cast<const bf16*>(x), static_cast<bf16*>(out), kv_len_dev, B, max_kv_len, cache,
                     static_cast<uint8_t*>(workspace), w, static_cast<cudaStream_t>(stream));
}

extern "C" pd_status pd_decode_attention_workspace_bytes(const pd_layer_cfg* cfg, int32_t B, int32_t max_kv_len,
                                                         size_t* out_bytes) {
  PD_TRY(check_cfg(cfg));
  if (!out_bytes || B < 0 || max_kv_len < 0) return PD_ERR_INVALID_ARG;
  const int splits = B ? pd::decode_attention_splits(B, cfg->n_kv_heads, max_kv_len) : 1;
  *out_bytes = pd::align_up(static_cast<size_t>(B) * cfg->n_kv_heads * splits * (cfg->n_q_heads / cfg->n_kv_heads) *
                                (cfg->head_dim + 2) * 4, 256);
  return PD_OK;
}

extern "C" pd_status pd_decode_attention(const pd_layer_cfg* cfg, const void* q, int32_t ldq, void* out,
                                         const int32_t* kv_len_dev, int32_t B, int32_t max_kv_len,
                                         const pd_kv_cache* cache, void* workspace, size_t workspace_bytes,
                                         void* stream) {
  PD_TRY(check_cfg(cfg));
  if (B < 0) return PD_ERR_INVALID_ARG;
  if (B == 0) return PD_OK;
  PD_TRY(check_cache(nullptr, cache));
  if (!q || !out || !kv_len_dev || ldq < cfg->n_q_heads * cfg->head_dim || ldq % 8 != 0) return PD_ERR_INVALID_ARG;
  if (B > cache->batch_cap || max_kv_len <= 0 || max_kv_len > cache->len_cap) return PD_ERR_INVALID_ARG;
  size_t need = 0;
  PD_TRY(pd_decode_attention_workspace_bytes(cfg, B, max_kv_len, &need));
  pd::DecodeAttnArgs a{};
  a.n_splits = pd::decode_attention_splits(B, cfg->n_kv_heads, max_kv_len);
  if (a.n_splits > 1) {
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return PD_ERR_INVALID_ARG;
    if (workspace_bytes < need) return PD_ERR_WORKSPACE_TOO_SMALL;
  }
  a.q = static_cast<const bf16*>(q); a.ldq = ldq;
  a.k_cache = static_cast<const bf16*>(cache->k); a.v_cache = static_cast<const bf16*>(cache->v);
  a.o = static_cast<bf16*>(out); a.kv_len = kv_len_dev; a.partial = static_cast<float*>(workspace);
  a.batch = B; a.max_kv_len = max_kv_len;
  a.n_q_heads = cfg->n_q_heads; a.n_kv_heads = cfg->n_kv_heads; a.head_dim = cfg->head_dim; a.len_cap = cache->len_cap;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  pd::TraceScope ts(PD_K_ATTN_DECODE, st);
  return pd::launch_decode_attention(a, st);
}

extern "C" pd_status pd_prefill_attention(const pd_layer_cfg* cfg, const void* q, int32_t ldq, void* out,
                                          const int32_t* cu_dev, const int32_t* cu_host, int32_t n_req,
                                          const int32_t* prefix_dev, const int32_t* prefix_host,
                                          const int32_t* slots_dev, const pd_kv_cache* cache, int32_t* err_word,
                                          void* stream) {
  PD_TRY(check_cfg(cfg));
  if (!cu_host || n_req < 0 || n_req > 4095 || (prefix_dev == nullptr) != (prefix_host == nullptr))
    return PD_ERR_INVALID_ARG;
  PD_TRY(check_cache(nullptr, cache));
  if (cu_host[0] != 0) return PD_ERR_INVALID_ARG;
  int max_len = 0;
  for (int r = 0; r < n_req; ++r) {
    const int len = cu_host[r + 1] - cu_host[r];
    const int pre = prefix_host ? prefix_host[r] : 0;
    if (len < 0 || pre < 0 || pre > cache->len_cap - len) return PD_ERR_INVALID_ARG;
    if (len > max_len) max_len = len;
  }
  if (!slots_dev && n_req > cache->batch_cap) return PD_ERR_INVALID_ARG;
  const int tokens = cu_host[n_req];
  if (tokens == 0) return PD_OK;
  if (!q || !out || !cu_dev || ldq < cfg->n_q_heads * cfg->head_dim || ldq % 8 != 0) return PD_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(out) & 31u) return PD_ERR_INVALID_ARG;
  pd::PrefillAttnArgs a{};
  a.q = static_cast<const bf16*>(q); a.ldq = ldq;
  a.k_cache = static_cast<const bf16*>(cache->k); a.v_cache = static_cast<const bf16*>(cache->v);
  a.o = static_cast<bf16*>(out); a.cu_seqlens = cu_dev; a.slots = slots_dev; a.prefix = prefix_dev;
  a.n_req = n_req; a.n_tokens = tokens; a.max_len = max_len;
  a.n_q_heads = cfg->n_q_heads; a.n_kv_heads = cfg->n_kv_heads; a.head_dim = cfg->head_dim;
  a.len_cap = cache->len_cap; a.batch_cap = cache->batch_cap;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  pd::TraceScope ts(PD_K_ATTN_PREFILL, st);
  return pd::launch_prefill_attention_tc(a, err_word, st);
}

extern "C" pd_status pd_prefill_stack(pd_layer* const* layers, const pd_kv_cache* caches, int32_t n_layers,
                                      int32_t n_caches, const void* x, void* out, int32_t io_on_host,
                                      const int32_t* cu_dev, const int32_t* cu_host, int32_t n_req, void* workspace,
                                      size_t workspace_bytes, void* stream) {
  if (!layers || !caches || n_layers <= 0 || n_caches <= 0 || !layers[0]) return PD_ERR_INVALID_ARG;
  int tokens = 0, max_len = 0;
  for (int i = 0; i < n_layers; ++i) {
    if (!layers[i] || !same_shape(layers[i]->cfg, layers[0]->cfg)) return PD_ERR_INVALID_ARG;
    PD_TRY(validate_prefill(layers[i], cu_host, n_req, &caches[i % n_caches], true, &tokens, &max_len));
  }
  if (tokens == 0) return PD_OK;
  if (!x || !out || !workspace || (!io_on_host && !cu_dev)) return PD_ERR_INVALID_ARG;
  const Workspace w = carve(layers[0]->cfg, tokens, 0, 0);
  if (workspace_bytes < w.total) return PD_ERR_WORKSPACE_TOO_SMALL;
  if (reinterpret_cast<uintptr_t>(workspace) & 255u) return PD_ERR_INVALID_ARG;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t act_bytes = static_cast<size_t>(tokens) * layers[0]->cfg.d_model * 2;
  bf16* buf[2] = {reinterpret_cast<bf16*>(ws + w.stage_a), reinterpret_cast<bf16*>(ws + w.stage_b)};
  const bf16* cur = static_cast<const bf16*>(x);
  if (io_on_host) {
    PD_CUDA_TRY(cudaMemcpyAsync(buf[0], x, act_bytes, cudaMemcpyHostToDevice, st));
    PD_CUDA_TRY(cudaMemcpyAsync(ws + w.meta, cu_host, (n_req + 1) * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    cu_dev = reinterpret_cast<const int32_t*>(ws + w.meta);
    cur = buf[0];
  }
  for (int i = 0; i < n_layers; ++i) {
    bf16* dst = (i == n_layers - 1 && !io_on_host) ? static_cast<bf16*>(out) : buf[(i + 1) & 1];
    PD_TRY(prefill_impl(layers[i], cur, dst, cu_dev, n_req, tokens, max_len, nullptr, &caches[i % n_caches], ws, w, st));
    cur = dst;
  }
  if (io_on_host) {
    PD_CUDA_TRY(cudaMemcpyAsync(out, cur, act_bytes, cudaMemcpyDeviceToHost, st));
    PD_CUDA_TRY(cudaStreamSynchronize(st));
  }
  return PD_OK;
}

extern "C" pd_status pd_prefill_chunk_stack(pd_layer* const* layers, const pd_kv_cache* caches, int32_t n_layers,
                                            int32_t n_caches, const void* x, void* out, const int32_t* cu_dev,
                                            const int32_t* cu_host, int32_t n_req, const int32_t* prefix_dev,
                                            const int32_t* prefix_host, void* workspace, size_t workspace_bytes,
                                            void* stream) {
  if (!layers || !caches || n_layers <= 0 || n_caches <= 0 || !layers[0] || !prefix_dev || !prefix_host)
    return PD_ERR_INVALID_ARG;
  int tokens = 0, max_len = 0;
  for (int i = 0; i < n_layers; ++i) {
    if (!layers[i] || !same_shape(layers[i]->cfg, layers[0]->cfg)) return PD_ERR_INVALID_ARG;
    PD_TRY(validate_prefill(layers[i], cu_host, n_req, &caches[i % n_caches], true, &tokens, &max_len, prefix_host));
  }
  if (tokens == 0) return PD_OK;
  if (!x || !out || !workspace || !cu_dev) return PD_ERR_INVALID_ARG;
  const Workspace w = carve(layers[0]->cfg, tokens, 0, 0);
  if (workspace_bytes < w.total) return PD_ERR_WORKSPACE_TOO_SMALL;
  if (reinterpret_cast<uintptr_t>(workspace) & 255u) return PD_ERR_INVALID_ARG;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  bf16* buf[2] = {reinterpret_cast<bf16*>(ws + w.stage_a), reinterpret_cast<bf16*>(ws + w.stage_b)};
  const bf16* cur = static_cast<const bf16*>(x);
  for (int i = 0; i < n_layers; ++i) {
    bf16* dst = (i == n_layers - 1) ? static_cast<bf16*>(out) : buf[(i + 1) & 1];
    PD_TRY(prefill_impl(layers[i], cur, dst, cu_dev, n_req, tokens, max_len, nullptr, &caches[i % n_caches], ws, w, st,
                        prefix_dev));
    cur = dst;
  }
  return PD_OK;
}

extern "C" pd_status pd_decode_stack(pd_layer* const* layers, const pd_kv_cache* caches, int32_t n_layers,
                                     int32_t n_caches, const void* x, void* out, int32_t io_on_host,
                                     const int32_t* kv_len, int32_t B, int32_t max_kv_len, void* workspace,
                                     size_t workspace_bytes, void* stream) {
  if (!layers || !caches || n_layers <= 0 || n_caches <= 0 || B < 0 || B > 4096) return PD_ERR_INVALID_ARG;
  if (B == 0) return PD_OK;
  for (int i = 0; i < n_layers; ++i) {
    if (!layers[i] || !layers[0] || !same_shape(layers[i]->cfg, layers[0]->cfg)) return PD_ERR_INVALID_ARG;
    const pd_kv_cache* c = &caches[i % n_caches];
    PD_TRY(check_cache(layers[i], c));
    if (B > c->batch_cap || max_kv_len <= 0 || max_kv_len > c->len_cap || max_kv_len > layers[i]->cfg.max_pos)
      return PD_ERR_INVALID_ARG;
  }
  if (!x || !out || !kv_len || !workspace) return PD_ERR_INVALID_ARG;
  const Workspace w = carve(layers[0]->cfg, B, B, max_kv_len);
  if (workspace_bytes < w.total) return PD_ERR_WORKSPACE_TOO_SMALL;
  if (reinterpret_cast<uintptr_t>(workspace) & 255u) return PD_ERR_INVALID_ARG;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t act_bytes = static_cast<size_t>(B) * layers[0]->cfg.d_model * 2;
  bf16* buf[2] = {reinterpret_cast<bf16*>(ws + w.stage_a), reinterpret_cast<bf16*>(ws + w.stage_b)};
  const bf16* cur = static_cast<const bf16*>(x);
  const int32_t* kv_dev = kv_len;
  if (io_on_host) {
    PD_CUDA_TRY(cudaMemcpyAsync(buf[0], x, act_bytes, cudaMemcpyHostToDevice, st));
    PD_CUDA_TRY(cudaMemcpyAsync(ws + w.meta, kv_len, B * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    kv_dev = reinterpret_cast<const int32_t*>(ws + w.meta);
    cur = buf[0];
  }
  // Between two layers of the same shape the first RMSNorm of the second runs inside the last row-wise kernel
  // of the first (one launch fewer per layer); PD_FUSE_NEXT_NORM=0 in the environment keeps them apart.
  static const bool fuse_next_norm = [] {
    const char* v = std::getenv("PD_FUSE_NEXT_NORM");
    return !(v && v[0] == '0');
  }();
  DecodeLink link{};
  for (int i = 0; i < n_layers; ++i) {
    bf16* dst = (i == n_layers - 1 && !io_on_host) ? static_cast<bf16*>(out) : buf[(i + 1) & 1];
    const bool fuse = fuse_next_norm && i + 1 < n_layers && B < wide_decode_batch() &&
                      std::memcmp(&layers[i]->cfg, &layers[i + 1]->cfg, sizeof(pd_layer_cfg)) == 0;
    link.next_gain = fuse ? layers[i + 1]->g_attn : nullptr;
    PD_TRY(decode_impl(layers[i], cur, dst, kv_dev, B, max_kv_len, &caches[i % n_caches], ws, w, st, link));
    link.norm_ready = fuse;
    cur = dst;
  }
  if (io_on_host) {
    PD_CUDA_TRY(cudaMemcpyAsync(out, cur, act_bytes, cudaMemcpyDeviceToHost, st));
    PD_CUDA_TRY(cudaStreamSynchronize(st));
  }
  return PD_OK;
}
