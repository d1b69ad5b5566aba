// Shared host-side helpers of the CUDA translation units: status plumbing, the
// layer object, tensor-map creation and kernel launcher declarations.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "pd.h"

namespace pd {

typedef __nv_bfloat16 bf16;

pd_status cuda_fail(cudaError_t e);  // records e for pd_last_cuda_error(), returns PD_ERR_CUDA

#define PD_CUDA_TRY(expr)                              \
  do {                                                 \
    cudaError_t pd_e_ = (expr);                        \
    if (pd_e_ != cudaSuccess) return ::pd::cuda_fail(pd_e_); \
  } while (0)

#define PD_TRY(expr)                    \
  do {                                  \
    pd_status pd_s_ = (expr);           \
    if (pd_s_ != PD_OK) return pd_s_;   \
  } while (0)

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Per-device memo for launch set-up.  The opt-in to large dynamic shared memory (cudaFuncSetAttribute) and the
// answers of the occupancy queries belong to one device, so a process that drives several GPUs needs them once
// per device ordinal, not once per process.  Slot = ordinal of the current device (ordinals >= kMaxDevices share
// the last slot's "unknown" state and simply redo the set-up on every call).
constexpr int kMaxDevices = 64;
inline int current_device_slot() {
  int d = 0;
  if (cudaGetDevice(&d) != cudaSuccess || d < 0 || d >= kMaxDevices) return -1;
  return d;
}
struct PerDeviceInt {
  std::atomic<int> v[kMaxDevices];
  PerDeviceInt() { for (auto& e : v) e.store(-1, std::memory_order_relaxed); }
  // -1 = not yet determined on the current device
  int get() const { const int s = current_device_slot(); return s < 0 ? -1 : v[s].load(std::memory_order_acquire); }
  void set(int value) { const int s = current_device_slot(); if (s >= 0) v[s].store(value, std::memory_order_release); }
};
// Opts `kern` in to `bytes` of dynamic shared memory on the current device, once per device.
template <class K>
pd_status opt_in_smem(PerDeviceInt& memo, K kern, int bytes) {
  if (memo.get() == 1) return PD_OK;
  PD_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
  memo.set(1);
  return PD_OK;
}

// Counts kernel launches made by this thread (reported by pd_measure).
extern thread_local long long g_launch_count;
inline void count_launch(int n = 1) { g_launch_count += n; }

// Launches `kern` so that it may begin while the previous kernel of `st` is still running (programmatic
// dependent launch).  Such a kernel must call ptx::grid_dependency_wait() before it touches anything an
// earlier kernel writes or still reads; everything before that call overlaps the predecessor's tail.
// PD_DISABLE_PDL=1 in the environment launches normally instead (for A/B timing).
bool pdl_enabled();
template <class... KArgs, class... Args>
cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl_enabled() ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

// Test hook behind pd_test_inject_wait_timeout: true (once) if the calling thread armed an injection for this
// kind of kernel; the launcher then gives the kernel the short wait bound and tells its producer to leave out
// one tile load.
bool take_wait_injection(int kind, unsigned long long* limit_ns);

// Brackets the kernels launched in its scope with CUDA events while a trace is active
// (pd_trace_begin .. pd_trace_end); free otherwise.
class TraceScope {
 public:
  TraceScope(int cls, cudaStream_t s);
  ~TraceScope();
  TraceScope(const TraceScope&) = delete;
  TraceScope& operator=(const TraceScope&) = delete;

 private:
  cudaStream_t stream_;
  int idx_;
};

// ------------------------------------------------------------ tensor maps
// 2-D bf16 row-major tensor [rows, cols] with row pitch `ld` elements, tiled in boxes of
// box_rows x 64 columns with the 128-byte shared-memory swizzle.
pd_status make_tmap_bf16(CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols, uint64_t ld,
                         uint32_t box_rows);

// The same for one-byte elements (FP8 codes): boxes of box_rows x 128 columns.
pd_status make_tmap_u8(CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols, uint64_t ld,
                       uint32_t box_rows);

// ------------------------------------------------------------------ GEMM
enum GemmEpilogue : int {
  EPI_STORE = 0,     // C = acc
  EPI_RESIDUAL = 1,  // C = R + acc
  EPI_SWIGLU = 2,    // C[M, N/2] = silu(gate) * up, B rows interleaved gate/up in blocks of 64
  EPI_ROPE_KV = 3,   // rotate-half RoPE on q and k heads; q -> C, k and v -> the KV cache
};

// What the RoPE / KV-write epilogue needs besides the accumulator.  Row t of the product is token t:
// prefill finds its request by binary search in cu_seqlens (position = offset in the request, cache
// sequence = slots[request] or the request index); decode uses position kv_len[t], sequence t.
struct RopeEpilogue {
  const float2* rope_tab;     // [max_pos, hd/2] (cos, sin)
  const int32_t* cu_seqlens;  // prefill: device [n_req + 1]; decode: NULL
  const int32_t* slots;       // prefill: device [n_req] or NULL
  const int32_t* prefix;      // chunked prefill: device [n_req] tokens already cached per request, or NULL
  const int32_t* kv_len;      // decode: device [B]
  bf16* k_cache;              // [batch_cap, Hkv, len_cap, hd]
  bf16* v_cache;
  int n_req, n_q_heads, n_kv_heads, head_dim, len_cap, batch_cap, max_pos;
};

struct GemmArgs {
  const bf16* a;  // [M, K], row pitch lda (FP8 operands: E4M3 codes, one byte per element, behind the same pointers)
  const bf16* b;  // [N, K], row pitch ldb
  bf16* c;        // [M, N] (EPI_SWIGLU: [M, N/2]; EPI_ROPE_KV: q heads only), row pitch ldc
  const bf16* r;  // residual [M, N], row pitch ldr (EPI_RESIDUAL); may alias c
  int m, n, k;
  int lda, ldb, ldc, ldr;
  int epilogue;
  int fp8;                    // 1: A and B hold E4M3 codes; the product is scaled by scale_a[row] * scale_b[column]
  const float* scale_a;       // [M]
  const float* scale_b;       // [N]
  const RopeEpilogue* rope;   // EPI_ROPE_KV
  int* err_word;              // device int32: 1 = a bounded wait gave up, 2 = a position or slot was out of range
  // Optional K split of the last partial wave (see gemm_tc_kernel): fp32 scratch of at least
  // kSplitMaxTiles * 128 * 256 * 4 bytes and kSplitMaxTiles * 4 flags that are zero between launches.
  // Launches sharing flags must be ordered on one stream.
  float* split_scratch;
  size_t split_scratch_bytes;
  int* split_flags;
};
constexpr int kSplitMaxTiles = 74;
constexpr size_t kSplitScratchBytes = static_cast<size_t>(kSplitMaxTiles) * 128 * 256 * 4;

// Tensor-core GEMM (tcgen05 + TMEM accumulators, operands staged by TMA).
pd_status gemm(const GemmArgs& g, cudaStream_t stream);
// Tile width (rows of B per tile) the GEMM will use for this problem.
int gemm_block_n(int m, int n, int epilogue);

// Decode-mode projection: acc[B, N] (fp32) = X[B, K] * W[N, K]^T, weight-streaming, K split over
// blocks (the buffer is zeroed and accumulated with atomics when it is split).
struct SkinnyGemmArgs {
  const bf16* x;  // [B, K], row pitch ldx
  const bf16* w;  // [N, K] contiguous
  float* acc;     // [B, N]
  int batch, n, k, ldx;
  int* err_word;
  bool acc_zeroed;  // the caller guarantees acc is zero when the kernel's epilogue runs (no memset is enqueued)
  int fp8;                 // 1: x and w hold E4M3 codes (one byte per element); sums are scaled by scale_x[b] * scale_w[n]
  const float* scale_x;    // [B]
  const float* scale_w;    // [N]
  // Not NULL: w is a gate/up matrix (64 gate rows, 64 up rows, alternating) and the kernel writes
  // silu(gate) * up as bf16 [B, N/2] here instead of the fp32 sums.  Only where gemm_skinny_fuses_swiglu() holds.
  bf16* swiglu_out;
};
pd_status gemm_skinny(const SkinnyGemmArgs& g, cudaStream_t stream);
// Number of K slices gemm_skinny will use (1: plain stores, acc need not be zero).
int gemm_skinny_splits(int batch, int n, int k, bool fp8 = false);
// True when the projection is not split along K for this batch, so that SwiGLU can be applied in its epilogue.
bool gemm_skinny_fuses_swiglu(int batch, int n, int k, bool fp8 = false);
// Row-wise kernels that turn the fp32 sums into the layer's stored tensors.
// Every row-wise kernel can also clear the fp32 sums of a LATER projection (zero_ptr[batch, zero_cols], NULL to
// skip): the buffer is idle while the kernel runs, and the projection then needs no memset of its own.
pd_status launch_skinny_rope_kv(const float* acc, bf16* qkv, const RopeEpilogue& rp, int batch, int* err_word,
                                float* zero_ptr, int zero_cols, cudaStream_t s);
// h = x + acc; if n != NULL also n = RMSNorm(h) * gain (and, with q_out / s_out, the E4M3 codes and scales of n).
pd_status launch_skinny_residual(const float* acc, const bf16* x, bf16* h, const bf16* gain, bf16* n, int batch, int d,
                                 float eps, float* zero_ptr, int zero_cols, cudaStream_t s, uint8_t* q_out = nullptr,
                                 float* s_out = nullptr);
// out[B, F] = silu(gate) * up from acc[B, 2F] whose columns follow the 64/64 interleaved weight rows.
pd_status launch_skinny_swiglu(const float* acc, bf16* out, int batch, int f, float* zero_ptr, int zero_cols,
                               cudaStream_t s);

// ------------------------------------------------------------ whole model
// Pieces of the whole-model step around the layer stack (the measurement harness times them alone).
pd_status model_embed(pd_model* m, const int32_t* tokens_dev, int n, bf16* x, cudaStream_t st);
// h -> logits -> greedy tokens; cu_dev != NULL selects the last row of each request first (into sel).
pd_status model_head(pd_model* m, const bf16* h, const int32_t* cu_dev, int rows, bf16* sel, bf16* norm,
                     float* logits, int32_t* next_dev, cudaStream_t st);

// ------------------------------------------------------------ elementwise
// q_out / s_out (both or neither): also emit the E4M3 codes [rows, d] and per-row scales of the stored result,
// identical to running launch_quantize_rows_fp8 on y.
pd_status launch_rmsnorm(const bf16* x, const bf16* gain, bf16* y, int rows, int d, float eps, cudaStream_t s,
                         uint8_t* q_out = nullptr, float* s_out = nullptr);
// The same as the first kernel of a decode layer: launched with programmatic serialization, and clears
// zero_ptr[rows, zero_cols] (fp32, NULL to skip) for a later projection.
pd_status launch_rmsnorm_decode(const bf16* x, const bf16* gain, bf16* y, int rows, int d, float eps, float* zero_ptr,
                                int zero_cols, cudaStream_t s, uint8_t* q_out = nullptr, float* s_out = nullptr);

// -------------------------------------------------------------- attention
struct PrefillAttnArgs {
  const bf16* q;       // [T, ldq] (head h at column h*hd)
  int ldq;
  const bf16* k_cache; // [batch_cap, Hkv, len_cap, hd]
  const bf16* v_cache;
  bf16* o;             // [T, Hq*hd]
  const int32_t* cu_seqlens;  // device [n_req+1]
  const int32_t* slots;       // device [n_req] or NULL
  const int32_t* prefix;      // device [n_req] cached tokens before each request's rows, or NULL
  int n_req, n_tokens, max_len;
  int n_q_heads, n_kv_heads, head_dim, len_cap, batch_cap;
  // Two device ints (work-item counter, finished-block counter) that are zero between launches; NULL takes a
  // pair from a pool inside the library.  Launches sharing a pair must be ordered on one stream.
  int* sched = nullptr;
  // Test hooks: a shorter bound (ns) for the kernel's waits (0 = the default of 4 s), and a producer that leaves
  // out one K tile load so that a wait runs into that bound.
  unsigned long long wait_limit_ns = 0;
  int test_skip_load = 0;
};
// Causal GQA attention of a packed ragged batch on tcgen05 / tensor memory.
pd_status launch_prefill_attention_tc(const PrefillAttnArgs& a, int* err_word, cudaStream_t s);

struct DecodeAttnArgs {
  const bf16* q;       // [B, ldq]
  int ldq;
  const bf16* k_cache;
  const bf16* v_cache;
  bf16* o;             // [B, Hq*hd]
  const int32_t* kv_len;  // device [B]; attention covers kv_len[b] + 1 entries
  float* partial;         // workspace [B, Hkv, n_splits, G, hd + 2] fp32 (when n_splits > 1)
  int batch, max_kv_len, n_splits;
  int n_q_heads, n_kv_heads, head_dim, len_cap;
};
int decode_attention_splits(int batch, int n_kv_heads, int max_kv_len);
pd_status launch_decode_attention(const DecodeAttnArgs& a, cudaStream_t s);

// Per-row dynamic FP8 quantisation: scale[r] = max|x[r, :]| / 448 (1 for an all-zero row),
// codes[r, k] = E4M3(x[r, k] / scale[r]), round to nearest even, saturating.  k a multiple of 16.
pd_status launch_quantize_rows_fp8(const bf16* x, int ldx, int rows, int k, uint8_t* codes, int ldq, float* scale,
                                   cudaStream_t s);

// Seeded N(mean, std) fill in bf16 (counter-based; value i depends only on seed, stream, i).
pd_status launch_fill_normal(bf16* dst, size_t n, uint64_t seed, uint64_t stream_id, float mean, float std,
                             cudaStream_t s);

}  // namespace pd

// The opaque layer object.
struct pd_layer {
  pd_layer_cfg cfg;
  int n_qkv;
  pd::bf16 *w_qkv, *w_o, *w_gu, *w_down;  // owned copies; w_gu = [2F, d]: 64 gate rows, 64 up rows, alternating
                                           // (released after quantisation when cfg.fp8_projections is set)
  uint8_t *q_qkv, *q_o, *q_gu, *q_down;    // FP8 mode: E4M3 codes in the same layouts
  float *s_qkv, *s_o, *s_gu, *s_down;      // FP8 mode: one scale per weight row
  pd::bf16 *g_attn, *g_mlp;
  float2* rope_tab;                        // [max_pos, hd/2]
  int* err_word;                           // device int32
  int* split_flags;                        // device int32[kSplitMaxTiles * 4], see GemmArgs
  int* attn_sched;                         // device int32[2], work counters of the prefill-attention kernel
};
