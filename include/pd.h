/*
 * pd.h - C ABI of the B200 (sm_100a) prefill/decode benchmarking library.
 *
 * The library measures one dense decoder layer in the two modes the allocation
 * method needs as inputs (paper, Method: "Acquire prefill throughput under TTFT
 * constraints" wants the maximum prefill throughput of a saturated instance;
 * "Acquire decode throughput under TPOT constraints" wants the TPOT-versus-batch
 * curve), and evaluates the allocation model itself (Eq. 1-13).
 *
 * Conventions
 *   - Every function returns a pd_status; nothing throws or aborts.
 *   - "device" pointers are CUDA global memory of the current device; "host"
 *     pointers are ordinary process memory.  The library never takes ownership of
 *     a caller's pointer; the only library-owned objects are pd_layer handles.
 *   - bf16 tensors are raw 16-bit patterns, row-major, innermost index contiguous.
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).  Layer calls
 *     only enqueue work: they neither allocate nor synchronise.
 *   - Structs start with `struct_size = sizeof(struct)` so that fields can be appended.
 */
#ifndef PD_H_
#define PD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  PD_OK = 0,
  PD_ERR_INVALID_ARG = -1,
  PD_ERR_UNSUPPORTED_SHAPE = -2,
  PD_ERR_WORKSPACE_TOO_SMALL = -3,
  PD_ERR_CUDA = -4,
  PD_ERR_DEVICE_TIMEOUT = -5,
  PD_ERR_INFEASIBLE_TTFT = -6,
  PD_ERR_INFEASIBLE_TPOT = -7,
  PD_ERR_ARCH = -8
} pd_status;

/* Static string for a status code. */
const char* pd_status_str(pd_status s);
/* cudaError_t (as int) recorded by the calling thread's last PD_ERR_CUDA. */
int pd_last_cuda_error(void);
/* Library version, for the binding's sanity check. */
int pd_version(void);

/* ------------------------------------------------------------------ layer */

/* Shape of one decoder layer.  Supported: head_dim 64 or 128, n_q_heads a multiple
 * of n_kv_heads with group size <= 16, d_model and d_ff multiples of 64,
 * max_pos = largest token position + 1 ever used (RoPE table length).
 * fp8_projections = 1 runs the five projections in FP8 (see pd_gemm_fp8 for the reading of the paper's
 * FP8 checkpoint): pd_layer_create quantises every weight matrix per output channel to E4M3 and keeps
 * only the codes and scales; each pass quantises the projection inputs per token.  Attention, norms,
 * residual stream and KV cache stay bf16.  Needs d_model, d_ff and n_q_heads * head_dim multiples of 128. */
typedef struct {
  uint32_t struct_size;
  int32_t d_model, n_q_heads, n_kv_heads, head_dim, d_ff;
  float rms_eps, rope_theta;
  int32_t max_pos;
  int32_t fp8_projections;
} pd_layer_cfg;

/* Caller's weights: device pointers, bf16, row-major [out_features, in_features]. */
typedef struct {
  uint32_t struct_size;
  const void* w_qkv;  /* [(Hq+2Hkv)*hd, d]: q heads, then k heads, then v heads */
  const void* w_o;    /* [d, Hq*hd] */
  const void* w_gate; /* [F, d] */
  const void* w_up;   /* [F, d] */
  const void* w_down; /* [d, F] */
  const void* g_attn; /* [d] RMSNorm gain before attention */
  const void* g_mlp;  /* [d] RMSNorm gain before the MLP */
} pd_layer_weights;

typedef struct pd_layer pd_layer; /* opaque; owns repacked weight copies, tensor maps, RoPE table */

/* Copies and repacks the weights on `stream` (cudaMalloc inside).  The caller may free
 * its own weight buffers once `stream` has been synchronised.  PD_ERR_ARCH if the
 * current device is not compute capability 10.x. */
pd_status pd_layer_create(const pd_layer_cfg* cfg, const pd_layer_weights* w, void* stream, pd_layer** out);
pd_status pd_layer_destroy(pd_layer* layer);

/* Bytes of scratch the layer calls need for at most `max_tokens` prefill tokens per
 * call, `max_batch` decode sequences and KV length `max_kv_len`. */
pd_status pd_workspace_bytes(const pd_layer_cfg* cfg, int32_t max_tokens, int32_t max_batch,
                             int32_t max_kv_len, size_t* out_bytes);

/* Caller-owned KV cache: K and V device bf16 [batch_cap, Hkv, len_cap, hd], one
 * contiguous run per (sequence, kv head). */
typedef struct {
  uint32_t struct_size;
  void* k;
  void* v;
  int32_t batch_cap, len_cap;
} pd_kv_cache;

/* Prefill mode (paper: the compute-bound phase whose saturated throughput is the
 * "maximum prefill throughput").  One layer over a packed ragged batch:
 *   x, out        device bf16 [T, d]; out may alias x
 *   cu_seqlens    n_req+1 int32, cu[0] = 0, cu[n_req] = T; request r owns rows cu[r]..cu[r+1]-1
 *                 at positions 0..len_r-1 and attends causally within itself.  Given twice:
 *                 `_dev` (device copy read by the kernels) and `_host` (validated, sizes grids).
 *   slots_dev     device int32[n_req] (NULL: slot r = r): K/V of request r are written to
 *                 cache sequence slots[r], positions 0..len_r-1.  A slot outside the cache is
 *                 skipped by the kernels and reported by pd_layer_check.
 * Errors: INVALID_ARG (NULL, non-monotone cu, length beyond the cache or the RoPE table; T = 0
 * is accepted and does nothing), WORKSPACE_TOO_SMALL, CUDA (launch failure). */
pd_status pd_prefill_layer(pd_layer* layer, const void* x, void* out, const int32_t* cu_seqlens_dev,
                           const int32_t* cu_seqlens_host, int32_t n_req, const int32_t* slots_dev,
                           const pd_kv_cache* cache, void* workspace, size_t workspace_bytes, void* stream);

/* Chunked prefill (paper, "Acquire prefill throughput ...": the maximum prefill throughput depends on
 * the chunked-prefill size, and the M/M/1 model holds when a request is at least one chunk long).
 * Same as pd_prefill_layer, but request r already has prefix[r] tokens in its cache sequence: its
 * rows take positions prefix[r], prefix[r]+1, ..., their K/V are appended there, and each row attends
 * to every cached position up to its own.  `prefix` is given twice like cu_seqlens (device copy read
 * by the kernels, host copy validated: prefix[r] + len_r must fit the cache and the RoPE table).
 * prefix = 0 reproduces pd_prefill_layer; one-token chunks reproduce pd_decode_layer. */
pd_status pd_prefill_chunk_layer(pd_layer* layer, const void* x, void* out, const int32_t* cu_seqlens_dev,
                                 const int32_t* cu_seqlens_host, int32_t n_req, const int32_t* prefix_dev,
                                 const int32_t* prefix_host, const int32_t* slots_dev, const pd_kv_cache* cache,
                                 void* workspace, size_t workspace_bytes, void* stream);

/* Decode mode (paper: the memory-bandwidth-bound phase measured as TPOT versus batch).
 *   x, out        device bf16 [B, d]; out may alias x
 *   kv_len_dev    device int32[B]: tokens already cached for sequence b (= position of the new
 *                 token).  The new K/V are appended at index kv_len[b]; attention covers
 *                 kv_len[b]+1 entries.  kv_len itself is not modified.
 *   max_kv_len    host upper bound of kv_len[b]+1 (sizes the split of the KV range); must be
 *                 <= cache->len_cap.  Sequence b uses cache slot b.
 * B = 0 is accepted and does nothing. */
pd_status pd_decode_layer(pd_layer* layer, const void* x, void* out, const int32_t* kv_len_dev, int32_t B,
                          int32_t max_kv_len, const pd_kv_cache* cache, void* workspace,
                          size_t workspace_bytes, void* stream);

/* The decode-attention kernel on its own (the HBM-bound part of decode mode; paper: decode is
 * memory-bandwidth-bound), for roofline measurement and unit tests.
 *   q, out        device bf16 [B, Hq*hd]; q has row pitch ldq elements (a multiple of 8)
 *   kv_len_dev    device int32[B]; sequence b attends over entries 0..kv_len[b] of cache slot b
 *                 (kv_len[b]+1 entries, all of which must already be in the cache)
 *   workspace     scratch for the partial results of the KV-range splits, at least
 *                 pd_decode_attention_workspace_bytes(cfg, B, max_kv_len) bytes, 256-byte aligned
 * Only n_q_heads, n_kv_heads and head_dim of cfg are used.  kv_len is read on the device and not validated by
 * this call: a range that reaches past the cache (kv_len[b] + 1 > len_cap) is clamped to len_cap entries, and a
 * sequence with kv_len[b] < 0 (no entry at all) gets an all-zero output row; neither is reported.  (The layer
 * calls do report an out-of-range position, through pd_layer_check.) */
pd_status pd_decode_attention_workspace_bytes(const pd_layer_cfg* cfg, int32_t B, int32_t max_kv_len,
                                              size_t* out_bytes);
pd_status pd_decode_attention(const pd_layer_cfg* cfg, const void* q, int32_t ldq, void* out,
                              const int32_t* kv_len_dev, int32_t B, int32_t max_kv_len, const pd_kv_cache* cache,
                              void* workspace, size_t workspace_bytes, void* stream);

/* The prefill-attention kernel on its own (causal grouped-query attention of the compute-bound prefill
 * mode; paper, "Acquire prefill throughput under TTFT constraints" benchmarks the pass this kernel is the
 * attention step of), for roofline measurement and unit tests.
 *   q, out        device bf16 [T, ldq] / [T, Hq*hd]: row t of request r is query cu[r] + t at position
 *                 prefix[r] + t; head h occupies columns h*hd .. of a row; ldq a multiple of 8, q 16-byte aligned
 *   cu_seqlens    as for pd_prefill_layer (device copy and host copy)
 *   prefix        tokens of each request already cached before its rows (device and host copy, both or
 *                 neither; NULL = 0)
 *   cache         must already hold K (after RoPE) and V of positions 0 .. prefix[r] + len_r - 1 of
 *                 request r in sequence slots[r] (NULL: r)
 *   err_word      optional device int32, set to 1 if a bounded wait inside the kernel gave up
 * Query t attends to positions 0 .. prefix[r] + t of its own request.  Only n_q_heads, n_kv_heads and
 * head_dim of cfg are used; out must be 32-byte aligned.  Enqueues one kernel; no workspace.  The kernel
 * keeps its work counter in a small pool inside the library: calls that follow each other on one stream
 * are always safe, and up to 64 calls may overlap on the GPU. */
pd_status pd_prefill_attention(const pd_layer_cfg* cfg, const void* q, int32_t ldq, void* out,
                               const int32_t* cu_seqlens_dev, const int32_t* cu_seqlens_host, int32_t n_req,
                               const int32_t* prefix_dev, const int32_t* prefix_host, const int32_t* slots_dev,
                               const pd_kv_cache* cache, int32_t* err_word, void* stream);

/* pd_decode_attention for callers that may not allocate device memory.  (The paper has no
 * counterpart of this call; it exists for the library's users.)
 *
 * Who needs it: a process whose own memory pool already owns the device, code that runs while
 * a stream is being captured, or a latency-critical loop that must stay out of the CUDA
 * allocator.  Such a caller cannot cudaMalloc the scratch that pd_decode_attention wants for
 * the partial results of its KV-range splits.  Here that scratch is a fixed array of
 * PD_NOALLOC_SCRATCH_BYTES inside the library image: every GPU that loads the library holds
 * it from load until the process exits, used or not.  The call itself performs no cudaMalloc,
 * cudaFree or other allocating routine.
 *
 * Arguments and results are those of pd_decode_attention without the workspace pair.
 * Limits and rules:
 *   - B * n_q_heads * splits * (head_dim + 2) * 4 bytes must fit the array.  splits is chosen
 *     from B, n_kv_heads and max_kv_len as in pd_decode_attention: small batches are split until
 *     about 110 blocks exist, and any batch is split so that a block covers at most about 2048
 *     keys; a problem that needs no split always fits.  With 32 query heads and head_dim 128
 *     the array holds B * splits up to 504, e.g. B = 256 at up to 3071 keys or B = 126 at up to
 *     9215.  Otherwise the call returns
 *     PD_ERR_WORKSPACE_TOO_SMALL and launches nothing.
 *   - The first call on each device looks up the array's device address (that device must be
 *     current); make this first call before any stream capture begins.
 *   - All calls on a device share the one array.  It still holds the previous call's partials
 *     when a call starts; nothing has to be cleared because each call overwrites every entry
 *     it later reads.  Two calls whose kernels can overlap on the GPU (different streams,
 *     different host threads) race on it: serialise them on one stream. */
#define PD_NOALLOC_SCRATCH_BYTES (8u << 20)
pd_status pd_decode_attention_noalloc(const pd_layer_cfg* cfg, const void* q, int32_t ldq, void* out,
                                      const int32_t* kv_len_dev, int32_t B, int32_t max_kv_len,
                                      const pd_kv_cache* cache, void* stream);

/* The same two modes over a stack of n_layers layers run back to back (layer i+1 reads layer
 * i's output), layer i using caches[i % n_caches].  With io_on_host = 0, x/out/cu_seqlens_dev/
 * kv_len are device pointers and the call only enqueues work.  With io_on_host = 1 they are
 * host pointers (pinned memory advised): the call copies the inputs to the device on `stream`,
 * runs the stack, copies `out` back and synchronises `stream` before returning; for prefill
 * `cu_seqlens_dev` is then ignored (the host copy is uploaded).  The workspace must come from
 * pd_workspace_bytes (it includes room for the staged activations).
 * Every layer of a stack must have the shape of layers[0] (d_model, head counts, head_dim, d_ff and the
 * fp8_projections switch: the workspace and the inter-layer buffers are laid out once, for that shape);
 * rms_eps, rope_theta and max_pos may differ.  A stack with a layer of another shape is refused with
 * PD_ERR_INVALID_ARG before anything is enqueued.
 * In decode mode, between two layers of the same shape, the first RMSNorm of the second layer is
 * computed by the last kernel of the first; the result equals that of chained pd_decode_layer calls
 * up to the summation order of that norm's sum of squares (at most one bf16 unit in the last place
 * of a normalised value). */
pd_status pd_prefill_stack(pd_layer* const* layers, const pd_kv_cache* caches, int32_t n_layers, int32_t n_caches,
                           const void* x, void* out, int32_t io_on_host, const int32_t* cu_seqlens_dev,
                           const int32_t* cu_seqlens_host, int32_t n_req, void* workspace,
                           size_t workspace_bytes, void* stream);
pd_status pd_decode_stack(pd_layer* const* layers, const pd_kv_cache* caches, int32_t n_layers, int32_t n_caches,
                          const void* x, void* out, int32_t io_on_host, const int32_t* kv_len, int32_t B,
                          int32_t max_kv_len, void* workspace, size_t workspace_bytes, void* stream);
/* pd_prefill_chunk_layer over a stack: one chunk of every request through all layers (the unit a
 * chunked-prefill engine schedules; paper, "Acquire prefill throughput under TTFT constraints": the maximum
 * prefill throughput is a function of the chunked-prefill size).  Device pointers only; request r uses cache
 * sequence r of caches[i % n_caches] in layer i; same shape rule as the other stack calls. */
pd_status pd_prefill_chunk_stack(pd_layer* const* layers, const pd_kv_cache* caches, int32_t n_layers,
                                 int32_t n_caches, const void* x, void* out, const int32_t* cu_seqlens_dev,
                                 const int32_t* cu_seqlens_host, int32_t n_req, const int32_t* prefix_dev,
                                 const int32_t* prefix_host, void* workspace, size_t workspace_bytes, void* stream);

/* Reads and clears the device-side error word of the layer (set when a bounded wait inside
 * a kernel gave up).  Synchronises `stream`.  PD_OK or PD_ERR_DEVICE_TIMEOUT. */
pd_status pd_layer_check(pd_layer* layer, void* stream);

/* ------------------------------------------------------------ whole model */

/* A whole-model step: token embedding, the layer stack, final RMSNorm, LM-head projection,
 * greedy sampling.  The paper's TTFT runs to the first output token and its TPOT from one
 * output token to the next ("Acquire prefill throughput under TTFT constraints", "Acquire
 * decode throughput under TPOT constraints"), so a measured step ends with a token id; the
 * paper does not define the network around the layers, this is the standard one:
 *   x = E[token];  h = layers(x);  n = RMSNorm(h_last) * g_final;  logits = n W_lm^T (fp32);
 *   next = argmax logits, the lowest index among equal maxima.
 * Prefill takes the last row of every request, decode every row. */
typedef struct pd_model pd_model;

/* Device pointers, bf16, row-major; copied at creation.  vocab must be a multiple of 4. */
typedef struct {
  uint32_t struct_size;
  int32_t vocab;
  const void* embed;   /* [vocab, d_model] */
  const void* g_final; /* [d_model] */
  const void* lm_head; /* [vocab, d_model] */
} pd_model_weights;

/* The layers (all of one shape) are borrowed: they must outlive the model.  The copies are
 * enqueued on `stream`. */
pd_status pd_model_create(pd_layer* const* layers, int32_t n_layers, const pd_model_weights* w, void* stream,
                          pd_model** out);
pd_status pd_model_destroy(pd_model* model);

/* Workspace for prefill passes of up to max_tokens tokens in max_requests requests and decode
 * steps of up to max_batch sequences over max_kv_len cached tokens (includes fp32 logits for
 * the case that the caller passes no logits buffer). */
pd_status pd_model_workspace_bytes(const pd_model* model, int32_t max_tokens, int32_t max_requests,
                                   int32_t max_batch, int32_t max_kv_len, size_t* out_bytes);

/* Prefill of a packed ragged batch of prompts up to the first output token.
 *   tokens_dev  device int32[T] token ids (T = cu_seqlens[n_req]); an id outside [0, vocab)
 *               gives a zero embedding row and makes pd_model_check return PD_ERR_INVALID_ARG
 *   cu_seqlens  as for pd_prefill_layer; request r is written to cache sequence r of
 *               caches[i % n_caches] for layer i
 *   next_dev    device int32[n_req]: the greedy token after each prompt, -1 for an empty one
 *   logits_dev  optional device fp32[n_req, vocab] (16-byte aligned); NULL keeps the logits
 *               in the workspace
 * Only enqueues work on `stream`; allocates nothing. */
pd_status pd_model_prefill(pd_model* model, const int32_t* tokens_dev, const int32_t* cu_seqlens_dev,
                           const int32_t* cu_seqlens_host, int32_t n_req, const pd_kv_cache* caches,
                           int32_t n_caches, int32_t* next_dev, float* logits_dev, void* workspace,
                           size_t workspace_bytes, void* stream);

/* One decode step: tokens_dev[b] is the newest token of sequence b whose kv_len_dev[b] earlier
 * tokens are cached; its K/V are appended in every layer and next_dev[b] receives the greedy
 * next token.  Captured in a CUDA graph this is the whole-model decode step. */
pd_status pd_model_decode_step(pd_model* model, const int32_t* tokens_dev, const int32_t* kv_len_dev, int32_t B,
                               int32_t max_kv_len, const pd_kv_cache* caches, int32_t n_caches, int32_t* next_dev,
                               float* logits_dev, void* workspace, size_t workspace_bytes, void* stream);

/* pd_layer_check over every layer plus the model's own error word (bad token id).
 * Synchronises `stream`. */
pd_status pd_model_check(pd_model* model, void* stream);

/* Plain C[M,N] = A[M,K] * B[N,K]^T in bf16 with fp32 accumulation on the tensor cores
 * (the contraction every projection of the layer uses), exposed for unit tests and
 * roofline measurement.  A, B, C device bf16 row-major; K a multiple of 64, N of 16.
 * `err_word` device int32 (may be NULL), set non-zero if a bounded wait gave up. */
pd_status pd_gemm_bf16(const void* a, const void* b, void* c, int32_t m, int32_t n, int32_t k,
                       int32_t* err_word, void* stream);

/* pd_gemm_bf16 with the scratch the layer calls give their projections: with it the kernel may cut tiles in two
 * along K and run the halves on different SMs (every tile when the problem has too few tiles to fill the SMs,
 * e.g. a few hundred tokens against N = d_model; otherwise only the tiles of the last, partly filled wave when K
 * is long).  The first half parks its fp32 partial tile in the workspace, the second adds it before the
 * epilogue; the wait between them is bounded like every other wait.  workspace: device, 256-byte aligned, at
 * least pd_gemm_workspace_bytes() bytes; the call clears the flags at its start, so calls sharing a workspace
 * must be ordered on one stream. */
pd_status pd_gemm_workspace_bytes(size_t* out_bytes);
pd_status pd_gemm_bf16_ws(const void* a, const void* b, void* c, int32_t m, int32_t n, int32_t k, void* workspace,
                          size_t workspace_bytes, int32_t* err_word, void* stream);

/* Where a layer pass leaves its intermediates.  Byte offsets, inside the workspace handed to
 * pd_prefill_layer / pd_prefill_chunk_layer over `tokens` rows (or pd_decode_layer with B = tokens), of the
 * bf16 tensors that are still there when the pass has finished: norm = RMSNorm output that fed the MLP
 * [tokens, d]; qkv = [tokens, Nqkv] of which the q columns (after RoPE) are written; attn_o = attention output
 * [tokens, Hq*hd]; resid = residual stream after the attention half [tokens, d]; act = SwiGLU output
 * [tokens, F].  For inspection and stage-by-stage parity checks (the layer is the unit the paper's benchmarks
 * time; the stages are this library's).  Host only. */
typedef struct {
  uint32_t struct_size;
  uint64_t norm, qkv, attn_o, resid, act;
} pd_workspace_layout;
pd_status pd_workspace_offsets(const pd_layer_cfg* cfg, int32_t tokens, pd_workspace_layout* out);

/* FP8 projections.  The paper's TTFT validation (Figure 1 experiment) runs an FP8 checkpoint but gives
 * neither the number format nor the scaling; the reading built here is OCP E4M3 codes with one fp32 scale
 * per row: a weight matrix is quantised per output channel, an activation matrix per token.
 *
 * pd_quantize_fp8_rows: x device bf16 [rows, k] with row pitch ldx elements -> codes device uint8
 * [rows, k] (contiguous), scales device fp32 [rows].  scale = max|row| / 448 (1 for an all-zero row),
 * code = E4M3(x / scale), both in fp32, round to nearest even, saturating.  k a multiple of 16.
 *
 * pd_gemm_fp8: C[M,N] (device bf16) = (dec(A)[M,K] * dec(B)[N,K]^T) * a_scales[m] * b_scales[n] with fp32
 * accumulation on the tensor cores (tcgen05 kind::f8f6f4).  Codes contiguous row-major, 16-byte aligned;
 * K a multiple of 128, N of 16.  `err_word` as in pd_gemm_bf16.  Both calls only enqueue work. */
pd_status pd_quantize_fp8_rows(const void* x, int32_t ldx, int32_t rows, int32_t k, void* codes, float* scales,
                               void* stream);
pd_status pd_gemm_fp8(const void* a_codes, const float* a_scales, const void* b_codes, const float* b_scales,
                      void* c, int32_t m, int32_t n, int32_t k, int32_t* err_word, void* stream);

/* FP8 (E4M3) with block-wise scales, the scaling scheme of checkpoints that state `weight_block_size = [128, 128]`
 * (reading of the paper's FP8 deployment, Evaluation section: the TTFT experiment on an FP8 checkpoint; the paper does
 * not say how that checkpoint is scaled):
 *   a weight matrix W[n, k] carries one fp32 scale per 128 x 128 block, an activation matrix X[rows, k] one per row and
 *   group of 128 consecutive k; scale = max|block| / 448 (1 for an all-zero block), code = E4M3(value / scale), both in
 *   fp32, round to nearest even, saturating;
 *   C[i, j] = sum over K blocks kb of ( sum_{k in kb} dec(A[i, k]) dec(B[j, k]) ) * a_scales[i, kb] * b_scales[j / 128, kb],
 *   the inner sums exact in fp32 on the tensor cores (tcgen05 kind::f8f6f4), the scaled partial sums added in fp32.
 *
 * pd_quantize_fp8_groups: x device bf16 [rows, k], row pitch ldx elements (a multiple of 8) -> codes device uint8
 * [rows, k] contiguous, scales device fp32 [rows, k / 128] contiguous.  k a multiple of 128.
 * pd_quantize_fp8_blocks: w device bf16 [n, k], row pitch ldw elements (a multiple of 8) -> codes device uint8 [n, k]
 * contiguous, scales device fp32 [ceil(n / 128), k / 128] contiguous (the last row of blocks may have fewer than 128
 * rows).  k a multiple of 128.
 * pd_gemm_fp8_blockwise: C[m, n] device bf16 contiguous from codes and scales laid out as above; code pointers 16-byte
 * aligned, k a multiple of 128, n of 16.  `err_word` as in pd_gemm_bf16.  The caller owns every buffer; the three calls
 * only enqueue work on `stream`; a shape outside these rules returns PD_ERR_UNSUPPORTED_SHAPE, a NULL pointer or a
 * negative size PD_ERR_INVALID_ARG, and zero rows return PD_OK without a launch. */
pd_status pd_quantize_fp8_groups(const void* x, int32_t ldx, int32_t rows, int32_t k, void* codes, float* scales,
                                 void* stream);
pd_status pd_quantize_fp8_blocks(const void* w, int32_t ldw, int32_t n, int32_t k, void* codes, float* scales,
                                 void* stream);
pd_status pd_gemm_fp8_blockwise(const void* a_codes, const float* a_scales, const void* b_codes, const float* b_scales,
                                void* c, int32_t m, int32_t n, int32_t k, int32_t* err_word, void* stream);

/* Failure-detection test hook.  Every wait inside the tensor-core kernels (on a tile load, an accumulator, a
 * partner block) is bounded by wall clock (4 s); when a wait gives up, the block raises its abort flag, leaves
 * through the normal teardown (tensor memory freed, cluster barrier of a CTA pair passed) and sets the error
 * word that pd_layer_check / the err_word arguments report as PD_ERR_DEVICE_TIMEOUT.  This call arms ONE such
 * event for the calling thread: the next launch of the named kernel kind runs with the bound wait_limit_ns
 * (between 0.1 ms and 4 s) and its producer leaves out one operand tile load, so that a wait runs into the
 * bound.  Nothing faults or spins without a limit; the output of that launch is undefined, later launches are
 * unaffected.  PD_INJECT_NONE disarms.  (The paper has no counterpart; it exists so that the timeout path can
 * be exercised without a real fault.) */
enum { PD_INJECT_NONE = 0, PD_INJECT_ATTN_PREFILL = 1, PD_INJECT_GEMM = 2, PD_INJECT_GEMM_PAIR = 3,
       PD_INJECT_GEMM_FP8_BLOCKWISE = 4 };
pd_status pd_test_inject_wait_timeout(int32_t kernel_kind, uint64_t wait_limit_ns);

/* Kernels launched so far by the calling thread through this library. */
int64_t pd_launch_count(void);

/* Optional per-kernel-class timing for roofline reports.  Between pd_trace_begin and
 * pd_trace_end every kernel the calling thread launches through the layer calls is bracketed
 * by a pair of CUDA events on its stream; pd_trace_end waits for them and sums the elapsed
 * time and the launch count per class.  Tracing adds two event records per kernel, so a
 * traced pass is for attribution, not for the headline time. */
#define PD_TRACE_CLASSES 16
enum {
  PD_K_GEMM_QKV = 0, PD_K_GEMM_O = 1, PD_K_GEMM_GATE_UP = 2, PD_K_GEMM_DOWN = 3, PD_K_ATTN_PREFILL = 4,
  PD_K_ATTN_DECODE = 5, PD_K_RMSNORM = 6, PD_K_EMBED = 7, PD_K_LM_HEAD = 8, PD_K_SAMPLE = 9
};
typedef struct {
  uint32_t struct_size;
  double time_s[PD_TRACE_CLASSES];
  int64_t launches[PD_TRACE_CLASSES];
} pd_trace_report;
pd_status pd_trace_begin(void);
pd_status pd_trace_end(pd_trace_report* out);

/* ---------------------------------------------------------------- measure */

/* One measurement job on the current device with synthetic seeded data.
 * Prefill (paper, "Acquire prefill throughput ..."): one batch of n_req requests with host
 * lengths l_in[] is pushed through n_layers_run distinct layers back to back, `reps` times;
 * the maximum prefill throughput is tokens / median time, scaled to n_layers_model layers.
 * Decode (paper, "Acquire decode throughput ..."): for every batch size, steps t = 0,
 * step_stride, ... < n_steps (and the last step) run the stack at kv_len = kv_len_start + t;
 * TPOT(B) is the mean step time scaled to n_layers_model layers.
 * Either part is skipped when its count (n_req / n_batch_sizes) is 0.
 * chunk_tokens > 0 measures the prefill pass as chunked prefill: step s pushes rows s*chunk .. (s+1)*chunk-1
 * of every request that still has rows through all layers (pd_prefill_chunk_stack), each chunk attending to
 * its cached prefix; the reported time is that of the whole batch, all chunks.
 * l_in_grid / n_grid (at most PD_MEASURE_GRID_MAX lengths): in addition every grid length is measured as one
 * request on its own (same layers, same chunk size) and reported in grid_l / grid_time_s: the service-time
 * curve t(L) that pd_interp_service_times, pd_mixture_throughput and pd_queue_replay take.
 * Every layer of a timed stack has its own weights.  KV buffers: one per layer when memory allows, otherwise a
 * ring of fewer buffers that the layers cycle through; the ring sizes are reported (prefill_kv_ring,
 * decode_kv_ring).  Where the K/V bytes one attention-only timing pass touches are below twice the L2 size
 * (small batches), attn_l2_resident is 1 and attn_frac_hbm_peak is left 0: the kernel time is then not an HBM
 * figure.
 * With vocab > 0 the step is the whole-model step: the time of the token embedding, the final
 * RMSNorm, the LM head over a vocabulary of that size and the greedy sampling (once per step,
 * not per layer; timed on their own, median of `reps`) is added to prefill_time_s and TPOT(B)
 * and reported in prefill_head_s / decode_head_s. */
typedef struct {
  uint32_t struct_size;
  int32_t n_layers_run, n_layers_model;
  int32_t warmup, reps;
  uint64_t seed;
  const int32_t* l_in; /* host int32[n_req] */
  int32_t n_req;
  const int32_t* batch_sizes; /* host int32[n_batch_sizes], at most 32 */
  int32_t n_batch_sizes;
  int32_t kv_len_start, n_steps, step_stride;
  const int32_t* kv_len_mix; /* optional host int32[max batch]: per-sequence start lengths (ragged); NULL = kv_len_start */
  int32_t vocab;             /* 0: layer stack only; > 0 (a multiple of 4): whole-model step */
  int32_t chunk_tokens;      /* 0: every request in one piece; > 0: chunked prefill with chunks of this many tokens */
  const int32_t* l_in_grid;  /* optional host int32[n_grid]: lengths measured one request at a time */
  int32_t n_grid;
} pd_measure_cfg;
#define PD_MEASURE_GRID_MAX 128

typedef struct {
  uint32_t struct_size;
  double prefill_time_s;   /* median, n_layers_model layers */
  double prefill_tok_s;    /* maximum prefill throughput */
  double prefill_flops;    /* algorithmic flops of that pass (causal half of attention) */
  double prefill_frac_bf16_peak;
  int32_t n_points;
  int32_t batch[32];
  double tpot_s[32];                /* TPOT(B), n_layers_model layers */
  double decode_bytes[32];          /* algorithmic bytes per step */
  double decode_frac_hbm_peak[32];
  double attn_time_s[32];           /* decode-attention kernel alone, per layer, mean over the steps */
  double attn_frac_hbm_peak[32];
  int32_t gpu_launches;             /* kernels launched inside the timed regions */
  double prefill_head_s;            /* embedding + final norm + LM head + sampling of the prefill pass (vocab > 0) */
  double decode_head_s[32];         /* the same for one decode step at batch[i] */
  int32_t prefill_chunks;           /* stack passes per prefill measurement (1 unless chunk_tokens > 0) */
  int32_t prefill_kv_ring;          /* distinct KV buffers the layers of the prefill stack cycle through */
  int32_t decode_kv_ring[32];       /* the same for the decode stack at batch[i] */
  int32_t attn_l2_resident[32];     /* 1: the attention-only pass fits L2, attn_frac_hbm_peak not reported */
  int32_t n_grid;
  int32_t grid_l[PD_MEASURE_GRID_MAX];
  double grid_time_s[PD_MEASURE_GRID_MAX]; /* median time of one request of grid_l[i] tokens, n_layers_model layers */
} pd_measurement;

pd_status pd_measure(const pd_layer_cfg* cfg, const pd_measure_cfg* mcfg, double peak_bf16_flops,
                     double peak_hbm_bytes_s, pd_measurement* out);

/* --------------------------------------------------------------- allocate */

/* Inputs of the allocation model.  Throughputs in tokens/s, times in seconds; l_in and
 * l_out are the mean input and output lengths (Eq. 1); the curve (batch[i], tpot_s[i]) is
 * the measured TPOT per decode batch size. */
typedef struct {
  uint32_t struct_size;
  double tp_total_tok_s, l_in, l_out, ttft_slo_s, tpot_slo_s, t_overhead_s;
  double prefill_max_tok_s;
  int32_t n_points;
  const int32_t* batch;
  const double* tpot_s;
} pd_alloc_in;

typedef struct {
  uint32_t struct_size;
  double tp_prefill_eff; /* Eq. 13 */
  double tp_decode_eff;  /* B* / TPOT(B*) */
  double mu, lambda, rho; /* Eq. 9-11 */
  int32_t feasible_batch; /* B*: largest sweep point whose whole prefix meets the TPOT SLO */
  int32_t sweep_capped;   /* 1 if B* is the largest measured batch */
  double n_prefill_frac, n_decode_frac; /* Eq. 5, 6 */
  double ratio_pd;                       /* Eq. 7 */
  int32_t n_prefill, n_decode;           /* nearest integer (half up), at least 1 */
  int32_t n_prefill_ceil, n_decode_ceil; /* ceiling, at least 1 */
  double achieved_total_tok_s;           /* Eq. 1 with T_total = max(Eq. 2, Eq. 3) at the integer counts */
} pd_alloc_out;

/* Pure host code, usable without a GPU.  PD_ERR_INFEASIBLE_TTFT when TTFT - T_overhead <= 0
 * or Eq. 13 is not positive; PD_ERR_INFEASIBLE_TPOT when no sweep point meets the TPOT SLO.
 * Fields that can still be computed are filled; the others are NaN / 0. */
pd_status pd_allocate(const pd_alloc_in* in, pd_alloc_out* out);

/* pd_allocate with the two extensions the paper names but does not work out ("Acquire prefill
 * throughput under TTFT constraints"):
 *   prefix_hit_frac in [0, 1): prefix caching; the input length is replaced, everywhere in
 *     Eq. 1-13, by the part that misses the cache, l_in * (1 - prefix_hit_frac), so the
 *     throughputs count computed tokens;
 *   dp_groups >= 1: data-parallel prefill; each of the G groups of an instance is its own
 *     M/M/1 queue with 1/G of prefill_max_tok_s, so Eq. 13 reads
 *     TP_prefill = TP_max - G * L_in / (TTFT - T_overhead); mu, lambda and rho in the result
 *     describe one group, everything else one instance.
 * (0, 1) gives pd_allocate's result bit for bit.  PD_ERR_INVALID_ARG outside those ranges. */
pd_status pd_allocate_ext(const pd_alloc_in* in, double prefix_hit_frac, int32_t dp_groups, pd_alloc_out* out);

/* FIFO single-server replay of n requests (host): request i arrives gaps[i] after request
 * i-1 and needs service[i] seconds.  Outputs the mean sojourn time (what Eq. 12 predicts as
 * 1/(mu - lambda)) and the mean waiting time. */
pd_status pd_queue_replay(const double* gaps, const double* service, int64_t n, double* mean_sojourn_s,
                          double* mean_wait_s);

/* ------------------------------------------------- workload statistics (host) */

/* Maximum prefill throughput of a mix of request lengths (paper, Preliminaries: L_in and L_out are
 * averages; "Acquire prefill throughput under TTFT constraints": the maximum throughput is that of a
 * continuously busy instance).  Request i has l_in[i] > 0 tokens and takes service_s[i] > 0 seconds when
 * served alone; the mix sustains tp_max = sum(l_in) / sum(service_s) tokens/s, and mean_l_in = sum(l_in) / n
 * is the L_in of Eq. 5-13 (so Eq. 9's mu = tp_max / mean_l_in is requests per busy second).  Sums run
 * left to right in double. */
pd_status pd_mixture_throughput(const int32_t* l_in, const double* service_s, int64_t n, double* tp_max_tok_s,
                                double* mean_l_in);

/* Service time of each request length by linear interpolation between measured prefill times
 * (grid_l strictly increasing; lengths outside the grid take the end values):
 * t = t_lo + (t_hi - t_lo) * ((l - l_lo) / (l_hi - l_lo)), where l is the request length rounded up to a multiple
 * of `quantum` >= 1: the prefill kernels work in tiles (256 rows per attention item and per GEMM tile pair), so the
 * time is a step function of the length and a grid of tile multiples with quantum = the tile size has no
 * interpolation error.  Feeds pd_mixture_throughput, pd_mg1_sojourn and pd_queue_replay when a length distribution
 * is served from a grid of measured lengths. */
pd_status pd_interp_service_times(const int32_t* grid_l, const double* grid_time_s, int32_t n_grid,
                                  const int32_t* l_in, int64_t n, int32_t quantum, double* service_s);

/* Eq. 12: mean sojourn time 1 / (mu - lambda) of the M/M/1 prefill queue.  PD_ERR_INFEASIBLE_TTFT when
 * lambda >= mu (no steady state). */
pd_status pd_mm1_sojourn(double mu, double lambda, double* sojourn_s);

/* Mean sojourn time of the same queue when the service times follow the given sample instead of the
 * exponential law Eq. 12 assumes (Pollaczek-Khinchine: E[S] + lambda E[S^2] / (2 (1 - lambda E[S]))); what
 * the replayed queue is compared with for fixed or log-normal request lengths.  PD_ERR_INFEASIBLE_TTFT when
 * lambda E[S] >= 1. */
pd_status pd_mg1_sojourn(const double* service_s, int64_t n, double lambda, double* sojourn_s);

/* One step of the integer refinement of the TPOT-feasible batch (paper, "Acquire decode throughput under
 * TPOT constraints": determine the batch size that satisfies the target TPOT).  Given every (batch, TPOT)
 * point measured so far, lo = the largest point whose whole prefix (in order of batch size) meets the SLO,
 * hi = the first point that does not; *next_batch = lo + (hi - lo) / 2 is where to measure next, or 0 when
 * nothing is left to measure (no feasible point, no infeasible point, or hi = lo + 1).  The caller measures,
 * appends the point and calls again; pd_allocate on the final point set then returns B* = lo. */
pd_status pd_refine_next_batch(const int32_t* batch, const double* tpot_s, int32_t n_points, double tpot_slo_s,
                               int32_t* next_batch);

#ifdef __cplusplus
}
#endif
#endif /* PD_H_ */
