// Decode attention for callers that are not allowed to allocate device memory.
//
// Some hosts of this library run under rules that forbid cudaMalloc once they are up: a
// serving process whose memory pool owns the whole device, code running while a CUDA graph is
// being captured, or a real-time loop that must not take the allocator's locks.  They cannot
// obtain the scratch buffer that pd_decode_attention needs for the partial results of its
// KV-range splits.  This variant keeps that scratch in a fixed array that is part of the
// library image: it exists on every GPU that loads the library, from load to exit, and costs
// PD_NOALLOC_SCRATCH_BYTES of device memory there whether or not the call is ever made.
#include <mutex>

#include "pd_common.cuh"

namespace {

// The scratch itself.  In host code this name is only a handle for the runtime, not a device
// address; the address is looked up once per device below.
static __device__ __align__(256) unsigned char g_noalloc_scratch[PD_NOALLOC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
void* g_scratch_ptr[kMaxDevices] = {};

// Device address of the array on the current device; resolved on the first call per device.
pd_status scratch_for_current_device(void** out) {
  int dev = 0;
  PD_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return PD_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_scratch_ptr[dev]) {
    void* p = nullptr;
    PD_CUDA_TRY(cudaGetSymbolAddress(&p, g_noalloc_scratch));
    if (!p) return PD_ERR_CUDA;
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return PD_OK;
}

}  // namespace

extern "C" pd_status pd_decode_attention_noalloc(const pd_layer_cfg* cfg, const void* q, int32_t ldq, void* out,
                                                 const int32_t* kv_len_dev, int32_t B, int32_t max_kv_len,
                                                 const pd_kv_cache* cache, void* stream) {
  if (!cfg || cfg->struct_size != sizeof(pd_layer_cfg)) return PD_ERR_INVALID_ARG;
  if (cfg->n_q_heads <= 0 || cfg->n_kv_heads <= 0) return PD_ERR_INVALID_ARG;
  if (cfg->head_dim != 64 && cfg->head_dim != 128) return PD_ERR_UNSUPPORTED_SHAPE;
  if (cfg->n_q_heads % cfg->n_kv_heads != 0 || cfg->n_q_heads / cfg->n_kv_heads > 16) return PD_ERR_UNSUPPORTED_SHAPE;
  if (B < 0) return PD_ERR_INVALID_ARG;
  if (B == 0) return PD_OK;
  if (!cache || cache->struct_size != sizeof(pd_kv_cache) || !cache->k || !cache->v || cache->batch_cap <= 0 ||
      cache->len_cap <= 0)
    return PD_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(cache->k) & 15u) || (reinterpret_cast<uintptr_t>(cache->v) & 15u))
    return PD_ERR_INVALID_ARG;
  if (!q || !out || !kv_len_dev || ldq < cfg->n_q_heads * cfg->head_dim || ldq % 8 != 0) return PD_ERR_INVALID_ARG;
  if (B > cache->batch_cap || max_kv_len <= 0 || max_kv_len > cache->len_cap) return PD_ERR_INVALID_ARG;

  pd::DecodeAttnArgs a{};
  a.n_splits = pd::decode_attention_splits(B, cfg->n_kv_heads, max_kv_len);
  const size_t need = static_cast<size_t>(B) * cfg->n_q_heads * a.n_splits * (cfg->head_dim + 2) * sizeof(float);
  // The problem does not fit the built-in scratch: refuse rather than overrun it.
  if (a.n_splits > 1 && need > static_cast<size_t>(PD_NOALLOC_SCRATCH_BYTES)) return PD_ERR_WORKSPACE_TOO_SMALL;
  void* scratch = nullptr;
  PD_TRY(scratch_for_current_device(&scratch));

  a.q = static_cast<const pd::bf16*>(q); a.ldq = ldq;
  a.k_cache = static_cast<const pd::bf16*>(cache->k); a.v_cache = static_cast<const pd::bf16*>(cache->v);
  a.o = static_cast<pd::bf16*>(out); a.kv_len = kv_len_dev;
  // Nothing in the scratch has to start at zero: every slot the merge step reads is written by
  // this same call first, so the previous call's leftovers are never observed.
  a.partial = static_cast<float*>(scratch);
  a.batch = B; a.max_kv_len = max_kv_len;
  a.n_q_heads = cfg->n_q_heads; a.n_kv_heads = cfg->n_kv_heads; a.head_dim = cfg->head_dim; a.len_cap = cache->len_cap;
  return pd::launch_decode_attention(a, static_cast<cudaStream_t>(stream));
}
