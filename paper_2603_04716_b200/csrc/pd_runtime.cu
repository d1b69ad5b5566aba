// Process-level plumbing of the library: last CUDA error, launch counter and the
// optional per-kernel-class CUDA-event trace used for roofline reporting.
#include <cstdlib>
#include <vector>

#include "pd_common.cuh"

namespace pd {

thread_local int g_last_cuda_error = 0;
thread_local long long g_launch_count = 0;

bool pdl_enabled() {
  static const bool on = [] {
    const char* v = std::getenv("PD_DISABLE_PDL");
    return !(v && v[0] == '1');
  }();
  return on;
}

namespace {
thread_local int t_inject_kind = 0;
thread_local unsigned long long t_inject_limit_ns = 0;
}  // namespace

bool take_wait_injection(int kind, unsigned long long* limit_ns) {
  if (t_inject_kind != kind) return false;
  t_inject_kind = 0;
  *limit_ns = t_inject_limit_ns;
  return true;
}

pd_status cuda_fail(cudaError_t e) {
  g_last_cuda_error = static_cast<int>(e);
  return PD_ERR_CUDA;
}

namespace {
struct TraceRec {
  int cls;
  cudaEvent_t a, b;
};
thread_local bool t_tracing = false;
thread_local std::vector<TraceRec> t_recs;
thread_local std::vector<cudaEvent_t> t_pool;

cudaEvent_t take_event() {
  if (!t_pool.empty()) {
    cudaEvent_t e = t_pool.back();
    t_pool.pop_back();
    return e;
  }
  cudaEvent_t e = nullptr;
  if (cudaEventCreate(&e) != cudaSuccess) return nullptr;
  return e;
}
}  // namespace

TraceScope::TraceScope(int cls, cudaStream_t s) : stream_(s), idx_(-1) {
  if (!t_tracing) return;
  TraceRec r{cls, take_event(), take_event()};
  if (!r.a || !r.b) return;
  cudaEventRecord(r.a, s);
  idx_ = static_cast<int>(t_recs.size());
  t_recs.push_back(r);
}

TraceScope::~TraceScope() {
  if (idx_ >= 0) cudaEventRecord(t_recs[idx_].b, stream_);
}

}  // namespace pd

extern "C" pd_status pd_test_inject_wait_timeout(int32_t kernel_kind, uint64_t wait_limit_ns) {
  if (kernel_kind < PD_INJECT_NONE || kernel_kind > PD_INJECT_GEMM_FP8_BLOCKWISE) return PD_ERR_INVALID_ARG;
  if (kernel_kind != PD_INJECT_NONE && (wait_limit_ns < 100000ull || wait_limit_ns > 4000000000ull)) return PD_ERR_INVALID_ARG;
  pd::t_inject_kind = kernel_kind;
  pd::t_inject_limit_ns = wait_limit_ns;
  return PD_OK;
}

extern "C" int pd_last_cuda_error(void) { return pd::g_last_cuda_error; }
extern "C" int64_t pd_launch_count(void) { return pd::g_launch_count; }

extern "C" pd_status pd_trace_begin(void) {
  for (auto& r : pd::t_recs) {
    pd::t_pool.push_back(r.a);
    pd::t_pool.push_back(r.b);
  }
  pd::t_recs.clear();
  pd::t_tracing = true;
  return PD_OK;
}

extern "C" pd_status pd_trace_end(pd_trace_report* out) {
  pd::t_tracing = false;
  if (!out || out->struct_size != sizeof(pd_trace_report)) return PD_ERR_INVALID_ARG;
  for (int i = 0; i < PD_TRACE_CLASSES; ++i) {
    out->time_s[i] = 0.0;
    out->launches[i] = 0;
  }
  pd_status st = PD_OK;
  for (auto& r : pd::t_recs) {
    float ms = 0.f;
    cudaError_t e = cudaEventSynchronize(r.b);
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, r.a, r.b);
    if (e != cudaSuccess) {
      st = pd::cuda_fail(e);
    } else if (r.cls >= 0 && r.cls < PD_TRACE_CLASSES) {
      out->time_s[r.cls] += ms * 1e-3;
      out->launches[r.cls] += 1;
    }
    pd::t_pool.push_back(r.a);
    pd::t_pool.push_back(r.b);
  }
  pd::t_recs.clear();
  return st;
}
