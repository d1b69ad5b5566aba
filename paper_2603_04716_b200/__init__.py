"""Python binding of libpd.so: argument marshalling only.

Every computational step runs inside the CUDA library; this module converts
Python/torch arguments to the plain pointers and structs of include/pd.h and
raises PdError on a non-zero status.  There is no fallback: if the shared
library has not been built, importing fails.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libpd.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2603_04716_b200.build` "
        "(there is no CPU or PyTorch fallback)")
_lib = C.CDLL(LIB_PATH)

PD_OK = 0
PD_ERR_INVALID_ARG = -1
PD_ERR_UNSUPPORTED_SHAPE = -2
PD_ERR_WORKSPACE_TOO_SMALL = -3
PD_ERR_CUDA = -4
PD_ERR_DEVICE_TIMEOUT = -5
PD_ERR_INFEASIBLE_TTFT = -6
PD_ERR_INFEASIBLE_TPOT = -7
PD_ERR_ARCH = -8

EXPORTS = [
    "pd_status_str", "pd_last_cuda_error", "pd_version", "pd_layer_create", "pd_layer_destroy",
    "pd_workspace_bytes", "pd_prefill_layer", "pd_decode_layer", "pd_prefill_stack", "pd_decode_stack",
    "pd_layer_check", "pd_gemm_bf16", "pd_measure", "pd_allocate", "pd_queue_replay",
    "pd_launch_count", "pd_trace_begin", "pd_trace_end", "pd_decode_attention", "pd_decode_attention_workspace_bytes",
    "pd_decode_attention_noalloc", "pd_prefill_chunk_layer",
    "pd_model_create", "pd_model_destroy", "pd_model_workspace_bytes", "pd_model_prefill", "pd_model_decode_step",
    "pd_model_check", "pd_allocate_ext", "pd_quantize_fp8_rows", "pd_gemm_fp8", "pd_workspace_offsets",
    "pd_prefill_attention", "pd_mixture_throughput", "pd_interp_service_times", "pd_mm1_sojourn", "pd_mg1_sojourn",
    "pd_refine_next_batch", "pd_prefill_chunk_stack", "pd_test_inject_wait_timeout",
    "pd_gemm_workspace_bytes", "pd_gemm_bf16_ws",
    "pd_quantize_fp8_groups", "pd_quantize_fp8_blocks", "pd_gemm_fp8_blockwise",
]

TRACE_CLASSES = ["gemm_qkv", "gemm_o", "gemm_gate_up", "gemm_down", "attn_prefill", "attn_decode", "rmsnorm",
                 "embed", "lm_head", "sample"]


class PdError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = _lib.pd_status_str(status).decode()
        if status == PD_ERR_CUDA:
            msg += f" (cudaError {_lib.pd_last_cuda_error()})"
        super().__init__(f"{where}: {msg} [{status}]")


class pd_layer_cfg(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("d_model", C.c_int32), ("n_q_heads", C.c_int32),
                ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("d_ff", C.c_int32),
                ("rms_eps", C.c_float), ("rope_theta", C.c_float), ("max_pos", C.c_int32),
                ("fp8_projections", C.c_int32)]


class pd_workspace_layout(C.Structure):
    _fields_ = [("struct_size", C.c_uint32)] + [(n, C.c_uint64) for n in ("norm", "qkv", "attn_o", "resid", "act")]


class pd_layer_weights(C.Structure):
    _fields_ = [("struct_size", C.c_uint32)] + [(n, C.c_void_p) for n in
                ("w_qkv", "w_o", "w_gate", "w_up", "w_down", "g_attn", "g_mlp")]


class pd_model_weights(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("vocab", C.c_int32), ("embed", C.c_void_p), ("g_final", C.c_void_p),
                ("lm_head", C.c_void_p)]


class pd_kv_cache(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("k", C.c_void_p), ("v", C.c_void_p),
                ("batch_cap", C.c_int32), ("len_cap", C.c_int32)]


MEASURE_GRID_MAX = 128


class pd_measure_cfg(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("n_layers_run", C.c_int32), ("n_layers_model", C.c_int32),
                ("warmup", C.c_int32), ("reps", C.c_int32), ("seed", C.c_uint64),
                ("l_in", C.POINTER(C.c_int32)), ("n_req", C.c_int32),
                ("batch_sizes", C.POINTER(C.c_int32)), ("n_batch_sizes", C.c_int32),
                ("kv_len_start", C.c_int32), ("n_steps", C.c_int32), ("step_stride", C.c_int32),
                ("kv_len_mix", C.POINTER(C.c_int32)), ("vocab", C.c_int32), ("chunk_tokens", C.c_int32),
                ("l_in_grid", C.POINTER(C.c_int32)), ("n_grid", C.c_int32)]


class pd_measurement(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("prefill_time_s", C.c_double), ("prefill_tok_s", C.c_double),
                ("prefill_flops", C.c_double), ("prefill_frac_bf16_peak", C.c_double),
                ("n_points", C.c_int32), ("batch", C.c_int32 * 32), ("tpot_s", C.c_double * 32),
                ("decode_bytes", C.c_double * 32), ("decode_frac_hbm_peak", C.c_double * 32),
                ("attn_time_s", C.c_double * 32), ("attn_frac_hbm_peak", C.c_double * 32),
                ("gpu_launches", C.c_int32), ("prefill_head_s", C.c_double), ("decode_head_s", C.c_double * 32),
                ("prefill_chunks", C.c_int32), ("prefill_kv_ring", C.c_int32), ("decode_kv_ring", C.c_int32 * 32),
                ("attn_l2_resident", C.c_int32 * 32), ("n_grid", C.c_int32), ("grid_l", C.c_int32 * MEASURE_GRID_MAX),
                ("grid_time_s", C.c_double * MEASURE_GRID_MAX)]


class pd_trace_report(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("time_s", C.c_double * 16), ("launches", C.c_int64 * 16)]


class pd_alloc_in(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("tp_total_tok_s", C.c_double), ("l_in", C.c_double),
                ("l_out", C.c_double), ("ttft_slo_s", C.c_double), ("tpot_slo_s", C.c_double),
                ("t_overhead_s", C.c_double), ("prefill_max_tok_s", C.c_double), ("n_points", C.c_int32),
                ("batch", C.POINTER(C.c_int32)), ("tpot_s", C.POINTER(C.c_double))]


class pd_alloc_out(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("tp_prefill_eff", C.c_double), ("tp_decode_eff", C.c_double),
                ("mu", C.c_double), ("lam", C.c_double), ("rho", C.c_double),
                ("feasible_batch", C.c_int32), ("sweep_capped", C.c_int32),
                ("n_prefill_frac", C.c_double), ("n_decode_frac", C.c_double), ("ratio_pd", C.c_double),
                ("n_prefill", C.c_int32), ("n_decode", C.c_int32), ("n_prefill_ceil", C.c_int32),
                ("n_decode_ceil", C.c_int32), ("achieved_total_tok_s", C.c_double)]


_lib.pd_status_str.restype = C.c_char_p
_lib.pd_status_str.argtypes = [C.c_int]
_lib.pd_last_cuda_error.restype = C.c_int
_lib.pd_version.restype = C.c_int
_P = C.c_void_p
_lib.pd_layer_create.argtypes = [C.POINTER(pd_layer_cfg), C.POINTER(pd_layer_weights), _P, C.POINTER(_P)]
_lib.pd_layer_destroy.argtypes = [_P]
_lib.pd_workspace_bytes.argtypes = [C.POINTER(pd_layer_cfg), C.c_int32, C.c_int32, C.c_int32, C.POINTER(C.c_size_t)]
_lib.pd_prefill_layer.argtypes = [_P, _P, _P, _P, C.POINTER(C.c_int32), C.c_int32, _P, C.POINTER(pd_kv_cache), _P,
                                  C.c_size_t, _P]
_lib.pd_prefill_chunk_layer.argtypes = [_P, _P, _P, _P, C.POINTER(C.c_int32), C.c_int32, _P, C.POINTER(C.c_int32), _P,
                                        C.POINTER(pd_kv_cache), _P, C.c_size_t, _P]
_lib.pd_decode_layer.argtypes = [_P, _P, _P, _P, C.c_int32, C.c_int32, C.POINTER(pd_kv_cache), _P, C.c_size_t, _P]
_lib.pd_prefill_stack.argtypes = [C.POINTER(_P), C.POINTER(pd_kv_cache), C.c_int32, C.c_int32, _P, _P, C.c_int32, _P,
                                  C.POINTER(C.c_int32), C.c_int32, _P, C.c_size_t, _P]
_lib.pd_prefill_chunk_stack.argtypes = [C.POINTER(_P), C.POINTER(pd_kv_cache), C.c_int32, C.c_int32, _P, _P, _P,
                                        C.POINTER(C.c_int32), C.c_int32, _P, C.POINTER(C.c_int32), _P, C.c_size_t, _P]
_lib.pd_decode_stack.argtypes = [C.POINTER(_P), C.POINTER(pd_kv_cache), C.c_int32, C.c_int32, _P, _P, C.c_int32, _P,
                                 C.c_int32, C.c_int32, _P, C.c_size_t, _P]
_lib.pd_layer_check.argtypes = [_P, _P]
_lib.pd_gemm_bf16.argtypes = [_P, _P, _P, C.c_int32, C.c_int32, C.c_int32, _P, _P]
_lib.pd_gemm_workspace_bytes.argtypes = [C.POINTER(C.c_size_t)]
_lib.pd_gemm_bf16_ws.argtypes = [_P, _P, _P, C.c_int32, C.c_int32, C.c_int32, _P, C.c_size_t, _P, _P]
_lib.pd_workspace_offsets.argtypes = [C.POINTER(pd_layer_cfg), C.c_int32, C.POINTER(pd_workspace_layout)]
_lib.pd_quantize_fp8_rows.argtypes = [_P, C.c_int32, C.c_int32, C.c_int32, _P, _P, _P]
_lib.pd_gemm_fp8.argtypes = [_P, _P, _P, _P, _P, C.c_int32, C.c_int32, C.c_int32, _P, _P]
_lib.pd_quantize_fp8_groups.argtypes = [_P, C.c_int32, C.c_int32, C.c_int32, _P, _P, _P]
_lib.pd_quantize_fp8_blocks.argtypes = [_P, C.c_int32, C.c_int32, C.c_int32, _P, _P, _P]
_lib.pd_gemm_fp8_blockwise.argtypes = [_P, _P, _P, _P, _P, C.c_int32, C.c_int32, C.c_int32, _P, _P]
_lib.pd_measure.argtypes = [C.POINTER(pd_layer_cfg), C.POINTER(pd_measure_cfg), C.c_double, C.c_double,
                            C.POINTER(pd_measurement)]
_lib.pd_allocate.argtypes = [C.POINTER(pd_alloc_in), C.POINTER(pd_alloc_out)]
_lib.pd_allocate_ext.argtypes = [C.POINTER(pd_alloc_in), C.c_double, C.c_int32, C.POINTER(pd_alloc_out)]
_lib.pd_queue_replay.argtypes = [C.POINTER(C.c_double), C.POINTER(C.c_double), C.c_int64, C.POINTER(C.c_double),
                                 C.POINTER(C.c_double)]
_DP, _IP = C.POINTER(C.c_double), C.POINTER(C.c_int32)
_lib.pd_mixture_throughput.argtypes = [_IP, _DP, C.c_int64, _DP, _DP]
_lib.pd_interp_service_times.argtypes = [_IP, _DP, C.c_int32, _IP, C.c_int64, C.c_int32, _DP]
_lib.pd_mm1_sojourn.argtypes = [C.c_double, C.c_double, _DP]
_lib.pd_mg1_sojourn.argtypes = [_DP, C.c_int64, C.c_double, _DP]
_lib.pd_refine_next_batch.argtypes = [_IP, _DP, C.c_int32, C.c_double, _IP]
_lib.pd_decode_attention_workspace_bytes.argtypes = [C.POINTER(pd_layer_cfg), C.c_int32, C.c_int32,
                                                     C.POINTER(C.c_size_t)]
_lib.pd_decode_attention.argtypes = [C.POINTER(pd_layer_cfg), _P, C.c_int32, _P, _P, C.c_int32, C.c_int32,
                                     C.POINTER(pd_kv_cache), _P, C.c_size_t, _P]
_lib.pd_prefill_attention.argtypes = [C.POINTER(pd_layer_cfg), _P, C.c_int32, _P, _P, C.POINTER(C.c_int32), C.c_int32,
                                      _P, C.POINTER(C.c_int32), _P, C.POINTER(pd_kv_cache), _P, _P]
_lib.pd_decode_attention_noalloc.argtypes = [C.POINTER(pd_layer_cfg), _P, C.c_int32, _P, _P, C.c_int32, C.c_int32,
                                             C.POINTER(pd_kv_cache), _P]
_lib.pd_model_create.argtypes = [C.POINTER(_P), C.c_int32, C.POINTER(pd_model_weights), _P, C.POINTER(_P)]
_lib.pd_model_destroy.argtypes = [_P]
_lib.pd_model_check.argtypes = [_P, _P]
_lib.pd_model_workspace_bytes.argtypes = [_P, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.POINTER(C.c_size_t)]
_lib.pd_model_prefill.argtypes = [_P, _P, _P, C.POINTER(C.c_int32), C.c_int32, C.POINTER(pd_kv_cache), C.c_int32, _P,
                                  _P, _P, C.c_size_t, _P]
_lib.pd_model_decode_step.argtypes = [_P, _P, _P, C.c_int32, C.c_int32, C.POINTER(pd_kv_cache), C.c_int32, _P, _P, _P,
                                      C.c_size_t, _P]
_lib.pd_launch_count.restype = C.c_int64
_lib.pd_trace_end.argtypes = [C.POINTER(pd_trace_report)]
for _n in EXPORTS:
    if _n not in ("pd_status_str", "pd_last_cuda_error", "pd_version", "pd_launch_count"):
        getattr(_lib, _n).restype = C.c_int


def _check(status: int, where: str, allow=()):
    if status != PD_OK and status not in allow:
        raise PdError(status, where)
    return status


def _ptr(t):
    """Device/host address of a torch tensor, a numpy array, an int, or None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if hasattr(t, "data_ptr"):
        return t.data_ptr()
    if hasattr(t, "ctypes"):
        return t.ctypes.data
    raise TypeError(type(t))


def _stream_ptr(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _i32_array(values):
    arr = (C.c_int32 * len(values))(*[int(v) for v in values])
    return arr


@dataclass(frozen=True)
class LayerConfig:
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ff: int
    rms_eps: float = 1e-6
    rope_theta: float = 1e4
    max_pos: int = 4096
    fp8_projections: bool = False

    def c_struct(self) -> pd_layer_cfg:
        return pd_layer_cfg(C.sizeof(pd_layer_cfg), self.d_model, self.n_q_heads, self.n_kv_heads, self.head_dim,
                            self.d_ff, self.rms_eps, self.rope_theta, self.max_pos, int(self.fp8_projections))

    @property
    def n_qkv(self) -> int:
        return (self.n_q_heads + 2 * self.n_kv_heads) * self.head_dim


INJECT_NONE, INJECT_ATTN_PREFILL, INJECT_GEMM, INJECT_GEMM_PAIR, INJECT_GEMM_FP8_BLOCKWISE = 0, 1, 2, 3, 4
_lib.pd_test_inject_wait_timeout.argtypes = [C.c_int32, C.c_uint64]


def pd_test_inject_wait_timeout(kernel_kind: int, wait_limit_ns: int):
    """Arms one injected wait timeout for the calling thread's next launch of that kernel kind."""
    _check(_lib.pd_test_inject_wait_timeout(kernel_kind, wait_limit_ns), "pd_test_inject_wait_timeout")


def pd_version() -> int:
    return _lib.pd_version()


def pd_launch_count() -> int:
    return _lib.pd_launch_count()


def pd_trace_begin():
    _check(_lib.pd_trace_begin(), "pd_trace_begin")


def pd_trace_end() -> dict:
    """{class name: (seconds, launches)} for the kernels launched since pd_trace_begin."""
    rep = pd_trace_report(C.sizeof(pd_trace_report))
    _check(_lib.pd_trace_end(C.byref(rep)), "pd_trace_end")
    return {name: (rep.time_s[i], rep.launches[i]) for i, name in enumerate(TRACE_CLASSES)}


def pd_workspace_bytes(cfg: LayerConfig, max_tokens: int, max_batch: int, max_kv_len: int) -> int:
    out = C.c_size_t(0)
    _check(_lib.pd_workspace_bytes(C.byref(cfg.c_struct()), max_tokens, max_batch, max_kv_len, C.byref(out)),
           "pd_workspace_bytes")
    return out.value


class Layer:
    """Owns a pd_layer handle."""

    def __init__(self, cfg: LayerConfig, weights: dict, stream=None):
        self.cfg = cfg
        w = pd_layer_weights(C.sizeof(pd_layer_weights), *[_ptr(weights[k]) for k in
                             ("w_qkv", "w_o", "w_gate", "w_up", "w_down", "g_attn", "g_mlp")])
        h = _P()
        _check(_lib.pd_layer_create(C.byref(cfg.c_struct()), C.byref(w), _stream_ptr(stream), C.byref(h)),
               "pd_layer_create")
        self.handle = h

    def close(self):
        if getattr(self, "handle", None):
            _lib.pd_layer_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def kv_cache_struct(k, v, batch_cap: int, len_cap: int) -> pd_kv_cache:
    return pd_kv_cache(C.sizeof(pd_kv_cache), _ptr(k), _ptr(v), batch_cap, len_cap)


def pd_prefill_layer(layer: Layer, x, out, cu_seqlens_dev, cu_seqlens_host, cache: pd_kv_cache, workspace,
                     workspace_bytes: int, slots_dev=None, stream=None):
    cu = _i32_array(cu_seqlens_host)
    _check(_lib.pd_prefill_layer(layer.handle, _ptr(x), _ptr(out), _ptr(cu_seqlens_dev), cu, len(cu_seqlens_host) - 1,
                                 _ptr(slots_dev), C.byref(cache), _ptr(workspace), workspace_bytes,
                                 _stream_ptr(stream)), "pd_prefill_layer")


def pd_prefill_chunk_layer(layer: Layer, x, out, cu_seqlens_dev, cu_seqlens_host, prefix_dev, prefix_host,
                           cache: pd_kv_cache, workspace, workspace_bytes: int, slots_dev=None, stream=None):
    cu = _i32_array(cu_seqlens_host)
    pre = _i32_array(prefix_host)
    _check(_lib.pd_prefill_chunk_layer(layer.handle, _ptr(x), _ptr(out), _ptr(cu_seqlens_dev), cu,
                                       len(cu_seqlens_host) - 1, _ptr(prefix_dev), pre, _ptr(slots_dev),
                                       C.byref(cache), _ptr(workspace), workspace_bytes, _stream_ptr(stream)),
           "pd_prefill_chunk_layer")


def pd_decode_layer(layer: Layer, x, out, kv_len_dev, batch: int, max_kv_len: int, cache: pd_kv_cache, workspace,
                    workspace_bytes: int, stream=None):
    _check(_lib.pd_decode_layer(layer.handle, _ptr(x), _ptr(out), _ptr(kv_len_dev), batch, max_kv_len,
                                C.byref(cache), _ptr(workspace), workspace_bytes, _stream_ptr(stream)),
           "pd_decode_layer")


def pd_decode_attention_workspace_bytes(cfg: LayerConfig, batch: int, max_kv_len: int) -> int:
    out = C.c_size_t(0)
    _check(_lib.pd_decode_attention_workspace_bytes(C.byref(cfg.c_struct()), batch, max_kv_len, C.byref(out)),
           "pd_decode_attention_workspace_bytes")
    return out.value


def pd_decode_attention(cfg: LayerConfig, q, ldq: int, out, kv_len_dev, batch: int, max_kv_len: int,
                        cache: pd_kv_cache, workspace, workspace_bytes: int, stream=None):
    _check(_lib.pd_decode_attention(C.byref(cfg.c_struct()), _ptr(q), ldq, _ptr(out), _ptr(kv_len_dev), batch,
                                    max_kv_len, C.byref(cache), _ptr(workspace), workspace_bytes,
                                    _stream_ptr(stream)), "pd_decode_attention")


def pd_prefill_attention(cfg: LayerConfig, q, ldq: int, out, cu_seqlens_dev, cu_seqlens_host, cache: pd_kv_cache,
                         prefix_dev=None, prefix_host=None, slots_dev=None, err_word=None, stream=None):
    cu = _i32_array(cu_seqlens_host)
    pre = _i32_array(prefix_host) if prefix_host is not None else None
    _check(_lib.pd_prefill_attention(C.byref(cfg.c_struct()), _ptr(q), ldq, _ptr(out), _ptr(cu_seqlens_dev), cu,
                                     len(cu_seqlens_host) - 1, _ptr(prefix_dev), pre, _ptr(slots_dev),
                                     C.byref(cache), _ptr(err_word), _stream_ptr(stream)), "pd_prefill_attention")


NOALLOC_SCRATCH_BYTES = 8 << 20


def pd_decode_attention_noalloc(cfg: LayerConfig, q, ldq: int, out, kv_len_dev, batch: int, max_kv_len: int,
                                cache: pd_kv_cache, stream=None):
    """pd_decode_attention without a workspace argument, for callers that must not allocate
    device memory: the split partials live in a fixed NOALLOC_SCRATCH_BYTES array inside the
    library.  Raises PdError(PD_ERR_WORKSPACE_TOO_SMALL) when the problem does not fit it.
    Calls on one device share that array, so keep them on one stream."""
    _check(_lib.pd_decode_attention_noalloc(C.byref(cfg.c_struct()), _ptr(q), ldq, _ptr(out), _ptr(kv_len_dev),
                                            batch, max_kv_len, C.byref(cache), _stream_ptr(stream)),
           "pd_decode_attention_noalloc")


def _layer_array(layers):
    return (_P * len(layers))(*[l.handle for l in layers])


def _cache_array(caches):
    return (pd_kv_cache * len(caches))(*caches)


def pd_prefill_stack(layers, caches, x, out, io_on_host: bool, cu_seqlens_dev, cu_seqlens_host, workspace,
                     workspace_bytes: int, stream=None):
    cu = _i32_array(cu_seqlens_host)
    _check(_lib.pd_prefill_stack(_layer_array(layers), _cache_array(caches), len(layers), len(caches), _ptr(x),
                                 _ptr(out), int(io_on_host), _ptr(cu_seqlens_dev), cu, len(cu_seqlens_host) - 1,
                                 _ptr(workspace), workspace_bytes, _stream_ptr(stream)), "pd_prefill_stack")


def pd_prefill_chunk_stack(layers, caches, x, out, cu_seqlens_dev, cu_seqlens_host, prefix_dev, prefix_host,
                           workspace, workspace_bytes: int, stream=None):
    cu = _i32_array(cu_seqlens_host)
    pre = _i32_array(prefix_host)
    _check(_lib.pd_prefill_chunk_stack(_layer_array(layers), _cache_array(caches), len(layers), len(caches), _ptr(x),
                                       _ptr(out), _ptr(cu_seqlens_dev), cu, len(cu_seqlens_host) - 1, _ptr(prefix_dev),
                                       pre, _ptr(workspace), workspace_bytes, _stream_ptr(stream)),
           "pd_prefill_chunk_stack")


def pd_decode_stack(layers, caches, x, out, io_on_host: bool, kv_len, batch: int, max_kv_len: int, workspace,
                    workspace_bytes: int, stream=None):
    _check(_lib.pd_decode_stack(_layer_array(layers), _cache_array(caches), len(layers), len(caches), _ptr(x),
                                _ptr(out), int(io_on_host), _ptr(kv_len), batch, max_kv_len, _ptr(workspace),
                                workspace_bytes, _stream_ptr(stream)), "pd_decode_stack")


class Model:
    """Owns a pd_model handle (embedding, final norm gain, LM head) over borrowed layers."""

    def __init__(self, layers, vocab: int, embed, g_final, lm_head, stream=None):
        self.layers = list(layers)          # keeps the borrowed layers alive
        self.vocab = vocab
        w = pd_model_weights(C.sizeof(pd_model_weights), vocab, _ptr(embed), _ptr(g_final), _ptr(lm_head))
        h = _P()
        _check(_lib.pd_model_create(_layer_array(self.layers), len(self.layers), C.byref(w), _stream_ptr(stream),
                                    C.byref(h)), "pd_model_create")
        self.handle = h

    def close(self):
        if getattr(self, "handle", None):
            _lib.pd_model_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def pd_model_workspace_bytes(model: Model, max_tokens: int, max_requests: int, max_batch: int,
                             max_kv_len: int) -> int:
    out = C.c_size_t(0)
    _check(_lib.pd_model_workspace_bytes(model.handle, max_tokens, max_requests, max_batch, max_kv_len,
                                         C.byref(out)), "pd_model_workspace_bytes")
    return out.value


def pd_model_prefill(model: Model, tokens_dev, cu_seqlens_dev, cu_seqlens_host, caches, next_dev, workspace,
                     workspace_bytes: int, logits_dev=None, stream=None):
    cu = _i32_array(cu_seqlens_host)
    _check(_lib.pd_model_prefill(model.handle, _ptr(tokens_dev), _ptr(cu_seqlens_dev), cu, len(cu_seqlens_host) - 1,
                                 _cache_array(caches), len(caches), _ptr(next_dev), _ptr(logits_dev),
                                 _ptr(workspace), workspace_bytes, _stream_ptr(stream)), "pd_model_prefill")


def pd_model_decode_step(model: Model, tokens_dev, kv_len_dev, batch: int, max_kv_len: int, caches, next_dev,
                         workspace, workspace_bytes: int, logits_dev=None, stream=None):
    _check(_lib.pd_model_decode_step(model.handle, _ptr(tokens_dev), _ptr(kv_len_dev), batch, max_kv_len,
                                     _cache_array(caches), len(caches), _ptr(next_dev), _ptr(logits_dev),
                                     _ptr(workspace), workspace_bytes, _stream_ptr(stream)), "pd_model_decode_step")


def pd_model_check(model: Model, stream=None):
    _check(_lib.pd_model_check(model.handle, _stream_ptr(stream)), "pd_model_check")


def pd_layer_check(layer: Layer, stream=None):
    _check(_lib.pd_layer_check(layer.handle, _stream_ptr(stream)), "pd_layer_check")


def pd_gemm_bf16(a, b, c, m: int, n: int, k: int, err_word=None, stream=None):
    _check(_lib.pd_gemm_bf16(_ptr(a), _ptr(b), _ptr(c), m, n, k, _ptr(err_word), _stream_ptr(stream)), "pd_gemm_bf16")


def pd_gemm_workspace_bytes() -> int:
    out = C.c_size_t(0)
    _check(_lib.pd_gemm_workspace_bytes(C.byref(out)), "pd_gemm_workspace_bytes")
    return out.value


def pd_gemm_bf16_ws(a, b, c, m: int, n: int, k: int, workspace, workspace_bytes: int, err_word=None, stream=None):
    """pd_gemm_bf16 with the K-split scratch (tiles may be cut in two along K and run on two SMs / CTA pairs)."""
    _check(_lib.pd_gemm_bf16_ws(_ptr(a), _ptr(b), _ptr(c), m, n, k, _ptr(workspace), workspace_bytes, _ptr(err_word),
                                _stream_ptr(stream)), "pd_gemm_bf16_ws")


def pd_workspace_offsets(cfg: LayerConfig, tokens: int) -> dict:
    """Byte offsets of the intermediates a layer pass over `tokens` rows leaves in its workspace."""
    out = pd_workspace_layout(C.sizeof(pd_workspace_layout))
    _check(_lib.pd_workspace_offsets(C.byref(cfg.c_struct()), tokens, C.byref(out)), "pd_workspace_offsets")
    return {n: int(getattr(out, n)) for n in ("norm", "qkv", "attn_o", "resid", "act")}


def pd_quantize_fp8_rows(x, rows: int, k: int, codes, scales, ldx: int = 0, stream=None):
    """x: device bf16 [rows, k] (row pitch ldx, default k) -> codes: device uint8 [rows, k], scales: device fp32 [rows]."""
    _check(_lib.pd_quantize_fp8_rows(_ptr(x), ldx or k, rows, k, _ptr(codes), _ptr(scales), _stream_ptr(stream)),
           "pd_quantize_fp8_rows")


def pd_gemm_fp8(a_codes, a_scales, b_codes, b_scales, c, m: int, n: int, k: int, err_word=None, stream=None):
    _check(_lib.pd_gemm_fp8(_ptr(a_codes), _ptr(a_scales), _ptr(b_codes), _ptr(b_scales), _ptr(c), m, n, k,
                            _ptr(err_word), _stream_ptr(stream)), "pd_gemm_fp8")


def pd_quantize_fp8_groups(x, rows: int, k: int, codes, scales, ldx: int = 0, stream=None):
    """x: device bf16 [rows, k] -> codes uint8 [rows, k], scales fp32 [rows, k / 128] (one per row and 128 channels)."""
    _check(_lib.pd_quantize_fp8_groups(_ptr(x), ldx or k, rows, k, _ptr(codes), _ptr(scales), _stream_ptr(stream)),
           "pd_quantize_fp8_groups")


def pd_quantize_fp8_blocks(w, n: int, k: int, codes, scales, ldw: int = 0, stream=None):
    """w: device bf16 [n, k] -> codes uint8 [n, k], scales fp32 [ceil(n / 128), k / 128] (one per 128 x 128 block)."""
    _check(_lib.pd_quantize_fp8_blocks(_ptr(w), ldw or k, n, k, _ptr(codes), _ptr(scales), _stream_ptr(stream)),
           "pd_quantize_fp8_blocks")


def pd_gemm_fp8_blockwise(a_codes, a_scales, b_codes, b_scales, c, m: int, n: int, k: int, err_word=None, stream=None):
    _check(_lib.pd_gemm_fp8_blockwise(_ptr(a_codes), _ptr(a_scales), _ptr(b_codes), _ptr(b_scales), _ptr(c), m, n, k,
                                      _ptr(err_word), _stream_ptr(stream)), "pd_gemm_fp8_blockwise")


def pd_measure(cfg: LayerConfig, *, n_layers_run: int, n_layers_model: int, warmup: int = 3, reps: int = 10,
               seed: int = 0, l_in=(), batch_sizes=(), kv_len_start: int = 0, n_steps: int = 1,
               step_stride: int = 1, kv_len_mix=None, peak_bf16_flops: float = 0.0,
               peak_hbm_bytes_s: float = 0.0, vocab: int = 0, chunk_tokens: int = 0, l_in_grid=()) -> dict:
    """vocab > 0 measures the whole-model step (embedding, final norm, LM head and greedy sampling added
    to the prefill time and to every TPOT); chunk_tokens > 0 measures chunked prefill; l_in_grid lists
    lengths to be timed one request at a time (the service-time curve)."""
    l_arr = _i32_array(l_in) if len(l_in) else None
    b_arr = _i32_array(batch_sizes) if len(batch_sizes) else None
    mix = _i32_array(kv_len_mix) if kv_len_mix is not None else None
    g_arr = _i32_array(l_in_grid) if len(l_in_grid) else None
    m = pd_measure_cfg(C.sizeof(pd_measure_cfg), n_layers_run, n_layers_model, warmup, reps, seed,
                       l_arr, len(l_in), b_arr, len(batch_sizes), kv_len_start, n_steps, step_stride, mix, vocab,
                       chunk_tokens, g_arr, len(l_in_grid))
    out = pd_measurement()
    _check(_lib.pd_measure(C.byref(cfg.c_struct()), C.byref(m), peak_bf16_flops, peak_hbm_bytes_s, C.byref(out)),
           "pd_measure")
    n = out.n_points
    return {
        "prefill_time_s": out.prefill_time_s, "prefill_tok_s": out.prefill_tok_s,
        "prefill_flops": out.prefill_flops, "prefill_frac_bf16_peak": out.prefill_frac_bf16_peak,
        "batch": list(out.batch[:n]), "tpot_s": list(out.tpot_s[:n]),
        "decode_bytes": list(out.decode_bytes[:n]), "decode_frac_hbm_peak": list(out.decode_frac_hbm_peak[:n]),
        "attn_time_s": list(out.attn_time_s[:n]), "attn_frac_hbm_peak": list(out.attn_frac_hbm_peak[:n]),
        "gpu_launches": out.gpu_launches,
        "prefill_head_s": out.prefill_head_s, "decode_head_s": list(out.decode_head_s[:n]),
        "prefill_chunks": out.prefill_chunks, "prefill_kv_ring": out.prefill_kv_ring,
        "decode_kv_ring": list(out.decode_kv_ring[:n]), "attn_l2_resident": list(out.attn_l2_resident[:n]),
        "grid_l": list(out.grid_l[:out.n_grid]), "grid_time_s": list(out.grid_time_s[:out.n_grid]),
    }


def pd_allocate(tp_total_tok_s: float, l_in: float, l_out: float, ttft_slo_s: float, tpot_slo_s: float,
                prefill_max_tok_s: float, batch, tpot_s, t_overhead_s: float = 0.0) -> dict:
    """Returns every field of pd_alloc_out plus `status` (0, PD_ERR_INFEASIBLE_TTFT or PD_ERR_INFEASIBLE_TPOT)."""
    n = len(batch)
    b = _i32_array(batch) if n else None
    t = (C.c_double * n)(*[float(v) for v in tpot_s]) if n else None
    inp = pd_alloc_in(C.sizeof(pd_alloc_in), tp_total_tok_s, l_in, l_out, ttft_slo_s, tpot_slo_s, t_overhead_s,
                      prefill_max_tok_s, n, b, t)
    out = pd_alloc_out()
    st = _check(_lib.pd_allocate(C.byref(inp), C.byref(out)), "pd_allocate",
                allow=(PD_ERR_INFEASIBLE_TTFT, PD_ERR_INFEASIBLE_TPOT))
    res = {name: getattr(out, name) for name, _ in pd_alloc_out._fields_ if name != "struct_size"}
    res["status"] = st
    return res


def pd_allocate_ext(tp_total_tok_s: float, l_in: float, l_out: float, ttft_slo_s: float, tpot_slo_s: float,
                    prefill_max_tok_s: float, batch, tpot_s, t_overhead_s: float = 0.0, prefix_hit_frac: float = 0.0,
                    dp_groups: int = 1) -> dict:
    """pd_allocate with a prefix-cache hit fraction and data-parallel prefill groups (mu, lam, rho per group)."""
    n = len(batch)
    b = _i32_array(batch) if n else None
    t = (C.c_double * n)(*[float(v) for v in tpot_s]) if n else None
    inp = pd_alloc_in(C.sizeof(pd_alloc_in), tp_total_tok_s, l_in, l_out, ttft_slo_s, tpot_slo_s, t_overhead_s,
                      prefill_max_tok_s, n, b, t)
    out = pd_alloc_out()
    st = _check(_lib.pd_allocate_ext(C.byref(inp), prefix_hit_frac, dp_groups, C.byref(out)), "pd_allocate_ext",
                allow=(PD_ERR_INFEASIBLE_TTFT, PD_ERR_INFEASIBLE_TPOT))
    res = {name: getattr(out, name) for name, _ in pd_alloc_out._fields_ if name != "struct_size"}
    res["status"] = st
    return res


def pd_queue_replay(gaps, service):
    """(mean sojourn, mean wait) of the FIFO single-server replay; numpy float64 arrays or sequences."""
    import numpy as np
    g = np.ascontiguousarray(gaps, dtype=np.float64)
    s = np.ascontiguousarray(service, dtype=np.float64)
    if g.shape != s.shape:
        raise ValueError("gaps and service must have the same length")
    soj, wait = C.c_double(), C.c_double()
    dp = C.POINTER(C.c_double)
    _check(_lib.pd_queue_replay(g.ctypes.data_as(dp), s.ctypes.data_as(dp), g.size, C.byref(soj), C.byref(wait)),
           "pd_queue_replay")
    return soj.value, wait.value


def _np_i32(a):
    import numpy as np
    return np.ascontiguousarray(a, dtype=np.int32)


def _np_f64(a):
    import numpy as np
    return np.ascontiguousarray(a, dtype=np.float64)


def pd_mixture_throughput(l_in, service_s):
    """(maximum prefill throughput of the request mix, mean input length)."""
    l, s = _np_i32(l_in), _np_f64(service_s)
    if l.shape != s.shape:
        raise ValueError("one service time per request")
    tp, mean_l = C.c_double(), C.c_double()
    _check(_lib.pd_mixture_throughput(l.ctypes.data_as(_IP), s.ctypes.data_as(_DP), l.size, C.byref(tp),
                                      C.byref(mean_l)), "pd_mixture_throughput")
    return tp.value, mean_l.value


def pd_interp_service_times(grid_l, grid_time_s, l_in, quantum: int = 1):
    """numpy float64 array: service time of each length (rounded up to a multiple of `quantum`), interpolated on
    the measured grid."""
    import numpy as np
    gl, gt, l = _np_i32(grid_l), _np_f64(grid_time_s), _np_i32(l_in)
    if gl.shape != gt.shape:
        raise ValueError("one time per grid length")
    out = np.empty(l.size, dtype=np.float64)
    _check(_lib.pd_interp_service_times(gl.ctypes.data_as(_IP), gt.ctypes.data_as(_DP), gl.size,
                                        l.ctypes.data_as(_IP), l.size, quantum, out.ctypes.data_as(_DP)),
           "pd_interp_service_times")
    return out


def pd_mm1_sojourn(mu: float, lam: float) -> float:
    out = C.c_double()
    _check(_lib.pd_mm1_sojourn(mu, lam, C.byref(out)), "pd_mm1_sojourn")
    return out.value


def pd_mg1_sojourn(service_s, lam: float) -> float:
    s = _np_f64(service_s)
    out = C.c_double()
    _check(_lib.pd_mg1_sojourn(s.ctypes.data_as(_DP), s.size, lam, C.byref(out)), "pd_mg1_sojourn")
    return out.value


def pd_refine_next_batch(batch, tpot_s, tpot_slo_s: float) -> int:
    """Next batch size to measure while refining the TPOT-feasible batch, 0 when done."""
    b, t = _np_i32(batch), _np_f64(tpot_s)
    if b.shape != t.shape:
        raise ValueError("one TPOT per batch size")
    out = C.c_int32()
    _check(_lib.pd_refine_next_batch(b.ctypes.data_as(_IP), t.ctypes.data_as(_DP), b.size, tpot_slo_s,
                                     C.byref(out)), "pd_refine_next_batch")
    return out.value
