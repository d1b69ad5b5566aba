"""CPU oracle for one dense decoder layer (prefill and decode mode).

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain statement of what the
GPU library computes.  It shares no code with the CUDA path and must never be
imported by it; only tests, the smoke check and the benchmark's CPU-baseline
leg call it.

The paper (Introduction; "Acquire prefill throughput under TTFT constraints";
"Acquire decode throughput under TPOT constraints") benchmarks an inference
engine in a compute-bound prefill mode and a memory-bandwidth-bound decode mode
but does not define the network.  The layer evaluated here is the standard
pre-norm dense decoder block: RMSNorm, fused QKV projection, rotate-half RoPE,
causal grouped-query attention, output projection with residual, RMSNorm,
SwiGLU MLP with residual.  Everything is evaluated in float64 (``dtype`` may be
set to float32 to show that the oracle's own rounding is far below the parity
tolerance); no intermediate is rounded to bf16.

Layouts (all row-major numpy arrays):
    x        [T, d_model]
    w_qkv    [(Hq + 2*Hkv) * hd, d_model]   rows: q heads, then k heads, then v heads
    w_o      [d_model, Hq * hd]
    w_gate   [d_ff, d_model]      w_up [d_ff, d_model]      w_down [d_model, d_ff]
    g_attn   [d_model]            g_mlp [d_model]
    KV cache [batch, Hkv, len_cap, hd]  (K and V separate)

Storage rounding.  The definition above is exact arithmetic on the given inputs.
The data layout the GPU library is measured with keeps every tensor that crosses
HBM between two operations in bf16 (normalised activations, q, the K/V cache, the
attention output, the residual stream, the SwiGLU output, the layer output).  Passing
``store=<rounding function>`` applies that function at exactly those hand-over
points and nowhere else (no rounding inside a contraction, the softmax or SwiGLU);
``store=None`` (default) is the unrounded definition.  With it the tests can separate
"the kernels compute the right function" (tight, against the rounded variant) from
"bf16 storage costs this much accuracy" (against the exact variant).

Projections.  ``proj=None`` (default) evaluates every projection as the plain product
x @ W^T.  A callable ``proj(x, name, lo, hi)`` replaces it (rows lo..hi of weight ``name``);
oracle/fp8.py provides the FP8 variant.  It changes how the five projections are evaluated
and nothing else.

Parity pins (see tests/test_oracle_layer.py): softmax rows sum to one, decode
step t equals prefill row t, zero-weight and single-token special cases,
rotation invariants of RoPE, permutation invariance over packed requests, a
pure-Python brute force on a tiny shape, and a textbook multi-head attention
for the G = 1 case.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


@dataclass(frozen=True)
class LayerConfig:
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ff: int
    rms_eps: float = 1e-6
    rope_theta: float = 1e4

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def n_qkv(self) -> int:
        return (self.n_q_heads + 2 * self.n_kv_heads) * self.head_dim


@dataclass
class LayerWeights:
    w_qkv: np.ndarray
    w_o: np.ndarray
    w_gate: np.ndarray
    w_up: np.ndarray
    w_down: np.ndarray
    g_attn: np.ndarray
    g_mlp: np.ndarray


def rmsnorm(x: np.ndarray, g: np.ndarray, eps: float) -> np.ndarray:
    """y = x * rsqrt(mean(x^2) + eps) * g, the mean taken over the feature axis."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * g


def rope_angles(pos: np.ndarray, head_dim: int, theta: float) -> np.ndarray:
    """angle[t, i] = pos[t] * theta^(-2 i / head_dim), i < head_dim / 2."""
    i = np.arange(head_dim // 2, dtype=np.float64)
    inv_freq = theta ** (-2.0 * i / head_dim)
    return pos.astype(np.float64)[:, None] * inv_freq[None, :]


def rope(u: np.ndarray, pos: np.ndarray, theta: float) -> np.ndarray:
    """Rotate-half RoPE on u[T, H, hd]: pairs (i, i + hd/2) rotate by angle[t, i]."""
    hd = u.shape[-1]
    half = hd // 2
    ang = rope_angles(pos, hd, theta).astype(u.dtype)
    c = np.cos(ang)[:, None, :]
    s = np.sin(ang)[:, None, :]
    a = u[..., :half]
    b = u[..., half:]
    return np.concatenate([a * c - b * s, b * c + a * s], axis=-1)


def softmax_rows(s: np.ndarray) -> np.ndarray:
    """Row softmax with the row maximum subtracted first."""
    m = np.max(s, axis=-1, keepdims=True)
    e = np.exp(s - m)
    return e / np.sum(e, axis=-1, keepdims=True)


def silu(z: np.ndarray) -> np.ndarray:
    return z / (1.0 + np.exp(-z))


def _attend(q: np.ndarray, k: np.ndarray, v: np.ndarray, q_pos: np.ndarray,
            k_pos: np.ndarray, cfg: LayerConfig, probs_out: list | None) -> np.ndarray:
    """Causal GQA attention of queries q[Tq, Hq, hd] over keys k,v[Tk, Hkv, hd].

    Query t sees key u iff k_pos[u] <= q_pos[t].  Query head h reads KV head
    h // G.  Returns o[Tq, Hq * hd].
    """
    tq = q.shape[0]
    scale = 1.0 / np.sqrt(float(cfg.head_dim))
    visible = k_pos[None, :] <= q_pos[:, None]
    o = np.empty((tq, cfg.n_q_heads, cfg.head_dim), dtype=q.dtype)
    for h in range(cfg.n_q_heads):
        j = h // cfg.group
        s = (q[:, h, :] @ k[:, j, :].T) * scale
        s = np.where(visible, s, -np.inf)
        p = softmax_rows(s)
        if probs_out is not None:
            probs_out.append(p)
        o[:, h, :] = p @ v[:, j, :]
    return o.reshape(tq, cfg.n_q_heads * cfg.head_dim)


def _identity(a: np.ndarray) -> np.ndarray:
    return a


class _ExactProjector:
    """Default projection: x @ W[name][lo:hi]^T in the working precision."""

    def __init__(self, w: LayerWeights, dt):
        self.w, self.dt, self.cast = w, dt, {}

    def __call__(self, x, name, lo=None, hi=None):
        if name not in self.cast:
            self.cast[name] = getattr(self.w, name).astype(self.dt)
        return x @ self.cast[name][lo:hi].T


def _mlp_and_residuals(x_rows: np.ndarray, o_rows: np.ndarray, w: LayerWeights,
                       cfg: LayerConfig, dt, st, pj, stages: dict | None = None) -> np.ndarray:
    h = st(x_rows + pj(o_rows, "w_o"))
    n2 = st(rmsnorm(h, w.g_mlp.astype(dt), cfg.rms_eps))
    a = st(silu(pj(n2, "w_gate")) * pj(n2, "w_up"))
    if stages is not None:
        stages.update(attn_o=o_rows, h=h, n2=n2, act=a)
    return st(h + pj(a, "w_down"))


def prefill_layer(cfg: LayerConfig, w: LayerWeights, x: np.ndarray, cu_seqlens,
                  rows=None, dtype=np.float64, probs_out: list | None = None, store=None, proj=None,
                  stages: dict | None = None):
    """One layer over a packed ragged batch of requests.

    ``cu_seqlens`` has n_req + 1 entries; request r owns rows cu[r]..cu[r+1]-1 at
    positions 0..len_r-1 and attends only within itself (block-diagonal causal).
    ``rows`` (optional, sorted global row indices) restricts the expensive part
    to those query rows: K and V are still produced for every row.

    ``stages`` (optional dict) receives the intermediates of the selected rows: q (after RoPE),
    attn_o, h (residual stream after attention), n2, act (SwiGLU output).

    Returns (out, k, v): out[len(rows) or T, d]; k, v[T, Hkv, hd] (k after RoPE).
    """
    dt = dtype
    st = store or _identity
    x = np.asarray(x, dtype=dt)
    cu = np.asarray(cu_seqlens, dtype=np.int64)
    t_total = x.shape[0]
    assert cu[0] == 0 and cu[-1] == t_total and np.all(np.diff(cu) >= 0)
    hq, hkv, hd = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    req = np.repeat(np.arange(len(cu) - 1), np.diff(cu))
    pos = np.arange(t_total) - cu[req]

    pj = proj or _ExactProjector(w, dt)
    n1 = st(rmsnorm(x, w.g_attn.astype(dt), cfg.rms_eps))
    k = st(rope(pj(n1, "w_qkv", hq * hd, (hq + hkv) * hd).reshape(t_total, hkv, hd), pos, cfg.rope_theta))
    v = st(pj(n1, "w_qkv", (hq + hkv) * hd, (hq + 2 * hkv) * hd).reshape(t_total, hkv, hd))

    sel = np.arange(t_total) if rows is None else np.asarray(rows, dtype=np.int64)
    q = st(rope(pj(n1[sel], "w_qkv", 0, hq * hd).reshape(len(sel), hq, hd), pos[sel], cfg.rope_theta))

    o = np.empty((len(sel), hq * hd), dtype=dt)
    for r in range(len(cu) - 1):
        mine = np.nonzero(req[sel] == r)[0]
        if mine.size == 0:
            continue
        lo, hi = cu[r], cu[r + 1]
        o[mine] = _attend(q[mine], k[lo:hi], v[lo:hi], pos[sel][mine], pos[lo:hi], cfg, probs_out)
    if stages is not None:
        stages["q"] = q
    out = _mlp_and_residuals(x[sel], st(o), w, cfg, dt, st, pj, stages)
    return out, k, v


def decode_layer(cfg: LayerConfig, w: LayerWeights, x: np.ndarray, kv_len,
                 k_cache: np.ndarray, v_cache: np.ndarray, dtype=np.float64,
                 probs_out: list | None = None, store=None, proj=None, stages: dict | None = None) -> np.ndarray:
    """One decode step for a batch of B sequences, one new token each.

    kv_len[b] tokens are already cached for sequence b; the new token has
    position kv_len[b], its K/V are appended IN PLACE at that index, and it
    attends over the kv_len[b] + 1 entries.  Caches are [B, Hkv, len_cap, hd].
    Returns out[B, d].
    """
    dt = dtype
    st = store or _identity
    x = np.asarray(x, dtype=dt)
    kv_len = np.asarray(kv_len, dtype=np.int64)
    b_sz = x.shape[0]
    hq, hkv, hd = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    assert np.all(kv_len < k_cache.shape[2])

    pj = proj or _ExactProjector(w, dt)
    n1 = st(rmsnorm(x, w.g_attn.astype(dt), cfg.rms_eps))
    qkv = pj(n1, "w_qkv")
    q = st(rope(qkv[:, :hq * hd].reshape(b_sz, hq, hd), kv_len, cfg.rope_theta))
    k = st(rope(qkv[:, hq * hd:(hq + hkv) * hd].reshape(b_sz, hkv, hd), kv_len, cfg.rope_theta))
    v = st(qkv[:, (hq + hkv) * hd:].reshape(b_sz, hkv, hd))

    o = np.empty((b_sz, hq * hd), dtype=dt)
    for b in range(b_sz):
        n = int(kv_len[b])
        k_cache[b, :, n, :] = k[b]
        v_cache[b, :, n, :] = v[b]
        keys = np.ascontiguousarray(k_cache[b, :, :n + 1, :].transpose(1, 0, 2)).astype(dt)
        vals = np.ascontiguousarray(v_cache[b, :, :n + 1, :].transpose(1, 0, 2)).astype(dt)
        o[b:b + 1] = _attend(q[b:b + 1], keys, vals, kv_len[b:b + 1], np.arange(n + 1), cfg, probs_out)
    if stages is not None:
        stages["q"] = q
    return _mlp_and_residuals(x, st(o), w, cfg, dt, st, pj, stages)


def extend_layer(cfg: LayerConfig, w: LayerWeights, x: np.ndarray, cu_seqlens, prefix_lens,
                 k_cache: np.ndarray, v_cache: np.ndarray, dtype=np.float64, store=None, proj=None) -> np.ndarray:
    """Chunked prefill: one layer over a packed batch of request CHUNKS.

    Request r already has prefix_lens[r] tokens in cache sequence r; its chunk rows
    cu[r]..cu[r+1]-1 sit at positions prefix_lens[r] + 0, 1, ...  Their K/V are appended
    IN PLACE at those positions and every row attends to all cached positions up to and
    including its own.  With prefix_lens = 0 this is prefill_layer; with chunks of one token
    it is decode_layer.  Caches are [batch, Hkv, len_cap, hd].  Returns out[T, d].
    """
    dt = dtype
    st = store or _identity
    x = np.asarray(x, dtype=dt)
    cu = np.asarray(cu_seqlens, dtype=np.int64)
    pre = np.asarray(prefix_lens, dtype=np.int64)
    t_total = x.shape[0]
    assert cu[0] == 0 and cu[-1] == t_total and np.all(np.diff(cu) >= 0) and len(pre) == len(cu) - 1
    hq, hkv, hd = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    req = np.repeat(np.arange(len(cu) - 1), np.diff(cu))
    pos = np.arange(t_total) - cu[req] + pre[req]
    assert np.all(pos < k_cache.shape[2])

    pj = proj or _ExactProjector(w, dt)
    n1 = st(rmsnorm(x, w.g_attn.astype(dt), cfg.rms_eps))
    qkv = pj(n1, "w_qkv")
    q = st(rope(qkv[:, :hq * hd].reshape(t_total, hq, hd), pos, cfg.rope_theta))
    k = st(rope(qkv[:, hq * hd:(hq + hkv) * hd].reshape(t_total, hkv, hd), pos, cfg.rope_theta))
    v = st(qkv[:, (hq + hkv) * hd:].reshape(t_total, hkv, hd))

    o = np.empty((t_total, hq * hd), dtype=dt)
    for r in range(len(cu) - 1):
        lo, hi = int(cu[r]), int(cu[r + 1])
        if hi == lo:
            continue
        p0, n = int(pre[r]), hi - lo
        k_cache[r, :, p0:p0 + n, :] = k[lo:hi].transpose(1, 0, 2)
        v_cache[r, :, p0:p0 + n, :] = v[lo:hi].transpose(1, 0, 2)
        keys = np.ascontiguousarray(k_cache[r, :, :p0 + n, :].transpose(1, 0, 2)).astype(dt)
        vals = np.ascontiguousarray(v_cache[r, :, :p0 + n, :].transpose(1, 0, 2)).astype(dt)
        o[lo:hi] = _attend(q[lo:hi], keys, vals, pos[lo:hi], np.arange(p0 + n), cfg, None)
    return _mlp_and_residuals(x, st(o), w, cfg, dt, st, pj)


def layer_flops_prefill(cfg: LayerConfig, lens) -> float:
    """Algorithmic flops of one prefill pass (causal half of attention only)."""
    t = float(sum(lens))
    hq, hd, d, f = cfg.n_q_heads, cfg.head_dim, cfg.d_model, cfg.d_ff
    gemm = 2.0 * t * (d * cfg.n_qkv + hq * hd * d + 3.0 * d * f)
    attn = sum(4.0 * hq * hd * (l * (l + 1) / 2.0) for l in lens)
    return gemm + attn
