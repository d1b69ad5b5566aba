"""Seeded synthetic inputs shared by the tests, the benchmark and the smoke check.

Only data generation and the bf16 storage format live here: none of the
decoder layer's or the allocation model's arithmetic.  Streams are numpy Philox
counters keyed by (seed, stream id), so a tensor's values do not depend on
which other tensors were drawn before it.
"""
from __future__ import annotations

import numpy as np

# stream ids (tensor kinds)
S_WQKV, S_WO, S_WGATE, S_WUP, S_WDOWN, S_GATTN, S_GMLP = range(7)
S_X, S_KCACHE, S_VCACHE, S_XSTEP, S_LENGTHS, S_ARRIVALS, S_SERVICE, S_ROWS = range(16, 24)
S_EMBED, S_LMHEAD, S_GFINAL, S_TOKENS = range(32, 36)


def _rng(seed: int, stream: int, sub: int = 0) -> np.random.Generator:
    key = np.array([np.uint64(seed), (np.uint64(stream) << np.uint64(32)) | np.uint64(sub)], dtype=np.uint64)
    return np.random.Generator(np.random.Philox(key=key))


def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit pattern (uint16), round to nearest even."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def from_bf16_bits(b: np.ndarray) -> np.ndarray:
    """bf16 bit pattern (uint16) -> float32 (exact)."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_round(a: np.ndarray) -> np.ndarray:
    """Round float values to the nearest bf16-representable float32."""
    return from_bf16_bits(to_bf16_bits(a))


def normal_bf16(seed: int, stream: int, shape, std: float = 1.0, mean: float = 0.0, sub: int = 0) -> np.ndarray:
    """N(mean, std) values rounded to bf16, returned as float32."""
    r = _rng(seed, stream, sub)
    a = r.standard_normal(size=shape, dtype=np.float32)
    if std != 1.0:
        a *= np.float32(std)
    if mean != 0.0:
        a += np.float32(mean)
    return bf16_round(a)


def layer_weights(d_model: int, n_q_heads: int, n_kv_heads: int, head_dim: int, d_ff: int,
                  seed: int = 0, layer: int = 0, std: float = 0.02) -> dict:
    """Random weights of one layer: matrices ~N(0, std), gains 1 + N(0, std); bf16 values as float32."""
    n_qkv = (n_q_heads + 2 * n_kv_heads) * head_dim
    return {
        "w_qkv": normal_bf16(seed, S_WQKV, (n_qkv, d_model), std, sub=layer),
        "w_o": normal_bf16(seed, S_WO, (d_model, n_q_heads * head_dim), std, sub=layer),
        "w_gate": normal_bf16(seed, S_WGATE, (d_ff, d_model), std, sub=layer),
        "w_up": normal_bf16(seed, S_WUP, (d_ff, d_model), std, sub=layer),
        "w_down": normal_bf16(seed, S_WDOWN, (d_model, d_ff), std, sub=layer),
        "g_attn": normal_bf16(seed, S_GATTN, (d_model,), std, mean=1.0, sub=layer),
        "g_mlp": normal_bf16(seed, S_GMLP, (d_model,), std, mean=1.0, sub=layer),
    }


def model_head_weights(vocab: int, d_model: int, seed: int = 0, std: float = 0.02) -> dict:
    """Embedding table ~N(0, 1) (the scale the layer inputs are drawn with), LM head ~N(0, std),
    final gain 1 + N(0, std); bf16 values as float32."""
    return {
        "embed": normal_bf16(seed, S_EMBED, (vocab, d_model), 1.0),
        "g_final": normal_bf16(seed, S_GFINAL, (d_model,), std, mean=1.0),
        "lm_head": normal_bf16(seed, S_LMHEAD, (vocab, d_model), std),
    }


def token_ids(seed: int, n: int, vocab: int, sub: int = 0) -> np.ndarray:
    """n token ids uniform in [0, vocab)."""
    return _rng(seed, S_TOKENS, sub).integers(0, vocab, size=n, dtype=np.int64).astype(np.int32)


def activations(seed: int, n_tokens: int, d_model: int, sub: int = 0, stream: int = S_X) -> np.ndarray:
    """Token embeddings ~N(0, 1), bf16 values as float32."""
    return normal_bf16(seed, stream, (n_tokens, d_model), 1.0, sub=sub)


def kv_cache(seed: int, batch: int, n_kv_heads: int, len_cap: int, head_dim: int, sub: int = 0):
    """Synthetic K and V caches ~N(0, 1) (the scale of projected, normalised activations)."""
    k = normal_bf16(seed, S_KCACHE, (batch, n_kv_heads, len_cap, head_dim), 1.0, sub=sub)
    v = normal_bf16(seed, S_VCACHE, (batch, n_kv_heads, len_cap, head_dim), 1.0, sub=sub)
    return k, v


def lognormal_lengths(seed: int, n: int, median: float, sigma: float, lo: int, hi: int) -> np.ndarray:
    """Request lengths: round(exp(N(ln median, sigma^2))) clipped to [lo, hi]."""
    z = _rng(seed, S_LENGTHS).standard_normal(n)
    return np.clip(np.rint(np.exp(np.log(median) + sigma * z)), lo, hi).astype(np.int32)


def uniform_lengths(seed: int, n: int, lo: int, hi: int, sub: int = 0) -> np.ndarray:
    return _rng(seed, S_LENGTHS, sub).integers(lo, hi + 1, size=n).astype(np.int32)


def exponential_gaps(seed: int, n: int, rate: float, stream: int = S_ARRIVALS) -> np.ndarray:
    """Inter-arrival gaps of a Poisson process of the given rate."""
    return _rng(seed, stream).exponential(1.0 / rate, size=n)


def sample_rows(seed: int, cu_seqlens, n_random: int = 48, tile: int = 128) -> np.ndarray:
    """Row subset for sampled parity: first/last row of every request, rows around
    multiples of `tile`, and seeded random rows.  Sorted, unique."""
    cu = np.asarray(cu_seqlens, dtype=np.int64)
    total = int(cu[-1])
    picks = set()
    for r in range(len(cu) - 1):
        lo, hi = int(cu[r]), int(cu[r + 1])
        if hi <= lo:
            continue
        for c in (lo, lo + 1, hi - 2, hi - 1):
            if lo <= c < hi:
                picks.add(c)
        for m in range(lo + tile, hi, max(tile, (hi - lo) // 8 // tile * tile or tile)):
            for c in (m - 1, m, m + 1):
                if lo <= c < hi:
                    picks.add(c)
    rnd = _rng(seed, S_ROWS).integers(0, total, size=n_random)
    picks.update(int(v) for v in rnd)
    return np.array(sorted(picks), dtype=np.int64)
