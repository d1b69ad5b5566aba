"""CPU oracle for a whole-model step: token embedding, the decoder layers, final
RMSNorm, LM-head projection and greedy sampling.

TEST INFRASTRUCTURE ONLY.  Slow, plain and independent of the CUDA path (it shares no
code with it and must never be imported by it); only tests, the smoke check and the
benchmark's CPU-baseline leg call it.

The paper's TTFT and TPOT are engine-level quantities ("Acquire prefill throughput
under TTFT constraints": time until the first output token; "Acquire decode throughput
under TPOT constraints": time per output token), so one measured step ends with a token,
not with a hidden state.  The paper does not define the network; the step evaluated
here is the standard one around the dense decoder layers of ``decoder_layer``:

    x      = E[token]                                  embedding rows, E [V, d]
    h      = layer_{L-1}( ... layer_0(x))              prefill / decode mode
    n      = RMSNorm(h_last) * g_final                 last row of each request (prefill),
                                                       every row (decode)
    logits = n @ W_lm^T                                W_lm [V, d]
    next   = argmax_v logits[v]                        lowest index among equal maxima

Everything is float64 unless ``dtype`` says otherwise.  ``store`` has the meaning it has
in ``decoder_layer``: a rounding function applied where a tensor crosses HBM between two
operations (here additionally: the final normalised rows); logits are never rounded.

Parity pins (tests/test_oracle_model.py): a permutation LM head on a zero-layer model
(catches a transposed head and a wrong gather), pure-Python brute force of the head on
tiny shapes, decode step t equal to the last prefill row of the sequence extended by one
token, zero-weight layers reducing the model to its head's closed form, the tie rule.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

from .decoder_layer import LayerConfig, LayerWeights, _identity, decode_layer, prefill_layer, rmsnorm


@dataclass
class ModelWeights:
    embed: np.ndarray      # [V, d]
    g_final: np.ndarray    # [d]
    lm_head: np.ndarray    # [V, d]
    layers: list = field(default_factory=list)   # LayerWeights, first layer first


def embed_tokens(tokens, embed: np.ndarray, dtype=np.float64) -> np.ndarray:
    """x[i, :] = E[tokens[i], :]."""
    tok = np.asarray(tokens, dtype=np.int64)
    assert tok.ndim == 1 and (tok.size == 0 or (tok.min() >= 0 and tok.max() < embed.shape[0]))
    return np.asarray(embed, dtype=dtype)[tok]


def head_logits(h: np.ndarray, mw: ModelWeights, eps: float, dtype=np.float64, store=None) -> np.ndarray:
    """Final RMSNorm followed by the LM-head projection: [rows, d] -> [rows, V]."""
    st = store or _identity
    n = st(rmsnorm(np.asarray(h, dtype=dtype), mw.g_final.astype(dtype), eps))
    return n @ mw.lm_head.astype(dtype).T


def greedy(logits: np.ndarray) -> np.ndarray:
    """Greedy sampling: the index of the largest logit of each row (the lowest such index)."""
    if logits.shape[0] == 0:
        return np.zeros(0, dtype=np.int64)
    return np.argmax(logits, axis=1).astype(np.int64)


def model_prefill(cfg: LayerConfig, mw: ModelWeights, tokens, cu_seqlens, k_caches=None, v_caches=None,
                  dtype=np.float64, store=None):
    """Prefill of a packed ragged batch of prompts up to the first output token.

    ``tokens`` [T] int; request r owns tokens cu[r]..cu[r+1]-1.  If caches are given
    (one [batch, Hkv, len_cap, hd] array per layer, K and V), the K/V of request r are
    written to cache sequence r at positions 0..len_r-1.  Returns (next, logits):
    next[r] = greedy token after the prompt (-1 for an empty request), logits [n_req, V]
    (rows of empty requests are zero).
    """
    cu = np.asarray(cu_seqlens, dtype=np.int64)
    n_req = len(cu) - 1
    x = embed_tokens(tokens, mw.embed, dtype)
    for li, lw in enumerate(mw.layers):
        x, k, v = prefill_layer(cfg, lw, x, cu, dtype=dtype, store=store)
        if k_caches is not None:
            for r in range(n_req):
                lo, hi = int(cu[r]), int(cu[r + 1])
                k_caches[li][r, :, :hi - lo, :] = k[lo:hi].transpose(1, 0, 2)
                v_caches[li][r, :, :hi - lo, :] = v[lo:hi].transpose(1, 0, 2)
    vocab = mw.lm_head.shape[0]
    logits = np.zeros((n_req, vocab), dtype=dtype)
    nxt = np.full(n_req, -1, dtype=np.int64)
    have = np.nonzero(np.diff(cu) > 0)[0]
    if have.size:
        last = cu[have + 1] - 1
        logits[have] = head_logits(x[last], mw, cfg.rms_eps, dtype, store)
        nxt[have] = greedy(logits[have])
    return nxt, logits


def model_decode_step(cfg: LayerConfig, mw: ModelWeights, tokens, kv_len, k_caches, v_caches,
                      dtype=np.float64, store=None):
    """One decode step of B sequences: tokens[b] is the newest token of sequence b, whose
    kv_len[b] earlier tokens are cached; its K/V are appended in place in every layer.
    Returns (next [B], logits [B, V])."""
    x = embed_tokens(tokens, mw.embed, dtype)
    for li, lw in enumerate(mw.layers):
        x = decode_layer(cfg, lw, x, kv_len, k_caches[li], v_caches[li], dtype=dtype, store=store)
    logits = head_logits(x, mw, cfg.rms_eps, dtype, store)
    return greedy(logits), logits
