"""Pins for the whole-model-step oracle (embedding, layers, final norm, LM head, greedy
sampling): special cases with a closed form, a scalar brute force, and the invariant
that ties decode mode to prefill mode."""
import math

import numpy as np

import pd_inputs as gen
from oracle import decoder_layer as L
from oracle import model_step as M

MICRO = L.LayerConfig(d_model=8, n_q_heads=2, n_kv_heads=1, head_dim=4, d_ff=12, rms_eps=1e-6, rope_theta=1e4)
SMALL = L.LayerConfig(d_model=64, n_q_heads=4, n_kv_heads=2, head_dim=16, d_ff=96)


def make_model(cfg, vocab, n_layers, seed=0, std=0.02):
    head = gen.model_head_weights(vocab, cfg.d_model, seed, std)
    layers = [L.LayerWeights(**gen.layer_weights(cfg.d_model, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim,
                                                 cfg.d_ff, seed, li, std)) for li in range(n_layers)]
    return M.ModelWeights(layers=layers, **head)


def empty_caches(cfg, n_layers, batch, cap):
    shape = (batch, cfg.n_kv_heads, cap, cfg.head_dim)
    return [np.zeros(shape) for _ in range(n_layers)], [np.zeros(shape) for _ in range(n_layers)]


def test_permutation_head_on_zero_layer_model():
    """E = c I, W_lm = a permutation matrix, no layers: RMSNorm keeps the one-hot direction,
    so the next token is perm(token).  A transposed head would give the inverse permutation,
    a wrong gather a different row."""
    d = 16
    cfg = L.LayerConfig(d_model=d, n_q_heads=2, n_kv_heads=1, head_dim=8, d_ff=16)
    perm = np.array([(5 * i + 3) % d for i in range(d)])      # not an involution
    assert not np.array_equal(perm[perm], np.arange(d))
    lm = np.zeros((d, d))
    lm[perm, np.arange(d)] = 1.0                                # logits[perm[j]] = n[j]
    mw = M.ModelWeights(embed=3.0 * np.eye(d), g_final=np.ones(d), lm_head=lm, layers=[])
    tokens = np.arange(d)
    nxt, logits = M.model_decode_step(cfg, mw, tokens, np.zeros(d, dtype=np.int64), [], [])
    assert np.array_equal(nxt, perm)
    # the one-hot row of scale c has mean square c^2/d: the normalised entry is sqrt(d) (up to eps)
    assert np.allclose(logits.max(axis=1), math.sqrt(d), rtol=1e-6)
    # prefill takes the LAST token of each request
    cu = np.array([0, 3, 3, 7, 16])
    nxt_p, logits_p = M.model_prefill(cfg, mw, tokens, cu)
    assert np.array_equal(nxt_p, [perm[2], -1, perm[6], perm[15]])
    assert np.all(logits_p[1] == 0.0)


def test_head_matches_scalar_brute_force():
    cfg = MICRO
    vocab = 11
    mw = make_model(cfg, vocab, 0, seed=3, std=0.5)
    h = gen.activations(4, 5, cfg.d_model).astype(np.float64)
    got = M.head_logits(h, mw, cfg.rms_eps)
    for r in range(h.shape[0]):
        ms = sum(float(v) ** 2 for v in h[r]) / cfg.d_model
        n = [float(h[r, i]) / math.sqrt(ms + cfg.rms_eps) * float(mw.g_final[i]) for i in range(cfg.d_model)]
        for v in range(vocab):
            want = sum(n[i] * float(mw.lm_head[v, i]) for i in range(cfg.d_model))
            assert abs(got[r, v] - want) < 1e-12
    best = [max(range(vocab), key=lambda v: (got[r, v], -v)) for r in range(h.shape[0])]
    assert np.array_equal(M.greedy(got), best)


def test_greedy_takes_lowest_index_among_ties():
    logits = np.array([[1.0, 3.0, 3.0, -1.0], [2.0, 2.0, 2.0, 2.0], [-5.0, -7.0, -5.0, -9.0]])
    assert np.array_equal(M.greedy(logits), [1, 0, 0])
    assert M.greedy(np.zeros((0, 4))).shape == (0,)


def test_zero_weight_layers_reduce_to_the_head():
    """With all projection weights zero every layer is the identity (both residual branches
    vanish), so the model is embedding -> final norm -> head."""
    cfg = SMALL
    vocab = 50
    mw = make_model(cfg, vocab, 2, seed=1, std=0.3)
    for lw in mw.layers:
        for name in ("w_qkv", "w_o", "w_gate", "w_up", "w_down"):
            getattr(lw, name)[...] = 0.0
    tokens = gen.token_ids(0, 9, vocab)
    cu = np.array([0, 4, 9])
    nxt, logits = M.model_prefill(cfg, mw, tokens, cu)
    e = mw.embed[tokens[[3, 8]]].astype(np.float64)
    n = e / np.sqrt((e * e).mean(axis=1, keepdims=True) + cfg.rms_eps) * mw.g_final
    want = n @ mw.lm_head.T.astype(np.float64)
    assert np.allclose(logits, want, atol=1e-12)
    assert np.array_equal(nxt, want.argmax(axis=1))


def test_decode_step_equals_prefill_of_the_extended_prompt():
    """Prefill n tokens (filling the caches), then decode token n: the logits equal those of
    the last row of a prefill over n + 1 tokens, in every request of a ragged batch."""
    cfg = SMALL
    vocab, n_layers = 97, 3
    mw = make_model(cfg, vocab, n_layers, seed=2, std=0.08)
    lens = [5, 1, 9]
    cu = np.concatenate([[0], np.cumsum(lens)])
    full = gen.token_ids(5, int(cu[-1]) + len(lens), vocab)
    prompts = [full[cu[r] + r: cu[r + 1] + r + 1] for r in range(len(lens))]    # len_r + 1 tokens each
    kc, vc = empty_caches(cfg, n_layers, len(lens), 16)
    head_tokens = np.concatenate([p[:-1] for p in prompts])
    M.model_prefill(cfg, mw, head_tokens, cu, kc, vc)
    newest = np.array([p[-1] for p in prompts])
    nxt_d, logits_d = M.model_decode_step(cfg, mw, newest, np.array(lens), kc, vc)
    cu1 = np.concatenate([[0], np.cumsum([n + 1 for n in lens])])
    nxt_p, logits_p = M.model_prefill(cfg, mw, np.concatenate(prompts), cu1)
    assert np.allclose(logits_d, logits_p, atol=1e-10)
    assert np.array_equal(nxt_d, nxt_p)
    # and the decode step appended exactly one K/V row per sequence and layer
    for li in range(n_layers):
        for r, n in enumerate(lens):
            assert np.any(kc[li][r, :, n, :] != 0.0) and np.all(kc[li][r, :, n + 1:, :] == 0.0)


def test_store_rounding_only_touches_the_normalised_rows():
    """With a rounding function the logits move by at most the rounding of n times the head's
    row norms; without layers nothing else is rounded."""
    cfg = SMALL
    mw = make_model(cfg, 40, 0, seed=7, std=0.1)
    tokens = gen.token_ids(1, 6, 40)
    _, exact = M.model_decode_step(cfg, mw, tokens, np.zeros(6, dtype=np.int64), [], [])
    _, rounded = M.model_decode_step(cfg, mw, tokens, np.zeros(6, dtype=np.int64), [], [],
                                     store=lambda a: gen.bf16_round(a).astype(np.float64))
    bound = 2.0 ** -8 * np.abs(mw.lm_head).sum(axis=1).max() * 4.0     # |n| stays below 4 here
    diff = np.abs(exact - rounded).max()
    assert 0.0 < diff < bound
