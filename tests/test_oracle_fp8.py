"""Pins of the FP8 (E4M3) oracle: the published format table, exhaustive round trips, ties and
saturation, a brute-force nearest-value search, an independent library conversion, quantisation
error bounds and GEMMs with exactly representable operands."""
import numpy as np
import pytest

import pd_inputs as gen
from conftest import read_golden
from oracle import decoder_layer as L
from oracle import fp8

FINITE = np.array([c for c in range(256) if (c & 0x7F) != 0x7F], dtype=np.uint8)


def test_format_table_constants():
    g = read_golden("e4m3_format.txt")
    dec = fp8.e4m3_decode(np.arange(256))
    assert dec[int(g["max_normal_code"])] == g["max_normal_value"] == fp8.E4M3_MAX
    assert dec[int(g["min_normal_code"])] == 2.0 ** g["min_normal_log2"]
    assert dec[int(g["max_subnormal_code"])] == g["max_subnormal_value"]
    assert dec[int(g["min_subnormal_code"])] == 2.0 ** g["min_subnormal_log2"]
    assert dec[int(g["one_code"])] == 1.0
    assert np.isnan(dec[int(g["nan_code"])]) and np.isnan(dec[int(g["nan_code"]) | 0x80])
    assert dec[0] == 0.0 and dec[0x80] == 0.0 and np.signbit(dec[0x80])
    assert np.all(np.isfinite(dec[FINITE]))                       # no infinities anywhere
    assert np.nanmax(np.abs(dec)) == g["max_normal_value"]
    # the value formula with the table's bias, written out for one normal and one subnormal code
    assert dec[0b0_1010_101] == 2.0 ** (0b1010 - g["exponent_bias"]) * (1 + 5 / 8)
    assert dec[0b1_0000_011] == -(3 / 8) * 2.0 ** (1 - g["exponent_bias"])


def test_codes_are_monotone_and_round_trip():
    pos = fp8.e4m3_decode(np.arange(0, 127))
    assert np.all(np.diff(pos) > 0)                               # code order = value order
    assert np.array_equal(fp8.e4m3_encode(fp8.e4m3_decode(FINITE)), FINITE)
    assert fp8.e4m3_encode(np.array([np.nan]))[0] == 0x7F


def test_ties_go_to_even_and_saturation():
    vals = fp8.e4m3_decode(np.arange(0, 127))
    mid = (vals[:-1] + vals[1:]) / 2                               # exact midpoints of neighbouring codes
    got = fp8.e4m3_encode(mid)
    want = np.array([c if c % 2 == 0 else c + 1 for c in range(126)], dtype=np.uint8)
    assert np.array_equal(got, want)
    assert np.array_equal(fp8.e4m3_encode(-mid), want | 0x80)
    eps = np.nextafter(mid, np.inf) - mid
    assert np.array_equal(fp8.e4m3_encode(mid + eps), np.arange(1, 127, dtype=np.uint8))
    assert np.array_equal(fp8.e4m3_encode(mid - eps), np.arange(0, 126, dtype=np.uint8))
    big = np.array([448.0, 449.0, 464.0, 480.0, 1e4, 3e38, np.inf])
    assert np.all(fp8.e4m3_encode(big) == 0x7E) and np.all(fp8.e4m3_encode(-big) == 0xFE)


def test_encode_matches_brute_force_nearest():
    rng = np.random.Generator(np.random.Philox(key=5))
    x = np.concatenate([rng.standard_normal(20000) * s for s in (1e-3, 0.02, 1.0, 30.0, 300.0)]).astype(np.float32)
    table = fp8.e4m3_decode(np.arange(0, 127))
    a = np.minimum(np.abs(x.astype(np.float64)), 448.0)
    d = np.abs(a[:, None] - table[None, :])
    best = d.min(axis=1)
    cand = d == best[:, None]                                       # one or (on a tie) two neighbouring codes
    idx = np.arange(127)
    even_first = np.where(cand & (idx % 2 == 0)[None, :], 0, 1) + np.where(cand, 0, 10)
    want = np.argmin(even_first, axis=1).astype(np.uint8) | np.where(np.signbit(x), 0x80, 0).astype(np.uint8)
    assert np.array_equal(fp8.e4m3_encode(x), want)


def test_encode_matches_library_conversion():
    torch = pytest.importorskip("torch")
    if not hasattr(torch, "float8_e4m3fn"):
        pytest.skip("torch build without float8_e4m3fn")
    rng = np.random.Generator(np.random.Philox(key=6))
    x = np.concatenate([rng.standard_normal(50000) * s for s in (1e-3, 0.05, 1.0, 100.0)]).astype(np.float32)
    x = x[np.abs(x) <= 448.0]                                       # the library does not saturate beyond the range
    lib = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(fp8.e4m3_encode(x), lib)
    codes = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).to(torch.float32).numpy()
    ours = fp8.e4m3_decode(np.arange(256))
    assert np.array_equal(np.isnan(codes), np.isnan(ours))
    assert np.array_equal(codes[FINITE].astype(np.float64), ours[FINITE])


def test_quantize_rows_bounds_and_special_rows():
    x = gen.normal_bf16(3, gen.S_X, (37, 200), 1.0)
    x[5] = 0.0
    x[6, :] = 0.0
    x[6, 17] = -3.5
    q, s = fp8.quantize_rows(x)
    assert q.dtype == np.uint8 and s.dtype == np.float32 and q.shape == x.shape and s.shape == (37,)
    amax = np.abs(x).max(axis=1)
    assert np.array_equal(s[amax > 0], (amax[amax > 0] / np.float32(448.0)).astype(np.float32))
    assert s[5] == 1.0 and np.all(q[5] == 0)
    assert q[6, 17] == 0xFE and np.all(np.delete(q[6], 17) == 0)    # the row maximum maps to +-448 exactly
    assert np.all((q & 0x7F).max(axis=1)[amax > 0] == 0x7E)
    back = fp8.dequantize_rows(q, s)
    # normal range: half a unit in the last of 3 mantissa bits (2^-4 relative); below it half a subnormal step
    bound = np.maximum(np.abs(x) * 2.0 ** -4, 0.5 * 2.0 ** -9 * s[:, None]) * (1 + 1e-6)
    assert np.all(np.abs(back - x) <= bound)


def test_gemm_with_exactly_representable_operands_is_the_plain_product():
    rng = np.random.Generator(np.random.Philox(key=7))
    # small integers times a power of two per row: every element and 448/amax scaling is exact in E4M3
    a = rng.integers(-7, 8, size=(9, 64)).astype(np.float64)
    b = rng.integers(-7, 8, size=(11, 64)).astype(np.float64)
    a[:, 0] = 7.0
    b[:, 0] = -7.0                                                 # every row has amax 7 -> scale 7/448 = 2^-6
    a *= np.exp2(rng.integers(-3, 4, size=(9, 1)).astype(np.float64))
    b *= np.exp2(rng.integers(-3, 4, size=(11, 1)).astype(np.float64))
    qa, sa = fp8.quantize_rows(a)
    qb, sb = fp8.quantize_rows(b)
    assert np.array_equal(fp8.dequantize_rows(qa, sa), a) and np.array_equal(fp8.dequantize_rows(qb, sb), b)
    assert np.array_equal(fp8.gemm_fp8(qa, sa, qb, sb), a @ b.T)


def test_gemm_error_against_unquantised_product():
    a = gen.normal_bf16(1, gen.S_X, (64, 512), 1.0).astype(np.float64)
    b = gen.normal_bf16(1, gen.S_WQKV, (96, 512), 0.02).astype(np.float64)
    y = fp8.gemm_fp8(*fp8.quantize_rows(a), *fp8.quantize_rows(b))
    ref = a @ b.T
    rel = np.linalg.norm(y - ref) / np.linalg.norm(ref)
    # two operands with independent relative rounding errors of rms about 2^-4 / sqrt(3) / sqrt(2) each
    assert 0.01 < rel < 0.06
    # transposed roles give the transposed result (scales commute)
    assert np.allclose(fp8.gemm_fp8(*fp8.quantize_rows(b), *fp8.quantize_rows(a)), y.T, rtol=0, atol=1e-12)


# ------------------------------------------------------------------- block-wise scales
def test_blockwise_reduces_to_per_row_scheme():
    """One K block and one output row per weight block: the block-wise scheme IS the per-row scheme."""
    a = gen.normal_bf16(3, gen.S_X, (7, 96), 1.0).astype(np.float64)
    b = gen.normal_bf16(3, gen.S_WQKV, (5, 96), 0.02).astype(np.float64)
    qa, sa = fp8.quantize_groups(a, group=96)
    qb, sb = fp8.quantize_blocks(b, block_n=1, block_k=96)
    qa_r, sa_r = fp8.quantize_rows(a)
    qb_r, sb_r = fp8.quantize_rows(b)
    assert np.array_equal(qa, qa_r) and np.array_equal(sa[:, 0], sa_r)
    assert np.array_equal(qb, qb_r) and np.array_equal(sb[:, 0], sb_r)
    assert np.array_equal(fp8.gemm_fp8_blockwise(qa, sa, qb, sb, block_n=1, block_k=96), fp8.gemm_fp8(qa_r, sa_r, qb_r, sb_r))


def test_blockwise_quantisers_by_element_loops():
    """Scales and codes against loops over single elements (ragged edge blocks included)."""
    rng = np.random.Generator(np.random.Philox(key=21))
    x = (rng.standard_normal((5, 21)) * np.exp2(rng.integers(-4, 5, size=(5, 21)))).astype(np.float32)
    x[2, 8:16] = 0.0                                               # an all-zero group
    w = (rng.standard_normal((11, 21)) * 0.05).astype(np.float32)
    qx, sx = fp8.quantize_groups(x, group=8)
    qw, sw = fp8.quantize_blocks(w, block_n=4, block_k=8)
    assert sx.shape == (5, 3) and sw.shape == (3, 3) and sx.dtype == np.float32 and sw.dtype == np.float32
    for t in range(5):
        for g in range(3):
            seg = x[t, g * 8:(g + 1) * 8]
            amax = np.float32(np.abs(seg).max())
            want = np.float32(amax / np.float32(448.0)) if amax > 0 else np.float32(1.0)
            assert sx[t, g] == want
            for i, v in enumerate(seg):
                assert qx[t, g * 8 + i] == fp8.e4m3_encode(np.float32(v / want))
    for i in range(3):
        for j in range(3):
            blk = w[i * 4:(i + 1) * 4, j * 8:(j + 1) * 8]
            amax = np.float32(np.abs(blk).max())
            assert sw[i, j] == np.float32(amax / np.float32(448.0))
            assert np.array_equal(qw[i * 4:(i + 1) * 4, j * 8:(j + 1) * 8], fp8.e4m3_encode((blk / sw[i, j]).astype(np.float32)))
    assert sx[2, 1] == 1.0 and np.all(qx[2, 8:16] == 0)


def test_blockwise_gemm_by_element_loops():
    rng = np.random.Generator(np.random.Philox(key=22))
    x = rng.standard_normal((4, 20)).astype(np.float32)
    w = rng.standard_normal((7, 20)).astype(np.float32)
    qx, sx = fp8.quantize_groups(x, group=8)
    qw, sw = fp8.quantize_blocks(w, block_n=3, block_k=8)
    dx, dw = fp8.e4m3_decode(qx), fp8.e4m3_decode(qw)
    want = np.zeros((4, 7))
    for t in range(4):
        for n in range(7):
            for k in range(20):
                want[t, n] += dx[t, k] * dw[n, k] * float(sx[t, k // 8]) * float(sw[n // 3, k // 8])
    got = fp8.gemm_fp8_blockwise(qx, sx, qw, sw, block_n=3, block_k=8)
    assert np.allclose(got, want, rtol=1e-13, atol=1e-13)


def test_blockwise_exact_for_blockwise_representable_operands():
    """Small integers times one power of two per block: codes, scales and the product are exact."""
    rng = np.random.Generator(np.random.Philox(key=23))
    a = rng.integers(-7, 8, size=(6, 256)).astype(np.float64)
    b = rng.integers(-7, 8, size=(256, 256)).astype(np.float64)
    a[:, 0::128] = 7.0                                             # every 1 x 128 group has amax 7
    b[0::128, 0::128] = -7.0                                       # every 128 x 128 block has amax 7
    a = a.reshape(6, 2, 128) * np.exp2(rng.integers(-3, 4, size=(6, 2, 1)).astype(np.float64))
    a = a.reshape(6, 256)
    pw = np.exp2(rng.integers(-3, 4, size=(2, 2)).astype(np.float64))
    b = b * np.kron(pw, np.ones((128, 128)))
    qa, sa = fp8.quantize_groups(a)
    qb, sb = fp8.quantize_blocks(b)
    assert np.array_equal(fp8.e4m3_decode(qa) * np.repeat(sa.astype(np.float64), 128, axis=1), a)
    assert np.array_equal(fp8.e4m3_decode(qb) * np.kron(sb.astype(np.float64), np.ones((128, 128))), b)
    assert np.array_equal(fp8.gemm_fp8_blockwise(qa, sa, qb, sb), a @ b.T)


def test_blockwise_scale_invariance_and_error_bound():
    a = gen.normal_bf16(4, gen.S_X, (48, 512), 1.0).astype(np.float64)
    b = gen.normal_bf16(4, gen.S_WQKV, (256, 512), 0.02).astype(np.float64)
    qa, sa = fp8.quantize_groups(a)
    qb, sb = fp8.quantize_blocks(b)
    y = fp8.gemm_fp8_blockwise(qa, sa, qb, sb)
    ref = a @ b.T
    rel = np.linalg.norm(y - ref) / np.linalg.norm(ref)
    assert 0.01 < rel < 0.06                                       # same error class as the per-row scheme
    # multiplying one weight block and one activation group by powers of two changes only their scales
    b2 = b.copy(); b2[128:256, 256:384] *= 8.0
    a2 = a.copy(); a2[:, 128:256] *= 0.25
    qb2, sb2 = fp8.quantize_blocks(b2)
    qa2, sa2 = fp8.quantize_groups(a2)
    assert np.array_equal(qb2, qb) and np.array_equal(qa2, qa)
    assert sb2[1, 2] == sb[1, 2] * 8 and np.array_equal(sa2[:, 1], sa[:, 1] * np.float32(0.25))
    # an outlier confined to one block leaves the codes of every other block untouched (what block scales are for)
    b3 = b.copy(); b3[5, 7] = 3.0
    qb3, sb3 = fp8.quantize_blocks(b3)
    keep = np.ones_like(b, dtype=bool); keep[0:128, 0:128] = False
    assert np.array_equal(qb3[keep], qb[keep]) and sb3[0, 0] > sb[0, 0] and np.array_equal(sb3.ravel()[1:], sb.ravel()[1:])


CFG = L.LayerConfig(d_model=64, n_q_heads=4, n_kv_heads=2, head_dim=16, d_ff=96)


def _weights(seed=0):
    return L.LayerWeights(**gen.layer_weights(64, 4, 2, 16, 96, seed=seed))


def test_projection_hook_default_is_the_plain_layer():
    w = _weights()
    x = gen.activations(0, 12, 64)
    ref, k0, v0 = L.prefill_layer(CFG, w, x, [0, 5, 12])
    got, k1, v1 = L.prefill_layer(CFG, w, x, [0, 5, 12], proj=L._ExactProjector(w, np.float64))
    assert np.array_equal(ref, got) and np.array_equal(k0, k1) and np.array_equal(v0, v1)


def test_fp8_layer_is_close_to_exact_layer_and_decode_matches_prefill_row():
    w = _weights(1)
    pj = fp8.Fp8Projector(w)
    x = gen.activations(1, 10, 64)
    exact, _, _ = L.prefill_layer(CFG, w, x, [0, 10])
    out, k, v = L.prefill_layer(CFG, w, x, [0, 10], proj=pj)
    # the residual stream passes through untouched, so the error is measured on the layer's update
    rel = np.linalg.norm(out - exact) / np.linalg.norm(exact - x)
    assert 5e-3 < rel < 0.1
    # per-token quantisation keeps rows independent: decode of token t on the prefix cache = prefill row t
    t = 7
    kc = np.zeros((1, 2, 16, 16)); vc = np.zeros((1, 2, 16, 16))
    kc[0, :, :t] = k[:t].transpose(1, 0, 2); vc[0, :, :t] = v[:t].transpose(1, 0, 2)
    dec = L.decode_layer(CFG, w, x[t:t + 1], [t], kc, vc, proj=pj)
    assert np.allclose(dec[0], out[t], rtol=0, atol=1e-10)
    # row subset = full
    sub, _, _ = L.prefill_layer(CFG, w, x, [0, 10], rows=[0, 3, 9], proj=pj)
    assert np.allclose(sub, out[[0, 3, 9]], rtol=0, atol=1e-12)
