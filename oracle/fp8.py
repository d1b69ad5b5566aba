"""CPU oracle for the FP8 (E4M3) projections.

TEST INFRASTRUCTURE ONLY: shares no code with the CUDA path and is imported only by
tests, the smoke check and the benchmark's CPU-baseline leg.

The paper validates its TTFT model on an FP8 checkpoint (the Qwen3-235B-A22B-FP8
deployment of the Figure 1 experiment) but does not describe the number format or the
scaling scheme.  The reading taken here is the common "dynamic W8A8" one:

  * number format: OCP 8-bit floating point E4M3 (1 sign, 4 exponent bits with bias 7,
    3 mantissa bits; no infinities; S.1111.111 is NaN; largest finite value 448;
    subnormals m/8 * 2^-6), which is what the tensor cores consume;
  * a weight matrix W[N, K] is quantised once per output channel (row): scale_n =
    max_k |W[n, k]| / 448, code = RNE_E4M3(W[n, k] / scale_n);
  * an activation matrix X[T, K] is quantised per token (row) the same way, every time
    it is fed to a projection;
  * the projection is Y[t, n] = (sum_k dec(qx[t, k]) * dec(qw[n, k])) * sx[t] * sw[n].

Scale and quotient are evaluated in IEEE float32 (one division each, round to nearest),
so that the integer codes are decided in the same precision as on the GPU; an all-zero
row gets scale 1.  Rounding to E4M3 is round-to-nearest-even with saturation to +-448.

A second scaling scheme, one scale per 128 x 128 weight block and per token and 128 channels
(quantize_groups, quantize_blocks, gemm_fp8_blockwise), is described where it is defined.

Pins: tests/test_oracle_fp8.py (format constants of the published table, exhaustive
decode/encode round trip, ties and saturation, brute-force nearest-value search, an
independent library conversion, error bounds, exactly representable GEMM; for the
block-wise scheme: reduction to the per-row scheme when K is one block and every output
row its own block, element-by-element loops on small cases, exactness for operands that
are representable block by block, scale invariance under per-block powers of two, and
the error bound of the scheme against the unquantised product).
"""
from __future__ import annotations

import numpy as np

E4M3_MAX = 448.0
E4M3_NAN = 0x7F


def e4m3_decode(codes) -> np.ndarray:
    """Value of each 8-bit code as float64 (NaN for S.1111.111)."""
    c = np.asarray(codes, dtype=np.uint8).astype(np.int64)
    sign = np.where(c & 0x80, -1.0, 1.0)
    e = (c >> 3) & 0xF
    m = (c & 0x7).astype(np.float64)
    sub = m / 8.0 * 2.0 ** -6
    nrm = (1.0 + m / 8.0) * np.exp2((e - 7).astype(np.float64))
    val = np.where(e == 0, sub, nrm)
    val = np.where((e == 15) & ((c & 0x7) == 7), np.nan, val)
    return sign * val


def e4m3_encode(x) -> np.ndarray:
    """Round float values to E4M3 codes: nearest, ties to even mantissa, finite overflow saturates to 448."""
    x = np.asarray(x, dtype=np.float64)
    a = np.abs(x)
    nan = np.isnan(a)
    a = np.where(nan, 0.0, a)
    a = np.minimum(a, E4M3_MAX)  # satfinite: everything beyond the largest finite value becomes it
    # binade of a (clamped to the subnormal binade), quantum = 2^(e - 3)
    with np.errstate(divide="ignore"):
        e = np.floor(np.log2(np.where(a > 0, a, 1.0)))
    e = np.clip(e, -6, 8)
    # guard against log2 rounding at binade edges
    e = np.where(a < np.exp2(e), e - 1, e)
    e = np.where(a >= np.exp2(e + 1), e + 1, e)
    e = np.clip(e, -6, 8)
    q = np.exp2(e - 3)
    steps = np.rint(a / q)            # numpy rint rounds halves to even; a / q is exact (power-of-two scaling)
    v = steps * q                     # may land on the next binade's first value, which is representable
    v = np.minimum(v, E4M3_MAX)
    # value -> code
    with np.errstate(divide="ignore"):
        ev = np.floor(np.log2(np.where(v > 0, v, 1.0)))
    ev = np.where(v < np.exp2(ev), ev - 1, ev)
    ev = np.where(v >= np.exp2(ev + 1), ev + 1, ev)
    normal = v >= 2.0 ** -6
    exp_field = np.where(normal, ev + 7, 0).astype(np.int64)
    man_field = np.where(normal, np.rint((v / np.exp2(ev) - 1.0) * 8.0), np.rint(v * 2.0 ** 9)).astype(np.int64)
    code = (exp_field << 3) | man_field
    code = np.where(np.signbit(x), code | 0x80, code)
    code = np.where(nan, E4M3_NAN, code)
    return code.astype(np.uint8)


def quantize_rows(x):
    """Per-row dynamic quantisation of x[T, K] -> (codes uint8 [T, K], scale float32 [T])."""
    x32 = np.ascontiguousarray(x, dtype=np.float32)
    amax = np.max(np.abs(x32), axis=-1) if x32.shape[-1] else np.zeros(x32.shape[:-1], np.float32)
    scale = (amax / np.float32(E4M3_MAX)).astype(np.float32)
    scale = np.where(amax > 0, scale, np.float32(1.0)).astype(np.float32)
    y = (x32 / scale[..., None]).astype(np.float32)
    return e4m3_encode(y), scale


def dequantize_rows(codes, scale) -> np.ndarray:
    return e4m3_decode(codes) * np.asarray(scale, dtype=np.float64)[..., None]


def gemm_fp8(qx, sx, qw, sw) -> np.ndarray:
    """Y[T, N] = (dec(qx) @ dec(qw)^T) * sx[:, None] * sw[None, :] in float64."""
    acc = e4m3_decode(qx) @ e4m3_decode(qw).T
    return acc * np.asarray(sx, np.float64)[:, None] * np.asarray(sw, np.float64)[None, :]


# ----------------------------------------------------------------------------- block-wise scales
# Reading for checkpoints that carry one scale per block instead of per channel (the public FP8 releases of
# the model families the paper deploys state `weight_block_size = [128, 128]`): a weight matrix W[N, K] has one
# fp32 scale per 128 x 128 block, an activation matrix X[T, K] one per token and group of 128 consecutive
# channels, and the products of the codes are summed per 128-wide K block and scaled block by block:
#   Y[t, n] = sum_kb ( sum_{k in kb} dec(qx[t, k]) dec(qw[n, k]) ) * sx[t, kb] * sw[n // 128, kb].
# Scales and quotients are evaluated in float32 like the per-row ones; an all-zero block gets scale 1; N and K
# need not be multiples of 128 (edge blocks are smaller).
BLOCK = 128


def quantize_groups(x, group: int = BLOCK):
    """Per-row, per-K-group dynamic quantisation of x[T, K] -> (codes uint8 [T, K], scale float32 [T, ceil(K / group)])."""
    x32 = np.ascontiguousarray(x, dtype=np.float32)
    t, k = x32.shape
    kb = (k + group - 1) // group
    codes = np.zeros((t, k), dtype=np.uint8)
    scale = np.ones((t, kb), dtype=np.float32)
    for b in range(kb):
        blk = x32[:, b * group:(b + 1) * group]
        amax = np.max(np.abs(blk), axis=1)
        sc = (amax / np.float32(E4M3_MAX)).astype(np.float32)
        sc = np.where(amax > 0, sc, np.float32(1.0)).astype(np.float32)
        codes[:, b * group:(b + 1) * group] = e4m3_encode((blk / sc[:, None]).astype(np.float32))
        scale[:, b] = sc
    return codes, scale


def quantize_blocks(w, block_n: int = BLOCK, block_k: int = BLOCK):
    """Per-block quantisation of w[N, K] -> (codes uint8 [N, K], scale float32 [ceil(N / block_n), ceil(K / block_k)])."""
    w32 = np.ascontiguousarray(w, dtype=np.float32)
    n, k = w32.shape
    nb, kb = (n + block_n - 1) // block_n, (k + block_k - 1) // block_k
    codes = np.zeros((n, k), dtype=np.uint8)
    scale = np.ones((nb, kb), dtype=np.float32)
    for i in range(nb):
        for j in range(kb):
            blk = w32[i * block_n:(i + 1) * block_n, j * block_k:(j + 1) * block_k]
            amax = np.float32(np.max(np.abs(blk))) if blk.size else np.float32(0)
            sc = np.float32(amax / np.float32(E4M3_MAX)) if amax > 0 else np.float32(1.0)
            codes[i * block_n:(i + 1) * block_n, j * block_k:(j + 1) * block_k] = e4m3_encode((blk / sc).astype(np.float32))
            scale[i, j] = sc
    return codes, scale


def gemm_fp8_blockwise(qx, sx, qw, sw, block_n: int = BLOCK, block_k: int = BLOCK) -> np.ndarray:
    """Y[T, N] with one partial product per K block, each scaled by the token's group scale and the weight block's scale."""
    dx, dw = e4m3_decode(qx), e4m3_decode(qw)
    t, k = dx.shape
    n = dw.shape[0]
    sx = np.asarray(sx, np.float64)
    sw = np.asarray(sw, np.float64)
    y = np.zeros((t, n), dtype=np.float64)
    row_block = np.arange(n) // block_n
    for j in range((k + block_k - 1) // block_k):
        part = dx[:, j * block_k:(j + 1) * block_k] @ dw[:, j * block_k:(j + 1) * block_k].T
        y += part * sx[:, j][:, None] * sw[row_block, j][None, :]
    return y


class Fp8Projector:
    """Projection hook for oracle.decoder_layer: x @ W[name][lo:hi]^T through the FP8 path.

    The weights are quantised once (per output channel) when the object is built; the
    activation rows are quantised at every call.
    """

    def __init__(self, weights):
        self.q = {}
        for name in ("w_qkv", "w_o", "w_gate", "w_up", "w_down"):
            self.q[name] = quantize_rows(getattr(weights, name))

    def __call__(self, x, name, lo=None, hi=None):
        qw, sw = self.q[name]
        qx, sx = quantize_rows(x)
        return gemm_fp8(qx, sx, qw[lo:hi], sw[lo:hi])
