"""GPU: the single-CTA GEMM and decode-projection kernels, which the library falls back to when clusters of two
cannot be placed (or PD_GEMM_PAIRS=0 / PD_SKINNY_PAIRS=0 is set), checked against the oracle in a fresh process with
the CTA-pair kernels switched off (the switches are read once per process)."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r'''
import sys, numpy as np, torch
sys.path.insert(0, "tests")
import pd_inputs as gen
import paper_2603_04716_b200 as pd
from gpu_util import to_dev, from_dev, empty_bf16, i32_dev, assert_close, DeviceLayer, store_bf16
from oracle import decoder_layer as L, fp8

def gemm_case(m, n, k):
    a = gen.normal_bf16(1, 40, (m, k), 1.0, sub=m); b = gen.normal_bf16(1, 41, (n, k), 0.05, sub=n)
    dc = empty_bf16(m, n); err = torch.zeros(1, dtype=torch.int32, device="cuda")
    pd.pd_gemm_bf16(to_dev(a), to_dev(b), dc, m, n, k, err_word=err); torch.cuda.synchronize()
    assert int(err.item()) == 0
    ref = (a @ b.T).astype(np.float64); got = from_dev(dc).astype(np.float64)
    assert np.all(np.abs(got - ref) <= 1e-2 * np.sqrt(k) * 0.05 + 8e-3 * np.abs(ref)), (m, n, k)

def gemm_fp8_case(m, n, k):
    a = gen.normal_bf16(2, 40, (m, k), 1.0, sub=m); b = gen.normal_bf16(2, 41, (n, k), 0.02, sub=n)
    def q(x):
        codes = torch.zeros(x.shape, dtype=torch.uint8, device="cuda"); sc = torch.zeros(x.shape[0], dtype=torch.float32, device="cuda")
        pd.pd_quantize_fp8_rows(to_dev(x), x.shape[0], x.shape[1], codes, sc); return codes, sc
    (qa, sa), (qb, sb) = q(a), q(b)
    dc = empty_bf16(m, n)
    pd.pd_gemm_fp8(qa, sa, qb, sb, dc, m, n, k); torch.cuda.synchronize()
    ref = fp8.gemm_fp8(*fp8.quantize_rows(a), *fp8.quantize_rows(b)); got = from_dev(dc).astype(np.float64)
    assert np.all(np.abs(got - ref) <= 2.0 ** -8 * np.abs(ref) + 1e-5 * np.sqrt(k) * 0.02), (m, n, k)

def decode_case(b, fp8_on):
    shape = dict(d_model=512, n_q_heads=8, n_kv_heads=2, head_dim=64, d_ff=1536); cap = 48
    w = gen.layer_weights(**shape, seed=3)
    ocfg, ow = L.LayerConfig(**shape), L.LayerWeights(**w)
    dl = DeviceLayer(pd, pd.LayerConfig(**shape, max_pos=64, fp8_projections=fp8_on), w, 0, b, cap)
    k0, v0 = gen.kv_cache(31, b, 2, cap, 64); k, v, cache = dl.make_cache(b, cap, k0, v0)
    x = gen.activations(31, b, 512, sub=b); kv_len = [int(t) for t in gen.uniform_lengths(31, b, 0, cap - 1, sub=b)]
    dout = empty_bf16(b, 512)
    pd.pd_decode_layer(dl.layer, to_dev(x), dout, i32_dev(kv_len), b, max(kv_len) + 1, cache, dl.ws, dl.ws_bytes)
    pd.pd_layer_check(dl.layer)
    kw = dict(store=store_bf16, proj=fp8.Fp8Projector(ow)) if fp8_on else {}
    ref = L.decode_layer(ocfg, ow, x, kv_len, k0.astype(np.float64), v0.astype(np.float64), **kw)
    assert_close(from_dev(dout), ref, f"decode B={b} fp8={fp8_on}")

gemm_case(1000, 6144, 4096); gemm_case(333, 4096, 14336); gemm_fp8_case(300, 3072, 512); gemm_fp8_case(1000, 6144, 4096)
decode_case(100, False); decode_case(256, False); decode_case(200, True)
print("single-CTA paths ok")
'''


def test_single_cta_kernels_match_oracle(pdlib):
    env = dict(os.environ, PD_GEMM_PAIRS="0", PD_SKINNY_PAIRS="0")
    res = subprocess.run([sys.executable, "-c", CHILD], cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)
    assert res.returncode == 0 and "single-CTA paths ok" in res.stdout, res.stdout[-2000:] + res.stderr[-4000:]
