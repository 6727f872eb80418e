"""The tcgen05 weight-streaming GEMM against the oracle's matmul, through the C ABI."""
import numpy as np
import pytest
import torch

import synth
from gpu_common import engine, requires_gpu


def _case(M, N, K, seed):
    x = synth.normal_bf16(seed, 100, (M, K), 1.0)
    w = synth.normal_bf16(seed, 101, (N, K), 0.05)
    return x, w


@requires_gpu
@pytest.mark.parametrize("M,N,K,splits", [
    (32, 768, 256, 1),        # tiny-model QKV
    (32, 768, 256, 2),
    (16, 256, 688, 1),        # K tail: 688 = 10 * 64 + 48
    (16, 256, 688, 3),
    (64, 1376, 256, 0),       # N tail: 1376 = 10 * 128 + 96; 64-row tile
    (100, 2048, 256, 0),      # ragged rows inside a 128-row tile
    (128, 512, 1024, 4),
    (300, 640, 512, 0),       # many rows, odd number of weight tiles (5): single-CTA tiles of 128 rows, last ragged
    (300, 768, 512, 0),       # many rows, even number of weight tiles: CTA pairs, two 256-row tiles, second ragged
    (700, 1024, 688, 2),      # CTA pairs with a K split and a K tail; three row tiles, last ragged (188 rows)
    (129, 256, 64, 1),        # CTA pair, one k-block, one row beyond the first half of the second CTA's rows
    (1, 128, 64, 1),          # smallest
    (48, 2048, 2048, 0),
])
def test_gemm_matches_oracle(M, N, K, splits):
    E = engine()
    xb, wb = _case(M, N, K, seed=M + N + K)
    x = E.bits_to_device(xb, "cuda")
    w = E.bits_to_device(wb, "cuda")
    out = E.debug_gemm(x, w, splits).cpu().numpy().astype(np.float64)
    xf = synth.bf16_bits_to_f32(xb).astype(np.float64)
    wf = synth.bf16_bits_to_f32(wb).astype(np.float64)
    ref = xf @ wf.T
    scale = (np.abs(xf) @ np.abs(wf).T).max()
    err = np.abs(out - ref).max()
    assert err <= 2e-6 * scale, (err, scale)          # fp32 accumulation of exact bf16 products
    out2 = E.debug_gemm(x, w, splits).cpu().numpy().astype(np.float64)
    assert np.array_equal(out, out2)                   # fixed-order split reduction: bitwise repeatable


@requires_gpu
def test_gemm_garbage_rows_do_not_leak():
    """Rows of x beyond M are never read into the result: a 32-row tile fed 5 rows."""
    E = engine()
    xb, wb = _case(32, 256, 256, seed=9)
    big = E.bits_to_device(xb, "cuda")
    big[5:] = float("nan")
    w = E.bits_to_device(wb, "cuda")
    out = E.debug_gemm(big[:5], w, 1).cpu().numpy()
    ref = synth.bf16_bits_to_f32(xb[:5]).astype(np.float64) @ synth.bf16_bits_to_f32(wb).astype(np.float64).T
    assert np.isfinite(out).all() and np.abs(out - ref).max() < 1e-3
