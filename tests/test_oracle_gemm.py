"""Pins for the oracle's fp64 dequantized GEMM reference (right-hand side of Eq. 8) and for
function preservation X W = (X P)(P^T W)."""
import numpy as np
import torch

from oracle import pq_oracle as O
from paper_2605_09503_b200 import inputs

E2M1 = np.array([0, .5, 1, 1.5, 2, 3, 4, 6, -0.0, -.5, -1, -1.5, -2, -3, -4, -6])


def decode(codes, sf):
    """Independent numpy decode: nibble -> value table, scale byte -> torch float8 cast."""
    lo, hi = codes & 15, codes >> 4
    nib = np.stack([lo, hi], axis=-1).reshape(codes.shape[0], -1)
    scale = torch.from_numpy(sf.copy()).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    return E2M1[nib] * np.repeat(scale, 16, axis=1)


def test_exact_integer_case():
    """codes in {0, +-1, +-2}, unit scales, K = 64: every product sum is a small integer."""
    rng = np.random.default_rng(0)
    M, N, K = 8, 12, 64
    pick = np.array([0, 2, 4, 10, 12], dtype=np.uint8)          # 0, 1, 2, -1, -2
    xn, wn = pick[rng.integers(0, 5, (M, K))], pick[rng.integers(0, 5, (N, K))]
    pack = lambda n: (n[:, 0::2] | (n[:, 1::2] << 4)).astype(np.uint8)
    sfx = np.full((M, K // 16), 0x38, dtype=np.uint8)
    sfw = np.full((N, K // 16), 0x38, dtype=np.uint8)
    Y = O.gemm_ref(pack(xn), sfx, 1.0, pack(wn), sfw, 1.0)
    want = E2M1[xn] @ E2M1[wn].T
    assert np.array_equal(Y, want) and np.abs(Y).max() <= 256
    # linear in the tensor scales
    assert np.array_equal(O.gemm_ref(pack(xn), sfx, 2.0, pack(wn), sfw, 0.25), want * 0.5)


def test_matches_numpy_matmul_of_independent_decode():
    cfg = inputs.CONFIGS["tiny"]
    x = inputs.bits(inputs.activations(cfg, 0, 1000, rows=40))[:, :128].copy()
    w = inputs.bits(inputs.weight(cfg, 0, N=24))[:, :128].copy()
    tsx = O.tensor_scale(O.calib_stats(x)[1])
    tsw = O.tensor_scale(O.calib_stats(w)[1])
    xq, sfx = O.quant_nvfp4(x, tsx)
    wq, sfw = O.quant_nvfp4(w, tsw)
    Y = O.gemm_ref(xq, sfx, tsx, wq, sfw, tsw)
    want = np.float64(np.float32(tsx)) * np.float64(np.float32(tsw)) * (decode(xq, sfx) @ decode(wq, sfw).T)
    assert np.allclose(Y, want, rtol=1e-12, atol=1e-300)
    # sampled entry point agrees with the full one
    ms = np.array([0, 5, 39, 17]); ns = np.array([23, 0, 11, 11])
    assert np.array_equal(O.gemm_ref_sampled(xq, sfx, tsx, wq, sfw, tsw, ms, ns), Y[ms, ns])
    # dequant_nvfp4 agrees with the independent decode
    assert np.allclose(O.dequant_nvfp4(xq, sfx, tsx), decode(xq, sfx) * np.float32(tsx), rtol=1e-6)
    # quantization is an approximation of the bf16 product (Eq. 8, "approx"): loose check
    exact = O.gemm_bf16_ref(x, w)
    assert np.linalg.norm(Y - exact) / np.linalg.norm(exact) < 0.2


def test_function_preservation_unquantized():
    """X W = X P P^T W exactly when nothing is quantized (Eq. 8, first equality)."""
    rng = np.random.default_rng(3)
    x = inputs.bits(torch.randn(6, 32, generator=torch.Generator().manual_seed(1)).to(torch.bfloat16))
    w = inputs.bits(torch.randn(5, 32, generator=torch.Generator().manual_seed(2)).to(torch.bfloat16))
    perm = rng.permutation(32).astype(np.int32)
    a, b = O.gemm_bf16_ref(x, w), O.gemm_bf16_ref(x, w, perm)
    assert np.allclose(a, b, rtol=1e-13, atol=1e-13)
    xf, wf = O.bf16_to_f32(x).astype(np.float64), O.bf16_to_f32(w).astype(np.float64)
    assert np.allclose(a, xf @ wf.T, rtol=1e-13, atol=1e-13)
