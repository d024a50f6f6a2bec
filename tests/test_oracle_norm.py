"""Pins of the oracle's fused normalization + reordering + NVFP4 quantization (App. C with the quantizer of
Eq. 8 attached): closed forms, a float64 restatement, and the invariants the absorbed permutation must keep."""
import numpy as np

from oracle import pq_oracle as O


def bf(a):
    """float array -> bf16 bit patterns (values chosen exactly representable, or truncated)."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    return (a.view(np.uint32) >> 16).astype(np.uint16).reshape(a.shape)


def test_rmsnorm_of_a_constant_row_is_the_weight():
    """x = 2 everywhere, eps = 0: mean(x^2) = 4, inv = 0.5, y = weight exactly; the codes are those of the weight."""
    K = 512
    w = (np.arange(K) % 13 - 6).astype(np.float32) * 0.5            # bf16-representable weights
    x = bf(np.full((3, K), 2.0))
    codes, sf, y = O.norm_quant_nvfp4(x, 0, w, None, 0.0, 0.01)
    want_c, want_s = O.quant_nvfp4(bf(np.tile(w, (3, 1))), 0.01)
    assert np.array_equal(y, bf(np.tile(w, (3, 1))))
    assert np.array_equal(codes, want_c) and np.array_equal(sf, want_s)


def test_adaptive_layernorm_of_an_alternating_row():
    """x = +-3: mu = 0, var = 9, normalized +-1, y = +-(1 + s) + b: small exact numbers."""
    K = 256
    x = np.where(np.arange(K) % 2 == 0, 3.0, -3.0)[None].astype(np.float32)
    s = (np.arange(K) % 4).astype(np.float32) * 0.25                 # 0, .25, .5, .75
    b = ((np.arange(K) % 3) - 1).astype(np.float32) * 0.5            # -.5, 0, .5
    want = np.where(np.arange(K) % 2 == 0, 1.0, -1.0) * (1.0 + s) + b
    codes, sf, y = O.norm_quant_nvfp4(bf(x), 1, s, b, 0.0, 0.004)
    assert np.array_equal(y, bf(want[None]))
    wc, ws = O.quant_nvfp4(bf(want[None]), 0.004)
    assert np.array_equal(codes, wc) and np.array_equal(sf, ws)


def test_against_a_float64_restatement():
    rng = np.random.default_rng(3)
    K = 768
    xb = bf(rng.standard_normal((9, K)) * np.exp(rng.standard_normal(K)) + 0.3)
    x = O.bf16_to_f32(xb).astype(np.float64)
    a = rng.standard_normal(K).astype(np.float32) * 0.3
    b = rng.standard_normal(K).astype(np.float32)
    eps = 1e-6
    rms = x / np.sqrt((x ** 2).mean(axis=1, keepdims=True) + eps) * a
    mu = x.mean(axis=1, keepdims=True)
    ln = (x - mu) / np.sqrt(((x - mu) ** 2).mean(axis=1, keepdims=True) + eps) * (1.0 + a) + b
    for kind, ref in ((0, rms), (1, ln)):
        codes, sf, y = O.norm_quant_nvfp4(xb, kind, a, b, eps, 0.01)
        got = O.bf16_to_f32(y).astype(np.float64)
        assert np.all(np.abs(got - ref) <= 2.0 ** -8 * np.abs(ref) + 1e-5)          # bf16 rounding of the output
        # the codes are the plain quantizer applied to the fp32 result: dequantized they stay within one
        # code step of it (step <= d = sf * ts, largest half-gap of E2M1 is one unit)
        dq = O.dequant_nvfp4(codes, sf, 0.01).astype(np.float64)
        d = O.dequant_nvfp4(np.full_like(codes, 0x22), sf, 0.01).astype(np.float64)   # code 2 = 1.0 -> d itself
        unsat = np.abs(ref) <= 6.0 * d
        assert np.all(np.abs(dq - ref)[unsat] <= d[unsat] * 1.001 + 1e-6)


def test_permutation_is_a_gather_of_the_unpermuted_result():
    rng = np.random.default_rng(5)
    K = 512
    xb = bf(rng.standard_normal((5, K)) * 3)
    a = rng.standard_normal(K).astype(np.float32)
    b = rng.standard_normal(K).astype(np.float32)
    perm = rng.permutation(K).astype(np.int32)
    for kind in (0, 1):
        c0, s0, y0 = O.norm_quant_nvfp4(xb, kind, a, b, 1e-5, 0.02)
        ci, si, yi = O.norm_quant_nvfp4(xb, kind, a, b, 1e-5, 0.02, perm=np.arange(K, dtype=np.int32))
        assert np.array_equal(c0, ci) and np.array_equal(s0, si) and np.array_equal(y0, yi)     # identity order
        # the parameters travel with their channels (they are indexed by output position)
        cp, sp, yp = O.norm_quant_nvfp4(xb, kind, a[perm], b[perm], 1e-5, 0.02, perm=perm)
        assert np.array_equal(yp, y0[:, perm])               # same statistics, channels read through the order
        # and parameters left in place act on whatever channel lands at their position
        cq, sq, yq = O.norm_quant_nvfp4(xb, kind, np.ones(K, np.float32) if kind == 0 else np.zeros(K, np.float32),
                                        np.zeros(K, np.float32), 1e-5, 0.02, perm=perm)
        c1, s1, y1 = O.norm_quant_nvfp4(xb, kind, np.ones(K, np.float32) if kind == 0 else np.zeros(K, np.float32),
                                        np.zeros(K, np.float32), 1e-5, 0.02)
        assert np.array_equal(yq, y1[:, perm])


def test_lane_order_of_the_row_sums():
    """A row built so that the order of the fp32 additions shows: lane l owns the elements i with
    (i // 8) % 32 == l, adds them in ascending i, then the lanes meet in a 16-8-4-2-1 butterfly."""
    rng = np.random.default_rng(8)
    K = 1024
    xf = O.bf16_to_f32(bf((rng.standard_normal((1, K)) * np.exp(3 * rng.standard_normal(K))).astype(np.float32)))
    x = xf[0]
    p = np.zeros(32, dtype=np.float32)
    for i in range(K):
        l = (i // 8) % 32
        p[l] = np.float32(np.float64(p[l]) + np.float64(x[i]) * np.float64(x[i]))      # fmaf
    for m in (16, 8, 4, 2, 1):
        p = np.array([np.float32(p[l] + p[l ^ m]) for l in range(32)], dtype=np.float32)
    ms = np.float32(p[0] / np.float32(K))
    inv = np.float32(np.float32(1.0) / np.sqrt(np.float32(ms + np.float32(0.0))))
    want = (x * inv).astype(np.float32)                      # weight 1
    _, _, y = O.norm_quant_nvfp4(bf(xf), 0, np.ones(K, dtype=np.float32), None, 0.0, 0.01)
    assert np.array_equal(y[0], (want.view(np.uint32) + 0x7FFF + ((want.view(np.uint32) >> 16) & 1) >> 16).astype(np.uint16))
    flat = np.float32(0.0)
    for i in range(K):
        flat = np.float32(np.float64(flat) + np.float64(x[i]) * np.float64(x[i]))
    assert flat != p[0]                                      # a plain left-to-right sum differs on this row
