"""Pins of the oracle's PermuQuant-H producer (App. D: Hadamard transform, then the reordering, then the
quantizer): hand-computed small transforms, an independent library matrix, the defining property
H H^T = K I in exact integer arithmetic, Paley's construction rebuilt from Euler's criterion, norm
preservation, the stated order of the additions, and "permuted output = gather of the unpermuted one"."""
import numpy as np
import pytest
import scipy.linalg

from oracle import pq_oracle as O


def bf(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return (a.view(np.uint32) >> 16).astype(np.uint16).reshape(a.shape)


def transform(x):
    """fp32 transformed rows of bf16-representable x (no reordering, no quantizer)."""
    return O.hadamard_quant_nvfp4(bf(x), 1.0, quantize=False)[3]


def matrix(K):
    """The transform's matrix recovered from unit vectors, divided by its scale: entries must be +-1."""
    M = transform(np.eye(K, dtype=np.float32)).astype(np.float64)       # row i = e_i H
    s = np.float32(1.0 / np.sqrt(np.float64(K)))
    assert np.array_equal(np.abs(M), np.full((K, K), np.float64(s)))
    return np.rint(M / np.float64(s)).astype(np.int64)


def test_hand_computed_width_16():
    # rows of the order-16 Sylvester matrix: H[i][j] = (-1)^popcount(i & j); scale 1/4 is exact
    x = np.zeros((3, 16), dtype=np.float32)
    x[0, :4] = [1, 2, 3, 4]
    x[1, 0] = 1
    x[2, 5] = 8
    y = transform(x)
    # (1,2,3,4,0,...) H: for output j only bits 0,1 of j matter: [10, -2, -4, 0] repeated 4 times, / 4
    assert np.array_equal(y[0], np.tile(np.array([10, -2, -4, 0], dtype=np.float32) / 4, 4))
    assert np.array_equal(y[1], np.full(16, 0.25, dtype=np.float32))
    signs = np.array([(-1) ** bin(5 & j).count("1") for j in range(16)], dtype=np.float32)
    assert np.array_equal(y[2], 2 * signs)


@pytest.mark.parametrize("K", [16, 64, 256])
def test_power_of_two_widths_are_the_sylvester_matrix_of_a_library(K):
    assert np.array_equal(matrix(K), scipy.linalg.hadamard(K).astype(np.int64))


def paley12():
    """Paley's first construction for q = 11 written independently: quadratic character by Euler's
    criterion r^((q-1)/2) mod q, H = I + [[0, 1^T], [-1, Q]], Q[i][j] = chi(i - j)."""
    chi = lambda r: 0 if r % 11 == 0 else (1 if pow(r % 11, 5, 11) == 1 else -1)
    S = np.zeros((12, 12), dtype=np.int64)
    S[0, 1:] = 1
    S[1:, 0] = -1
    for i in range(11):
        for j in range(11):
            S[1 + i, 1 + j] = chi(i - j)
    assert np.array_equal(S.T, -S)
    return np.eye(12, dtype=np.int64) + S


@pytest.mark.parametrize("K", [48, 192, 768])
def test_widths_12_times_a_power_of_two(K):
    H = matrix(K)
    assert np.array_equal(H @ H.T, K * np.eye(K, dtype=np.int64))          # the defining property, exactly
    H12 = paley12()
    assert np.array_equal(H12 @ H12.T, 12 * np.eye(12, dtype=np.int64))
    # Kronecker structure: channel i = a * (K/12) + b, entry = H12[a][a'] * Sylvester[b][b']
    assert np.array_equal(H, np.kron(H12, scipy.linalg.hadamard(K // 12).astype(np.int64)))


def test_widths_the_transform_is_not_defined_for_are_refused():
    with pytest.raises(ValueError):
        transform(np.zeros((1, 80), dtype=np.float32))                      # 5 * 16
    with pytest.raises(ValueError):
        transform(np.zeros((1, 96 * 3), dtype=np.float32))                  # 9 * 32


def test_norm_is_preserved_and_float64_agrees():
    rng = np.random.default_rng(2)
    for K in (512, 3072):
        xb = bf(rng.standard_normal((4, K)) * np.exp(1.5 * rng.standard_normal(K)))
        x = O.bf16_to_f32(xb).astype(np.float64)
        y = O.hadamard_quant_nvfp4(xb, 1.0, quantize=False)[3].astype(np.float64)
        H = matrix(K).astype(np.float64) if K == 512 else np.kron(paley12(), scipy.linalg.hadamard(256)).astype(np.float64)
        ref = x @ H / np.sqrt(K)
        assert np.allclose(y, ref, rtol=0, atol=2e-6 * np.abs(x).sum(axis=1, keepdims=True) / np.sqrt(K))
        assert np.allclose((y ** 2).sum(axis=1), (x ** 2).sum(axis=1), rtol=1e-5)
        # applying the transpose brings the row back: x H H^T / K = x
        assert np.allclose(ref @ H.T / np.sqrt(K), x, atol=1e-9 * np.abs(x).max())


def test_stated_order_of_the_additions():
    """Values spread over many binades so that the order of the fp32 additions shows: segments are
    combined first (terms added one by one in ascending segment), then butterflies with strides
    1, 2, 4, ..., then one multiplication by fl(1 / sqrt(K))."""
    rng = np.random.default_rng(7)
    K, seg = 192, 16
    xb = bf(rng.standard_normal((1, K)) * np.exp(4 * rng.standard_normal(K)))
    x = O.bf16_to_f32(xb)[0]
    H12 = paley12()
    f = np.float32
    u = np.zeros(K, dtype=np.float32)
    for b in range(seg):
        for ap in range(12):
            acc = f(H12[0, ap]) * x[b]
            for a in range(1, 12):
                acc = f(acc + x[a * seg + b]) if H12[a, ap] > 0 else f(acc - x[a * seg + b])
            u[ap * seg + b] = acc
    for a in range(12):
        h = 1
        while h < seg:
            for i in range(seg):
                if not i & h:
                    p, q = u[a * seg + i], u[a * seg + i + h]
                    u[a * seg + i], u[a * seg + i + h] = f(p + q), f(p - q)
            h *= 2
    want = (u * f(1.0 / np.sqrt(np.float64(K)))).astype(np.float32)
    got = O.hadamard_quant_nvfp4(xb, 1.0, quantize=False)[3][0]
    assert np.array_equal(got, want)
    # butterflies before the segment combination give different bits on this row: the order is observable
    v = x.copy()
    for a in range(12):
        h = 1
        while h < seg:
            for i in range(seg):
                if not i & h:
                    p, q = v[a * seg + i], v[a * seg + i + h]
                    v[a * seg + i], v[a * seg + i + h] = f(p + q), f(p - q)
            h *= 2
    w = np.zeros(K, dtype=np.float32)
    for b in range(seg):
        for ap in range(12):
            acc = f(H12[0, ap]) * v[b]
            for a in range(1, 12):
                acc = f(acc + v[a * seg + b]) if H12[a, ap] > 0 else f(acc - v[a * seg + b])
            w[ap * seg + b] = acc
    assert not np.array_equal((w * f(1.0 / np.sqrt(np.float64(K)))).astype(np.float32), want)


def test_reordered_output_is_a_gather_and_the_quantizer_sees_fp32():
    rng = np.random.default_rng(4)
    K = 768
    xb = bf(rng.standard_normal((6, K)) * np.exp(rng.standard_normal(K)))
    perm = rng.permutation(K).astype(np.int32)
    ts = 0.02
    c0, s0, y0, f0 = O.hadamard_quant_nvfp4(xb, ts)
    ci, si, yi, fi = O.hadamard_quant_nvfp4(xb, ts, perm=np.arange(K, dtype=np.int32))
    assert all(np.array_equal(a, b) for a, b in ((c0, ci), (s0, si), (y0, yi), (f0, fi)))       # identity order
    cp, sp, yp, fp = O.hadamard_quant_nvfp4(xb, ts, perm=perm)
    assert np.array_equal(fp, f0[:, perm]) and np.array_equal(yp, y0[:, perm])
    # bf16 output = the fp32 values rounded to nearest even
    u = f0.view(np.uint32)
    assert np.array_equal(y0, ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16))
    # codes: the plain quantizer on the fp32 values.  Where the transformed values happen to be bf16-exact the
    # existing quantizer on the bf16 tensor must give the same codes; construct such a case: +-1 inputs, K = 256
    # -> outputs are integers / 16, |value| <= 16, exact in bf16 when the integer has <= 8 significant bits
    xs = bf(np.where(rng.random((4, 256)) < 0.5, -1.0, 1.0))
    c, s, y, f = O.hadamard_quant_nvfp4(xs, 0.01)
    assert np.array_equal(O.bf16_to_f32(y), f)
    wc, ws = O.quant_nvfp4(y, 0.01)
    assert np.array_equal(c, wc) and np.array_equal(s, ws)
    # and in general the dequantized codes stay within the largest half-gap of the E2M1 grid (one unit of the group scale) of the fp32 values
    dq = O.dequant_nvfp4(cp, sp, ts).astype(np.float64)
    d = O.dequant_nvfp4(np.full_like(cp, 0x22), sp, ts).astype(np.float64)
    unsat = np.abs(fp) <= 6.0 * d
    assert np.all(np.abs(dq - fp)[unsat] <= d[unsat] * 1.001 + 1e-7)
