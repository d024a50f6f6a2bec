"""Pins for the oracle's group quantizers (NVFP4 and the integer quantizer of Eq. 1-2), the
per-group error of Eq. 3 and the deterministic bound of Eq. 4."""
import os

import numpy as np
import pytest
import torch

from oracle import pq_oracle as O
from paper_2605_09503_b200 import inputs

GOLD = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def bf(values):
    """python floats -> bf16 bit patterns [1, n] (rounded by torch, not by the oracle)."""
    t = torch.tensor([values], dtype=torch.float32).to(torch.bfloat16)
    return inputs.bits(t)


def unpack(codes):
    lo, hi = codes & 15, codes >> 4
    return np.stack([lo, hi], axis=-1).reshape(codes.shape[0], -1)


def _rows(name):
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                yield [part.strip() for part in line.split("|")]


def test_nvfp4_golden_groups():
    for ts, xs, sf, codes in _rows("nvfp4_group_examples.txt"):
        x = bf([float(v) for v in xs.split()])
        c, s = O.quant_nvfp4(x, float(ts))
        assert s.shape == (1, 1) and s[0, 0] == int(sf, 16), (xs, hex(s[0, 0]))
        assert list(unpack(c)[0]) == [int(v, 16) for v in codes.split()], xs


def test_nvfp4_dequant_of_amax7_example():
    x = bf([7.0] + [1.0] * 15)
    c, s = O.quant_nvfp4(x, 1.0)
    dq = O.dequant_nvfp4(c, s, 1.0)
    assert dq[0, 0] == 6.75 and dq[0, 1] == 1.125      # 6 * 1.125, 1 * 1.125


def test_tensor_scale():
    assert O.tensor_scale(np.array([1.0, 2688.0, 3.0], dtype=np.float32)) == 1.0
    assert O.tensor_scale(np.zeros(4, dtype=np.float32)) == 1.0
    assert O.tensor_scale(np.array([0.5, 1344.0], dtype=np.float32)) == 0.5


def _random_tensor(rows, K, seed):
    cfg = inputs.LayerConfig("t", rows, K, K, 1.0, 4, 30.0, 0.02, 1.0, False, 1)
    return inputs.bits(inputs.activations(cfg, seed, 0))


def test_nvfp4_sign_symmetry():
    x = _random_tensor(32, 128, 3)
    c1, s1 = O.quant_nvfp4(x, 0.01)
    c2, s2 = O.quant_nvfp4(x ^ np.uint16(0x8000), 0.01)
    assert np.array_equal(s1, s2)
    assert np.array_equal(unpack(c1) ^ 8, unpack(c2))


def test_nvfp4_power_of_two_scaling():
    x = _random_tensor(32, 128, 4)
    xs = inputs.bits(inputs.from_bits(x).to(torch.float32).mul(8.0).to(torch.bfloat16))  # exact
    c1, s1 = O.quant_nvfp4(x, 0.01)
    c2, s2 = O.quant_nvfp4(xs, 0.08)
    assert np.array_equal(c1, c2) and np.array_equal(s1, s2)


def test_nvfp4_within_group_permutation():
    """Shuffling channels inside each group of 16 shuffles the codes, keeps the scale bytes."""
    x = _random_tensor(16, 64, 5)
    rng = np.random.default_rng(0)
    perm = np.concatenate([16 * k + rng.permutation(16) for k in range(4)]).astype(np.int32)
    c1, s1 = O.quant_nvfp4(x, 0.02)
    c2, s2 = O.quant_nvfp4(x, 0.02, perm)
    assert np.array_equal(s1, s2)
    assert np.array_equal(unpack(c1)[:, perm], unpack(c2))


def test_identity_permutation_reproduces_unpermuted():
    x = _random_tensor(70, 128, 6)
    ident = np.arange(128, dtype=np.int32)
    for a, b in zip(O.quant_nvfp4(x, 0.02), O.quant_nvfp4(x, 0.02, ident)):
        assert np.array_equal(a, b)
    assert np.array_equal(O.fakequant_int(x, 3, 32), O.fakequant_int(x, 3, 32, ident))
    e0 = O.group_error(x, 0, 4, 16, 0.02)
    e1 = O.group_error(x, 0, 4, 16, 0.02, ident)
    assert np.array_equal(e0, e1)


def test_gather_convention():
    """out[:, j] = in[:, perm[j]]  (App. C: position j reads channel pi(j))."""
    x = _random_tensor(8, 64, 7)
    perm = np.random.default_rng(1).permutation(64).astype(np.int32)
    gathered = np.ascontiguousarray(x[:, perm])
    for a, b in zip(O.quant_nvfp4(x, 0.02, perm), O.quant_nvfp4(gathered, 0.02)):
        assert np.array_equal(a, b)
    assert np.array_equal(O.fakequant_int(x, 4, 32, perm), O.fakequant_int(gathered, 4, 32))
    assert np.array_equal(O.group_error(x, 1, 3, 32, 1.0, perm), O.group_error(gathered, 1, 3, 32))


def test_int_golden_groups():
    for bits, xs, s, zs, sse in _rows("int_group_examples.txt"):
        vals = [float(v) for v in xs.split()]
        x = bf(vals)
        g = len(vals)
        out = O.bf16_to_f32(O.fakequant_int(x, int(bits), g))[0]
        want = [float(z) * float(s) for z in zs.split()]
        assert list(out) == want, xs
        err = O.group_error(x, 1, int(bits), g)
        assert err.shape == (1, 1) and err[0, 0] == float(sse), xs


@pytest.mark.parametrize("bits,g", [(3, 32), (3, 64), (4, 128), (4, 32), (8, 64), (2, 16)])
def test_int_matches_numpy_restatement_and_bound(bits, g):
    """Eq. 1-2 written with numpy fp32 ops, and the per-vector bound of Eq. 4:
    ||e||^2 <= g / (4 Q^2) * sum_k max|x|^2."""
    x = _random_tensor(48, 256, 10 + bits)
    xf = O.bf16_to_f32(x).reshape(48, 256 // g, g)
    Q = np.float32(2 ** (bits - 1) - 1)
    amax = np.abs(xf).max(axis=-1, keepdims=True)
    s = (amax / Q).astype(np.float32)
    r = np.where(s > 0, np.float32(1) / np.where(s > 0, s, 1), 0).astype(np.float32)
    z = np.clip(np.rint((xf * r).astype(np.float32)), -Q, Q)
    xhat = (z * s).astype(np.float32)
    want = torch.from_numpy(xhat.reshape(48, 256)).to(torch.bfloat16)
    assert np.array_equal(O.fakequant_int(x, bits, g), inputs.bits(want))
    # the element carrying the group maximum maps to +-Q exactly
    at_max = np.abs(xf) == amax
    assert np.all(np.abs(z[at_max & (amax > 0)]) == Q)
    # Eq. 4, per group (error before the bf16 rounding of the output)
    err = O.group_error(x, 1, bits, g)[0]
    bound = (g / (4.0 * float(Q) ** 2)) * (amax.astype(np.float64) ** 2).sum(axis=0).reshape(-1)
    assert np.all(err <= bound * (1 + 1e-6))
    # and the reduction agrees with a float64 straight sum
    exact = ((xf.astype(np.float64) - xhat.astype(np.float64)) ** 2).sum(axis=(0, 2))
    assert np.allclose(err, exact, rtol=1e-5, atol=0)


def test_nvfp4_group_error_matches_dequant_difference():
    x = _random_tensor(130, 128, 20)     # 3 chunks, ragged tail
    ts = 0.03
    c, s = O.quant_nvfp4(x, ts)
    dq = O.dequant_nvfp4(c, s, ts).astype(np.float64)
    exact = ((O.bf16_to_f32(x).astype(np.float64) - dq) ** 2).reshape(130, 8, 16).sum(axis=(0, 2))
    err = O.group_error(x, 0, 4, 16, ts)[0]
    assert np.allclose(err, exact, rtol=2e-6, atol=0)
    # NVFP4 grid is non-uniform: |e| <= d (largest half-gap is one code unit) when unsaturated
    assert np.all(err >= 0)


def test_group_error_row_order_is_chunks_then_slabs():
    """One call on 300 rows = slab sums (128 rows, fp64 from zero, over 16-row chunk partials)
    added in order; a one-chunk call returns that chunk's fp32 partial exactly."""
    rng = np.random.default_rng(11)
    xf = (rng.standard_normal((300, 64)) * np.where(np.arange(300)[:, None] < 128, 3e4, 1e-3)).astype(np.float32)
    x = np.ascontiguousarray((xf.view(np.uint32) >> 16).astype(np.uint16))
    for fmt in ((1, 4, 32, 1.0), (0, 4, 16, 2.0)):
        whole = O.group_error(x, *fmt)
        total = np.zeros_like(whole)
        flat = np.zeros_like(whole)
        for s0 in range(0, 300, 128):
            slab = np.zeros_like(whole)
            for r0 in range(s0, min(s0 + 128, 300), 16):
                part = O.group_error(np.ascontiguousarray(x[r0:min(r0 + 16, s0 + 128, 300)]), *fmt)
                assert np.array_equal(part, part.astype(np.float32).astype(np.float64))
                slab += part
                flat += part
            total += slab
        assert np.array_equal(whole, total)
        assert fmt[0] == 0 or np.any(flat != total)      # the integer case separates the two orders


def test_group_error_accumulates_across_calls():
    x1, x2 = _random_tensor(64, 64, 30), _random_tensor(40, 64, 31)
    e = O.group_error(x1, 1, 3, 32)
    e = O.group_error(x2, 1, 3, 32, err=e)
    assert np.array_equal(e, O.group_error(x1, 1, 3, 32) + O.group_error(x2, 1, 3, 32))


def test_saturating_runtime_group():
    """A group whose absmax exceeds 448 * 6 * ts saturates the scale byte, then the codes."""
    x = bf([5000.0, 3000.0] + [1.0] * 14)
    c, s = O.quant_nvfp4(x, 1.0)
    assert s[0, 0] == 0x7E
    assert list(unpack(c)[0][:2]) == [7, 7]          # 5000/448 = 11.2 -> 6;  3000/448 = 6.7 -> 6
