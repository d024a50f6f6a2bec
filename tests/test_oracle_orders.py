"""Pins of the oracle's additional candidate orders of the reordering ablation (Tab. 2(a)): the first
moments behind the variance criterion, the variance order, the round-robin order, and group size 256
(Tab. 2(d)) in the error / fake-quant routines."""
import numpy as np

from oracle import pq_oracle as O


def bf(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return (a.view(np.uint32) >> 16).astype(np.uint16).reshape(a.shape)


def test_first_moment_closed_forms_and_float64():
    rows, K = 300, 24
    c = (np.arange(K) - 7).astype(np.float32) * 0.25                       # bf16-exact constants per column
    x = bf(np.tile(c, (rows, 1)))
    assert np.array_equal(O.calib_sum(x), rows * c.astype(np.float64))     # exact: small multiples of 1/4
    alt = bf(np.where(np.arange(rows)[:, None] % 2 == 0, 1.0, -1.0) * np.ones((rows, K)))
    assert np.array_equal(O.calib_sum(alt), np.zeros(K))                   # +1 -1 +1 -1 ... cancels exactly
    rng = np.random.default_rng(0)
    xb = bf(rng.standard_normal((1000, 40)) * np.exp(rng.standard_normal(40)) + 0.5)
    xf = O.bf16_to_f32(xb).astype(np.float64)
    got = O.calib_sum(xb)
    assert np.allclose(got, xf.sum(axis=0), rtol=0, atol=2e-6 * np.abs(xf).sum(axis=0))
    # accumulation across batches continues the same totals
    assert np.array_equal(O.calib_sum(xb[512:], O.calib_sum(xb[:512])), got)     # 512 = a whole number of slabs


def test_first_moment_order_of_additions():
    """Chunks of 16 rows in fp32 in row order, the 8 chunks of a 128-row slab in fp64 from zero, slabs in order."""
    rng = np.random.default_rng(3)
    xb = bf(rng.standard_normal((300, 1)) * np.exp(4 * rng.standard_normal((300, 1))))
    x = O.bf16_to_f32(xb)[:, 0]
    total = 0.0
    for s0 in range(0, 300, 128):
        slab = 0.0
        for r0 in range(s0, min(s0 + 128, 300), 16):
            p = np.float32(0.0)
            for t in range(r0, min(r0 + 16, s0 + 128, 300)):
                p = np.float32(p + x[t])
            slab += float(p)
        total += slab
    assert O.calib_sum(xb)[0] == total
    flat = np.float32(0.0)
    for t in range(300):
        flat = np.float32(flat + x[t])
    assert float(flat) != total                                             # the blocking is observable


def test_variance_order():
    # hand case, 4 rows: column sums / sums of squares chosen so that variance and second moment disagree
    x = np.array([[10, 1, 0, 3], [10, -1, 0, 3], [10, 1, 4, -3], [10, -1, -4, -3]], dtype=np.float32)
    xb = bf(x)
    S, _ = O.calib_stats(xb)
    total = O.calib_sum(xb)
    assert total.tolist() == [40.0, 0.0, 0.0, 0.0] and S.tolist() == [400.0, 4.0, 32.0, 36.0]
    # variances: 0, 1, 8, 9 -> order 3, 2, 1, 0; second moments 100, 1, 8, 9 -> order 0, 3, 2, 1
    assert O.order_by_variance(total, S, 4).tolist() == [3, 2, 1, 0]
    assert O.select_perm(S, 4, np.ones(4), 1, J=1)[1].tolist() == [0, 3, 2, 1]
    # against numpy on random data, ties (duplicated columns) resolved by ascending channel
    rng = np.random.default_rng(5)
    xr = rng.standard_normal((256, 64)) * np.exp(rng.standard_normal(64)) + rng.standard_normal(64)
    xr[:, 10] = xr[:, 40]
    xb = bf(xr)
    S, _ = O.calib_stats(xb)
    total = O.calib_sum(xb)
    var = S / 256.0 - (total / 256.0) * (total / 256.0)
    want = np.lexsort((np.arange(64), -var))
    got = O.order_by_variance(total, S, 256)
    assert np.array_equal(got, want) and list(got).index(10) + 1 == list(got).index(40)
    # zero-mean channels: the variance order is the second-moment order
    z = np.zeros(64)
    assert np.array_equal(O.order_by_variance(z, S, 256), O.select_perm(S, 256, np.ones(64), 1, J=1)[1])


def test_round_robin_order():
    S = np.array([5.0, 9.0, 1.0, 7.0, 3.0, 8.0, 2.0, 6.0])          # sorted descending: 1, 5, 3, 7, 0, 4, 6, 2
    # two groups of four: ranks 0, 2, 4, 6 -> group 0, ranks 1, 3, 5, 7 -> group 1
    assert O.order_round_robin(S, 4).tolist() == [1, 3, 0, 6, 5, 7, 4, 2]
    # four groups of two: group k gets ranks k and k + 4
    assert O.order_round_robin(S, 2).tolist() == [1, 0, 5, 4, 3, 6, 7, 2]
    # one group: plain descending sort; groups of one: plain descending sort as well
    assert O.order_round_robin(S, 8).tolist() == [1, 5, 3, 7, 0, 4, 6, 2]
    assert O.order_round_robin(S, 1).tolist() == [1, 5, 3, 7, 0, 4, 6, 2]
    rng = np.random.default_rng(1)
    S = rng.random(96)
    p = O.order_round_robin(S, 16)
    assert sorted(p.tolist()) == list(range(96))
    # every group holds one channel from each block of 6 consecutive ranks: its maxima are spread evenly
    rank = np.empty(96, dtype=int)
    rank[np.argsort(-S, kind="stable")] = np.arange(96)
    assert all(sorted(rank[p[g * 16:(g + 1) * 16]] // 6) == list(range(16)) for g in range(6))


def test_group_size_256():
    """Tab. 2(d)'s largest group: scale from the absmax of 256 channels, Eq. 4's bound on every group, and
    the error of a 256-group against the straight definition in float64."""
    rng = np.random.default_rng(2)
    K = 512
    xb = bf(rng.standard_normal((40, K)) * np.exp(rng.standard_normal(K)))
    x = O.bf16_to_f32(xb).astype(np.float64)
    for bits in (3, 4):
        Q = 2 ** (bits - 1) - 1
        fq = O.bf16_to_f32(O.fakequant_int(xb, bits, 256)).astype(np.float64)
        err = O.group_error(xb, 1, bits, 256)
        for k in range(2):
            g = x[:, 256 * k:256 * (k + 1)]
            s = np.abs(g).max(axis=1, keepdims=True) / Q
            ref = np.clip(np.rint(g / s), -Q, Q) * s
            assert np.allclose(fq[:, 256 * k:256 * (k + 1)], ref, rtol=2.0 ** -8, atol=1e-6)
            sse = ((g - ref) ** 2).sum()
            assert abs(err[0, k] - sse) <= 1e-3 * sse
            assert (((g - ref) ** 2).sum(axis=1) <= 256 * (s[:, 0] * Q) ** 2 / (4 * Q * Q) + 1e-9).all()   # Eq. 4
    # a 256-group whose channels are all equal in magnitude quantizes exactly
    c = bf(np.where(rng.random((8, 256)) < 0.5, -3.0, 3.0))          # scale = 3 / Q = 1 exactly
    assert np.array_equal(O.fakequant_int(c, 3, 256), c) and O.group_error(c, 1, 3, 256)[0, 0] == 0.0
