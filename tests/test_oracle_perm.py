"""Pins for the oracle's calibration statistics, sort candidates (Eq. 9, Prop. 3.2) and the
acceptance rule (Eq. 10): closed forms, brute force over all permutations on tiny inputs."""
import itertools

import numpy as np
import pytest
import torch

from oracle import pq_oracle as O
from paper_2605_09503_b200 import inputs


def bf(a):
    return inputs.bits(torch.tensor(np.asarray(a, dtype=np.float32)).to(torch.bfloat16))


# ---------------------------------------------------------------- statistics
def test_stats_closed_form_constant_columns():
    T, K = 200, 8
    c = np.array([0.5, 1, 2, 3, -4, 0, 1.5, 8], dtype=np.float32)
    sign = np.where(np.arange(T)[:, None] % 2 == 0, 1.0, -1.0)
    S, A = O.calib_stats(bf(sign * c[None, :]))
    assert np.array_equal(S, T * c.astype(np.float64) ** 2)      # exact: small integers / quarters
    assert np.array_equal(A, np.abs(c))


def test_stats_against_float64_sum_and_accumulation():
    cfg = inputs.CONFIGS["tiny"]
    x0, x1 = (inputs.bits(inputs.activations(cfg, 0, b, rows=150)) for b in (0, 1))
    S, A = O.calib_stats(x0)
    S, A = O.calib_stats(x1, S, A)
    both = np.concatenate([O.bf16_to_f32(x0), O.bf16_to_f32(x1)]).astype(np.float64)
    assert np.allclose(S, (both ** 2).sum(axis=0), rtol=1e-6, atol=0)
    assert np.array_equal(A, np.abs(both).max(axis=0).astype(np.float32))


def _fold(xf, rows, chunk=16, slab=128, flat=False):
    """Column sums of squares of float32 xf in the stated order, written out with numpy scalars."""
    want = np.zeros(xf.shape[1])
    for s0 in range(0, rows, slab):
        acc = np.zeros(xf.shape[1])
        for r0 in range(s0, min(s0 + slab, rows), chunk):
            p = np.zeros(xf.shape[1], dtype=np.float32)
            for t in range(r0, min(r0 + chunk, s0 + slab, rows)):
                p = (p.astype(np.float64) + xf[t].astype(np.float64) ** 2).astype(np.float32)  # = fmaf
            if flat:
                want += p.astype(np.float64)
            else:
                acc += p.astype(np.float64)
        if not flat:
            want += acc
    return want


def test_stats_chunk_order_is_the_stated_one():
    """Rows in chunks of 16 (fp32 fused accumulate), chunks in slabs of 128 rows (fp64 from zero),
    slab sums added to the fp64 total in order."""
    assert O.chunk_rows() == 16 and O.slab_rows() == 128
    x = inputs.bits(inputs.activations(inputs.CONFIGS["tiny"], 1, 0, rows=150))[:, :16]
    x = np.ascontiguousarray(x)
    S, _ = O.calib_stats(x)
    assert np.array_equal(S, _fold(O.bf16_to_f32(x), 150))


def test_stats_slab_sums_start_from_zero():
    """A column whose first slab is huge and whose later rows are tiny: adding the later chunk
    partials one by one to the running total rounds differently from adding their slab sum."""
    rng = np.random.default_rng(5)
    xf = np.zeros((400, 16), dtype=np.float32)
    xf[:128] = 2.0 ** 14 * (1 + rng.random((128, 16)))
    xf[128:] = 2.0 ** -9 * (1 + rng.random((272, 16)))
    x = np.ascontiguousarray((xf.view(np.uint32) >> 16).astype(np.uint16))     # exact bf16 truncation
    xf = O.bf16_to_f32(x)
    want, flat = _fold(xf, 400), _fold(xf, 400, flat=True)
    assert np.any(want != flat)                  # the case separates the two orders
    S, _ = O.calib_stats(x)
    assert np.array_equal(S, want)
    # starting from an earlier total, slab sums are added to it one by one
    S2, _ = O.calib_stats(x, S.copy(), np.zeros(16, dtype=np.float32))
    again = want.copy()
    for s0 in range(0, 400, 128):
        again += _fold(xf[s0:s0 + 128], min(128, 400 - s0))
    assert np.array_equal(S2, again)


# ---------------------------------------------------------------- sorting
def phi(mu2, order, g):
    """Sum over contiguous groups of the group maximum of mu^2 (the bound of Eq. 6)."""
    v = np.asarray(mu2)[list(order)]
    return v.reshape(-1, g).max(axis=1).sum()


@pytest.mark.parametrize("K,g", [(6, 2), (6, 3), (8, 2), (8, 4)])
def test_sorted_partition_minimises_bound_brute_force(K, g):
    """Prop. 3.2: among all K! orders the descending sort minimises sum_k max mu_i^2."""
    rng = np.random.default_rng(K * 10 + g)
    for trial in range(3):
        mu2 = rng.lognormal(0, 2, K)
        perms = O.select_perm(mu2 * 10, 10, np.ones(K), 1, J=1)
        act_sorted = perms[1]                                  # alpha = 1: activation only
        best = min(phi(mu2, p, g) for p in itertools.permutations(range(K)))
        assert np.isclose(phi(mu2, act_sorted, g), best, rtol=1e-12)
        # closed form: the group maxima of the sorted order are a_1, a_{g+1}, a_{2g+1}, ...
        a = np.sort(mu2)[::-1]
        assert np.isclose(best, a[::g].sum(), rtol=1e-12)


def test_alpha_endpoints_are_single_side_sorts_and_ties_are_stable():
    rng = np.random.default_rng(5)
    K = 64
    Sa = rng.lognormal(0, 2, K)
    Sw = rng.lognormal(0, 1, K)
    Sa[10] = Sa[3]
    Sa[40] = Sa[3]                       # three equal activation moments
    perms = O.select_perm(Sa, 7, Sw, 3, J=5)
    assert perms.shape == (6, K)
    for p in perms:
        assert sorted(p) == list(range(K))
    assert np.array_equal(perms[5], np.argsort(-Sa, kind="stable"))   # alpha = 1
    assert np.array_equal(perms[0], np.argsort(-Sw, kind="stable"))   # alpha = 0
    pos = {c: i for i, c in enumerate(perms[5])}
    assert pos[3] < pos[10] < pos[40]


def test_intermediate_alpha_orders_like_fractional_powers():
    """The integer-power key a^j w^(J-j) orders channels like (a)^alpha (w)^(1-alpha), Eq. 9."""
    rng = np.random.default_rng(6)
    K = 200
    Sa, Sw = rng.lognormal(0, 2, K), rng.lognormal(0, 1, K)
    perms = O.select_perm(Sa * 4, 4, Sw * 9, 9, J=5)
    for j in range(6):
        alpha = j / 5
        v = Sa ** alpha * Sw ** (1 - alpha)
        got = v[perms[j]]
        assert np.all(got[:-1] >= got[1:] * (1 - 1e-9))


# ---------------------------------------------------------------- acceptance
def true_error(x, order, kind, bits, g, ts=1.0):
    return O.group_error(x, kind, bits, g, ts, np.asarray(order, dtype=np.int32)).sum()


def _tiny_layer(seed, rows=24, K=8):
    rng = np.random.default_rng(seed)
    scale = rng.lognormal(0, 1.5, K)
    x = bf(rng.standard_normal((rows, K)) * scale[None, :])
    w = bf(0.02 * rng.standard_normal((rows, K)))
    return x, w


@pytest.mark.parametrize("g", [2, 4])
def test_accept_equals_brute_force_decision(g):
    """Eq. 10 at tau = 0 on layers small enough to enumerate all 8! orders: the decision is
    [E(best candidate) < E(original)], and no order beats the global optimum."""
    K = 8
    for seed in range(4):
        x, w = _tiny_layer(seed)
        Sa, _ = O.calib_stats(x)
        Sw, _ = O.calib_stats(w)
        perms = O.select_perm(Sa, x.shape[0], Sw, w.shape[0], J=5)
        cand = np.concatenate([np.arange(K, dtype=np.int32)[None], perms])
        ex = O.group_error(x, 1, 3, g, 1.0, cand)
        ew = O.group_error(w, 1, 3, g, 1.0, cand)
        lx, lw = O.error_weight(Sa), O.error_weight(Sw)
        best, acc, E = O.accept(ex, lx, ew, lw, 0.0)
        # E of every candidate recomputed one by one
        for p in range(7):
            want = lx * true_error(x, cand[p], 1, 3, g) + lw * true_error(w, cand[p], 1, 3, g)
            assert np.isclose(E[p], want, rtol=1e-12)
        assert best == 1 + int(np.argmin(E[1:]))
        assert acc == int(E[best] < E[0])
        # brute force over ALL orders: the error depends only on which channels share a group,
        # so the 8! orders collapse to 105 (g=2) or 35 (g=4) distinct partitions
        best_a, acc_a, Ea = O.accept(ex, 1.0, ew, 0.0, 0.0)
        parts = all_partitions(K, g)
        assert len(parts) == {2: 105, 4: 35}[g]
        all_err = np.array([true_error(x, p, 1, 3, g) for p in parts])
        assert all_err.min() <= Ea.min() * (1 + 1e-6)          # no candidate beats the optimum
        assert acc_a == int(Ea[best_a] < Ea[0])
        ident_is_optimal = true_error(x, range(K), 1, 3, g) <= all_err.min() * (1 + 1e-6)
        if ident_is_optimal:
            assert acc_a == 0


def all_partitions(K, g):
    """Every way to split range(K) into K/g unordered groups of size g, as channel orders."""
    out = []

    def rec(rest, acc):
        if not rest:
            out.append([c for grp in acc for c in grp])
            return
        first, others = rest[0], rest[1:]
        for combo in itertools.combinations(others, g - 1):
            left = [c for c in others if c not in combo]
            rec(left, acc + [[first, *combo]])

    rec(list(range(K)), [])
    return out


def test_presorted_layer_is_rejected_and_clustered_outliers_accepted():
    rows, K, g = 64, 16, 4
    rng = np.random.default_rng(11)
    x_any = bf(rng.standard_normal((rows, K)) * rng.lognormal(0, 2, K)[None, :])
    S_any, _ = O.calib_stats(x_any)
    # put the columns in descending order of their SAMPLED second moments (a column's sum moves with the
    # column, bit for bit), so the layer is sorted in exactly the sense the criterion uses
    x_sorted = np.ascontiguousarray(x_any[:, np.argsort(-S_any, kind="stable")])
    w = bf(np.ones((8, K)))                                   # weight side indifferent
    Sa, _ = O.calib_stats(x_sorted)
    assert (np.diff(Sa) < 0).all()
    Sw, _ = O.calib_stats(w)
    perms = O.select_perm(Sa, rows, Sw, 8, J=5)
    cand = np.concatenate([np.arange(K, dtype=np.int32)[None], perms])
    ex = O.group_error(x_sorted, 1, 3, g, 1.0, cand)
    ew = O.group_error(w, 1, 3, g, 1.0, cand)
    # every candidate of a sorted layer is the original order again (the weight-only sort too: equal
    # keys keep their order), so no candidate can lower the error and the strict '>' rejects
    assert all(np.array_equal(p_, np.arange(K)) for p_ in perms)
    _, acc, E = O.accept(ex, 1.0, ew, 0.0, 0.0)
    assert acc == 0 and (E[1:] == E[0]).all()
    # one 8x channel per group in the original order drowns its three neighbours (their
    # share of a 4-bit grid spanning the large channel is ~1 level); sorting puts the four
    # large channels into one group and gives the small ones grids of their own -> accepted
    scale = np.ones(K)
    scale[::g] = 8.0
    x_out = bf(rng.standard_normal((rows, K)) * scale[None, :])
    Sa, _ = O.calib_stats(x_out)
    perms = O.select_perm(Sa, rows, Sw, 8, J=5)
    cand = np.concatenate([np.arange(K, dtype=np.int32)[None], perms])
    ex = O.group_error(x_out, 1, 4, g, 1.0, cand)
    ew = O.group_error(w, 1, 4, g, 1.0, cand)
    best, acc, E = O.accept(ex, 1.0, ew, 0.0, 0.0)
    assert acc == 1 and E[best] < 0.8 * E[0]
    assert E[best] == true_error(x_out, cand[best], 1, 4, g)
    assert set(perms[5][:4]) == {0, 4, 8, 12}


def test_tau_monotone_and_zero_error_rejects():
    ex = np.array([[4.0, 4.0], [3.0, 3.0], [3.5, 3.5]])
    ew = np.zeros_like(ex)
    best, acc, E = O.accept(ex, 1.0, ew, 1.0, 0.0)
    assert (best, acc) == (1, 1) and list(E) == [8.0, 6.0, 7.0]
    assert O.accept(ex, 1.0, ew, 1.0, 0.24)[1] == 1            # relative drop is exactly 0.25
    assert O.accept(ex, 1.0, ew, 1.0, 0.25)[1] == 0            # strict inequality
    assert O.accept(ex, 1.0, ew, 1.0, 0.5)[1] == 0
    z = np.zeros((3, 2))
    assert O.accept(z, 1.0, z, 1.0, 0.0)[1] == 0               # E_orig = 0: nothing to gain
    tie = np.array([[4.0], [2.0], [2.0]])
    assert O.accept(tie, 1.0, np.zeros_like(tie), 0.0, 0.0)[0] == 1   # first of equal candidates
    # a candidate good for X but bad for W is judged on the weighted sum
    ex2 = np.array([[4.0], [1.0]])
    ew2 = np.array([[1.0], [5.0]])
    assert O.accept(ex2, 1.0, ew2, 1.0, 0.0)[1] == 0
    assert O.accept(ex2, 1.0, ew2, 0.1, 0.0)[1] == 1


def test_error_weight():
    assert O.error_weight(np.array([1.0, 3.0])) == 0.25


# ---------------------------------------------------------------- absmax criterion (Tab. 2(a))
def test_absmax_order_against_a_stable_library_sort_and_by_hand():
    a = np.array([3.0, 0.5, 3.0, 7.25, 0.0, 0.5, 1e-30, 7.25], dtype=np.float32)
    # by hand: 7.25 (ch 3), 7.25 (ch 7), 3 (ch 0), 3 (ch 2), .5 (ch 1), .5 (ch 5), 1e-30 (ch 6), 0 (ch 4)
    assert O.order_by_absmax(a).tolist() == [3, 7, 0, 2, 1, 5, 6, 4]
    g = np.random.default_rng(3)
    big = np.round(np.abs(g.standard_normal(5000)) * 8).astype(np.float32) / 8      # many ties
    got = O.order_by_absmax(big)
    assert np.array_equal(got, np.argsort(-big.astype(np.float64), kind="stable"))
    assert sorted(got.tolist()) == list(range(5000))


def test_absmax_order_of_real_statistics_differs_from_the_second_moment_order():
    """Heavy-tailed columns: a rare spike raises a channel's absmax but hardly its second moment, so
    the two criteria of Tab. 2(a) are different orders (and each is sorted by its own key)."""
    g = np.random.default_rng(9)
    x = g.standard_normal((512, 64)).astype(np.float32) * np.linspace(0.5, 2.0, 64, dtype=np.float32)
    x[7, 5] = 12.0
    xb = bf(x)
    S, A = O.calib_stats(xb)
    by_max = O.order_by_absmax(A)
    by_moment = O.select_perm(S, 512, np.ones(64), 1, J=1)[1]
    assert by_max[0] == 5 and by_moment[0] != 5
    assert np.all(np.diff(A[by_max]) <= 0) and np.all(np.diff(S[by_moment]) <= 0)
