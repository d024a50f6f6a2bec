"""GPU parity, offline half: statistics, sort candidates, calibration error, acceptance,
weight quantization, integer fake-quant -- every output compared bit for bit with the CPU
oracle on the same seeded inputs, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import pq_oracle as O
from paper_2605_09503_b200 import binding as B
from paper_2605_09503_b200 import inputs

pytestmark = pytest.mark.gpu
DEV = "cuda"


def dev(t):
    return t.to(DEV)


def small_cfg(rows, K, seed_outliers=4):
    return inputs.LayerConfig("t", rows, K, K, 1.0, seed_outliers, 30.0, 0.02, 5.0, False, 1)


def gpu_stats(batches):
    K = batches[0].shape[1]
    S = torch.zeros(K, dtype=torch.float64, device=DEV)
    A = torch.zeros(K, dtype=torch.float32, device=DEV)
    for x in batches:
        ws = B.workspace(B.OP_CALIB_STATS, x.shape[0], K)
        B.pq_calib_stats(x, S, A, ws)
    return S, A


@pytest.mark.parametrize("rows,K", [(256, 512), (130, 1032), (64, 8), (1, 2048), (200, 3072)])
def test_calib_stats_bit_exact(rows, K):
    cfg = small_cfg(rows, K)
    xs = [inputs.activations(cfg, 0, b) for b in range(2)]
    S, A = gpu_stats([dev(x) for x in xs])
    So, Ao = None, None
    for x in xs:
        So, Ao = O.calib_stats(inputs.bits(x), So, Ao)
    assert np.array_equal(S.cpu().numpy(), So)
    assert np.array_equal(A.cpu().numpy(), Ao)


def test_calib_stats_strided_input():
    cfg = small_cfg(100, 256)
    x = inputs.activations(cfg, 1, 0)
    big = torch.zeros(100, 320, dtype=torch.bfloat16)
    big[:, :256] = x
    S, A = gpu_stats([dev(big)[:, :256]])
    So, Ao = O.calib_stats(inputs.bits(x))
    assert np.array_equal(S.cpu().numpy(), So) and np.array_equal(A.cpu().numpy(), Ao)


def test_tensor_scale_and_error_weights():
    A = torch.tensor([0.5, 77.25, 3.0], dtype=torch.float32)
    ts = torch.zeros(1, dtype=torch.float32, device=DEV)
    B.pq_tensor_scale(dev(A), ts)
    assert ts.item() == O.tensor_scale(A.numpy())
    B.pq_tensor_scale(torch.zeros(5, dtype=torch.float32, device=DEV), ts)
    assert ts.item() == 1.0
    rng = np.random.default_rng(0)
    sa, sw = rng.lognormal(0, 2, 1000), rng.lognormal(0, 1, 1000)
    lam = torch.zeros(2, dtype=torch.float64, device=DEV)
    B.pq_error_weights(dev(torch.from_numpy(sa)), dev(torch.from_numpy(sw)), lam)
    assert lam.cpu().tolist() == [O.error_weight(sa), O.error_weight(sw)]


@pytest.mark.parametrize("K,J", [(512, 5), (3072, 5), (1000, 3), (16384, 5), (8, 1)])
def test_select_perm_bit_exact(K, J):
    rng = np.random.default_rng(K + J)
    sa, sw = rng.lognormal(0, 3, K), rng.lognormal(-8, 1, K)
    sa[K // 2] = sa[0]
    sw[K // 2] = sw[0]           # an exact tie in every candidate
    sa[K // 3] = 0.0             # zero moment: keys collapse to 0 for j >= 1
    perms = torch.empty(J + 1, K, dtype=torch.int32, device=DEV)
    ws = B.workspace(B.OP_SELECT_PERM, 0, K, 0, J + 1)
    B.pq_select_perm(dev(torch.from_numpy(sa)), 1024, dev(torch.from_numpy(sw)), 77, J, perms, ws)
    want = O.select_perm(sa, 1024, sw, 77, J)
    assert np.array_equal(perms.cpu().numpy(), want)


FORMATS = [(0, 4, 16), (1, 3, 32), (1, 3, 64), (1, 4, 128), (1, 4, 16), (1, 8, 32)]


@pytest.mark.parametrize("fmt", FORMATS)
@pytest.mark.parametrize("rows,K", [(130, 512), (64, 3072), (7, 128)])
def test_group_error_original_order_bit_exact(fmt, rows, K):
    x = inputs.activations(small_cfg(rows, K), 2, 0)
    ts = torch.tensor([0.013], dtype=torch.float32)
    err = torch.zeros(1, K // fmt[2], dtype=torch.float64, device=DEV)
    ws = B.workspace(B.OP_GROUP_ERROR, rows, K, 0, 1)
    B.pq_group_error(dev(x), fmt, dev(ts), None, err, ws)
    B.pq_group_error(dev(x), fmt, dev(ts), None, err, ws)        # accumulates across calls
    want = O.group_error(inputs.bits(x), *fmt, ts=ts.item())
    want = O.group_error(inputs.bits(x), *fmt, ts=ts.item(), err=want)
    assert np.array_equal(err.cpu().numpy(), want)


@pytest.mark.parametrize("fmt", FORMATS)
@pytest.mark.parametrize("rows,K,P", [(130, 512, 7), (70, 3072, 3), (5, 4096, 1), (64, 12288, 2),
                                      (33, 8192, 2), (40, 16384, 2), (21, 48 * 16, 8)])   # two and four runs per thread
def test_group_error_candidates_bit_exact(fmt, rows, K, P):
    x = inputs.activations(small_cfg(rows, K), 3, 0)
    rng = np.random.default_rng(K + P)
    perms = np.stack([rng.permutation(K) for _ in range(P)]).astype(np.int32)
    perms[0] = np.arange(K)                                   # identity as a candidate
    ts = torch.tensor([0.02], dtype=torch.float32)
    err = torch.zeros(P, K // fmt[2], dtype=torch.float64, device=DEV)
    ws = B.workspace(B.OP_GROUP_ERROR, rows, K, 0, P)
    B.pq_group_error(dev(x), fmt, dev(ts), dev(torch.from_numpy(perms)), err, ws)
    want = O.group_error(inputs.bits(x), *fmt, ts=ts.item(), perms=perms)
    got = err.cpu().numpy()
    assert np.array_equal(got, want)
    # identity candidate == original-order path (the invariant the method relies on)
    err0 = torch.zeros(1, K // fmt[2], dtype=torch.float64, device=DEV)
    B.pq_group_error(dev(x), fmt, dev(ts), None, err0, ws)
    assert np.array_equal(err0.cpu().numpy()[0], got[0])


def test_accept_bit_exact_and_edge_cases():
    rng = np.random.default_rng(4)
    for P, Kg, tau in [(6, 192, 0.0), (6, 32, 0.025), (1, 1, 0.0), (3, 768, 0.5)]:
        ex, ew = rng.lognormal(0, 1, (P + 1, Kg)), rng.lognormal(0, 1, (P + 1, Kg))
        lam = np.array([0.37, 1.9])
        best = torch.zeros(1, dtype=torch.int32, device=DEV)
        acc = torch.zeros(1, dtype=torch.int32, device=DEV)
        E = torch.zeros(P + 1, dtype=torch.float64, device=DEV)
        B.pq_accept(dev(torch.from_numpy(ex)), dev(torch.from_numpy(ew)), dev(torch.from_numpy(lam)), tau,
                    best, acc, E)
        b, a, Eo = O.accept(ex, lam[0], ew, lam[1], tau)
        assert (best.item(), acc.item()) == (b, a)
        assert np.array_equal(E.cpu().numpy(), Eo)
    # equal error is rejected (strict inequality); zero error is rejected; NULL lambda = (1, 1)
    for ex in (np.array([[4.0], [4.0]]), np.zeros((2, 1)), np.array([[4.0], [3.0]])):
        best = torch.zeros(1, dtype=torch.int32, device=DEV)
        acc = torch.zeros(1, dtype=torch.int32, device=DEV)
        B.pq_accept(dev(torch.from_numpy(ex)), dev(torch.zeros(2, 1, dtype=torch.float64)), None, 0.0, best, acc)
        assert (best.item(), acc.item()) == O.accept(ex, 1.0, np.zeros((2, 1)), 1.0, 0.0)[:2]


def unpack(codes):
    lo, hi = codes & 15, codes >> 4
    return np.stack([lo, hi], axis=-1).reshape(codes.shape[0], -1)


@pytest.mark.parametrize("layout", [B.PQ_SF_LINEAR, B.PQ_SF_TCGEN05])
@pytest.mark.parametrize("N,K,with_perm", [(512, 512, True), (130, 3072, True), (96, 1024, False),
                                           (3, 16384, True)])
def test_quant_weight_bit_exact(layout, N, K, with_perm):
    cfg = small_cfg(N, K)
    w = inputs.weight(cfg, 5, N=N)
    perm = np.random.default_rng(N).permutation(K).astype(np.int32) if with_perm else None
    codes = torch.empty(N, K // 2, dtype=torch.uint8, device=DEV)
    sf = torch.full((B.sf_bytes(N, K, layout),), 0xAA, dtype=torch.uint8, device=DEV)
    ts = torch.zeros(1, dtype=torch.float32, device=DEV)
    ws = B.workspace(B.OP_QUANT_WEIGHT, N, K)
    B.pq_quant_weight(dev(w), None if perm is None else dev(torch.from_numpy(perm)), None, codes, sf, layout,
                      ts, ws)
    wb = inputs.bits(w)
    ts_o = O.tensor_scale(O.calib_stats(wb)[1])
    assert ts.item() == ts_o
    co, so = O.quant_nvfp4(wb, ts_o, perm)
    assert np.array_equal(codes.cpu().numpy(), co)
    if layout == B.PQ_SF_TCGEN05:
        lin = torch.empty(N, K // 16, dtype=torch.uint8, device=DEV)
        B.pq_sf_to_linear(sf, N, K, lin)
        assert np.array_equal(lin.cpu().numpy(), so)
        # padding rows of the last 128-row block are zero
        raw = sf.cpu().numpy().reshape(-1, K // 64, 32, 4, 4)      # [rb][cb][r%32][r/32][c]
        rows_pad = raw.shape[0] * 128
        full = raw.transpose(0, 3, 2, 1, 4).reshape(rows_pad, K // 16)
        assert np.array_equal(full[:N], so) and not full[N:].any()
    else:
        assert np.array_equal(sf.cpu().numpy().reshape(N, K // 16), so)


@pytest.mark.parametrize("N,K", [(64, 256), (5, 8192)])  # four rows per warp / one block per row
def test_quant_weight_device_side_decision(N, K):
    """perm_select = {best, accept} on the device picks the candidate row or the original order."""
    w = inputs.weight(small_cfg(N, K), 6, N=N)
    rng = np.random.default_rng(9)
    table = np.stack([rng.permutation(K) for _ in range(6)]).astype(np.int32)
    for best, accept in [(3, 1), (6, 1), (2, 0)]:
        sel = torch.tensor([best, accept], dtype=torch.int32, device=DEV)
        codes = torch.empty(N, K // 2, dtype=torch.uint8, device=DEV)
        sf = torch.empty(N * K // 16, dtype=torch.uint8, device=DEV)
        ts = torch.zeros(1, dtype=torch.float32, device=DEV)
        B.pq_quant_weight(dev(w), dev(torch.from_numpy(table)), sel, codes, sf, B.PQ_SF_LINEAR, ts,
                          B.workspace(B.OP_QUANT_WEIGHT, N, K))
        co, so = O.quant_nvfp4(inputs.bits(w), ts.item(), table[best - 1] if accept else None)
        assert np.array_equal(codes.cpu().numpy(), co)
        assert np.array_equal(sf.cpu().numpy().reshape(N, -1), so)


@pytest.mark.parametrize("bits,group", [(3, 32), (3, 64), (3, 128), (4, 32), (4, 64), (4, 128), (4, 16), (8, 32)])
@pytest.mark.parametrize("rows,K,with_perm", [(130, 512, False), (33, 3072, True), (4, 16384, True), (40, 16384, True)])
def test_fakequant_int_bit_exact(bits, group, rows, K, with_perm):
    x = inputs.activations(small_cfg(rows, K), 7, 0)
    perm = np.random.default_rng(K).permutation(K).astype(np.int32) if with_perm else None
    out = torch.empty(rows, K, dtype=torch.bfloat16, device=DEV)
    B.pq_fakequant_int(dev(x), (1, bits, group), None if perm is None else dev(torch.from_numpy(perm)), out)
    want = O.fakequant_int(inputs.bits(x), bits, group, perm)
    assert np.array_equal(inputs.bits(out.cpu()), want)
    if perm is not None:        # identity gather == no gather
        ident = torch.arange(K, dtype=torch.int32, device=DEV)
        a = torch.empty_like(out)
        b = torch.empty_like(out)
        B.pq_fakequant_int(dev(x), (1, bits, group), ident, a)
        B.pq_fakequant_int(dev(x), (1, bits, group), None, b)
        assert torch.equal(a.view(torch.int16), b.view(torch.int16))


@pytest.mark.parametrize("rows,K", [(5, 4096), (16, 512), (17, 512), (129, 3072), (300, 1024)])
def test_workspaces_are_not_overrun(rows, K):
    """The reductions write only inside the bytes pq_workspace_bytes asks for (guard words behind them stay)."""
    x = dev(inputs.activations(small_cfg(rows, K), 5, 0))
    ts = dev(torch.tensor([0.02], dtype=torch.float32))
    perms = dev(torch.stack([torch.randperm(K) for _ in range(3)]).to(torch.int32))

    def guarded(op, P=0):
        need = B.workspace_bytes(op, rows, K, 0, P)
        buf = torch.full((need + 4096,), 0xA5, dtype=torch.uint8, device=DEV)
        return buf, buf[:need], need

    buf, ws, need = guarded(B.OP_CALIB_STATS)
    B.pq_calib_stats(x, torch.zeros(K, dtype=torch.float64, device=DEV), torch.zeros(K, dtype=torch.float32, device=DEV), ws)
    assert bool((buf[need:] == 0xA5).all())
    for fmt in FORMATS:
        for pm, P in ((None, 1), (perms, 3)):
            buf, ws, need = guarded(B.OP_GROUP_ERROR, P)
            err = torch.zeros(P, K // fmt[2], dtype=torch.float64, device=DEV)
            B.pq_group_error(x, fmt, ts, pm, err, ws)
            assert bool((buf[need:] == 0xA5).all())


@pytest.mark.parametrize("K", [16, 3072, 16384])
def test_absmax_order_bit_exact_with_ties(K):
    """Tab. 2(a) absmax criterion: same permutation as the oracle, ties included."""
    g = torch.Generator().manual_seed(K)
    amax = (torch.randn(K, generator=g).abs() * 8).round() / 8          # many equal values
    perm = torch.empty(K, dtype=torch.int32, device=DEV)
    B.pq_order_by_absmax(dev(amax.float()), perm, B.workspace(B.OP_SELECT_PERM, 0, K, 0, 1))
    assert np.array_equal(perm.cpu().numpy(), O.order_by_absmax(amax.numpy()))


def test_absmax_order_as_an_extra_candidate_of_the_error_pass():
    rows, K = 200, 512
    x = inputs.activations(small_cfg(rows, K), 3, 0)
    S = torch.zeros(K, dtype=torch.float64, device=DEV)
    A = torch.zeros(K, dtype=torch.float32, device=DEV)
    B.pq_calib_stats(dev(x), S, A, B.workspace(B.OP_CALIB_STATS, rows, K))
    perm = torch.empty(1, K, dtype=torch.int32, device=DEV)
    B.pq_order_by_absmax(A, perm[0], B.workspace(B.OP_SELECT_PERM, 0, K, 0, 1))
    _, A_o = O.calib_stats(inputs.bits(x))
    perm_o = O.order_by_absmax(A_o)
    assert np.array_equal(perm.cpu().numpy()[0], perm_o)
    ts = torch.tensor([0.02], dtype=torch.float32)
    err = torch.zeros(1, K // 16, dtype=torch.float64, device=DEV)
    B.pq_group_error(dev(x), (0, 4, 16), dev(ts), perm, err, B.workspace(B.OP_GROUP_ERROR, rows, K, 0, 1))
    want = O.group_error(inputs.bits(x), 0, 4, 16, ts=ts.item(), perms=perm_o[None, :])
    assert np.array_equal(err.cpu().numpy(), want)
