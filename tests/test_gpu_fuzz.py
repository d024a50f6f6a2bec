"""Seeded random shapes, leading dimensions and formats through every streaming entry point, each compared
bit for bit with the oracle, with guard bytes behind every output and workspace (nothing may be written
outside what the header says).  The GEMM gets random small shapes against the fp64 reference."""
import numpy as np
import pytest
import torch

from oracle import pq_oracle as O
from paper_2605_09503_b200 import binding as B
from paper_2605_09503_b200 import inputs
from test_gpu_gemm import assert_close, to_tc

pytestmark = pytest.mark.gpu
DEV = "cuda"
GUARD = 0x5A


def guarded(nbytes, dtype=torch.uint8):
    """(whole buffer, view of the first nbytes as dtype): 512 guard bytes follow the view."""
    buf = torch.full((nbytes + 512,), GUARD, dtype=torch.uint8, device=DEV)
    return buf, buf[:nbytes].view(dtype)


def intact(buf, nbytes):
    return bool((buf[nbytes:] == GUARD).all())


def strided_input(rng, rows, K, ld):
    """bf16 [rows, K] with leading dimension ld (device view and the contiguous host bits)."""
    scale = np.exp(rng.standard_normal(K)).astype(np.float32)
    x = torch.from_numpy((rng.standard_normal((rows, K)).astype(np.float32) * scale)).to(torch.bfloat16)
    full = torch.full((rows, ld), float("nan"), dtype=torch.bfloat16)
    full[:, :K] = x
    return full.to(DEV)[:, :K], inputs.bits(x)


CASES = list(range(12))


@pytest.mark.parametrize("case", CASES)
def test_streaming_entry_points_on_random_shapes(case):
    rng = np.random.default_rng(1000 + case)
    rows = int(rng.integers(1, 400))
    K = int(rng.choice([64, 128, 192, 320, 512, 1024, 1536, 3072, 4096]))
    ld = K + 8 * int(rng.integers(0, 5))
    xd, xb = strided_input(rng, rows, K, ld)
    ts = float(np.float32(rng.uniform(0.003, 0.05)))
    tsd = torch.tensor([ts], dtype=torch.float32, device=DEV)
    perm = rng.permutation(K).astype(np.int32)
    permd = torch.from_numpy(perm).to(DEV)

    # statistics (accumulating onto earlier totals)
    S0, A0 = rng.random(K) * 10, rng.random(K).astype(np.float32)
    S = torch.from_numpy(S0.copy()).to(DEV)
    A = torch.from_numpy(A0.copy()).to(DEV)
    need = B.workspace_bytes(B.OP_CALIB_STATS, rows, K)
    wbuf, ws = guarded(need)
    B.pq_calib_stats(xd, S, A, ws)
    So, Ao = O.calib_stats(xb, S0.copy(), A0.copy())
    assert np.array_equal(S.cpu().numpy(), So) and np.array_equal(A.cpu().numpy(), Ao) and intact(wbuf, need)

    # activation quantizer, both layouts
    for layout in (B.PQ_SF_LINEAR, B.PQ_SF_TCGEN05):
        cbuf, codes = guarded(rows * K // 2)
        nsf = B.sf_bytes(rows, K, layout)
        sbuf, sf = guarded(nsf)
        B.pq_quant_act_nvfp4(xd, tsd, codes.view(rows, K // 2), sf, layout)
        c_o, s_o = O.quant_nvfp4(xb, ts)
        assert np.array_equal(codes.cpu().numpy().reshape(rows, K // 2), c_o)
        want = s_o.reshape(-1) if layout == B.PQ_SF_LINEAR else to_tc(s_o)
        assert np.array_equal(sf.cpu().numpy(), want) and intact(cbuf, rows * K // 2) and intact(sbuf, nsf)

    # group errors, original order and two candidate orders, one random format
    fmt = [(B.KIND_NVFP4, 4, 16), (B.KIND_INT, 3, 32), (B.KIND_INT, 4, 64), (B.KIND_INT, 4, 16)][case % 4]
    for pm, P in ((None, 1), (np.stack([perm, np.arange(K, dtype=np.int32)]), 2)):
        need = B.workspace_bytes(B.OP_GROUP_ERROR, rows, K, 0, P)
        wbuf, ws = guarded(need)
        ebuf, err = guarded(P * (K // fmt[2]) * 8, torch.float64)
        err.zero_()
        B.pq_group_error(xd, fmt, tsd, None if pm is None else torch.from_numpy(pm).to(DEV), err.view(P, -1), ws)
        e_o = O.group_error(xb, *fmt, ts=ts, perms=pm)
        assert np.array_equal(err.cpu().numpy().reshape(P, -1), e_o)
        assert intact(wbuf, need) and intact(ebuf, P * (K // fmt[2]) * 8)

    # integer fake-quant with and without the gather, output with its own leading dimension
    bits, group = [(3, 32), (4, 64), (4, 16), (8, 32)][case % 4]
    for pm in (None, perm):
        ldo = K + 8
        obuf, out = guarded(rows * ldo * 2, torch.bfloat16)
        out = out.view(rows, ldo)
        B.pq_fakequant_int(xd, (B.KIND_INT, bits, group), None if pm is None else permd, out[:, :K])
        got = inputs.bits(out.cpu())
        assert np.array_equal(got[:, :K], O.fakequant_int(xb, bits, group, pm))
        assert np.all(got[:, K:] == (GUARD | (GUARD << 8))) and intact(obuf, rows * ldo * 2)

    # fused producer
    a = rng.standard_normal(K).astype(np.float32) * 0.3
    b = rng.standard_normal(K).astype(np.float32)
    kind = case % 2
    cbuf, codes = guarded(rows * K // 2)
    nsf = B.sf_bytes(rows, K, B.PQ_SF_TCGEN05)
    sbuf, sf = guarded(nsf)
    B.pq_norm_quant_nvfp4(xd, kind, torch.from_numpy(a).to(DEV), torch.from_numpy(b).to(DEV), 1e-6, permd, tsd,
                          codes.view(rows, K // 2), sf, B.PQ_SF_TCGEN05)
    c_o, s_o, _ = O.norm_quant_nvfp4(xb, kind, a, b, 1e-6, ts, perm)
    assert np.array_equal(codes.cpu().numpy().reshape(rows, K // 2), c_o)
    assert np.array_equal(sf.cpu().numpy(), to_tc(s_o)) and intact(cbuf, rows * K // 2) and intact(sbuf, nsf)


@pytest.mark.parametrize("case", range(8))
def test_weight_quantizer_and_gemm_on_random_shapes(case):
    rng = np.random.default_rng(2000 + case)
    M = int(rng.integers(1, 700))
    N = 8 * int(rng.integers(1, 90))
    K = 64 * int(rng.integers(1, 24))
    xd, xb = strided_input(rng, M, K, K)
    wd, wb = strided_input(rng, N, K, K + 8 * int(rng.integers(0, 3)))
    perm = rng.permutation(K).astype(np.int32) if case % 2 else None
    ts_x = float(np.float32(np.abs(O.bf16_to_f32(xb)).max() / 2688.0))
    cbuf, wq = guarded(N * K // 2)
    nsf = B.sf_bytes(N, K, B.PQ_SF_TCGEN05)
    sbuf, sfw = guarded(nsf)
    ts_w = torch.empty(1, dtype=torch.float32, device=DEV)
    B.pq_quant_weight(wd, None if perm is None else torch.from_numpy(perm).to(DEV), None, wq.view(N, K // 2), sfw,
                      B.PQ_SF_TCGEN05, ts_w, B.workspace(B.OP_QUANT_WEIGHT, N, K))
    assert ts_w.item() == O.tensor_scale(np.abs(O.bf16_to_f32(wb)).max(axis=0))
    wq_o, sfw_o = O.quant_nvfp4(wb, ts_w.item(), perm)
    assert np.array_equal(wq.cpu().numpy().reshape(N, K // 2), wq_o) and np.array_equal(sfw.cpu().numpy(), to_tc(sfw_o))
    assert intact(cbuf, N * K // 2) and intact(sbuf, nsf)
    # runtime path on activations already in the permuted order
    xpb = xb if perm is None else np.ascontiguousarray(xb[:, perm])
    xq = torch.empty(M, K // 2, dtype=torch.uint8, device=DEV)
    sfx = torch.empty(B.sf_bytes(M, K, 1), dtype=torch.uint8, device=DEV)
    ybuf, Y = guarded(M * N * 2, torch.bfloat16)
    tsd = torch.tensor([ts_x], dtype=torch.float32, device=DEV)
    ws = B.workspace(B.OP_GEMM, M, K, N)
    B.pq_linear_w4a4(inputs.from_bits(xpb).to(DEV), tsd, xq, sfx, wq.view(N, K // 2), sfw, ts_w, Y.view(M, N), ws)
    assert B.pq_device_status(ws) == B.PQ_OK and intact(ybuf, M * N * 2)
    xq_o, sfx_o = O.quant_nvfp4(xpb, ts_x)
    assert np.array_equal(xq.cpu().numpy(), xq_o)
    ref = O.gemm_ref(xq_o, sfx_o, ts_x, wq_o, sfw_o, ts_w.item())
    assert_close(Y.view(M, N).float().cpu().numpy().astype(np.float64), ref, min_exact=0.95)


@pytest.mark.parametrize("case", list(range(10)))
def test_hadamard_producer_and_orders_on_random_shapes(case):
    """Random row counts, widths (powers of two and 12 * 2^n), leading dimensions and scale layouts through
    the PermuQuant-H producer, plus the first-moment pass and the variance / round-robin orders, with guard
    bytes behind every output."""
    rng = np.random.default_rng(5000 + case)
    rows = int(rng.integers(1, 300))
    K = int(rng.choice([64, 96, 128, 192, 384, 512, 768, 1536, 2048, 3072, 6144]))
    ld = K + 8 * int(rng.integers(0, 5))
    xd, xb = strided_input(rng, rows, K, ld)
    ts = float(np.float32(rng.uniform(0.003, 0.05)))
    tsd = torch.tensor([ts], dtype=torch.float32, device=DEV)
    perm = rng.permutation(K).astype(np.int32)
    layout = B.PQ_SF_TCGEN05 if K % 64 == 0 and rng.random() < 0.5 else B.PQ_SF_LINEAR
    cbuf, codes = guarded(rows * K // 2)
    nsf = B.sf_bytes(rows, K, layout)
    sbuf, sf = guarded(nsf)
    ybuf, y = guarded(rows * K * 2, torch.bfloat16)
    B.pq_hadamard_quant_nvfp4(xd, torch.from_numpy(perm).to(DEV), tsd, codes.view(rows, K // 2), sf, layout, y.view(rows, K))
    c_o, s_o, y_o, _ = O.hadamard_quant_nvfp4(xb, ts, perm)
    assert np.array_equal(codes.view(rows, K // 2).cpu().numpy(), c_o)
    assert np.array_equal(inputs.bits(y.view(rows, K).cpu()), y_o)
    want_sf = to_tc(s_o) if layout == B.PQ_SF_TCGEN05 else s_o.reshape(-1)
    assert np.array_equal(sf.cpu().numpy(), want_sf)
    assert intact(cbuf, rows * K // 2) and intact(sbuf, nsf) and intact(ybuf, rows * K * 2)

    T0 = rng.standard_normal(K)
    T = torch.from_numpy(T0.copy()).to(DEV)
    need = B.workspace_bytes(B.OP_CALIB_STATS, rows, K)
    wbuf, ws = guarded(need)
    B.pq_calib_sum(xd, T, ws)
    To = O.calib_sum(xb, T0.copy())
    assert np.array_equal(T.cpu().numpy(), To) and intact(wbuf, need)
    So, _ = O.calib_stats(xb)
    need = B.workspace_bytes(B.OP_SELECT_PERM, 0, K, 0, 1)
    wbuf, ws = guarded(need)
    pbuf, p = guarded(K * 4, torch.int32)
    Sd = torch.from_numpy(So).to(DEV)
    B.pq_order_by_variance(T, Sd, rows, p, ws)
    assert np.array_equal(p.cpu().numpy(), O.order_by_variance(To, So, rows)) and intact(pbuf, K * 4)
    group = int(rng.choice([16, 32, 64]))
    B.pq_order_round_robin(Sd, group, p, ws)
    assert np.array_equal(p.cpu().numpy(), O.order_round_robin(So, group)) and intact(pbuf, K * 4) and intact(wbuf, need)
