"""GPU parity, W4A4 GEMM and the whole layer: exact cases bit for bit, general cases against
the fp64 dequantized reference.

Tolerance.  The output is bf16, and rounding a value to bf16 (8 significant bits, nearest even)
alone moves it by up to 2^-8 = 3.9e-3 of its magnitude, so no bf16 result can sit within 2e-3
of the reference element by element.  The 2e-3 budget is therefore applied to what the kernel
computes before that rounding (products are exact, accumulation is fp32), ACC_TOL = 1e-4 of the
largest output, twenty times tighter than the 2e-3 allowed:
  - every output satisfies |Y - Yref| <= 2^-8 |Yref| + ACC_TOL * max|Yref|;
  - counted in bf16 steps: an output whose reference lies further than ACC_TOL * max|Yref| from
    every bf16 rounding boundary EQUALS bf16(Yref); the others (the reference is within the
    accumulation allowance of a boundary, so either neighbour is a correct rounding of a value
    that close) are at most one step away -- for outputs of at least 2^-6 of the largest one, where
    a step is still larger than the allowance;
  - nearly all outputs equal bf16(Yref) exactly."""
import numpy as np
import pytest
import torch

from oracle import compare
from oracle import pq_oracle as O
from paper_2605_09503_b200 import binding as B
from paper_2605_09503_b200 import inputs, pipeline

pytestmark = pytest.mark.gpu
DEV = "cuda"
ACC_TOL = 1e-4          # accumulation error allowed, as a fraction of max|Yref| (budget: 2e-3)


def assert_close(Y, ref, min_exact=0.97):
    ref = np.asarray(ref, dtype=np.float64)
    scale = np.abs(ref).max()
    assert np.isfinite(Y).all()
    assert (np.abs(Y - ref) <= 2.0 ** -8 * np.abs(ref) + ACC_TOL * scale).all()
    bits = torch.from_numpy(np.asarray(Y, dtype=np.float64)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    rep = compare.bf16_step_report(bits, ref, ACC_TOL * scale)
    assert rep["off_clear"] == 0, rep["off_clear"]       # away from a rounding boundary: the very same bf16 value
    big = np.abs(ref) >= 2.0 ** -6 * scale
    assert rep["steps"][big].max(initial=0) <= 1          # near a boundary: the neighbouring value at most
    assert rep["exact"] >= min_exact, rep["exact"]
    return rep


def to_tc(sf_lin):
    """[rows, K/16] scale bytes -> tensor-core layout (host-side restatement of the layout in pq.h)."""
    rows, cols = sf_lin.shape
    rp, cp = (rows + 127) // 128 * 128, (cols + 3) // 4 * 4
    full = np.zeros((rp, cp), np.uint8)
    full[:rows, :cols] = sf_lin
    blk = full.reshape(rp // 128, 4, 32, cp // 4, 4).transpose(0, 3, 2, 1, 4)
    return np.ascontiguousarray(blk).reshape(-1)


def gemm(xq, sfx, tsx, wq, sfw, tsw, ldy=None):
    M, N, K = xq.shape[0], wq.shape[0], xq.shape[1] * 2
    ldy = N if ldy is None else ldy
    buf = torch.full((M, ldy), float("nan"), dtype=torch.bfloat16, device=DEV)
    Y = buf[:, :N]
    ws = B.workspace(B.OP_GEMM, M, K, N)
    d = lambda a: torch.from_numpy(a).to(DEV)
    B.pq_gemm_w4a4(d(xq), d(to_tc(sfx)), torch.tensor([tsx], dtype=torch.float32, device=DEV), d(wq),
                   d(to_tc(sfw)), torch.tensor([tsw], dtype=torch.float32, device=DEV), Y, ws)
    assert B.pq_device_status(ws) == B.PQ_OK
    if ldy > N:
        assert torch.isnan(buf[:, N:].float()).all()          # nothing written outside the tile
    return Y.float().cpu().numpy().astype(np.float64)


def pack(n):
    return (n[:, 0::2] | (n[:, 1::2] << 4)).astype(np.uint8)


def bf16_round(a):
    return torch.from_numpy(np.asarray(a, dtype=np.float64)).to(torch.bfloat16).double().numpy()


@pytest.mark.parametrize("M,N,K", [(128, 192, 64), (8, 8, 64), (1, 192, 128), (130, 200, 320), (256, 384, 512),
                                   (300, 1000, 1024), (129, 3072, 3072)])
def test_exact_cases_bitwise(M, N, K):
    """Codes in {0, +-1, +-2}, power-of-two group scales: every partial sum is exactly
    representable, so the result must equal the reference bit for bit.  Random scales per group
    make any misplacement of a scale byte visible."""
    rng = np.random.default_rng(M + N + K)
    pick = np.array([0, 2, 4, 10, 12], np.uint8)
    xn, wn = pick[rng.integers(0, 5, (M, K))], pick[rng.integers(0, 5, (N, K))]
    pow2 = np.array([0x30, 0x38, 0x40, 0x48], np.uint8)             # 0.5, 1, 2, 4
    sfx, sfw = pow2[rng.integers(0, 4, (M, K // 16))], pow2[rng.integers(0, 4, (N, K // 16))]
    Y = gemm(pack(xn), sfx, 0.5, pack(wn), sfw, 4.0)
    ref = O.gemm_ref(pack(xn), sfx, 0.5, pack(wn), sfw, 4.0)
    assert np.array_equal(Y, bf16_round(ref))


def test_leading_dimension_and_linearity_in_tensor_scale():
    rng = np.random.default_rng(3)
    M, N, K = 140, 264, 192
    xq = rng.integers(0, 256, (M, K // 2)).astype(np.uint8)
    wq = rng.integers(0, 256, (N, K // 2)).astype(np.uint8)
    sfx = rng.integers(0x20, 0x50, (M, K // 16)).astype(np.uint8)
    sfw = rng.integers(0x20, 0x50, (N, K // 16)).astype(np.uint8)
    a = gemm(xq, sfx, 0.25, wq, sfw, 1.0, ldy=272)
    b = gemm(xq, sfx, 0.5, wq, sfw, 1.0)
    assert np.array_equal(2 * a, b)                             # doubling ts_x doubles Y exactly
    ref = O.gemm_ref(xq, sfx, 0.25, wq, sfw, 1.0)
    assert_close(a, ref)


@pytest.mark.parametrize("M,N,K", [(256, 512, 512), (200, 392, 832), (64, 3072, 12288)])
def test_random_codes_and_scales_within_tolerance(M, N, K):
    rng = np.random.default_rng(K)
    xq = rng.integers(0, 256, (M, K // 2)).astype(np.uint8)
    wq = rng.integers(0, 256, (N, K // 2)).astype(np.uint8)
    sfx = rng.integers(0, 0x7F, (M, K // 16)).astype(np.uint8)       # every finite scale byte
    sfw = rng.integers(0, 0x7F, (N, K // 16)).astype(np.uint8)
    Y = gemm(xq, sfx, 1e-3, wq, sfw, 2e-4)
    ref = O.gemm_ref(xq, sfx, 1e-3, wq, sfw, 2e-4)
    assert_close(Y, ref)


@pytest.mark.parametrize("seed,fmt,expect_accept", [(0, (0, 4, 16), 0), (1, (1, 4, 32), 1), (2, (1, 3, 64), 1)])
def test_tiny_layer_end_to_end_against_oracle(seed, fmt, expect_accept):
    """The small configuration, every stage compared with the oracle: statistics, candidates,
    errors, decision, weight codes, activation codes, GEMM.  The error format that drives the
    decision is NVFP4 (rejected on this layer: clustering the outlier channels costs more on
    the activation side than it gains) or an integer format (accepted through the weight side);
    the deployed weight is NVFP4 in the chosen order either way."""
    cfg = inputs.CONFIGS["tiny"]
    group = 16 if fmt[0] == 0 else fmt[2]
    xs = [inputs.activations(cfg, seed, b) for b in range(cfg.calib_batches)]
    w = inputs.weight(cfg, seed)
    cal = pipeline.calibrate([x.to(DEV) for x in xs], w.to(DEV), fmt=fmt)
    # oracle, step by step
    Sa, Aa = None, None
    for x in xs:
        Sa, Aa = O.calib_stats(inputs.bits(x), Sa, Aa)
    Sw, Aw = O.calib_stats(inputs.bits(w))
    ts_x, ts_w = O.tensor_scale(Aa), O.tensor_scale(Aw)
    rows_a = sum(x.shape[0] for x in xs)
    perms = O.select_perm(Sa, rows_a, Sw, w.shape[0], 5)
    cand = np.concatenate([np.arange(cfg.K, dtype=np.int32)[None], perms])
    ex = np.zeros((7, cfg.K // group))
    for x in xs:
        ex = O.group_error(inputs.bits(x), *fmt, ts_x, cand, err=ex)
    ew = O.group_error(inputs.bits(w), *fmt, ts_w, cand)
    best, acc, E = O.accept(ex, O.error_weight(Sa), ew, O.error_weight(Sw), 0.0)
    assert np.array_equal(cal.sumsq_a.cpu().numpy(), Sa) and np.array_equal(cal.sumsq_w.cpu().numpy(), Sw)
    assert cal.ts_x.item() == ts_x and cal.ts_w.item() == ts_w
    assert np.array_equal(cal.perms.cpu().numpy(), perms)
    assert np.array_equal(cal.err_x.cpu().numpy(), ex) and np.array_equal(cal.err_w.cpu().numpy(), ew)
    assert np.array_equal(cal.E.cpu().numpy(), E)
    assert cal.select.tolist() == [best, acc]
    assert acc == expect_accept
    chosen = perms[best - 1] if acc else None
    wq_o, sfw_o = O.quant_nvfp4(inputs.bits(w), ts_w, chosen)
    assert np.array_equal(cal.wq.cpu().numpy(), wq_o)
    # runtime: the producer hands over activations already in permuted order
    x_rt = inputs.activations(cfg, seed, 1000)
    order = cal.chosen_perm().cpu()
    x_perm = x_rt[:, order].contiguous()
    layer = pipeline.QuantLinear(cal.wq, cal.sfw, cal.ts_w, cal.ts_x, cfg.M)
    Y = layer(x_perm.to(DEV))
    layer.check()
    xq_o, sfx_o = O.quant_nvfp4(inputs.bits(x_rt), ts_x, chosen)
    assert np.array_equal(layer.xq.cpu().numpy(), xq_o)
    ref = O.gemm_ref(xq_o, sfx_o, ts_x, wq_o, sfw_o, ts_w)
    got = Y.float().cpu().numpy().astype(np.float64)
    assert_close(got, ref)
    # the quantized product approximates the unquantized one (Eq. 8), better with the chosen order
    exact = O.gemm_bf16_ref(inputs.bits(x_rt), inputs.bits(w))
    rel = np.linalg.norm(got - exact) / np.linalg.norm(exact)
    xq_i, sfx_i = O.quant_nvfp4(inputs.bits(x_rt), ts_x)
    wq_i, sfw_i = O.quant_nvfp4(inputs.bits(w), ts_w)
    rel_ident = np.linalg.norm(O.gemm_ref(xq_i, sfx_i, ts_x, wq_i, sfw_i, ts_w) - exact) / np.linalg.norm(exact)
    assert rel < 0.25
    if not acc:
        assert abs(rel - rel_ident) < 1e-3       # same operands; only the bf16 output rounding differs


def test_identity_order_reproduces_unpermuted_layer():
    """Identity permutation == no permutation, bit for bit, through quantize and GEMM."""
    cfg = inputs.CONFIGS["tiny"]
    x, w = inputs.activations(cfg, 1, 1000).to(DEV), inputs.weight(cfg, 1).to(DEV)
    K, N = cfg.K, cfg.N
    ident = torch.arange(K, dtype=torch.int32, device=DEV)
    outs = []
    for perm in (None, ident):
        wq = torch.empty(N, K // 2, dtype=torch.uint8, device=DEV)
        sfw = torch.empty(B.sf_bytes(N, K, B.PQ_SF_TCGEN05), dtype=torch.uint8, device=DEV)
        ts_w = torch.empty(1, dtype=torch.float32, device=DEV)
        B.pq_quant_weight(w, perm, None, wq, sfw, B.PQ_SF_TCGEN05, ts_w, B.workspace(B.OP_QUANT_WEIGHT, N, K))
        layer = pipeline.QuantLinear(wq, sfw, ts_w, torch.tensor([0.05], device=DEV), cfg.M)
        outs.append((wq.clone(), sfw.clone(), layer(x).clone()))
        layer.check()
    for a, b in zip(*outs):
        assert torch.equal(a.view(torch.uint8) if a.dtype == torch.uint8 else a.view(torch.int16),
                           b.view(torch.uint8) if b.dtype == torch.uint8 else b.view(torch.int16))


def test_full_size_qkv_layer_sampled():
    """The benchmark's workload and launch configuration: 4608 x 3072 -> 9216, sampled outputs
    plus full rows and columns against the fp64 reference, codes against the oracle."""
    cfg = inputs.CONFIGS["qkv"]
    x = inputs.activations(cfg, 0, 1000)
    w = inputs.weight(cfg, 0)
    xb, wb = inputs.bits(x), inputs.bits(w)
    ts_x = O.tensor_scale(O.calib_stats(inputs.bits(inputs.activations(cfg, 0, 0)))[1])
    wq = torch.empty(cfg.N, cfg.K // 2, dtype=torch.uint8, device=DEV)
    sfw = torch.empty(B.sf_bytes(cfg.N, cfg.K, B.PQ_SF_TCGEN05), dtype=torch.uint8, device=DEV)
    ts_w = torch.empty(1, dtype=torch.float32, device=DEV)
    B.pq_quant_weight(w.to(DEV), None, None, wq, sfw, B.PQ_SF_TCGEN05, ts_w,
                      B.workspace(B.OP_QUANT_WEIGHT, cfg.N, cfg.K))
    layer = pipeline.QuantLinear(wq, sfw, ts_w, torch.tensor([ts_x], dtype=torch.float32, device=DEV), cfg.M)
    Y = layer(x.to(DEV)).float().cpu().numpy().astype(np.float64)
    layer.check()
    xq_o, sfx_o = O.quant_nvfp4(xb, ts_x)
    wq_o, sfw_o = O.quant_nvfp4(wb, ts_w.item())
    assert np.array_equal(layer.xq.cpu().numpy(), xq_o)
    assert np.array_equal(wq.cpu().numpy(), wq_o)
    rng = np.random.default_rng(0)
    ms = np.concatenate([rng.integers(0, cfg.M, 16384), np.repeat([0, 127, 128, 4607], cfg.N // 4),
                         rng.integers(0, cfg.M, 4096)])
    ns = np.concatenate([rng.integers(0, cfg.N, 16384), np.tile(np.arange(cfg.N // 4) * 4, 4),
                         np.repeat([0, 191, 192, 9215], 1024)])
    ref = O.gemm_ref_sampled(xq_o, sfx_o, ts_x, wq_o, sfw_o, ts_w.item(), ms, ns)
    assert_close(Y[ms, ns], ref)


def test_bounded_wait_runs_out_and_the_context_stays_usable():
    """The failure path of the GEMM's device-side waits, exercised without a hang or a fault: a wait
    (the helper every role of the kernel uses) on a barrier that nobody arrives at gives up after its
    limit, raises the abort flag, records PQ_ERR_TIMEOUT in the status word and the kernel returns.  The
    word stays set until the caller clears it; after that the same workspace serves a correct GEMM."""
    ws = B.workspace(B.OP_GEMM, 256, 512, 256)
    assert B.pq_device_status(ws) == B.PQ_OK
    waited, abort = B.pq_selftest_wait_expiry(ws, 1_000_000)        # about half a millisecond of SM clock
    assert (waited, abort) == (0, 1)
    assert B.pq_device_status(ws) == 7                               # PQ_ERR_TIMEOUT
    assert B.status_string(7) != "ok"
    ws.zero_()
    assert B.pq_device_status(ws) == B.PQ_OK
    rng = np.random.default_rng(5)
    M, N, K = 256, 256, 512
    pick = np.array([0, 2, 4, 10, 12], np.uint8)
    xn, wn = pick[rng.integers(0, 5, (M, K))], pick[rng.integers(0, 5, (N, K))]
    pow2 = np.array([0x30, 0x38, 0x40, 0x48], np.uint8)
    sfx, sfw = pow2[rng.integers(0, 4, (M, K // 16))], pow2[rng.integers(0, 4, (N, K // 16))]
    d = lambda a: torch.from_numpy(a).to(DEV)
    one = torch.tensor([1.0], dtype=torch.float32, device=DEV)
    Y = torch.empty(M, N, dtype=torch.bfloat16, device=DEV)
    B.pq_gemm_w4a4(d(pack(xn)), d(to_tc(sfx)), one, d(pack(wn)), d(to_tc(sfw)), one, Y, ws)
    assert B.pq_device_status(ws) == B.PQ_OK
    ref = O.gemm_ref(pack(xn), sfx, 1.0, pack(wn), sfw, 1.0)
    assert np.array_equal(Y.float().cpu().numpy().astype(np.float64), bf16_round(ref))
