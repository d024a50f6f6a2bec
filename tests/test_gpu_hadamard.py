"""GPU parity of the PermuQuant-H producer (App. D: Hadamard transform, reordered read-out, NVFP4 quantizer)
against the oracle: codes, scale bytes and the bf16 output bit for bit; and the layer identity
(x H P)(Wt H P)^T = x Wt^T through the W4A4 GEMM."""
import numpy as np
import pytest
import torch

from oracle import pq_oracle as O
from paper_2605_09503_b200 import binding as B
from paper_2605_09503_b200 import inputs
from test_gpu_gemm import assert_close, to_tc

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _case(M, K, seed):
    g = torch.Generator().manual_seed(seed)
    scale = torch.exp(1.5 * torch.randn(K, generator=g))
    x = (torch.randn(M, K, generator=g) * scale).to(torch.bfloat16)
    perm = torch.randperm(K, generator=g).to(torch.int32)
    return x, perm


# widths: powers of two (one pass, two passes, none), 12 * 2^n (FLUX: 3072 and 12288), ragged row counts
@pytest.mark.parametrize("layout", [B.PQ_SF_LINEAR, B.PQ_SF_TCGEN05])
@pytest.mark.parametrize("M,K,with_perm", [(37, 3072, True), (130, 3072, False), (9, 12288, True), (300, 1024, True),
                                           (5, 64, False), (23, 1536, True), (17, 192, True), (3, 16384, True),
                                           (70, 256, True), (12, 768, True), (1, 4096, True),
                                           # blocks of three rows (16384 channels) and of six (8192), more than one batch
                                           (8, 16384, True), (13, 8192, True)])
def test_hadamard_quant_bit_exact(layout, M, K, with_perm):
    x, perm = _case(M, K, seed=M + K)
    ts = 0.02
    codes = torch.empty(M, K // 2, dtype=torch.uint8, device=DEV)
    sf = torch.full((B.sf_bytes(M, K, layout),), 0xEE, dtype=torch.uint8, device=DEV)
    y = torch.empty(M, K, dtype=torch.bfloat16, device=DEV)
    B.pq_hadamard_quant_nvfp4(x.to(DEV), perm.to(DEV) if with_perm else None,
                              torch.tensor([ts], dtype=torch.float32, device=DEV), codes, sf, layout, y)
    c_o, s_o, y_o, _ = O.hadamard_quant_nvfp4(inputs.bits(x), ts, perm.numpy() if with_perm else None)
    assert np.array_equal(inputs.bits(y.cpu()), y_o)
    assert np.array_equal(codes.cpu().numpy(), c_o)
    if layout == B.PQ_SF_LINEAR:
        assert np.array_equal(sf.cpu().numpy().reshape(M, K // 16), s_o)
    else:
        assert np.array_equal(sf.cpu().numpy(), to_tc(s_o))      # padding rows hold zero scale bytes


def test_transform_only_and_small_widths():
    for M, K in ((7, 16), (4, 32), (33, 96), (2, 48 * 4)):
        x, perm = _case(M, K, seed=K)
        y = torch.empty(M, K, dtype=torch.bfloat16, device=DEV)
        B.pq_hadamard_quant_nvfp4(x.to(DEV), perm.to(DEV), None, None, None, B.PQ_SF_LINEAR, y)
        _, _, y_o, _ = O.hadamard_quant_nvfp4(inputs.bits(x), 1.0, perm.numpy(), quantize=False)
        assert np.array_equal(inputs.bits(y.cpu()), y_o)
    x, _ = _case(4, 80, seed=1)                                   # 5 * 16: no transform defined for it
    with pytest.raises(B.PqError):
        B.pq_hadamard_quant_nvfp4(x.to(DEV), None, None, None, None, B.PQ_SF_LINEAR,
                                  torch.empty(4, 80, dtype=torch.bfloat16, device=DEV))
    with pytest.raises(B.PqError):                                # 12 * 4: segments shorter than one 16-byte load
        B.pq_hadamard_quant_nvfp4(x[:, :48].contiguous().to(DEV), None, None, None, None, B.PQ_SF_LINEAR,
                                  torch.empty(4, 48, dtype=torch.bfloat16, device=DEV))


def test_strided_rows():
    M, K = 40, 3072
    x, perm = _case(M, 2 * K, seed=9)
    xv = x.to(DEV)[:, :K]                                        # leading dimension 2 K
    codes = torch.empty(M, K // 2, dtype=torch.uint8, device=DEV)
    sf = torch.empty(M * K // 16, dtype=torch.uint8, device=DEV)
    p = torch.randperm(K, generator=torch.Generator().manual_seed(3)).to(torch.int32)
    B.pq_hadamard_quant_nvfp4(xv, p.to(DEV), torch.tensor([0.05], dtype=torch.float32, device=DEV), codes, sf,
                              B.PQ_SF_LINEAR, None)
    c_o, s_o, _, _ = O.hadamard_quant_nvfp4(inputs.bits(x[:, :K].contiguous()), 0.05, p.numpy())
    assert np.array_equal(codes.cpu().numpy(), c_o) and np.array_equal(sf.cpu().numpy().reshape(M, K // 16), s_o)


def test_transformed_layer_reproduces_the_plain_product():
    """PermuQuant-H end to end on a small layer: activations and weight rows go through the same transform
    and the same order, so the quantized product approximates x Wt^T, and the GEMM on the transformed
    operands equals the fp64 reference built from the oracle's transformed codes."""
    cfg = inputs.CONFIGS["tiny"]
    M, K, N = 256, 512, 384
    x, perm = _case(M, K, seed=21)
    w = (0.02 * torch.randn(N, K, generator=torch.Generator().manual_seed(22))).to(torch.bfloat16)
    d = lambda t: t.to(DEV)
    # weight side: transform rows, then the ordinary permuted weight quantizer
    wh = torch.empty(N, K, dtype=torch.bfloat16, device=DEV)
    B.pq_hadamard_quant_nvfp4(d(w), None, None, None, None, B.PQ_SF_LINEAR, wh)
    wq = torch.empty(N, K // 2, dtype=torch.uint8, device=DEV)
    sfw = torch.empty(B.sf_bytes(N, K, 1), dtype=torch.uint8, device=DEV)
    ts_w = torch.empty(1, dtype=torch.float32, device=DEV)
    B.pq_quant_weight(wh, d(perm), None, wq, sfw, B.PQ_SF_TCGEN05, ts_w, B.workspace(B.OP_QUANT_WEIGHT, N, K))
    # activation side: transform + order + quantize in one kernel, tensor scale from the transformed absmax
    xh = torch.empty(M, K, dtype=torch.bfloat16, device=DEV)
    B.pq_hadamard_quant_nvfp4(d(x), None, None, None, None, B.PQ_SF_LINEAR, xh)
    ts_x = (xh.float().abs().max() / 2688.0).reshape(1).contiguous()
    xq = torch.empty(M, K // 2, dtype=torch.uint8, device=DEV)
    sfx = torch.empty(B.sf_bytes(M, K, 1), dtype=torch.uint8, device=DEV)
    B.pq_hadamard_quant_nvfp4(d(x), d(perm), ts_x, xq, sfx, B.PQ_SF_TCGEN05, None)
    Y = torch.empty(M, N, dtype=torch.bfloat16, device=DEV)
    ws = B.workspace(B.OP_GEMM, M, K, N)
    B.pq_gemm_w4a4(xq, sfx, ts_x, wq, sfw, ts_w, Y, ws)
    assert B.pq_device_status(ws) == B.PQ_OK
    # oracle route for the same operands
    _, _, wh_o, _ = O.hadamard_quant_nvfp4(inputs.bits(w), 1.0, quantize=False)
    assert np.array_equal(inputs.bits(wh.cpu()), wh_o)
    tsw_o = O.tensor_scale(O.calib_stats(wh_o)[1])
    wq_o, sfw_o = O.quant_nvfp4(wh_o, tsw_o, perm.numpy())
    xq_o, sfx_o, _, _ = O.hadamard_quant_nvfp4(inputs.bits(x), float(ts_x.item()), perm.numpy())
    assert np.array_equal(xq.cpu().numpy(), xq_o) and np.array_equal(wq.cpu().numpy(), wq_o)
    ref = O.gemm_ref(xq_o, sfx_o, float(ts_x.item()), wq_o, sfw_o, tsw_o)
    assert_close(Y.float().cpu().numpy().astype(np.float64), ref)
    # and the transformed, quantized layer is close to the unquantized product (the rotation cancels)
    plain = x.double().numpy() @ w.double().numpy().T
    rel = np.linalg.norm(ref - plain) / np.linalg.norm(plain)
    assert rel < 0.15, rel


def test_permuquant_h_pipeline_against_the_oracle_route():
    """calibrate_h + QuantLinearH on the small layer: every decision equals the oracle's taken on the
    oracle's own transformed tensors, and the layer output stays within the GEMM tolerance of the fp64
    reference of the transformed, reordered, quantized operands."""
    from paper_2605_09503_b200 import pipeline
    cfg = inputs.CONFIGS["tiny"]
    seed, fmt = 1, (B.KIND_INT, 4, 32)
    xs = [inputs.activations(cfg, seed, b) for b in range(2)]
    w = inputs.weight(cfg, seed)
    cal = pipeline.calibrate_h([x.to(DEV) for x in xs], w.to(DEV), fmt=fmt)
    # oracle: transform, then the ordinary offline pass
    xh = [O.hadamard_quant_nvfp4(inputs.bits(x), 1.0, quantize=False)[2] for x in xs]
    wh = O.hadamard_quant_nvfp4(inputs.bits(w), 1.0, quantize=False)[2]
    Sa = Aa = None
    for x in xh:
        Sa, Aa = O.calib_stats(x, Sa, Aa)
    Sw, Aw = O.calib_stats(wh)
    ts_x, ts_w = O.tensor_scale(Aa), O.tensor_scale(Aw)
    perms = O.select_perm(Sa, sum(x.shape[0] for x in xh), Sw, wh.shape[0], 5)
    cand = np.concatenate([np.arange(cfg.K, dtype=np.int32)[None], perms])
    ex = np.zeros((7, cfg.K // fmt[2]))
    for x in xh:
        ex = O.group_error(x, *fmt, ts_x, cand, err=ex)
    ew = O.group_error(wh, *fmt, ts_w, cand)
    best, acc, _ = O.accept(ex, O.error_weight(Sa), ew, O.error_weight(Sw), 0.0)
    assert np.array_equal(cal.sumsq_a.cpu().numpy(), Sa) and np.array_equal(cal.perms.cpu().numpy(), perms)
    assert np.array_equal(cal.err_x.cpu().numpy(), ex) and cal.select.tolist() == [best, acc]
    chosen = perms[best - 1] if acc else None
    wq_o, sfw_o = O.quant_nvfp4(wh, ts_w, chosen)
    assert np.array_equal(cal.wq.cpu().numpy(), wq_o)
    # runtime
    x_rt = inputs.activations(cfg, seed, 1000)
    order = cal.chosen_perm() if acc else None
    layer = pipeline.QuantLinearH(cal.wq, cal.sfw, cal.ts_w, cal.ts_x, cfg.M, order)
    Y = layer(x_rt.to(DEV)).float().cpu().numpy().astype(np.float64)
    layer.check()
    xq_o, sfx_o, _, _ = O.hadamard_quant_nvfp4(inputs.bits(x_rt), ts_x, chosen)
    assert np.array_equal(layer.xq.cpu().numpy(), xq_o)
    assert_close(Y, O.gemm_ref(xq_o, sfx_o, ts_x, wq_o, sfw_o, ts_w))
