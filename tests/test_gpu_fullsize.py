"""GPU parity at the workloads' full sizes, in the launch configurations bench.py times: the streaming
kernels bit for bit against the oracle on whole tensors, the long-K and the many-token GEMM on
sampled outputs against the fp64 reference, the batched path against the serial one."""
import numpy as np
import pytest
import torch

from oracle import pq_oracle as O
from paper_2605_09503_b200 import binding as B
from paper_2605_09503_b200 import inputs, pipeline
from test_gpu_gemm import assert_close

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _weights(cfg, seed=0):
    w = inputs.weight(cfg, seed)
    wq = torch.empty(cfg.N, cfg.K // 2, dtype=torch.uint8, device=DEV)
    sfw = torch.empty(B.sf_bytes(cfg.N, cfg.K, B.PQ_SF_TCGEN05), dtype=torch.uint8, device=DEV)
    ts_w = torch.empty(1, dtype=torch.float32, device=DEV)
    B.pq_quant_weight(w.to(DEV), None, None, wq, sfw, B.PQ_SF_TCGEN05, ts_w, B.workspace(B.OP_QUANT_WEIGHT, cfg.N, cfg.K))
    return w, wq, sfw, ts_w


def test_statistics_and_errors_on_a_full_calibration_batch():
    cfg = inputs.CONFIGS["qkv"]
    x = inputs.activations(cfg, 0, 0)
    xb, xd = inputs.bits(x), x.to(DEV)
    S = torch.zeros(cfg.K, dtype=torch.float64, device=DEV)
    A = torch.zeros(cfg.K, dtype=torch.float32, device=DEV)
    B.pq_calib_stats(xd, S, A, B.workspace(B.OP_CALIB_STATS, cfg.M, cfg.K))
    So, Ao = O.calib_stats(xb)
    assert np.array_equal(S.cpu().numpy(), So) and np.array_equal(A.cpu().numpy(), Ao)
    ts = O.tensor_scale(Ao)
    tsd = torch.tensor([ts], dtype=torch.float32, device=DEV)
    ws = B.workspace(B.OP_GROUP_ERROR, cfg.M, cfg.K, 0, 1)
    for fmt in ((B.KIND_NVFP4, 4, 16), (B.KIND_INT, 4, 64), (B.KIND_INT, 3, 128)):
        err = torch.zeros(1, cfg.K // fmt[2], dtype=torch.float64, device=DEV)
        B.pq_group_error(xd, fmt, tsd, None, err, ws)
        assert np.array_equal(err.cpu().numpy(), O.group_error(xb, *fmt, ts=ts)), fmt
    # activation quantizer, both scale layouts, whole tensor
    xq = torch.empty(cfg.M, cfg.K // 2, dtype=torch.uint8, device=DEV)
    sf = torch.empty(B.sf_bytes(cfg.M, cfg.K, B.PQ_SF_LINEAR), dtype=torch.uint8, device=DEV)
    B.pq_quant_act_nvfp4(xd, tsd, xq, sf, B.PQ_SF_LINEAR)
    xq_o, sf_o = O.quant_nvfp4(xb, ts)
    assert np.array_equal(xq.cpu().numpy(), xq_o)
    assert np.array_equal(sf.cpu().numpy().reshape(cfg.M, cfg.K // 16), sf_o)
    # integer fake-quant, whole tensor
    out = torch.empty(cfg.M, cfg.K, dtype=torch.bfloat16, device=DEV)
    B.pq_fakequant_int(xd, (B.KIND_INT, 4, 64), None, out)
    assert np.array_equal(inputs.bits(out.cpu()), O.fakequant_int(xb, 4, 64))


def test_eight_stacked_batches_equal_eight_calls():
    """One call on 8 stacked batches gives the same statistics and errors as 8 calls only when the batch
    rows are a multiple of the 128-row slab (4608 = 36 slabs): the stacked call is what bench.py times."""
    cfg = inputs.CONFIGS["qkv"]
    xs = [inputs.activations(cfg, 0, b).to(DEV) for b in range(8)]
    big = torch.cat(xs)
    K = cfg.K
    ts = torch.tensor([0.05], dtype=torch.float32, device=DEV)

    def run(tensors):
        rows = tensors[0].shape[0]
        S = torch.zeros(K, dtype=torch.float64, device=DEV)
        A = torch.zeros(K, dtype=torch.float32, device=DEV)
        E = torch.zeros(1, K // 16, dtype=torch.float64, device=DEV)
        ws_s = B.workspace(B.OP_CALIB_STATS, rows, K)
        ws_e = B.workspace(B.OP_GROUP_ERROR, rows, K, 0, 1)
        for t in tensors:
            B.pq_calib_stats(t, S, A, ws_s)
            B.pq_group_error(t, (B.KIND_NVFP4, 4, 16), ts, None, E, ws_e)
        return S.cpu(), A.cpu(), E.cpu()

    one, eight = run([big]), run(xs)
    for a, b in zip(one, eight):
        assert torch.equal(a, b)
    # and one of the batches against the oracle, through the accumulating path
    So, _ = O.calib_stats(inputs.bits(xs[0].cpu()))
    S = torch.zeros(K, dtype=torch.float64, device=DEV)
    A = torch.zeros(K, dtype=torch.float32, device=DEV)
    B.pq_calib_stats(xs[0], S, A, B.workspace(B.OP_CALIB_STATS, cfg.M, K))
    assert np.array_equal(S.cpu().numpy(), So)


def test_full_size_mlp_down_layer_sampled():
    """Long K: 4608 x 12288 -> 3072.  Codes of sampled rows bit for bit, sampled outputs within tolerance."""
    cfg = inputs.CONFIGS["mlp_down"]
    x = inputs.activations(cfg, 0, 1000)
    w, wq, sfw, ts_w = _weights(cfg)
    ts_x = float(np.float32(np.float32(x.float().abs().max().item()) / np.float32(2688.0)))
    layer = pipeline.QuantLinear(wq, sfw, ts_w, torch.tensor([ts_x], dtype=torch.float32, device=DEV), cfg.M)
    Y = layer(x.to(DEV)).float().cpu().numpy().astype(np.float64)
    layer.check()
    rows = np.array([0, 1, 127, 128, 2047, 2304, 4479, 4607])
    xq_o, sfx_o = O.quant_nvfp4(np.ascontiguousarray(inputs.bits(x)[rows]), ts_x)
    assert np.array_equal(layer.xq.cpu().numpy()[rows], xq_o)
    wq_o, sfw_o = O.quant_nvfp4(inputs.bits(w), ts_w.item())
    assert np.array_equal(wq.cpu().numpy(), wq_o)
    ref = O.gemm_ref(xq_o, sfx_o, ts_x, wq_o, sfw_o, ts_w.item())          # 8 full rows
    assert_close(Y[rows], ref)


def test_many_token_qkv_gemm_sampled():
    """M = 18432 (the largest token count of the DiT-block sweep): 72 x 48 tiles, several rounds per CTA pair."""
    cfg = inputs.CONFIGS["qkv"]
    M = 18432
    x = inputs.plain_activations(M, cfg.K, 5)
    w, wq, sfw, ts_w = _weights(cfg)
    ts_x = float(np.float32(np.float32(x.float().abs().max().item()) / np.float32(2688.0)))
    layer = pipeline.QuantLinear(wq, sfw, ts_w, torch.tensor([ts_x], dtype=torch.float32, device=DEV), M)
    Y = layer(x.to(DEV)).float().cpu().numpy().astype(np.float64)
    layer.check()
    rows = np.array([0, 255, 256, 9215, 9216, 13000, 18175, 18431])
    xq_o, sfx_o = O.quant_nvfp4(np.ascontiguousarray(inputs.bits(x)[rows]), ts_x)
    assert np.array_equal(layer.xq.cpu().numpy()[rows], xq_o)
    wq_o, sfw_o = O.quant_nvfp4(inputs.bits(w), ts_w.item())
    assert_close(Y[rows], O.gemm_ref(xq_o, sfx_o, ts_x, wq_o, sfw_o, ts_w.item()))


def test_full_size_batched_equals_serial():
    cfg = inputs.CONFIGS["qkv"]
    w, wq, sfw, ts_w = _weights(cfg)
    xs = [inputs.activations(cfg, 0, 1000 + i).to(DEV) for i in range(6)]
    ts_x = torch.tensor([0.3], dtype=torch.float32, device=DEV)
    layer = pipeline.QuantLinear(wq, sfw, ts_w, ts_x, cfg.M)
    ref = [layer(x).clone() for x in xs]
    ys = [torch.zeros(cfg.M, cfg.N, dtype=torch.bfloat16, device=DEV) for _ in xs]
    layer.forward_batches(xs, ys, n_sets=4)
    torch.cuda.synchronize()
    layer.check()
    for y, r in zip(ys, ref):
        assert torch.equal(y.view(torch.int16), r.view(torch.int16))


def test_repeated_launches_give_the_same_bits():
    """The same product 1200 times, serial and batched: every launch must reproduce the first one
    bit for bit (a rare ordering fault inside the kernel shows up as a few wrong 32-row blocks in one
    launch out of several hundred, which a single comparison against the oracle does not catch)."""
    cfg = inputs.CONFIGS["qkv"]
    w, wq, sfw, ts_w = _weights(cfg)
    xs = [inputs.activations(cfg, 0, 2000 + i).to(DEV) for i in range(4)]
    ts_x = torch.tensor([0.3], dtype=torch.float32, device=DEV)
    layer = pipeline.QuantLinear(wq, sfw, ts_w, ts_x, cfg.M)
    ref = [layer(x).clone() for x in xs]
    ys = [torch.zeros(cfg.M, cfg.N, dtype=torch.bfloat16, device=DEV) for _ in xs]
    wrong = 0
    for rep in range(150):
        layer.forward_batches(xs, ys, n_sets=4)
        wrong += sum(int(not torch.equal(y.view(torch.int16), r.view(torch.int16))) for y, r in zip(ys, ref))
        for x, r in zip(xs, ref):
            wrong += int(not torch.equal(layer(x).view(torch.int16), r.view(torch.int16)))
    layer.check()
    assert wrong == 0


def test_hadamard_producer_and_new_statistics_on_a_full_batch():
    """The bench's stage sizes for the kernels added after the first set: the PermuQuant-H producer on the whole
    4608 x 3072 batch (codes, scales in the tensor-core layout, bf16 output), the first-moment pass and the
    group-256 error, all bit for bit."""
    from test_gpu_gemm import to_tc
    cfg = inputs.CONFIGS["qkv"]
    x = inputs.activations(cfg, 0, 3)
    xb, xd = inputs.bits(x), x.to(DEV)
    g = torch.Generator().manual_seed(11)
    perm = torch.randperm(cfg.K, generator=g).to(torch.int32)
    _, _, yh, _ = O.hadamard_quant_nvfp4(xb, 1.0, quantize=False)
    ts = O.tensor_scale(O.calib_stats(yh)[1])
    tsd = torch.tensor([ts], dtype=torch.float32, device=DEV)
    xq = torch.empty(cfg.M, cfg.K // 2, dtype=torch.uint8, device=DEV)
    sf = torch.empty(B.sf_bytes(cfg.M, cfg.K, B.PQ_SF_TCGEN05), dtype=torch.uint8, device=DEV)
    y = torch.empty(cfg.M, cfg.K, dtype=torch.bfloat16, device=DEV)
    B.pq_hadamard_quant_nvfp4(xd, perm.to(DEV), tsd, xq, sf, B.PQ_SF_TCGEN05, y)
    c_o, s_o, y_o, _ = O.hadamard_quant_nvfp4(xb, ts, perm.numpy())
    assert np.array_equal(xq.cpu().numpy(), c_o)
    assert np.array_equal(sf.cpu().numpy(), to_tc(s_o))
    assert np.array_equal(inputs.bits(y.cpu()), y_o)
    T = torch.zeros(cfg.K, dtype=torch.float64, device=DEV)
    B.pq_calib_sum(xd, T, B.workspace(B.OP_CALIB_STATS, cfg.M, cfg.K))
    assert np.array_equal(T.cpu().numpy(), O.calib_sum(xb))
    err = torch.zeros(1, cfg.K // 256, dtype=torch.float64, device=DEV)
    B.pq_group_error(xd, (B.KIND_INT, 4, 256), None, None, err, B.workspace(B.OP_GROUP_ERROR, cfg.M, cfg.K, 0, 1))
    assert np.array_equal(err.cpu().numpy(), O.group_error(xb, 1, 4, 256))


def test_a_full_batch_through_the_kernels_that_apply_a_channel_order():
    """The bench's stage sizes for the kernels that gather through a permutation, whole 4608 x 3072 tensors bit for
    bit: the fused adaptive-LayerNorm producer (tensor-core scale layout), the quantizer with a candidate order,
    the error of six candidate orders in one call, and the integer fake-quant with an order."""
    from test_gpu_gemm import to_tc
    cfg = inputs.CONFIGS["qkv"]
    M, K = cfg.M, cfg.K
    x = inputs.activations(cfg, 0, 5)
    xb, xd = inputs.bits(x), x.to(DEV)
    g = torch.Generator().manual_seed(23)
    perms = torch.stack([torch.randperm(K, generator=g) for _ in range(6)]).to(torch.int32)
    perm = perms[2].contiguous()
    ts = O.tensor_scale(O.calib_stats(xb)[1])
    tsd = torch.tensor([ts], dtype=torch.float32, device=DEV)
    xq = torch.empty(M, K // 2, dtype=torch.uint8, device=DEV)
    sf = torch.empty(B.sf_bytes(M, K, B.PQ_SF_TCGEN05), dtype=torch.uint8, device=DEV)
    # quantizer with a candidate order
    B.pq_quant_act_nvfp4_perm(xd, perm.to(DEV), tsd, xq, sf, B.PQ_SF_TCGEN05)
    c_o, s_o = O.quant_nvfp4(xb, ts, perm.numpy())
    assert np.array_equal(xq.cpu().numpy(), c_o) and np.array_equal(sf.cpu().numpy(), to_tc(s_o))
    # fused producer
    a = (0.3 * torch.randn(K, generator=g)).float()
    b = torch.randn(K, generator=g).float()
    ts_n = torch.tensor([0.011], dtype=torch.float32, device=DEV)
    B.pq_norm_quant_nvfp4(xd, B.NORM_ADALN, a.to(DEV), b.to(DEV), 1e-6, perm.to(DEV), ts_n, xq, sf, B.PQ_SF_TCGEN05, None)
    c_o, s_o, _ = O.norm_quant_nvfp4(xb, 1, a.numpy(), b.numpy(), 1e-6, 0.011, perm.numpy())
    assert np.array_equal(xq.cpu().numpy(), c_o) and np.array_equal(sf.cpu().numpy(), to_tc(s_o))
    # six candidate orders in one error pass
    err = torch.zeros(6, K // 16, dtype=torch.float64, device=DEV)
    B.pq_group_error(xd, (B.KIND_NVFP4, 4, 16), tsd, perms.to(DEV), err, B.workspace(B.OP_GROUP_ERROR, M, K, 0, 6))
    assert np.array_equal(err.cpu().numpy(), O.group_error(xb, 0, 4, 16, ts=ts, perms=perms.numpy()))
    # integer fake-quant with an order
    out = torch.empty(M, K, dtype=torch.bfloat16, device=DEV)
    B.pq_fakequant_int(xd, (B.KIND_INT, 4, 64), perm.to(DEV), out)
    assert np.array_equal(inputs.bits(out.cpu()), O.fakequant_int(xb, 4, 64, perm.numpy()))
