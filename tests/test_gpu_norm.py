"""GPU parity of the fused normalization + reordering + NVFP4 quantization against the oracle: codes, scale
bytes and the optional bf16 output bit for bit."""
import numpy as np
import pytest
import torch

from oracle import pq_oracle as O
from paper_2605_09503_b200 import binding as B
from paper_2605_09503_b200 import inputs
from test_gpu_gemm import to_tc

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _case(M, K, seed):
    g = torch.Generator().manual_seed(seed)
    scale = torch.exp(torch.randn(K, generator=g))
    h = (torch.randn(M, K, generator=g) * scale + 0.25).to(torch.bfloat16)
    a = (0.3 * torch.randn(K, generator=g)).float()
    b = torch.randn(K, generator=g).float()
    perm = torch.randperm(K, generator=g).to(torch.int32)
    return h, a, b, perm


@pytest.mark.parametrize("kind", [B.NORM_RMS, B.NORM_ADALN])
@pytest.mark.parametrize("layout", [B.PQ_SF_LINEAR, B.PQ_SF_TCGEN05])
@pytest.mark.parametrize("M,K,with_perm", [(130, 512, True), (37, 3072, True), (64, 3072, False), (5, 12288, True),
                                           (300, 1024, True), (1, 64, False), (23, 1536, True), (18, 6400, True),
                                           # channels already in output order: the register-resident kernel at each of
                                           # its four register sizes, and the fall-back for rows wider than 4096
                                           (150, 1024, False), (33, 2048, False), (20, 4096, False), (7, 6400, False),
                                           (129, 2560, False),
                                           # the widest rows (three and six warps per block), several blocks
                                           (29, 16384, True), (10, 32768, True), (10, 32768, False)])
def test_norm_quant_bit_exact(kind, layout, M, K, with_perm):
    h, a, b, perm = _case(M, K, seed=M + K + kind)
    ts, eps = 0.011, 1e-6
    codes = torch.empty(M, K // 2, dtype=torch.uint8, device=DEV)
    sf = torch.full((B.sf_bytes(M, K, layout),), 0xEE, dtype=torch.uint8, device=DEV)
    y = torch.empty(M, K, dtype=torch.bfloat16, device=DEV)
    B.pq_norm_quant_nvfp4(h.to(DEV), kind, a.to(DEV), b.to(DEV), eps, perm.to(DEV) if with_perm else None,
                          torch.tensor([ts], dtype=torch.float32, device=DEV), codes, sf, layout, y)
    c_o, s_o, y_o = O.norm_quant_nvfp4(inputs.bits(h), kind, a.numpy(), b.numpy(), eps, ts,
                                       perm.numpy() if with_perm else None)
    assert np.array_equal(codes.cpu().numpy(), c_o)
    assert np.array_equal(inputs.bits(y.cpu()), y_o)
    if layout == B.PQ_SF_LINEAR:
        assert np.array_equal(sf.cpu().numpy().reshape(M, K // 16), s_o)
    else:
        assert np.array_equal(sf.cpu().numpy(), to_tc(s_o))      # padding rows hold zero scale bytes


def test_linear_layout_with_k_not_a_multiple_of_64_and_no_bf16_output():
    M, K = 19, 1040
    h, a, b, perm = _case(M, K, seed=2)
    codes = torch.empty(M, K // 2, dtype=torch.uint8, device=DEV)
    sf = torch.empty(M * K // 16, dtype=torch.uint8, device=DEV)
    B.pq_norm_quant_nvfp4(h.to(DEV), B.NORM_ADALN, a.to(DEV), b.to(DEV), 1e-5, perm.to(DEV),
                          torch.tensor([0.02], dtype=torch.float32, device=DEV), codes, sf, B.PQ_SF_LINEAR, None)
    c_o, s_o, _ = O.norm_quant_nvfp4(inputs.bits(h), 1, a.numpy(), b.numpy(), 1e-5, 0.02, perm.numpy())
    assert np.array_equal(codes.cpu().numpy(), c_o) and np.array_equal(sf.cpu().numpy().reshape(M, K // 16), s_o)


def test_fused_producer_feeds_the_gemm():
    """Full-size rows of the QKV workload: the fused producer's codes and scales go straight into the GEMM
    and the result matches the fp64 reference built from the oracle's codes."""
    from test_gpu_gemm import assert_close
    cfg = inputs.CONFIGS["qkv"]
    M = 512
    h = inputs.activations(cfg, 0, 7, rows=M)
    g = torch.Generator().manual_seed(9)
    a = (0.2 * torch.randn(cfg.K, generator=g)).float()
    b = (0.5 * torch.randn(cfg.K, generator=g)).float()
    perm = torch.randperm(cfg.K, generator=g).to(torch.int32)
    w = inputs.weight(cfg, 0)
    wq = torch.empty(cfg.N, cfg.K // 2, dtype=torch.uint8, device=DEV)
    sfw = torch.empty(B.sf_bytes(cfg.N, cfg.K, 1), dtype=torch.uint8, device=DEV)
    ts_w = torch.empty(1, dtype=torch.float32, device=DEV)
    B.pq_quant_weight(w.to(DEV), perm.to(DEV), None, wq, sfw, B.PQ_SF_TCGEN05, ts_w, B.workspace(B.OP_QUANT_WEIGHT, cfg.N, cfg.K))
    ts_x = 0.004
    xq = torch.empty(M, cfg.K // 2, dtype=torch.uint8, device=DEV)
    sfx = torch.empty(B.sf_bytes(M, cfg.K, 1), dtype=torch.uint8, device=DEV)
    tsd = torch.tensor([ts_x], dtype=torch.float32, device=DEV)
    B.pq_norm_quant_nvfp4(h.to(DEV), B.NORM_ADALN, a.to(DEV), b.to(DEV), 1e-6, perm.to(DEV), tsd, xq, sfx, B.PQ_SF_TCGEN05)
    Y = torch.empty(M, cfg.N, dtype=torch.bfloat16, device=DEV)
    ws = B.workspace(B.OP_GEMM, M, cfg.K, cfg.N)
    B.pq_gemm_w4a4(xq, sfx, tsd, wq, sfw, ts_w, Y, ws)
    assert B.pq_device_status(ws) == B.PQ_OK
    c_o, s_o, _ = O.norm_quant_nvfp4(inputs.bits(h), 1, a.numpy(), b.numpy(), 1e-6, ts_x, perm.numpy())
    assert np.array_equal(xq.cpu().numpy(), c_o)
    wq_o, sfw_o = O.quant_nvfp4(inputs.bits(w), ts_w.item(), perm.numpy())
    rows = np.array([0, 100, 255, 511])
    ref = O.gemm_ref(c_o[rows], s_o[rows], ts_x, wq_o, sfw_o, ts_w.item())
    assert_close(Y.float().cpu().numpy().astype(np.float64)[rows], ref)
