"""GPU parity, runtime activation quantizer: codes and scale bytes bit-exact with the oracle,
in both scale layouts, including the exhaustive sweep over every bf16 value."""
import numpy as np
import pytest
import torch

from oracle import pq_oracle as O
from paper_2605_09503_b200 import binding as B
from paper_2605_09503_b200 import inputs

pytestmark = pytest.mark.gpu
DEV = "cuda"


def run_quant(x, ts, layout):
    M, K = x.shape
    codes = torch.empty(M, K // 2, dtype=torch.uint8, device=DEV)
    sf = torch.full((B.sf_bytes(M, K, layout),), 0x55, dtype=torch.uint8, device=DEV)
    tsd = torch.tensor([ts], dtype=torch.float32, device=DEV)
    B.pq_quant_act_nvfp4(x.to(DEV), tsd, codes, sf, layout)
    if layout == B.PQ_SF_TCGEN05:
        lin = torch.empty(M, K // 16, dtype=torch.uint8, device=DEV)
        B.pq_sf_to_linear(sf, M, K, lin)
        return codes.cpu().numpy(), lin.cpu().numpy(), sf.cpu().numpy()
    return codes.cpu().numpy(), sf.cpu().numpy().reshape(M, K // 16), None


@pytest.mark.parametrize("layout", [B.PQ_SF_LINEAR, B.PQ_SF_TCGEN05])
@pytest.mark.parametrize("M,K", [(256, 512), (130, 3072), (1, 64), (300, 12288), (77, 1024)])
def test_quant_act_bit_exact(layout, M, K):
    cfg = inputs.LayerConfig("t", M, K, K, 1.5, 4, 50.0, 0.02, 1.0, False, 1)
    x = inputs.activations(cfg, 0, 1000)
    xb = inputs.bits(x)
    ts = O.tensor_scale(O.calib_stats(inputs.bits(inputs.activations(cfg, 0, 0)))[1])
    codes, sf, raw = run_quant(x, ts, layout)
    co, so = O.quant_nvfp4(xb, ts)
    assert np.array_equal(sf, so)
    assert np.array_equal(codes, co)
    if raw is not None:       # padding rows of the tensor-core layout are zero, nothing else is touched
        blocks = raw.reshape(-1, K // 64, 32, 4, 4).transpose(0, 3, 2, 1, 4).reshape(-1, K // 16)
        assert not blocks[M:].any()


def test_quant_act_linear_layout_k_not_multiple_of_64():
    cfg = inputs.LayerConfig("t", 50, 48, 48, 1.0, 2, 30.0, 0.02, 1.0, False, 1)
    x = inputs.activations(cfg, 1, 1000)
    codes, sf, _ = run_quant(x, 0.01, B.PQ_SF_LINEAR)
    co, so = O.quant_nvfp4(inputs.bits(x), 0.01)
    assert np.array_equal(codes, co) and np.array_equal(sf, so)


def test_quant_act_every_bf16_value():
    """All 65536 bit patterns, finite ones kept: each value is placed in a group whose absmax
    is 6.0 (scale byte 0x38, decode scale 1), so the code is the plain E2M1 rounding; a second
    pass lets every value be its own group's maximum."""
    pats = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    vals = O.bf16_to_f32(pats)
    finite = pats[np.isfinite(vals)]
    small = finite[np.abs(O.bf16_to_f32(finite)) <= 6.0]
    # pass 1: 15 probes + one 6.0 per group
    n = (len(small) + 14) // 15 * 15
    probes = np.resize(small, n).reshape(-1, 15)
    six = np.full((probes.shape[0], 1), 0x40C0, dtype=np.uint16)           # 6.0 in bf16
    groups = np.concatenate([six, probes], axis=1).reshape(1, -1)
    pad = (-groups.shape[1]) % 64
    groups = np.concatenate([groups, np.zeros((1, pad), dtype=np.uint16)], axis=1)
    x = inputs.from_bits(groups)
    for layout in (B.PQ_SF_LINEAR, B.PQ_SF_TCGEN05):
        codes, sf, _ = run_quant(x, 1.0, layout)
        co, so = O.quant_nvfp4(groups, 1.0)
        assert np.array_equal(codes, co) and np.array_equal(sf, so)
    # pass 2: every finite value alone in its group (rest zeros), three tensor scales
    rows = finite.reshape(-1, 1)
    g2 = np.concatenate([rows, np.zeros((len(finite), 15), dtype=np.uint16)], axis=1).reshape(1, -1)
    pad = (-g2.shape[1]) % 64
    g2 = np.concatenate([g2, np.zeros((1, pad), dtype=np.uint16)], axis=1)
    for ts in (1.0, 3.7e-3, 2.0 ** -60):
        codes, sf, _ = run_quant(inputs.from_bits(g2), ts, B.PQ_SF_LINEAR)
        co, so = O.quant_nvfp4(g2, ts)
        assert np.array_equal(sf, so), ts
        assert np.array_equal(codes, co), ts


def test_identity_invariants_on_device():
    """Sign symmetry and power-of-two scaling hold on the device exactly as in the definition."""
    cfg = inputs.LayerConfig("t", 64, 256, 256, 1.0, 2, 30.0, 0.02, 1.0, False, 1)
    x = inputs.activations(cfg, 2, 1000)
    c1, s1, _ = run_quant(x, 0.01, B.PQ_SF_LINEAR)
    c2, s2, _ = run_quant(-x, 0.01, B.PQ_SF_LINEAR)
    assert np.array_equal(s1, s2) and np.array_equal(c1 ^ 0x88, c2)
    c3, s3, _ = run_quant((x.float() * 4).to(torch.bfloat16), 0.04, B.PQ_SF_LINEAR)
    assert np.array_equal(c1, c3) and np.array_equal(s1, s3)
