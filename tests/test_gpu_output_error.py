"""pq_output_error, pq_quant_act_nvfp4_perm and the output-side acceptance (Sec. 3.3 / Eq. 10 read on
the layer output) against the oracle: bit-exact sums, bit-exact codes, and the same decision."""
import numpy as np
import pytest
import torch

from oracle import pq_oracle as O
from paper_2605_09503_b200 import binding as B, inputs, pipeline

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _pair(rows, N, seed, ld_extra=0):
    g = torch.Generator().manual_seed(seed)
    yref = torch.randn(rows, N + ld_extra, generator=g) * torch.exp(2 * torch.randn(rows, N + ld_extra, generator=g))
    yq = (yref * (1 + 0.05 * torch.randn(rows, N + ld_extra, generator=g))).to(torch.bfloat16)
    return yref.float(), yq


@pytest.mark.parametrize("rows,N,ld_extra", [(1, 8, 0), (37, 264, 0), (300, 1024, 24), (129, 4104, 0), (2048, 512, 8)])
def test_output_error_bit_exact(rows, N, ld_extra):
    yref, yq = _pair(rows, N, rows + N, ld_extra)
    err = torch.full((N,), 0.5, dtype=torch.float64, device=DEV)
    ws = B.workspace(B.OP_OUTPUT_ERROR, rows, N)
    B.pq_output_error(yref.to(DEV)[:, :N], yq.to(DEV)[:, :N], err, ws)
    want = O.output_error(yref[:, :N].numpy(), inputs.bits(yq[:, :N].contiguous()), np.full(N, 0.5))
    assert np.array_equal(err.cpu().numpy(), want)


def test_output_error_accumulates_over_batches_and_checks_its_arguments():
    N = 256
    err = torch.zeros(N, dtype=torch.float64, device=DEV)
    want = np.zeros(N)
    ws = B.workspace(B.OP_OUTPUT_ERROR, 500, N)
    for seed, rows in ((1, 500), (2, 77)):
        yref, yq = _pair(rows, N, seed)
        B.pq_output_error(yref.to(DEV), yq.to(DEV), err, ws)
        want = O.output_error(yref.numpy(), inputs.bits(yq), want)
    assert np.array_equal(err.cpu().numpy(), want)
    yref, yq = _pair(500, N, 3)
    small = torch.zeros(256, dtype=torch.uint8, device=DEV)
    with pytest.raises(B.PqError):
        B.pq_output_error(yref.to(DEV), yq.to(DEV), err, small)                      # workspace too small
    with pytest.raises(B.PqError):
        B.pq_output_error(yref.to(DEV)[:, :12], yq.to(DEV)[:, :12], err[:12], ws)    # N % 8 != 0


def test_output_error_full_size_output_of_the_bench_layer():
    cfg = inputs.CONFIGS["qkv"]
    yref, yq = _pair(cfg.M, cfg.N, 17)
    err = torch.zeros(cfg.N, dtype=torch.float64, device=DEV)
    B.pq_output_error(yref.to(DEV), yq.to(DEV), err, B.workspace(B.OP_OUTPUT_ERROR, cfg.M, cfg.N))
    assert np.array_equal(err.cpu().numpy(), O.output_error(yref.numpy(), inputs.bits(yq)))


@pytest.mark.parametrize("layout", [B.PQ_SF_LINEAR, B.PQ_SF_TCGEN05])
@pytest.mark.parametrize("M,K", [(130, 512), (37, 3072), (5, 16384), (129, 6400), (3, 6464), (2, 64), (40, 8192)])
def test_quant_act_with_an_order_is_bit_exact(layout, M, K):
    g = torch.Generator().manual_seed(M + K)
    x = (torch.randn(M, K, generator=g) * torch.exp(torch.randn(K, generator=g))).to(torch.bfloat16)
    perm = torch.randperm(K, generator=g).to(torch.int32)
    ts = float(x.float().abs().max()) / 2688.0
    codes = torch.empty(M, K // 2, dtype=torch.uint8, device=DEV)
    sf = torch.full((B.sf_bytes(M, K, layout),), 0xEE, dtype=torch.uint8, device=DEV)
    B.pq_quant_act_nvfp4_perm(x.to(DEV), perm.to(DEV), torch.tensor([ts], dtype=torch.float32, device=DEV), codes, sf, layout)
    c_o, s_o = O.quant_nvfp4(inputs.bits(x), ts, perm.numpy())
    assert np.array_equal(codes.cpu().numpy(), c_o)
    if layout == B.PQ_SF_LINEAR:
        assert np.array_equal(sf.cpu().numpy().reshape(M, K // 16), s_o)
    else:
        lin = torch.empty(M * K // 16, dtype=torch.uint8, device=DEV)
        B.pq_sf_to_linear(sf, M, K, lin)
        assert np.array_equal(lin.cpu().numpy().reshape(M, K // 16), s_o)


def test_quant_act_with_an_order_whose_index_vector_is_only_4_byte_aligned():
    """The four-rows-per-warp kernel loads indices 16 bytes at a time; an index vector that is not 16-byte
    aligned takes the one-block-per-row kernel.  Same codes and scales either way."""
    M, K = 70, 3072
    g = torch.Generator().manual_seed(5)
    x = (torch.randn(M, K, generator=g) * torch.exp(torch.randn(K, generator=g))).to(torch.bfloat16)
    perm = torch.randperm(K, generator=g).to(torch.int32)
    ts = torch.tensor([float(x.float().abs().max()) / 2688.0], dtype=torch.float32, device=DEV)
    buf = torch.zeros(K + 4, dtype=torch.int32, device=DEV)
    buf[1:K + 1] = perm.to(DEV)
    shifted = buf[1:K + 1]
    assert shifted.data_ptr() % 16 == 4
    out = []
    for pm in (perm.to(DEV), shifted):
        codes = torch.empty(M, K // 2, dtype=torch.uint8, device=DEV)
        sf = torch.full((B.sf_bytes(M, K, B.PQ_SF_TCGEN05),), 0xEE, dtype=torch.uint8, device=DEV)
        B.pq_quant_act_nvfp4_perm(x.to(DEV), pm, ts, codes, sf, B.PQ_SF_TCGEN05)
        out.append((codes.cpu().numpy(), sf.cpu().numpy()))
    c_o, _ = O.quant_nvfp4(inputs.bits(x), float(ts.item()), perm.numpy())
    assert np.array_equal(out[0][0], c_o) and np.array_equal(out[1][0], c_o)
    assert np.array_equal(out[0][1], out[1][1])


def test_selection_by_output_error_matches_the_oracle_route():
    """Small layer with strong channel outliers: E of the original order and of the Eq. 9 candidates,
    computed through quantizer -> W4A4 GEMM -> pq_output_error, against the oracle's quantizer,
    dequantized fp64 product rounded to bf16, and output error; same best candidate and decision."""
    cfg = inputs.CONFIGS["tiny"]
    M, K, N = 256, cfg.K, cfg.N
    xs = [inputs.activations(cfg, 0, b, rows=M) for b in (0, 1)]
    w = inputs.weight(cfg, 0)
    refs = [(x.double() @ w.double().T).float() for x in xs]
    S, A = None, None
    for x in xs:
        S, A = O.calib_stats(inputs.bits(x), S, A)
    Sw, Aw = O.calib_stats(inputs.bits(w))
    perms = O.select_perm(S, 2 * M, Sw, N, J=3)
    ts_x = float(O.tensor_scale(A))
    ts_w = float(O.tensor_scale(Aw))

    E, select = pipeline.select_by_output_error([x.to(DEV) for x in xs], [r.to(DEV) for r in refs], w.to(DEV),
                                                torch.tensor(perms, device=DEV),
                                                torch.tensor([ts_x], dtype=torch.float32, device=DEV))
    E = E.cpu().numpy()
    E_o = np.zeros(perms.shape[0] + 1)
    for p in range(perms.shape[0] + 1):
        order = None if p == 0 else perms[p - 1]
        wq, sfw = O.quant_nvfp4(inputs.bits(w), ts_w, order)
        for x, ref in zip(xs, refs):
            xq, sfx = O.quant_nvfp4(inputs.bits(x), ts_x, order)
            y = O.gemm_ref(xq, sfx, ts_x, wq, sfw, ts_w)
            yq = inputs.bits(torch.tensor(y).to(torch.bfloat16))
            E_o[p] += O.output_error(ref.numpy(), yq).sum()
    assert np.allclose(E, E_o, rtol=2e-3, atol=0)
    best_o = 1 + int(np.argmin(E_o[1:]))
    gaps = np.abs(E_o[1:] - E_o[best_o]) / E_o[best_o]
    if np.sort(gaps)[1] > 1e-2:                                        # a clear winner: same choice
        assert int(select[0]) == best_o
    if abs(E_o[0] - E_o[best_o]) > 1e-2 * E_o[0]:
        assert int(select[1]) == int(E_o[0] - E_o[best_o] > 0)
