"""pq_linear_w4a4_batched: n batches through one layer give exactly what n calls of pq_linear_w4a4 give."""
import pytest
import torch

from paper_2605_09503_b200 import binding as B

pytestmark = pytest.mark.gpu


def _layer(M, K, N, n, seed):
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    scale = torch.exp(torch.randn(K, device="cuda", generator=g))
    Xs = [(torch.randn(M, K, device="cuda", generator=g) * scale).to(torch.bfloat16) for _ in range(n)]
    Wt = (0.02 * torch.randn(N, K, device="cuda", generator=g)).to(torch.bfloat16)
    S = torch.zeros(K, dtype=torch.float64, device="cuda")
    A = torch.zeros(K, dtype=torch.float32, device="cuda")
    for x in Xs:
        B.pq_calib_stats(x, S, A, B.workspace(B.OP_CALIB_STATS, M, K))
    ts_x = torch.empty(1, dtype=torch.float32, device="cuda")
    B.pq_tensor_scale(A, ts_x)
    wq = torch.empty(N, K // 2, dtype=torch.uint8, device="cuda")
    sfw = torch.empty(B.sf_bytes(N, K, 1), dtype=torch.uint8, device="cuda")
    ts_w = torch.empty(1, dtype=torch.float32, device="cuda")
    B.pq_quant_weight(Wt, None, None, wq, sfw, B.PQ_SF_TCGEN05, ts_w, B.workspace(B.OP_QUANT_WEIGHT, N, K))
    return Xs, ts_x, wq, sfw, ts_w


@pytest.mark.parametrize("M,K,N,n,n_sets", [(300, 256, 320, 5, 2), (1024, 512, 768, 7, 3), (130, 128, 64, 1, 2),
                                            (2048, 1024, 1536, 9, 4)])
def test_batched_equals_one_by_one(M, K, N, n, n_sets):
    Xs, ts_x, wq, sfw, ts_w = _layer(M, K, N, n, seed=M + n)
    ws = B.workspace(B.OP_GEMM, M, K, N)
    mk = lambda: (torch.empty(M, K // 2, dtype=torch.uint8, device="cuda"),
                  torch.empty(B.sf_bytes(M, K, 1), dtype=torch.uint8, device="cuda"))
    ref = []
    xq, sfx = mk()
    for x in Xs:
        y = torch.empty(M, N, dtype=torch.bfloat16, device="cuda")
        B.pq_linear_w4a4(x, ts_x, xq, sfx, wq, sfw, ts_w, y, ws)
        ref.append(y)
    sets = [mk() for _ in range(n_sets)]
    Ys = [torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda") for _ in range(n)]
    # work queued before and after the call on the caller's stream must stay ordered around it
    marker = torch.zeros(1, device="cuda")
    B.pq_linear_w4a4_batched(Xs, ts_x, [a for a, _ in sets], [b for _, b in sets], wq, sfw, ts_w, Ys, ws)
    total = sum(y.float().abs().sum() for y in Ys) + marker          # reads every Y on the caller's stream
    torch.cuda.synchronize()
    assert B.pq_device_status(ws) == B.PQ_OK
    assert torch.isfinite(total).all()
    for y, r in zip(Ys, ref):
        assert torch.equal(y.view(torch.int16), r.view(torch.int16))


def test_batched_inside_a_cuda_graph():
    M, K, N, n = 512, 256, 384, 4
    Xs, ts_x, wq, sfw, ts_w = _layer(M, K, N, n, seed=3)
    ws = B.workspace(B.OP_GEMM, M, K, N)
    sets = [(torch.empty(M, K // 2, dtype=torch.uint8, device="cuda"),
             torch.empty(B.sf_bytes(M, K, 1), dtype=torch.uint8, device="cuda")) for _ in range(2)]
    Ys = [torch.zeros(M, N, dtype=torch.bfloat16, device="cuda") for _ in range(n)]
    call = lambda: B.pq_linear_w4a4_batched(Xs, ts_x, [a for a, _ in sets], [b for _, b in sets], wq, sfw, ts_w, Ys, ws)
    call()
    torch.cuda.synchronize()
    ref = [y.clone() for y in Ys]
    for y in Ys:
        y.zero_()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        call()
    graph.replay()
    torch.cuda.synchronize()
    for y, r in zip(Ys, ref):
        assert torch.equal(y.view(torch.int16), r.view(torch.int16))


def test_batched_rejects_bad_arguments():
    M, K, N = 128, 128, 64
    Xs, ts_x, wq, sfw, ts_w = _layer(M, K, N, 2, seed=1)
    ws = B.workspace(B.OP_GEMM, M, K, N)
    one = [torch.empty(M, K // 2, dtype=torch.uint8, device="cuda")]
    sf = [torch.empty(B.sf_bytes(M, K, 1), dtype=torch.uint8, device="cuda")]
    Ys = [torch.empty(M, N, dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    with pytest.raises(B.PqError):
        B.pq_linear_w4a4_batched(Xs, ts_x, one, sf, wq, sfw, ts_w, Ys, ws)      # a single set of intermediates


def test_host_batched_equals_one_by_one():
    M, K, N, n = 384, 256, 320, 5
    Xs, ts_x, wq, sfw, ts_w = _layer(M, K, N, n, seed=11)
    ws = B.workspace(B.OP_GEMM, M, K, N)
    xq = torch.empty(M, K // 2, dtype=torch.uint8, device="cuda")
    sfx = torch.empty(B.sf_bytes(M, K, 1), dtype=torch.uint8, device="cuda")
    ref = []
    for x in Xs:
        y = torch.empty(M, N, dtype=torch.bfloat16, device="cuda")
        B.pq_linear_w4a4(x, ts_x, xq, sfx, wq, sfw, ts_w, y, ws)
        ref.append(y.cpu())
    xh = [x.cpu().pin_memory() for x in Xs]
    yh = [torch.zeros(M, N, dtype=torch.bfloat16).pin_memory() for _ in range(n)]
    xd = [torch.empty(M, K, dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    yd = [torch.empty(M, N, dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    B.pq_linear_w4a4_host_batched(xh, ts_x, xd, yd, xq, sfx, wq, sfw, ts_w, yh, ws)
    torch.cuda.synchronize()
    assert B.pq_device_status(ws) == B.PQ_OK
    for y, r in zip(yh, ref):
        assert torch.equal(y.view(torch.int16), r.view(torch.int16))
