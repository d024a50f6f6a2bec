"""GPU parity of the additional candidate orders of the reordering ablation (Tab. 2(a): variance,
round-robin) with their first-moment statistics, and of group size 256 (Tab. 2(d)) in the error and
fake-quant kernels: everything bit for bit against the oracle."""
import numpy as np
import pytest
import torch

from oracle import pq_oracle as O
from paper_2605_09503_b200 import binding as B
from paper_2605_09503_b200 import inputs

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _acts(M, K, seed, shift=True):
    g = torch.Generator().manual_seed(seed)
    scale = torch.exp(1.5 * torch.randn(K, generator=g))
    x = torch.randn(M, K, generator=g) * scale
    if shift:
        x = x + torch.randn(K, generator=g) * scale        # channel means of the order of the spread
    return x.to(torch.bfloat16)


@pytest.mark.parametrize("M,K", [(300, 512), (4608, 3072), (130, 1024), (17, 64)])
def test_first_moments_and_variance_order(M, K):
    batches = [_acts(M, K, 10 + b) for b in range(2)]
    ws = B.workspace(B.OP_CALIB_STATS, M, K)
    S = torch.zeros(K, dtype=torch.float64, device=DEV)
    A = torch.zeros(K, dtype=torch.float32, device=DEV)
    T = torch.zeros(K, dtype=torch.float64, device=DEV)
    So = To = Ao = None
    for x in batches:
        B.pq_calib_stats(x.to(DEV), S, A, ws)
        B.pq_calib_sum(x.to(DEV), T, ws)
        So, Ao = O.calib_stats(inputs.bits(x), So, Ao)
        To = O.calib_sum(inputs.bits(x), To)
    assert np.array_equal(T.cpu().numpy(), To) and np.array_equal(S.cpu().numpy(), So)
    perm = torch.empty(K, dtype=torch.int32, device=DEV)
    wsp = B.workspace(B.OP_SELECT_PERM, 0, K, 0, 1)
    B.pq_order_by_variance(T, S, 2 * M, perm, wsp)
    assert np.array_equal(perm.cpu().numpy(), O.order_by_variance(To, So, 2 * M))
    for group in (16, 64, 256):
        if K % group:
            continue
        B.pq_order_round_robin(S, group, perm, wsp)
        assert np.array_equal(perm.cpu().numpy(), O.order_round_robin(So, group))


def test_variance_order_with_ties_and_constant_channels():
    K = 256
    x = _acts(200, K, 3)
    x[:, 5] = x[:, 77]                                           # equal variance: lower channel first
    x[:, 100] = 2.5                                              # constant channels: variance zero up to rounding
    x[:, 101] = -0.375
    x[:, 102] = 0.0
    T = torch.zeros(K, dtype=torch.float64, device=DEV)
    S = torch.zeros(K, dtype=torch.float64, device=DEV)
    A = torch.zeros(K, dtype=torch.float32, device=DEV)
    ws = B.workspace(B.OP_CALIB_STATS, 200, K)
    B.pq_calib_stats(x.to(DEV), S, A, ws)
    B.pq_calib_sum(x.to(DEV), T, ws)
    perm = torch.empty(K, dtype=torch.int32, device=DEV)
    B.pq_order_by_variance(T, S, 200, perm, B.workspace(B.OP_SELECT_PERM, 0, K, 0, 1))
    So, _ = O.calib_stats(inputs.bits(x))
    To = O.calib_sum(inputs.bits(x))
    want = O.order_by_variance(To, So, 200)
    got = perm.cpu().numpy()
    assert np.array_equal(got, want)
    assert list(got).index(5) + 1 == list(got).index(77)
    assert set(got[-3:].tolist()) == {100, 101, 102}


@pytest.mark.parametrize("bits", [3, 4])
@pytest.mark.parametrize("M,K", [(300, 512), (1000, 3072)])
def test_group_256_error_and_fakequant(bits, M, K):
    x = _acts(M, K, 40 + bits, shift=False)
    fmt = (B.KIND_INT, bits, 256)
    g = torch.Generator().manual_seed(5)
    perms = torch.stack([torch.randperm(K, generator=g) for _ in range(3)]).to(torch.int32)
    # error in the original order (streaming kernel) and of candidate orders (gather kernel)
    e1 = torch.zeros(1, K // 256, dtype=torch.float64, device=DEV)
    B.pq_group_error(x.to(DEV), fmt, None, None, e1, B.workspace(B.OP_GROUP_ERROR, M, K, 0, 1))
    assert np.array_equal(e1.cpu().numpy(), O.group_error(inputs.bits(x), 1, bits, 256))
    e3 = torch.zeros(3, K // 256, dtype=torch.float64, device=DEV)
    B.pq_group_error(x.to(DEV), fmt, None, perms.to(DEV), e3, B.workspace(B.OP_GROUP_ERROR, M, K, 0, 3))
    assert np.array_equal(e3.cpu().numpy(), O.group_error(inputs.bits(x), 1, bits, 256, perms=perms.numpy()))
    # fake-quant, plain and through an order
    out = torch.empty(M, K, dtype=torch.bfloat16, device=DEV)
    B.pq_fakequant_int(x.to(DEV), fmt, None, out)
    assert np.array_equal(inputs.bits(out.cpu()), O.fakequant_int(inputs.bits(x), bits, 256))
    B.pq_fakequant_int(x.to(DEV), fmt, perms[1].contiguous().to(DEV), out)
    assert np.array_equal(inputs.bits(out.cpu()), O.fakequant_int(inputs.bits(x), bits, 256, perms[1].numpy()))


def test_ablation_orders_as_candidates_of_the_acceptance_rule():
    """The three ablation orders appended to the candidate table: errors and the Eq. 10 decision as the oracle's."""
    cfg = inputs.CONFIGS["tiny"]
    K, g = cfg.K, 32
    x = inputs.activations(cfg, 2, 0)
    S = torch.zeros(K, dtype=torch.float64, device=DEV)
    A = torch.zeros(K, dtype=torch.float32, device=DEV)
    T = torch.zeros(K, dtype=torch.float64, device=DEV)
    ws = B.workspace(B.OP_CALIB_STATS, x.shape[0], K)
    B.pq_calib_stats(x.to(DEV), S, A, ws)
    B.pq_calib_sum(x.to(DEV), T, ws)
    cand = torch.empty(3, K, dtype=torch.int32, device=DEV)
    wsp = B.workspace(B.OP_SELECT_PERM, 0, K, 0, 1)
    B.pq_order_by_absmax(A, cand[0], wsp)
    B.pq_order_by_variance(T, S, x.shape[0], cand[1], wsp)
    B.pq_order_round_robin(S, g, cand[2], wsp)
    fmt = (B.KIND_INT, 4, g)
    err = torch.zeros(4, K // g, dtype=torch.float64, device=DEV)
    B.pq_group_error(x.to(DEV), fmt, None, None, err[:1], B.workspace(B.OP_GROUP_ERROR, x.shape[0], K, 0, 1))
    B.pq_group_error(x.to(DEV), fmt, None, cand, err[1:], B.workspace(B.OP_GROUP_ERROR, x.shape[0], K, 0, 3))
    best = torch.zeros(1, dtype=torch.int32, device=DEV)
    acc = torch.zeros(1, dtype=torch.int32, device=DEV)
    E = torch.zeros(4, dtype=torch.float64, device=DEV)
    B.pq_accept(err, torch.zeros_like(err), None, 0.0, best, acc, E)
    xb = inputs.bits(x)
    So, Ao = O.calib_stats(xb)
    To = O.calib_sum(xb)
    cand_o = np.stack([O.order_by_absmax(Ao), O.order_by_variance(To, So, x.shape[0]), O.order_round_robin(So, g)])
    assert np.array_equal(cand.cpu().numpy(), cand_o)
    err_o = O.group_error(xb, 1, 4, g, perms=np.concatenate([np.arange(K, dtype=np.int32)[None], cand_o]))
    assert np.array_equal(err.cpu().numpy(), err_o)
    b_o, a_o, E_o = O.accept(err_o, 1.0, np.zeros_like(err_o), 1.0, 0.0)
    assert (int(best.item()), int(acc.item())) == (b_o, a_o) and np.array_equal(E.cpu().numpy(), E_o)
