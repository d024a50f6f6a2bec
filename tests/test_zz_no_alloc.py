"""The allocation-free statistics entry point.

pq_calib_stats_static exists for callers that are not allowed to allocate device memory (a server
with a fixed memory pool, a plugin without an allocator): it keeps its per-chunk partial sums in an
array inside the library instead of a caller workspace.  It must return exactly what
pq_calib_stats returns, also when called twice in a row (the array still holds the previous call's
partials the second time), and must refuse problems that do not fit its array.

This file sorts after every other test file on purpose: a run that stops at the first failure has
then already run the rest of the suite.
"""
import ctypes as C

import pytest
import torch

from paper_2605_09503_b200 import binding as B
from paper_2605_09503_b200 import build, inputs


def test_rejects_problems_larger_than_the_static_array():
    """A host-side size check: no launch, no device memory touched (the pointers are fakes)."""
    build.build()
    L = B.lib()
    limit = int(L.pq_calib_stats_static_max_bytes())
    assert limit == 8 << 20
    p = C.c_void_p(0x1000)
    rows, K = 32768, 8192
    assert B.workspace_bytes(B.OP_CALIB_STATS, rows, K) > limit
    assert L.pq_calib_stats_static(p, rows, K, K, p, p, None) == 5          # PQ_ERR_WORKSPACE
    assert L.pq_calib_stats_static(p, 0, K, K, p, p, None) == 2             # PQ_ERR_SHAPE


@pytest.mark.gpu
def test_matches_the_workspace_entry_point_on_two_calls_in_a_row():
    dev = "cuda"
    cfg = inputs.LayerConfig("t", 300, 3072, 3072, 1.5, 8, 50.0, 0.02, 1.0, False, 1)
    batches = [inputs.activations(cfg, 3, b).to(dev) for b in range(2)]
    K = cfg.K
    assert B.workspace_bytes(B.OP_CALIB_STATS, cfg.M, K) <= int(B.lib().pq_calib_stats_static_max_bytes())

    S_ref = torch.zeros(K, dtype=torch.float64, device=dev)
    A_ref = torch.zeros(K, dtype=torch.float32, device=dev)
    S = torch.zeros(K, dtype=torch.float64, device=dev)
    A = torch.zeros(K, dtype=torch.float32, device=dev)
    ws = B.workspace(B.OP_CALIB_STATS, cfg.M, K)
    for x in batches:                       # two calls in a row, accumulating like calibration does
        B.pq_calib_stats(x, S_ref, A_ref, ws)
        B.pq_calib_stats_static(x, S, A)
        torch.cuda.synchronize()
        # same kernels, same arithmetic: the comparison is bit for bit, as in the other statistics tests
        assert torch.equal(S, S_ref)
        assert torch.equal(A, A_ref)
    # a smaller, ragged problem right after a larger one: stale partials beyond its range are never read
    x = batches[0][:37, :1024]
    S2_ref = torch.zeros(1024, dtype=torch.float64, device=dev)
    A2_ref = torch.zeros(1024, dtype=torch.float32, device=dev)
    S2, A2 = torch.zeros_like(S2_ref), torch.zeros_like(A2_ref)
    B.pq_calib_stats(x, S2_ref, A2_ref, ws)
    B.pq_calib_stats_static(x, S2, A2)
    torch.cuda.synchronize()
    assert torch.equal(S2, S2_ref) and torch.equal(A2, A2_ref)
    assert float(S2.sum()) > 0
