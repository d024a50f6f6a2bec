"""The reductions of the library compared with plain float64 sums computed by numpy, independent of any row
blocking: the bit-for-bit parity tests compare with an oracle that states the same chunk / slab order as the
kernels, so these tests pin the VALUES of the GPU results without reference to that order (a wrong blocking,
a dropped row block or a double count would show here whatever the oracle does)."""
import numpy as np
import pytest
import torch

from paper_2605_09503_b200 import binding as B
from paper_2605_09503_b200 import inputs

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _x(M, K, seed):
    g = torch.Generator().manual_seed(seed)
    return (torch.randn(M, K, generator=g) * torch.exp(1.5 * torch.randn(K, generator=g)) + 0.1).to(torch.bfloat16)


@pytest.mark.parametrize("M,K", [(4608, 3072), (1000, 512), (130, 192)])
def test_moments_and_absmax_against_float64(M, K):
    x = _x(M, K, M + K)
    xf = x.double().numpy()
    S = torch.zeros(K, dtype=torch.float64, device=DEV)
    A = torch.zeros(K, dtype=torch.float32, device=DEV)
    T = torch.zeros(K, dtype=torch.float64, device=DEV)
    ws = B.workspace(B.OP_CALIB_STATS, M, K)
    B.pq_calib_stats(x.to(DEV), S, A, ws)
    B.pq_calib_sum(x.to(DEV), T, ws)
    assert np.allclose(S.cpu().numpy(), (xf ** 2).sum(axis=0), rtol=2e-6, atol=0)
    assert np.array_equal(A.cpu().numpy().astype(np.float64), np.abs(xf).max(axis=0))
    assert np.allclose(T.cpu().numpy(), xf.sum(axis=0), rtol=0, atol=2e-6 * np.abs(xf).sum(axis=0))


@pytest.mark.parametrize("bits,group", [(4, 32), (3, 64), (4, 256)])
def test_integer_group_error_against_float64(bits, group):
    """Eq. 1-3 restated in float64 with numpy: scale = absmax / Q, round half to even, clip, squared residual."""
    M, K = 1536, 1024
    x = _x(M, K, bits * 1000 + group)
    xf = x.double().numpy().reshape(M, K // group, group)
    Q = 2 ** (bits - 1) - 1
    s = np.abs(xf).max(axis=2, keepdims=True) / Q
    with np.errstate(invalid="ignore", divide="ignore"):
        z = np.where(s > 0, np.clip(np.rint(xf / s), -Q, Q), 0.0)
    want = ((xf - z * s) ** 2).sum(axis=(0, 2))
    err = torch.zeros(1, K // group, dtype=torch.float64, device=DEV)
    B.pq_group_error(x.to(DEV), (B.KIND_INT, bits, group), None, None, err, B.workspace(B.OP_GROUP_ERROR, M, K, 0, 1))
    # fp32 scales and reciprocals move a value across a rounding tie once in a while: the sums agree to 1e-3
    assert np.allclose(err.cpu().numpy()[0], want, rtol=2e-3)


def test_nvfp4_group_error_against_a_numpy_restatement():
    """NVFP4 per-group error restated with numpy in float64 from the format's definition (E2M1 grid, E4M3 scale of
    absmax / (6 ts), codes of x / (scale ts)); agreement to 1e-3 (ties decided in fp32 on the device)."""
    M, K = 1024, 512
    x = _x(M, K, 7)
    xf = x.double().numpy().reshape(M, K // 16, 16)
    ts = float(np.float32(np.abs(xf).max() / 2688.0))
    grid = np.array([0, 0.5, 1, 1.5, 2, 3, 4, 6])
    e4m3 = np.array(sorted({0.0} | {m / 8 * 2.0 ** -6 for m in range(1, 8)} | {(1 + m / 8) * 2.0 ** (e - 7) for e in range(1, 16) for m in range(8)}))
    e4m3 = e4m3[e4m3 <= 448]
    u = np.abs(xf).max(axis=2) / (6.0 * ts)
    sf = e4m3[np.abs(u[..., None] - e4m3).argmin(axis=-1)]
    d = (sf * ts)[..., None]
    with np.errstate(invalid="ignore", divide="ignore"):
        y = np.where(d > 0, np.abs(xf) / d, 0.0)
    q = grid[np.abs(np.minimum(y, 6.0)[..., None] - grid).argmin(axis=-1)]
    want = ((np.abs(xf) - q * d) ** 2).sum(axis=(0, 2))
    err = torch.zeros(1, K // 16, dtype=torch.float64, device=DEV)
    B.pq_group_error(x.to(DEV), (B.KIND_NVFP4, 4, 16), torch.tensor([ts], dtype=torch.float32, device=DEV), None, err,
                     B.workspace(B.OP_GROUP_ERROR, M, K, 0, 1))
    assert np.allclose(err.cpu().numpy()[0], want, rtol=5e-3)


def test_hadamard_output_against_a_float64_matrix_product():
    import scipy.linalg
    M, K = 64, 3072
    x = _x(M, K, 5)
    chi = lambda r: 0 if r % 11 == 0 else (1 if pow(r % 11, 5, 11) == 1 else -1)
    S = np.zeros((12, 12))
    S[0, 1:], S[1:, 0] = 1, -1
    for i in range(11):
        for j in range(11):
            S[1 + i, 1 + j] = chi(i - j)
    H = np.kron(np.eye(12) + S, scipy.linalg.hadamard(256)).astype(np.float64)
    want = x.double().numpy() @ H / np.sqrt(K)
    y = torch.empty(M, K, dtype=torch.bfloat16, device=DEV)
    B.pq_hadamard_quant_nvfp4(x.to(DEV), None, None, None, None, B.PQ_SF_LINEAR, y)
    got = y.double().cpu().numpy()
    assert np.allclose(got, want, rtol=2.0 ** -8, atol=1e-5 * np.abs(x.double().numpy()).sum(axis=1, keepdims=True) / np.sqrt(K))
