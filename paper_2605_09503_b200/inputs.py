"""Seeded synthetic inputs shared by the tests, the smoke check and the benchmark.

This module holds none of the method's arithmetic: it only draws random tensors with the
shapes and channel statistics of the workloads (FLUX-like linear layers whose activations have
log-normal per-channel scales and a few outlier channels) and casts them to bf16.  The same
bytes are handed to the CUDA library and to the CPU oracle.

Everything is generated on the host with torch.Generator(device="cpu"), so a given
(config, layer seed, batch seed) yields identical bits on any machine.
"""
from dataclasses import dataclass

import numpy as np
import torch


@dataclass(frozen=True)
class LayerConfig:
    name: str
    M: int            # runtime tokens / calibration rows per batch
    K: int            # input channels (quantization axis)
    N: int            # output channels
    sigma: float      # std of log channel scale
    outlier_count: int
    outlier_gain: float
    w_std: float
    w_outlier_gain: float   # gain applied to the same input channels of W (1 = none)
    gelu: bool
    calib_batches: int


CONFIGS = {
    # tiny layer: everything is checked against the oracle
    "tiny": LayerConfig("tiny", 256, 512, 512, 1.0, 8, 30.0, 0.02, 5.0, False, 4),
    # FLUX-like attention QKV projection (4096 image + 512 text tokens)
    "qkv": LayerConfig("qkv", 4608, 3072, 9216, 1.5, 31, 50.0, 0.02, 1.0, False, 8),
    # FLUX-like MLP down-projection: GELU output, long K
    "mlp_down": LayerConfig("mlp_down", 4608, 12288, 3072, 2.0, 0, 1.0, 0.01, 1.0, True, 1),
    # INT fake-quant / acceptance sweep layer (statistics of "qkv")
    "int_sweep": LayerConfig("int_sweep", 4608, 3072, 3072, 1.5, 31, 50.0, 0.02, 1.0, False, 1),
}

# The eight linear layers of one double-stream DiT block (hidden 3072, MLP ratio 4), K -> N.
DIT_BLOCK_LINEARS = [
    ("img_qkv", 3072, 9216), ("img_out", 3072, 3072), ("img_mlp_up", 3072, 12288),
    ("img_mlp_down", 12288, 3072),
    ("txt_qkv", 3072, 9216), ("txt_out", 3072, 3072), ("txt_mlp_up", 3072, 12288),
    ("txt_mlp_down", 12288, 3072),
]
DIT_BLOCK_TOKENS = [512, 1024, 4608, 9216, 18432]


def _gen(seed: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed))
    return g


def channel_scales(cfg: LayerConfig, layer_seed: int):
    """Per-channel activation scale (fp32 [K]) and the outlier channel indices of one layer."""
    g = _gen(1_000_003 * (layer_seed + 1))
    scale = torch.exp(cfg.sigma * torch.randn(cfg.K, generator=g))
    idx = torch.randperm(cfg.K, generator=g)[: cfg.outlier_count]
    scale[idx] *= cfg.outlier_gain
    return scale, idx


def activations(cfg: LayerConfig, layer_seed: int, batch_seed: int, rows: int = None) -> torch.Tensor:
    """One batch X [rows, K] in bf16 (CPU).  Calibration batches use batch_seed 0, 1, ...;
    the runtime batch uses batch_seed + 1000."""
    rows = cfg.M if rows is None else rows
    scale, _ = channel_scales(cfg, layer_seed)
    g = _gen(7919 * (layer_seed + 1) + 104_729 * (batch_seed + 1))
    x = torch.randn(rows, cfg.K, generator=g)
    if cfg.gelu:
        x = torch.nn.functional.gelu(x)
    x *= scale[None, :]
    return x.to(torch.bfloat16)


def weight(cfg: LayerConfig, layer_seed: int, N: int = None) -> torch.Tensor:
    """Weight stored as Wt [N, K] in bf16 (CPU): the transpose of the K x N matrix of Y = XW."""
    N = cfg.N if N is None else N
    g = _gen(15_485_863 * (layer_seed + 1) + 17)
    w = cfg.w_std * torch.randn(N, cfg.K, generator=g)
    if cfg.w_outlier_gain != 1.0:
        _, idx = channel_scales(cfg, layer_seed)
        w[:, idx] *= cfg.w_outlier_gain
    return w.to(torch.bfloat16)


def plain_activations(M: int, K: int, seed: int, sigma: float = 1.5) -> torch.Tensor:
    """N(0,1) times a log-normal channel scale, no outliers: the DiT-block sweep inputs."""
    g = _gen(2_750_159 + seed)
    scale = torch.exp(sigma * torch.randn(K, generator=g))
    return (torch.randn(M, K, generator=g) * scale[None, :]).to(torch.bfloat16)


def plain_weight(N: int, K: int, seed: int, std: float = 0.02) -> torch.Tensor:
    g = _gen(3_497_861 + seed)
    return (std * torch.randn(N, K, generator=g)).to(torch.bfloat16)


def bits(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> uint16 numpy array of its bit patterns (for the oracle)."""
    assert t.dtype == torch.bfloat16
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def from_bits(a: np.ndarray) -> torch.Tensor:
    """uint16 bit patterns -> bf16 tensor."""
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16)
