"""Host-side plumbing for running the runtime path on several GPUs of one node.

The quantized linear layer shards by tokens: every rank holds the whole quantized weight and a
contiguous block of the rows of X; outputs stay row-sharded, so the data path needs no collective.
What the ranks do exchange is bookkeeping: the timing reduction of the benchmark (maximum over
ranks of a device-measured time).  Nothing here touches the GPU, so it is tested with `gloo`.
"""
import torch
import torch.distributed as dist

ROW_QUANTUM = 128  # rows per scale-factor block of the tensor-core layout


def shard_rows(M: int, world: int, rank: int, quantum: int = ROW_QUANTUM):
    """Rows [lo, hi) of an M-row activation owned by `rank`: contiguous, whole scale
    blocks (every shard but the last ends on a block boundary), block counts differing by at most one."""
    assert 0 <= rank < world and M >= 0
    blocks = (M + quantum - 1) // quantum
    base, extra = divmod(blocks, world)
    lo_b = rank * base + min(rank, extra)
    hi_b = lo_b + base + (1 if rank < extra else 0)
    return min(lo_b * quantum, M), min(hi_b * quantum, M)


def max_over_ranks(value: float, device="cpu") -> float:
    """Maximum of a per-rank scalar (a device-measured time) over the default process group."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank: float, seconds: float, world: int) -> float:
    """Whole-job throughput when every rank processed `units_per_rank` in (max over ranks) `seconds`."""
    return world * units_per_rank / seconds
