"""Host-side plumbing for running the runtime path on several GPUs of one node.

The quantized linear layer shards by tokens: every rank holds the whole quantized weight and a
contiguous block of the rows of X; outputs stay row-sharded, so the data path needs no collective.
What the ranks do exchange is bookkeeping: the timing reduction of the benchmark (maximum over
ranks of a device-measured time), and, when the calibration batches are spread over the ranks, the
per-rank partial statistics and group errors (a few hundred KB), combined in rank order so that the
totals do not depend on the collective's reduction order.  Nothing here launches a kernel of the
library, so it is tested with `gloo` on CPU tensors; with NCCL the same calls run on device tensors.
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


def ordered_sum_over_ranks(partial: torch.Tensor) -> torch.Tensor:
    """Sum of every rank's `partial` (same shape and dtype on all ranks), added in rank order
    starting from rank 0's value: ((p0 + p1) + p2) + ...  An all-reduce may add in any order and
    floating-point addition is not associative, so the per-rank arrays are gathered and added here;
    every rank returns the same bits.  Used for the fp64 second moments and group errors of a
    calibration set whose batches were processed on different GPUs (each rank starts from zero)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return partial.clone()
    parts = [torch.empty_like(partial) for _ in range(dist.get_world_size())]
    dist.all_gather(parts, partial.contiguous())
    total = parts[0].clone()
    for p in parts[1:]:
        total += p
    return total


def max_over_ranks_tensor(partial: torch.Tensor) -> torch.Tensor:
    """Element-wise maximum over ranks (the per-channel absmax: exact in any order)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return partial.clone()
    out = partial.clone()
    dist.all_reduce(out, op=dist.ReduceOp.MAX)
    return out


def combine_calibration(sumsq: torch.Tensor, amax: torch.Tensor, rows: int, errors=()):
    """Per-rank calibration partials -> totals every rank agrees on bit for bit.
    sumsq fp64 [K] and each tensor of `errors` (fp64 [P, K/g]) are added in rank order, amax fp32 [K]
    is maximised, the row counts are added.  Returns (sumsq, amax, rows, [errors...])."""
    rows_t = torch.tensor([int(rows)], dtype=torch.int64, device=sumsq.device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(rows_t)
    return (ordered_sum_over_ranks(sumsq), max_over_ranks_tensor(amax), int(rows_t.item()),
            [ordered_sum_over_ranks(e) for e in errors])
