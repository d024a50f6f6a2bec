"""World-size-2 checks of the multi-GPU host logic, on CPU with the gloo backend."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2605_09503_b200 import sharding


def test_shards_partition_the_rows_on_block_boundaries():
    for M in (4608, 4609, 130, 1, 18432, 127):
        for world in (1, 2, 3, 8):
            spans = [sharding.shard_rows(M, world, r) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == M
            for (lo, hi), (lo2, _) in zip(spans, spans[1:]):
                assert hi == lo2 and lo <= hi
            for lo, hi in spans[:-1]:
                assert (lo % sharding.ROW_QUANTUM == 0 or lo == M) and (hi % sharding.ROW_QUANTUM == 0 or hi == M)
            sizes = [hi - lo for lo, hi in spans]
            assert max(sizes) - min(sizes) < 2 * sharding.ROW_QUANTUM


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
        worst = sharding.max_over_ranks(ms)
        lo, hi = sharding.shard_rows(4608, world, rank)
        rows = torch.tensor([hi - lo], dtype=torch.int64)
        dist.all_reduce(rows)                        # every row is owned exactly once
        dist.barrier()
        out.put((rank, worst, int(rows.item()), sharding.aggregate_throughput(100.0, worst * 1e-3, world)))
    finally:
        dist.destroy_process_group()


def test_timing_reduction_and_sharding_across_two_ranks():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, worst, rows, agg in got:
        assert worst == 15.0                         # max over ranks, seen by both
        assert rows == 4608
        assert abs(agg - 2 * 100.0 / 15e-3) < 1e-6


def _calib_worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        g = torch.Generator().manual_seed(100 + rank)
        # partials built so that the order of the additions shows in the last bits
        sumsq = torch.rand(64, generator=g, dtype=torch.float64) * (1e12 if rank == 0 else 1e-3)
        amax = torch.rand(64, generator=g, dtype=torch.float32) * (rank + 1)
        err = torch.rand(3, 8, generator=g, dtype=torch.float64) * 10.0 ** (3 * rank)
        S, A, rows, (E,) = sharding.combine_calibration(sumsq, amax, 1000 + rank, [err])
        out.put((rank, sumsq, amax, err, S, A, rows, E))
    finally:
        dist.destroy_process_group()


def test_calibration_partials_combine_in_rank_order():
    world = 3
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_calib_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted((out.get(timeout=120) for _ in procs), key=lambda t: t[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    S_want = (got[0][1] + got[1][1]) + got[2][1]                 # rank order, written out
    E_want = (got[0][3] + got[1][3]) + got[2][3]
    A_want = torch.maximum(torch.maximum(got[0][2], got[1][2]), got[2][2])
    for _, _, _, _, S, A, rows, E in got:
        assert torch.equal(S, S_want) and torch.equal(E, E_want) and torch.equal(A, A_want)
        assert rows == 1000 + 1001 + 1002
    assert not torch.equal(S_want, got[0][1] + (got[1][1] + got[2][1]))   # the case does depend on the order


def test_bench_starts_its_own_ranks():
    """`python bench.py --gpus 2` without a launcher starts two ranks itself (torch.distributed.run on
    127.0.0.1).  On a machine without a GPU each rank must stop at the explicit "needs a CUDA device"
    exit (there is no CPU fallback), which shows that the ranks were started and reached the GPU arm."""
    import subprocess
    import sys
    if torch.cuda.is_available():
        pytest.skip("the two ranks would run the whole benchmark")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    out = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--steps", "2", "--warmup", "1"],
                         env=env, capture_output=True, text=True, timeout=600)
    assert out.returncode != 0
    text = out.stdout + out.stderr
    # the launcher ends the other rank as soon as one has failed, so one or two ranks get to say it
    assert 1 <= text.count("bench.py needs a CUDA device") <= 2
    # the launcher prints this notice only when it starts more than one process per node
    assert "OMP_NUM_THREADS environment variable for each process" in text
