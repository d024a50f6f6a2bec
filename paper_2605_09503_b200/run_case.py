"""Run one entry point of the library on one shape, a few times, and print its device time.

    python -m paper_2605_09503_b200.run_case --case gemm --M 4608 --N 9216 --K 3072 --iters 20

The driver for profiler captures and size sweeps: inputs are random bytes / seeded synthetic
activations created on the device side of the binding, buffers rotate over `--rot` copies so that
repeated launches do not find their operands in L2, timing is by CUDA events on the current stream.
No result is checked here (parity lives in tests/).
"""
import argparse
import json

import torch

from . import binding as B

CASES = ["hadamard", "output_error", "norm_quant", "gemm", "quant", "linear", "batched", "stats", "error", "error_perm", "fakequant", "fakequant_perm", "quant_weight",
         "quant_weight_perm", "select_perm"]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--case", required=True, choices=CASES)
    ap.add_argument("--M", type=int, default=4608)
    ap.add_argument("--N", type=int, default=9216)
    ap.add_argument("--K", type=int, default=3072)
    ap.add_argument("--P", type=int, default=6)
    ap.add_argument("--bits", type=int, default=4)
    ap.add_argument("--group", type=int, default=16, help="16 with --kind 0 (NVFP4); 16..128 with --kind 1")
    ap.add_argument("--kind", type=int, default=0)
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--rot", type=int, default=4)
    ap.add_argument("--ordered", action="store_true", help="norm_quant: channels already in output order (no permutation)")
    ap.add_argument("--graph", action="store_true",
                    help="capture the timed launches in one CUDA graph (takes the host's launch rate out of the number)")
    args = ap.parse_args()
    dev = "cuda"
    M, N, K, R = args.M, args.N, args.K, args.rot
    g = torch.Generator(device=dev)
    g.manual_seed(0)
    fmt = (args.kind, args.bits, 16 if args.kind == 0 else args.group)

    def acts(rows):
        scale = torch.exp(1.5 * torch.randn(K, device=dev, generator=g))
        return (torch.randn(rows, K, device=dev, generator=g) * scale).to(torch.bfloat16)

    def rbytes(*shape, hi=256):
        return torch.randint(0, hi, shape, dtype=torch.uint8, device=dev, generator=g)

    ts = torch.tensor([0.01], dtype=torch.float32, device=dev)
    tsw = torch.tensor([2e-5], dtype=torch.float32, device=dev)
    perms = torch.stack([torch.randperm(K, device=dev, generator=g) for _ in range(max(args.P, 1))]).to(torch.int32)
    work = bytes_moved = 0

    if args.case == "batched":
        # one call = `rot` independent batches through the layer; time is reported per batch
        X = [acts(M) for _ in range(R)]
        xq = [torch.empty(M, K // 2, dtype=torch.uint8, device=dev) for _ in range(4)]
        sfx = [torch.empty(B.sf_bytes(M, K, 1), dtype=torch.uint8, device=dev) for _ in range(4)]
        wq, sfw = rbytes(N, K // 2), rbytes(B.sf_bytes(N, K, 1), hi=0x60)
        Y = [torch.empty(M, N, dtype=torch.bfloat16, device=dev) for _ in range(R)]
        ws = B.workspace(B.OP_GEMM, M, K, N)
        work = 2.0 * M * N * K * R
        fn = lambda i: B.pq_linear_w4a4_batched(X, ts, xq, sfx, wq, sfw, tsw, Y, ws)
    elif args.case in ("gemm", "linear"):
        xq = [rbytes(M, K // 2) for _ in range(R)]
        sfx = [rbytes(B.sf_bytes(M, K, 1), hi=0x60) for _ in range(R)]
        wq = [rbytes(N, K // 2) for _ in range(R)]
        sfw = [rbytes(B.sf_bytes(N, K, 1), hi=0x60) for _ in range(R)]
        Y = [torch.empty(M, N, dtype=torch.bfloat16, device=dev) for _ in range(R)]
        ws = B.workspace(B.OP_GEMM, M, K, N)
        work = 2.0 * M * N * K
        if args.case == "gemm":
            fn = lambda i: B.pq_gemm_w4a4(xq[i % R], sfx[i % R], ts, wq[i % R], sfw[i % R], tsw, Y[i % R], ws)
        else:
            X = [acts(M) for _ in range(R)]
            fn = lambda i: B.pq_linear_w4a4(X[i % R], ts, xq[i % R], sfx[i % R], wq[i % R], sfw[i % R], tsw,
                                            Y[i % R], ws)
    elif args.case == "norm_quant":
        X = [acts(M) for _ in range(R)]
        xq = [torch.empty(M, K // 2, dtype=torch.uint8, device=dev) for _ in range(R)]
        sfx = [torch.empty(B.sf_bytes(M, K, 1), dtype=torch.uint8, device=dev) for _ in range(R)]
        av = torch.randn(K, device=dev, generator=g) * 0.2
        bv = torch.randn(K, device=dev, generator=g)
        pm = None if args.ordered else perms[0].contiguous()
        bytes_moved = M * K * 2 + M * K // 2 + M * K // 16
        fn = lambda i: B.pq_norm_quant_nvfp4(X[i % R], args.kind, av, bv, 1e-6, pm, ts, xq[i % R], sfx[i % R],
                                             B.PQ_SF_TCGEN05)
    elif args.case == "hadamard":
        X = [acts(M) for _ in range(R)]
        xq = [torch.empty(M, K // 2, dtype=torch.uint8, device=dev) for _ in range(R)]
        sfx = [torch.empty(B.sf_bytes(M, K, 1), dtype=torch.uint8, device=dev) for _ in range(R)]
        pm = perms[0].contiguous()
        bytes_moved = M * K * 2 + M * K // 2 + M * K // 16
        fn = lambda i: B.pq_hadamard_quant_nvfp4(X[i % R], pm, ts, xq[i % R], sfx[i % R], B.PQ_SF_TCGEN05)
    elif args.case == "quant":
        X = [acts(M) for _ in range(R)]
        xq = [torch.empty(M, K // 2, dtype=torch.uint8, device=dev) for _ in range(R)]
        sfx = [torch.empty(B.sf_bytes(M, K, 1), dtype=torch.uint8, device=dev) for _ in range(R)]
        bytes_moved = M * K * 2 + M * K // 2 + M * K // 16
        fn = lambda i: B.pq_quant_act_nvfp4(X[i % R], ts, xq[i % R], sfx[i % R], B.PQ_SF_TCGEN05)
    elif args.case == "output_error":
        yref = [torch.randn(M, N, device=dev, generator=g) for _ in range(2)]
        yq = [(r * 1.01).to(torch.bfloat16) for r in yref]
        eo = torch.zeros(N, dtype=torch.float64, device=dev)
        ws = B.workspace(B.OP_OUTPUT_ERROR, M, N)
        bytes_moved = M * N * 6
        fn = lambda i: B.pq_output_error(yref[i % 2], yq[i % 2], eo, ws)
    elif args.case == "stats":
        X = [acts(M) for _ in range(R)]
        S = torch.zeros(K, dtype=torch.float64, device=dev)
        A = torch.zeros(K, dtype=torch.float32, device=dev)
        ws = B.workspace(B.OP_CALIB_STATS, M, K)
        bytes_moved = M * K * 2
        fn = lambda i: B.pq_calib_stats(X[i % R], S, A, ws)
    elif args.case in ("error", "error_perm"):
        X = [acts(M) for _ in range(R)]
        P = 1 if args.case == "error" else args.P
        err = torch.zeros(P, K // fmt[2], dtype=torch.float64, device=dev)
        ws = B.workspace(B.OP_GROUP_ERROR, M, K, 0, P)
        bytes_moved = M * K * 2
        pm = None if args.case == "error" else perms[:P].contiguous()
        fn = lambda i: B.pq_group_error(X[i % R], fmt, ts, pm, err, ws)
    elif args.case in ("fakequant", "fakequant_perm"):
        X = [acts(M) for _ in range(R)]
        out = [torch.empty(M, K, dtype=torch.bfloat16, device=dev) for _ in range(R)]
        bytes_moved = M * K * 4
        pm = perms[0].contiguous() if args.case == "fakequant_perm" else None
        f = (B.KIND_INT, args.bits, max(args.group, 16))
        fn = lambda i: B.pq_fakequant_int(X[i % R], f, pm, out[i % R])
    elif args.case in ("quant_weight", "quant_weight_perm"):
        W = [(0.02 * torch.randn(N, K, device=dev, generator=g)).to(torch.bfloat16) for _ in range(R)]
        wq = torch.empty(N, K // 2, dtype=torch.uint8, device=dev)
        sfw = torch.empty(B.sf_bytes(N, K, 1), dtype=torch.uint8, device=dev)
        t = torch.empty(1, dtype=torch.float32, device=dev)
        ws = B.workspace(B.OP_QUANT_WEIGHT, N, K)
        bytes_moved = 2 * N * K * 2 + N * K // 2 + N * K // 16
        pm = perms[0].contiguous() if args.case == "quant_weight_perm" else None
        fn = lambda i: B.pq_quant_weight(W[i % R], pm, None, wq, sfw, B.PQ_SF_TCGEN05, t, ws)
    else:  # select_perm
        sa = torch.rand(K, dtype=torch.float64, device=dev, generator=g)
        sw = torch.rand(K, dtype=torch.float64, device=dev, generator=g)
        out = torch.empty(6, K, dtype=torch.int32, device=dev)
        ws = B.workspace(B.OP_SELECT_PERM, 0, K, 0, 6)
        fn = lambda i: B.pq_select_perm(sa, 1000, sw, 1000, 5, out, ws)

    for i in range(args.warmup):
        fn(i)
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if args.graph:
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            for i in range(args.iters):
                fn(i)
        graph.replay()
        torch.cuda.synchronize()
        a.record()
        graph.replay()
        b.record()
    else:
        a.record()
        for i in range(args.iters):
            fn(i)
        b.record()
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / args.iters
    line = {"case": args.case, "M": M, "N": N, "K": K, "ms": ms, "graph": args.graph}
    if args.case == "batched":
        line["ms_per_batch"] = ms / R
    if work:
        line["TFLOP/s"] = work / ms / 1e9
    if bytes_moved:
        line["GB/s"] = bytes_moved / ms / 1e6
    print(json.dumps(line))


if __name__ == "__main__":
    main()
