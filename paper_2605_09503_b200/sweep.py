"""Sweeps over the two multi-layer workloads, printed as tables (one JSON line per row with --json).

    python -m paper_2605_09503_b200.sweep dit_block     # every linear of a double-stream DiT block, M swept
    python -m paper_2605_09503_b200.sweep int_sweep     # INT3/INT4 x group 32/64/128/256 acceptance over 16 layers

dit_block: the eight linears (QKV 3072->9216, out 3072->3072, MLP up 3072->12288, down 12288->3072, image
and text stream) with random-init N(0, 0.02) weights quantized to NVFP4, run at M tokens each through the
runtime path (activation quantize + W4A4 GEMM, pq_linear_w4a4); per block: time, TFLOP/s, fraction of the
FP4 peak passed with --peak (TFLOP/s).  Timings are CUDA-graph replays of the eight launches of a block.

int_sweep: sixteen seeded layers (X 4608 x 3072 with the QKV activation statistics, W 3072 x 3072); for
INT3 and INT4 with groups of 32, 64, 128 and 256 (Tab. 2(d)'s largest) the offline pipeline runs with that format driving Eq. 10;
reported per format: mean per-group MSE of the activations without and with the chosen order, layers
accepted, and the throughput of the per-group error reduction.
"""
import argparse
import json

import torch

from . import binding as B
from . import inputs, pipeline


def _graph_ms(fn, iters=10, replays=3):
    fn()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for _ in range(iters):
            fn()
    graph.replay()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(replays):
        graph.replay()
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) / (iters * replays)


def dit_block(args):
    dev = "cuda"
    layers = {}
    for i, (name, K, N) in enumerate(inputs.DIT_BLOCK_LINEARS):
        w = inputs.plain_weight(N, K, i).to(dev)
        wq = torch.empty(N, K // 2, dtype=torch.uint8, device=dev)
        sfw = torch.empty(B.sf_bytes(N, K, 1), dtype=torch.uint8, device=dev)
        ts_w = torch.empty(1, dtype=torch.float32, device=dev)
        B.pq_quant_weight(w, None, None, wq, sfw, B.PQ_SF_TCGEN05, ts_w, B.workspace(B.OP_QUANT_WEIGHT, N, K))
        layers[name] = (K, N, wq, sfw, ts_w)
    rows = []
    for M in inputs.DIT_BLOCK_TOKENS:
        xs, ys, lins = {}, {}, {}
        for i, (name, (K, N, wq, sfw, ts_w)) in enumerate(layers.items()):
            x = inputs.plain_activations(M, K, 100 + i).to(dev)
            ts_x = (x.abs().max().float() / 2688.0).reshape(1)
            xs[name], ys[name] = x, torch.empty(M, N, dtype=torch.bfloat16, device=dev)
            lins[name] = pipeline.QuantLinear(wq, sfw, ts_w, ts_x, M)
        per_layer = {name: _graph_ms(lambda n=name: lins[n](xs[n], ys[n])) for name in layers}

        def block():
            for name in layers:
                lins[name](xs[name], ys[name])

        ms = _graph_ms(block)
        for lin in lins.values():
            lin.check()
        flops = sum(2.0 * M * K * N for _, K, N in inputs.DIT_BLOCK_LINEARS)
        row = {"M": M, "block_ms": ms, "TFLOP/s": flops / ms / 1e9, "frac_fp4_peak": flops / ms / 1e9 / args.peak,
               "layer_ms": per_layer}
        rows.append(row)
        if args.json:
            print(json.dumps(row))
    if not args.json:
        print("| M | block ms | TFLOP/s | of FP4 peak | qkv | out | mlp up | mlp down (ms, image stream) |")
        print("|---|---|---|---|---|---|---|---|")
        for r in rows:
            l = r["layer_ms"]
            print(f"| {r['M']} | {r['block_ms']:.3f} | {r['TFLOP/s']:.0f} | {100 * r['frac_fp4_peak']:.1f} % | "
                  f"{l['img_qkv']:.4f} | {l['img_out']:.4f} | {l['img_mlp_up']:.4f} | {l['img_mlp_down']:.4f} |")


def int_sweep(args):
    dev = "cuda"
    cfg = inputs.CONFIGS["int_sweep"]
    rows = []
    for bits in (3, 4):
        for group in (32, 64, 128, 256):
            fmt = (B.KIND_INT, bits, group)
            mse0 = mse1 = 0.0
            accepted = 0
            for seed in range(args.layers):
                x = inputs.activations(cfg, seed, 0).to(dev)
                w = inputs.weight(cfg, seed).to(dev)
                cal = pipeline.calibrate([x], w, fmt=fmt)
                best, acc = cal.select.tolist()
                n_el = x.shape[0] * cfg.K
                e0 = cal.err_x[0].sum().item() / n_el
                e1 = cal.err_x[best].sum().item() / n_el if acc else e0
                mse0, mse1, accepted = mse0 + e0, mse1 + e1, accepted + int(acc)
            x = inputs.activations(cfg, 0, 0).to(dev)
            err = torch.zeros(1, cfg.K // group, dtype=torch.float64, device=dev)
            ws = B.workspace(B.OP_GROUP_ERROR, x.shape[0], cfg.K, 0, 1)
            ms = _graph_ms(lambda: B.pq_group_error(x, fmt, None, None, err, ws), iters=20)
            row = {"format": f"INT{bits} g{group}", "mse_original": mse0 / args.layers, "mse_chosen": mse1 / args.layers,
                   "accepted": accepted, "layers": args.layers, "group_error_GB/s": x.numel() * 2 / ms / 1e6}
            rows.append(row)
            if args.json:
                print(json.dumps(row))
    if not args.json:
        print("| format | MSE, original order | MSE, chosen order | accepted | pq_group_error GB/s (28 MB, L2-warm) |")
        print("|---|---|---|---|---|")
        for r in rows:
            print(f"| {r['format']} | {r['mse_original']:.5g} | {r['mse_chosen']:.5g} | {r['accepted']}/{r['layers']} | "
                  f"{r['group_error_GB/s']:.0f} |")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("which", choices=["dit_block", "int_sweep"])
    ap.add_argument("--peak", type=float, default=9000.0, help="dense FP4 peak in TFLOP/s for the fraction column")
    ap.add_argument("--layers", type=int, default=16)
    ap.add_argument("--json", action="store_true")
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device: there is no CPU fallback")
    (dit_block if args.which == "dit_block" else int_sweep)(args)


if __name__ == "__main__":
    main()
