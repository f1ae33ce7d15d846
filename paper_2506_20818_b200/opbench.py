"""Operator-level timing of the library's single-operator entry points on a synthetic graph.

    python -m paper_2506_20818_b200.opbench --op aggregate --nodes 1000000 --mean-degree 16 --width 256

times `lp_op_aggregate` (AGG of Eq. 1 and, with --transpose, its adjoint; `--op gather-ceiling`: the bare gather of the
same index stream, `lp_op_gather_ceiling`, the floor of any such kernel) with CUDA events and prints one JSON
line: microseconds per launch, the algorithmic bytes of the launch in the gather convention (every stored entry
reads one source row; offsets, indices and the output once) and in the compulsory convention (every source row
once), and both divided by the time.  The graph is the Chung-Lu power-law generator of the benchmark workloads;
with --nodes 1000000 --mean-degree 16 it is the graph of the partitioned configuration, whose 512 MB BF16 source
matrix does not fit the L2 cache, so the launch is bound by HBM rather than by L2 gathers.  Used for the ncu
captures of single kernels (few launches, small process).

    python -m paper_2506_20818_b200.opbench --op step --config c2_chunglu_sage2 --batch 10240 --fanout 25,10 --iters 5

runs whole training steps (negatives, step, Adam) of one of the named workload configurations, optionally scaled
down and over sampled blocks, and prints the time per step: a small process around any kernel of the step.
"""
from __future__ import annotations

import argparse
import json

import numpy as np


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--op", choices=["aggregate", "gather-ceiling", "step"], default="aggregate")
    ap.add_argument("--config", default="c2_chunglu_sage2", help="--op step: workload configuration")
    ap.add_argument("--scale", type=float, default=1.0, help="--op step: shrink the configuration's graph")
    ap.add_argument("--batch", type=int, default=65536, help="--op step: positives per step")
    ap.add_argument("--fanout", default="", help="--op step: comma-separated fan-outs (hop 1 first); empty = full-graph training")
    ap.add_argument("--prec", choices=["bf16", "fp32"], default="bf16")
    ap.add_argument("--nodes", type=int, default=1_000_000)
    ap.add_argument("--mean-degree", type=float, default=16.0)
    ap.add_argument("--exponent", type=float, default=2.1)
    ap.add_argument("--width", type=int, default=256)
    ap.add_argument("--arch", choices=["sage", "gcn"], default="sage")
    ap.add_argument("--transpose", action="store_true")
    ap.add_argument("--fp32", action="store_true")
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--seed", type=int, default=5)
    args = ap.parse_args()

    import torch
    import workloads as wl
    from . import Context

    if args.op == "step":
        g, X, params, pos, cfg = wl.make_config(args.config, scale=args.scale)
        fanout = [int(x) for x in args.fanout.split(",") if x] or None
        B = min(args.batch, len(pos[0]))
        ctx = Context(0)
        ctx.load_graph(g.n, g.rowptr, g.col, g.w, X)
        ctx.set_model(cfg["arch"], cfg["dims"], prec=args.prec, fanout=fanout, max_batch=B, max_k=1)
        dev = "cuda:0"
        pu, pv = torch.from_numpy(pos[0]).to(dev), torch.from_numpy(pos[1]).to(dev)
        p = torch.from_numpy(params).to(dev)
        m, v, grads, loss = torch.zeros_like(p), torch.zeros_like(p), torch.zeros_like(p), torch.zeros(1, device=dev)
        nb = max(1, len(pos[0]) // B)
        times = []
        for i in range(args.warmup + args.iters):
            lo = (i % nb) * B
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            _, nd = ctx.sample_negatives(args.seed, i, 1, pu[lo:lo + B], edge_index_base=lo)
            ctx.train_step(p, pu[lo:lo + B], pv[lo:lo + B], None, nd, 1, loss, grads, seed=args.seed, step=i)
            ctx.adam_step(p, m, v, grads, i + 1)
            b.record()
            torch.cuda.synchronize()
            if i >= args.warmup:
                times.append(a.elapsed_time(b) * 1e3)
        print(json.dumps({"op": "step", "config": args.config, "scale": args.scale, "nodes": g.n, "entries": int(g.nnz), "batch_pos": B, "fanout": fanout,
                          "dtype": args.prec, "us_per_step": round(float(np.median(times)), 1), "loss": float(loss.item()),
                          "launches_per_step": int(ctx.stats().kernel_launches // max(1, args.warmup + args.iters))}))
        ctx.close()
        return

    g = wl.chung_lu(args.nodes, args.mean_degree, args.exponent, seed=args.seed)
    ctx = Context(0)
    ctx.load_graph(g.n, g.rowptr, g.col, g.w, wl.node_features(g.n, 8, args.seed))
    torch.manual_seed(args.seed)
    H = torch.randn(g.n, args.width, device="cuda:0")
    if not args.fp32:
        H = H.to(torch.bfloat16)
    es = H.element_size()
    if args.op == "gather-ceiling":
        run = lambda: ctx.op_gather_ceiling(H, transpose=args.transpose)  # noqa: E731
    else:
        run = lambda: ctx.op_aggregate(args.arch, H, transpose=args.transpose)  # noqa: E731
    for _ in range(args.warmup):
        run()
    torch.cuda.synchronize()
    times = []
    for _ in range(args.iters):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        run()
        b.record()
        torch.cuda.synchronize()
        times.append(a.elapsed_time(b) * 1e3)
    us = float(np.median(times))
    if args.op == "gather-ceiling":
        moved = g.nnz * (args.width * es + 4) + ((g.nnz + 63) // 64) * args.width * es
        print(json.dumps({"op": "gather-ceiling", "transpose": args.transpose, "nodes": g.n, "entries": int(g.nnz), "row_bytes": args.width * es,
                          "us_per_launch": round(us, 1), "gather_bytes": moved, "gather_GBps": round(moved / us / 1e3, 1),
                          "source_matrix_MB": round(g.n * args.width * es / 1e6, 1)}))
        ctx.close()
        return
    per_entry = 4 + (4 if (args.arch == "gcn" or args.transpose) else 0)
    fixed = (g.n + 1) * 4 + g.n * args.width * es + (g.n * 4 if args.arch == "sage" and not args.transpose else 0)
    if args.arch == "gcn":
        fixed += g.n * args.width * es + g.n * 4  # self term
    gather = g.nnz * (args.width * es + per_entry) + fixed
    compulsory = g.n * args.width * es + g.nnz * per_entry + fixed
    print(json.dumps({"op": "aggregate", "arch": args.arch, "transpose": args.transpose, "dtype": "fp32" if args.fp32 else "bf16",
                      "nodes": g.n, "entries": int(g.nnz), "width": args.width, "us_per_launch": round(us, 1),
                      "gather_bytes": gather, "gather_GBps": round(gather / us / 1e3, 1),
                      "compulsory_bytes": compulsory, "compulsory_GBps": round(compulsory / us / 1e3, 1),
                      "source_matrix_MB": round(g.n * args.width * es / 1e6, 1)}))
    ctx.close()


if __name__ == "__main__":
    main()
