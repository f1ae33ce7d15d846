#!/usr/bin/env python
"""Benchmark of the link-prediction training step.

One "step" = everything a worker does for one batch in Algorithm 1: draw the negatives, run the
encoder forward, score positives and negatives, take the loss, back-propagate, update the weights
with Adam.  The metric is training edges per second (positives + negatives) over the whole job.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line.  Keys beyond the usual ones:
  roofline      the aggregation launches of the timed region (the dominant kernel), algorithmic bytes / time
  hbm_roofline  the same kernel on a graph whose source matrix does not fit the L2 cache (HBM-bound)
  configs       the other workload configurations at full size (parity-tested elsewhere; timed here)
  cpu_baseline  the CPU oracle on the host cores, one thread and all cores
  e2e           the same metric through the host-buffer entry point, copies inside the timed region
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import socket
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

WORKLOAD = "c2_chunglu_sage2"
METRIC = "training edges/sec (pos+neg) per step"
UNIT = "edges/s"
K_NEG = 1
SEED = 1234

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of the aggregation launches of one step on the
# benchmark workload, from one ncu capture of a whole step at full size (layer-1 forward 124.1 MB, layer-2 forward
# 409.5 MB, adjoint 406.3 MB): mean per timed launch.  Valid only for the kernel source it was taken with (sha1 of
# csrc/spmm.cuh + csrc/common.cuh); reported as null otherwise.
NCU_TRAFFIC = {"spmm_sha1": "78f78a3c22a0f25d5b0710a2e5a8e287eb3db256", "bytes_per_launch": (124.1e6 + 409.5e6 + 406.3e6) / 3.0,
               # the forward mean aggregation (F = 256, BF16) on the 1 M-node graph of the HBM-bound roofline run: 3414.8 MB read + 560.8 MB written
               "hbm_forward_bytes_per_launch": 3414.8e6 + 560.8e6}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), float(d.get("bf16_tflops_sustained", d.get("bf16_tflops", 0))), "measured"
    return 6650.0, 1400.0, "fallback"


def spmm_source_hash():
    h = hashlib.sha1()
    for name in ("spmm.cuh", "common.cuh"):  # the kernel and the vector load / store forms it uses
        with open(os.path.join(ROOT, "paper_2506_20818_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


class ClockSampler:
    """nvidia-smi sampling of SM clocks and throttle reasons while the timed region runs."""

    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.device_index = device_index
        self.proc = None
        self.path = f"/tmp/lp_bench_clocks_{os.getpid()}.csv"

    def start(self):
        try:
            self.out = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100",
                                          "-i", str(self.device_index)], stdout=self.out, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.out.close()
        sm, smax, reasons, power = [], [], set(), []
        for line in open(self.path):
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1]))
                smax.append(float(parts[2]))
                power.append(float(parts[3]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        try:
            os.remove(self.path)
        except OSError:
            pass
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        busy = [c for c, p in zip(sm, power) if p >= 0.5 * max(power)] or sm
        return {"sm_mhz": statistics.median(busy), "sm_max_mhz": max(smax), "reasons": sorted(reasons), "samples": len(sm),
                "power_w_max": max(power)}


def cpu_cores():
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def run_oracle_steps(g, X, params, dims, pos, B, steps, warmup):
    """Times the CPU oracle, as it stands, on full steps of the benchmark workload."""
    import oracle
    times = []
    p = params.astype(np.float64)
    m = np.zeros_like(p)
    v = np.zeros_like(p)
    nb = max(1, len(pos[0]) // B)
    for i in range(warmup + steps):
        lo = (i % nb) * B
        u, w = pos[0][lo:lo + B], pos[1][lo:lo + B]
        t0 = time.perf_counter()
        ns, nd, _ = oracle.sample_negatives(g.n, g.rowptr, g.col, u, SEED, i, K_NEG, edge_index_base=lo)
        out = oracle.train_step(g, X, p, "sage", dims, u, w, ns, nd)
        p, m, v = oracle.adam_step(p, m, v, out["grads"], i + 1)
        dt = time.perf_counter() - t0
        if i >= warmup:
            times.append(dt)
    return times


def oracle_baseline(g, X, params, dims, pos, B, steps_all_cores):
    """The oracle on the host: the requested number of steps with every core the process may use, and one step held to a
    single thread (numpy's BLAS pool and the C part's OpenMP team both limited to 1)."""
    out = {"unit": UNIT, "cores": cpu_cores(), "kind": "oracle"}
    times = run_oracle_steps(g, X, params, dims, pos, B, steps_all_cores, 0)
    out["value"] = len(times) * B * (1 + K_NEG) / sum(times)
    out["s_per_step"] = sum(times) / len(times)
    out["sample"] = (f"{len(times)} full steps of the same workload on all {out['cores']} cores (full-graph encoder, {B} positives + "
                     f"{B * K_NEG} negatives each); 1 such step on one thread")
    try:
        from threadpoolctl import threadpool_limits
        with threadpool_limits(limits=1):
            t1 = run_oracle_steps(g, X, params, dims, pos, B, 1, 0)
        out["single_thread"] = {"value": B * (1 + K_NEG) / t1[0], "unit": UNIT, "cores": 1, "s_per_step": t1[0]}
    except Exception as ex:  # the single-thread figure is additional: never lose the other one over it
        out["single_thread"] = {"value": None, "note": f"failed: {ex}"}
    return out


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


# ------------------------------------------------------------------------------------------------------------------
# the other configurations, timed at full size after the headline region (N = 1, rank 0)
# ------------------------------------------------------------------------------------------------------------------
def _events(torch):
    return torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)


def time_steps(torch, ctx, params, pu, pv, B, k, steps, warmup, seed=SEED):
    """ms per step of negatives + step + Adam on consecutive batches of B positives (wrapping around)."""
    dev = pu.device
    p = params.clone()
    m, v, grads = torch.zeros_like(p), torch.zeros_like(p), torch.zeros_like(p)
    loss = torch.zeros(1, device=dev)
    nb = max(1, pu.numel() // B)

    def one(i):
        lo = (i % nb) * B
        su, sv = pu[lo:lo + B], pv[lo:lo + B]
        _, nd = ctx.sample_negatives(seed, i, k, su, edge_index_base=lo)
        ctx.train_step(p, su, sv, None, nd, k, loss, grads, seed=seed, step=i)
        ctx.adam_step(p, m, v, grads, i + 1)

    for i in range(warmup):
        one(i)
    torch.cuda.synchronize()
    a, b = _events(torch)
    a.record()
    for i in range(steps):
        one(warmup + i)
    b.record()
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / steps
    Bq = min(B, pu.numel())
    return {"ms_per_step": ms, "edges_per_s": Bq * (1 + k) / (ms * 1e-3), "batch_pos": Bq, "steps": steps, "loss_last": float(loss.item())}


def bench_other_configs(torch, pkg, wl, dev):
    out = {}
    t_all = time.perf_counter()

    def t(a):
        return torch.from_numpy(np.ascontiguousarray(a)).to(dev)

    # ---- config 1: tiny graph, 2-layer GCN, FP32, every edge a positive
    g, X, params, pos, cfg = wl.make_config("c1_tiny_er_gcn2")
    ctx = pkg.Context(0)
    ctx.load_graph(g.n, g.rowptr, g.col, g.w, X)
    ctx.set_model("gcn", cfg["dims"], prec="fp32", max_batch=len(pos[0]), max_k=1)
    out["c1_tiny_er_gcn2"] = dict(time_steps(torch, ctx, t(params), t(pos[0]), t(pos[1]), len(pos[0]), 1, 100, 5), nodes=g.n, entries=g.nnz, dtype="f32")
    ctx.close()

    # ---- config 2 variants: every training positive behind one encoder pass; mini-batches over sampled blocks
    g, X, params, pos, cfg = wl.make_config("c2_chunglu_sage2")
    ctx = pkg.Context(0)
    ctx.load_graph(g.n, g.rowptr, g.col, g.w, X)
    pu, pv, pp = t(pos[0]), t(pos[1]), t(params)
    ctx.set_model("sage", cfg["dims"], prec="bf16", max_batch=len(pos[0]), max_k=1)
    out["c2_one_pass_all_positives"] = dict(time_steps(torch, ctx, pp, pu, pv, len(pos[0]), 1, 20, 3), nodes=g.n, entries=g.nnz, dtype="bf16")
    for B in (256, 10240, 51200):
        ctx.set_model("sage", cfg["dims"], prec="bf16", fanout=[25, 10], max_batch=B, max_k=1)
        out[f"c2_minibatch_fanout25_10_B{B}"] = dict(time_steps(torch, ctx, pp, pu, pv, B, 1, 30, 5), dtype="bf16")
    ctx.close()

    # ---- config 3: weighted 3-layer GCN, full graph (every training edge a positive; B = 65,536) and mini-batches
    g, X, params, pos, cfg = wl.make_config("c3_coauthor_gcn3")
    ctx = pkg.Context(0)
    ctx.load_graph(g.n, g.rowptr, g.col, g.w, X)
    pu, pv, pp = t(pos[0]), t(pos[1]), t(params)
    ctx.set_model("gcn", cfg["dims"], prec="bf16", max_batch=len(pos[0]), max_k=1)
    out["c3_coauthor_gcn3"] = dict(time_steps(torch, ctx, pp, pu, pv, len(pos[0]), 1, 20, 3), nodes=g.n, entries=g.nnz, dtype="bf16")
    out["c3_coauthor_gcn3_B65536"] = dict(time_steps(torch, ctx, pp, pu, pv, 65536, 1, 30, 3), dtype="bf16")
    for B in (256, 10240, 51200):
        ctx.set_model("gcn", cfg["dims"], prec="bf16", fanout=[25, 10, 5], max_batch=B, max_k=1)
        out[f"c3_minibatch_fanout25_10_5_B{B}"] = dict(time_steps(torch, ctx, pp, pu, pv, B, 1, 30, 5), dtype="bf16")
    ctx.close()

    # ---- config 4: directed 2.9 M-node graph, 3-layer SAGE-mean over sampled blocks (fan-outs 15/10/5)
    g, X, params, pos, cfg = wl.make_config("c4_citation_sage3_sampled")
    ctx = pkg.Context(0)
    ctx.load_graph(g.n, g.rowptr, g.col, None, X)
    ctx.set_model("sage", cfg["dims"], prec="bf16", fanout=cfg["fanout"], max_batch=65536, max_k=1)
    sel = np.random.default_rng(4).permutation(len(pos[0]))[: 16 * 65536]
    r = time_steps(torch, ctx, t(params), t(pos[0][sel]), t(pos[1][sel]), 65536, 1, 12, 3)
    st = ctx.stats()
    out["c4_citation_sage3_sampled"] = dict(r, nodes=g.n, entries=g.nnz, dtype="bf16", frontier_nodes=[int(st.block_nodes[h]) for h in range(3)],
                                           block_entries=[int(st.block_edges[h]) for h in range(3)])
    ctx.close()
    del X

    # ---- config 5: 8 emulated workers in sequence, gradients accumulated, one update; local vs global negatives
    g, X, params, pos, cfg = wl.make_config("c5_partitioned_sage2")
    p_workers, B = cfg["partitions"], 65536
    part = wl.random_partition(g.n, p_workers, seed=5)
    ctxG = pkg.Context(0)
    ctxG.load_graph(g.n, g.rowptr, g.col, None, X)
    a, b = _events(torch)
    a.record()
    ctxG.sparsify(cfg["alpha"], 5)
    b.record()
    torch.cuda.synchronize()
    sparsify_ms = a.elapsed_time(b)
    dpart, X_dev, pp = t(part), t(X), t(params)
    rows = np.repeat(np.arange(g.n, dtype=np.int64), np.diff(g.rowptr))
    upper = g.col > rows
    prow, pcol = part[rows], part[g.col]
    for negatives in ("local", "global"):
        acc = torch.zeros_like(pp)
        scratch = torch.zeros_like(pp)
        loss = torch.zeros(1, device=dev)
        total_ms, edges, n_batches, view_entries = 0.0, 0, 0, 0
        for i in range(p_workers):
            inside = (prow == i) & (pcol == i)
            ctx = pkg.Context(0)
            if negatives == "local":
                # local negatives never leave the partition: the worker holds its induced subgraph as a graph of its own
                # (nodes renumbered in ascending order of their ids; every node of it is a candidate)
                own = np.nonzero(part == i)[0]
                new_id = np.full(g.n, -1, dtype=np.int64)
                new_id[own] = np.arange(own.shape[0])
                sub = wl.csr_from_edges(own.shape[0], new_id[rows[inside]], new_id[g.col[inside]], presorted=True)
                ctx.load_graph(sub.n, sub.rowptr, sub.col, None, np.ascontiguousarray(X[own]))
                view_entries += sub.nnz
                keep = inside & upper  # the partition's own undirected edges, each once
                pu, pv = t(new_id[rows[keep]].astype(np.int32)), t(new_id[g.col[keep]].astype(np.int32))
            else:
                # global negatives: own rows from the partition, foreign rows from the sparsified global graph (built on the GPU)
                rp, col, vstats = ctxG.worker_view(dpart, i, keep_cross_edges=False, foreign_mode=1)
                view_entries += int(col.numel())
                ctx.load_graph(g.n, rp, col, None, X_dev, on_device=True)
                keep = inside & upper
                pu, pv = t(rows[keep].astype(np.int32)), t(g.col[keep].astype(np.int32))
            ctx.set_model("sage", cfg["dims"], prec="bf16", max_batch=B, max_k=1)
            nbat = (pu.numel() + B - 1) // B
            _, nd = ctx.sample_negatives(SEED, 10_000 + i, 1, pu[:B])  # warm-up step into a scratch gradient
            ctx.train_step(pp, pu[:B], pv[:B], None, nd, 1, loss, scratch, seed=SEED, step=0)
            torch.cuda.synchronize()
            a, b = _events(torch)
            a.record()
            for j in range(nbat):
                su, sv = pu[j * B:(j + 1) * B], pv[j * B:(j + 1) * B]
                _, nd = ctx.sample_negatives(SEED, i * 64 + j, 1, su, edge_index_base=j * B)
                ctx.train_step(pp, su, sv, None, nd, 1, loss, acc, seed=SEED, step=i * 64 + j, accumulate=True)
            if i == p_workers - 1:  # Algorithm 1: average over the workers, then one update
                m, v = torch.zeros_like(pp), torch.zeros_like(pp)
                ctx.adam_step(pp.clone(), m, v, acc, 1, grad_scale=1.0 / p_workers)
            b.record()
            torch.cuda.synchronize()
            total_ms += a.elapsed_time(b)
            edges += 2 * int(pu.numel())
            n_batches += nbat
            ctx.close()
        out[f"c5_partitioned_sage2_{negatives}_negatives"] = {"ms_per_pass": total_ms, "edges_per_s": edges / (total_ms * 1e-3), "batches": n_batches, "scored_edges": edges,
                                                             "workers": p_workers, "nodes": g.n, "entries_global": g.nnz, "entries_all_views": view_entries, "dtype": "bf16",
                                                             "note": "one pass over every partition's own positives in batches of 65,536, gradients accumulated "
                                                                     "in partition order, one Adam update; graph loading and view building outside the timed spans; "
                                                                     + ("each worker trains on its induced subgraph alone (about 125,000 nodes)" if negatives == "local" else
                                                                        "each worker trains on its view of all 1 M nodes (own rows induced, foreign rows sparsified)")}
    out["c5_sparsify_global_graph_ms"] = sparsify_ms
    ctxG.close()
    out["wall_s"] = time.perf_counter() - t_all
    return out


def bench_hbm_roofline(torch, pkg, wl, dev, hbm_peak, peak_kind):
    """The aggregation kernel where it is bound by HBM: the 1 M-node graph of the partitioned configuration, whose
    512 MB BF16 source matrix does not fit the 126 MB L2 (mean aggregation, F = 256, forward and adjoint)."""
    g = wl.chung_lu(1_000_000, 16.0, 2.1, seed=5)
    ctx = pkg.Context(0)
    ctx.load_graph(g.n, g.rowptr, g.col, None, wl.node_features(g.n, 8, 5))
    F, es = 256, 2
    H = torch.randn(g.n, F, device=dev).to(torch.bfloat16)
    out = {"graph": "Chung-Lu, 1,000,000 nodes, mean degree 16", "entries": g.nnz, "width": F, "dtype": "bf16", "source_matrix_MB": g.n * F * es / 1e6,
           "peak": hbm_peak, "peak_source": f"of {peak_kind}", "unit": "GB/s", "bound": "hbm",
           "note": "time includes the combine launch of the hub rows; dram_frac = ncu DRAM bytes of the launch / live time / peak"}
    for name, transpose in (("forward", False), ("adjoint_with_coefficients", True)):  # the operator-level adjoint carries 1/|N(v)| per entry
        for _ in range(3):
            ctx.op_aggregate("sage", H, transpose=transpose)
        torch.cuda.synchronize()
        ev = []
        for _ in range(20):
            a, b = _events(torch)
            a.record()
            ctx.op_aggregate("sage", H, transpose=transpose)
            b.record()
            ev.append((a, b))
        torch.cuda.synchronize()
        us = 1e3 * statistics.median(a.elapsed_time(b) for a, b in ev)
        per_entry = 4 + (4 if transpose else 0)
        fixed = (g.n + 1) * 4 + g.n * F * es + (0 if transpose else g.n * 4)
        gather = g.nnz * (F * es + per_entry) + fixed
        compulsory = g.n * F * es + g.nnz * per_entry + fixed
        out[name] = {"us_per_launch": us, "launches": 20, "gather_bytes": gather, "compulsory_bytes": compulsory,
                     "achieved_gather": gather / us / 1e3, "frac_gather": gather / us / 1e3 / hbm_peak,
                     "achieved_compulsory": compulsory / us / 1e3, "frac_compulsory": compulsory / us / 1e3 / hbm_peak}
        if not transpose:  # DRAM traffic of this launch from ncu (valid for the kernel source it was captured with)
            traffic = NCU_TRAFFIC["hbm_forward_bytes_per_launch"] if NCU_TRAFFIC["spmm_sha1"] == spmm_source_hash() else None
            out[name]["traffic"] = traffic
            out[name]["dram_achieved"] = traffic / us / 1e3 if traffic else None
            out[name]["dram_frac"] = traffic / us / 1e3 / hbm_peak if traffic else None
    ctx.close()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--scale", type=float, default=1.0, help="shrink the workload (for quick checks and ncu captures)")
    ap.add_argument("--batch", type=int, default=65536)
    ap.add_argument("--cpu-baseline-steps", type=int, default=2)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip the HBM-bound roofline run and the other configurations")
    ap.add_argument("--cache-input-agg", action="store_true", help="reuse the weight-independent first-layer aggregation across steps (not the default, not the headline)")
    ap.add_argument("--predictor", default="dot", choices=["dot", "mlp"], help="mlp: the 3-layer MLP predictor of width 256 instead of the dot product (not the headline)")
    ap.add_argument("--breakdown", action="store_true", help="print a per-category time breakdown to stderr")
    args = ap.parse_args()

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours":
        # started as a plain process: start one rank per GPU of this node and let rank 0 print the line
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}", "--master-addr", "127.0.0.1",
               "--master-port", str(free_port()), os.path.abspath(__file__)] + sys.argv[1:]
        return subprocess.call(cmd)

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    import workloads as wl

    if args.impl == "reference":
        # the CPU oracle, as it stands, on the host cores: rank 0 alone
        if rank != 0:
            return 0
        g, X, params, pos, cfg = wl.make_config(WORKLOAD, scale=args.scale)
        B = min(args.batch, len(pos[0]))
        steps = max(1, min(args.steps, 4))
        warm = min(args.warmup, 1)
        times = run_oracle_steps(g, X, params, cfg["dims"], pos, B, steps, warm)
        t = sum(times)
        val = steps * B * (1 + K_NEG) / t
        line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": steps, "warmup": warm,
                "ms_per_step": 1e3 * t / steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
                "data": "synthetic", "config": {"workload": WORKLOAD, "nodes": g.n, "entries": g.nnz, "batch_pos": B, "neg_per_pos": K_NEG,
                                                "scale": args.scale},
                "cpu_baseline": {"value": val, "unit": UNIT, "cores": cpu_cores(), "kind": "oracle",
                                 "sample": f"{steps} full steps of the workload (requested {args.steps}, bounded to keep the run to minutes)"},
                "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
        print(json.dumps(line))
        return 0

    import torch
    import paper_2506_20818_b200 as pkg
    from paper_2506_20818_b200 import build as lpbuild
    from paper_2506_20818_b200.dp import batch_for, sync_gradients

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (no CPU fall-back exists)")
    dist = None
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local_rank}"))
    if rank == 0:
        lpbuild.build()
    if world > 1:
        dist.barrier()  # no rank loads the library before rank 0 has (re)built it
    dev = f"cuda:{local_rank}"
    torch.cuda.set_device(local_rank)

    g, X, params, pos, cfg = wl.make_config(WORKLOAD, scale=args.scale)
    dims = cfg["dims"]
    B = min(args.batch, len(pos[0]))
    nb = max(1, len(pos[0]) // B)

    pred_hidden = 256 if args.predictor == "mlp" else 0
    if pred_hidden:
        params = wl.glorot_params("sage", dims, SEED, pred_hidden=pred_hidden)
        args.no_cpu_baseline = True  # the baseline leg times the headline (dot-product) workload only

    stream = torch.cuda.Stream(device=dev)
    with torch.cuda.stream(stream):
        ctx = pkg.Context(local_rank, stream=stream)
        ctx.load_graph(g.n, g.rowptr, g.col, g.w, X)
        ctx.set_model("sage", dims, prec="bf16", max_batch=B, max_k=K_NEG, cache_input_aggregation=args.cache_input_agg, pred_hidden=pred_hidden)
        pu = torch.from_numpy(pos[0]).to(dev)
        pv = torch.from_numpy(pos[1]).to(dev)
        p = torch.from_numpy(params).to(dev)
        m = torch.zeros_like(p)
        v = torch.zeros_like(p)
        grads = torch.zeros_like(p)
        loss = torch.zeros(1, device=dev)
        neg = torch.empty(B * K_NEG, dtype=torch.int32, device=dev)
    lib = ctx.lib
    import ctypes as C

    def one_step(i, t_adam):
        # data-parallel over batches: rank r takes batches r, r + world, ...
        b = batch_for(i, rank, world, nb)
        lo = b * B
        su, sv = pu[lo:lo + B], pv[lo:lo + B]
        ctx._ck(lib.lp_sample_negatives(ctx.h, C.c_uint64(SEED), C.c_uint64(i), C.c_int32(K_NEG), C.c_int32(0), C.c_void_p(su.data_ptr()),
                                        C.c_int64(B), C.c_int64(lo), None, C.c_void_p(neg.data_ptr())))
        ctx.train_step(p, su, sv, None, neg, K_NEG, loss, grads, seed=SEED, step=i)
        with torch.cuda.stream(stream):
            scale = sync_gradients(grads, world, dist)  # gradient synchronisation of Algorithm 1 (sum; 1/p folded into the update)
        ctx.adam_step(p, m, v, grads, t_adam, grad_scale=scale)

    # ---- warm-up
    with torch.cuda.stream(stream):
        for i in range(args.warmup):
            one_step(i, i + 1)
    stream.synchronize()

    # ---- timed region: K steps, events on the launching stream, aggregation launches timed inside
    launches0 = ctx.stats().kernel_launches
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.2)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    # the aggregation launches are timed inside the region on every 8th step only: an event record between two kernels
    # keeps the second from being made resident while the first still runs (a timed step is about 3 % slower)
    PROF_EVERY = 8
    ctx.profile_sample_every(PROF_EVERY)
    ctx.profile_begin(["agg_fwd", "agg_bwd"])
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(stream):
        e0.record(stream)
        for i in range(args.steps):
            one_step(args.warmup + i, args.warmup + i + 1)
        e1.record(stream)
    stream.synchronize()
    prof = ctx.profile_end()
    ctx.profile_sample_every(1)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    elapsed_ms = e0.elapsed_time(e1)
    clocks = sampler.stop() if rank == 0 else None
    launches = ctx.stats().kernel_launches - launches0
    loss_value = float(loss.item())
    if world > 1:
        t = torch.tensor([elapsed_ms], device=dev, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        elapsed_ms = float(t.item())
    edges_per_step = B * (1 + K_NEG) * world
    value = args.steps * edges_per_step / (elapsed_ms * 1e-3)

    # ---- roofline of the dominant kernel (aggregation launches timed inside the region above)
    hbm_peak, bf16_peak, peak_kind = measured_peaks()
    agg_ms = prof["agg_fwd"]["ms"] + prof["agg_bwd"]["ms"]
    agg_bytes = prof["agg_fwd"]["bytes"] + prof["agg_bwd"]["bytes"]
    agg_spans = prof["agg_fwd"]["spans"] + prof["agg_bwd"]["spans"]
    achieved = agg_bytes / (agg_ms * 1e-3) / 1e9 if agg_ms > 0 else None
    traffic = NCU_TRAFFIC["bytes_per_launch"] if NCU_TRAFFIC["spmm_sha1"] == spmm_source_hash() and args.scale == 1.0 else None
    # compulsory bytes of the same launches: every source row read once instead of once per stored entry
    # (three aggregation launches per step: widths dims[0], dims[1], dims[1]; BF16)
    widths = [dims[0]] + [dims[k] for k in range(1, len(dims) - 1) for _ in (0, 1)]
    gather_minus_min = sum((g.nnz - g.n) * f * 2 for f in widths) / max(len(widths), 1)
    avg_launch_s = 1e-3 * agg_ms / max(agg_spans, 1)
    agg_steps = max(1, agg_spans // max(len(widths), 1))  # steps of the timed region whose aggregation launches carried events
    min_bytes = agg_bytes / max(agg_spans, 1) - gather_minus_min
    fits_l2 = bool(g.n * max(widths) * 2 <= 126e6)
    roofline = {"bound": "l2" if fits_l2 else "hbm",
                "bound_note": ("the gathered source matrices (51-102 MB) stay in the 126 MB L2, so the launches are bound by L2 gathers, not by HBM: "
                               "`achieved` (gather convention) may exceed the HBM peak; read dram_frac, t_bound_over_t and gather_ceiling, and "
                               "hbm_roofline for the same kernel on an input that does not fit L2") if fits_l2 else "source matrix larger than L2",
                "kernel": "spmm_padded_kernel (aggregation forward + adjoint)", "achieved": achieved, "peak": hbm_peak,
                "unit": "GB/s", "frac": (achieved / hbm_peak) if achieved else None, "peak_source": f"of {peak_kind} (HBM copy bandwidth)",
                "frac_of_nominal_8000": (achieved / 8000.0) if achieved else None, "traffic": traffic,
                "dram_frac": (traffic / avg_launch_s / 1e9 / hbm_peak) if traffic and avg_launch_s > 0 else None,
                "min_bytes_per_launch": min_bytes,
                "t_bound_over_t": (min_bytes / (hbm_peak * 1e9) / avg_launch_s) if avg_launch_s > 0 else None,
                "source_rows_fit_l2": fits_l2,
                "launches_timed": agg_spans, "avg_launch_us": 1e3 * agg_ms / max(agg_spans, 1),
                "timed_every_nth_step": PROF_EVERY,
                "bytes_per_launch": agg_bytes / max(agg_spans, 1), "share_of_step": (agg_ms / agg_steps) / (elapsed_ms / args.steps),
                "note": "algorithmic bytes, gather convention (each stored entry reads one source row, nothing assumed cached)"}

    # ---- gather ceiling of the same launches (outside the timed region): the bare gather of the index streams the
    # three aggregation launches of a step walk (lp_op_gather_ceiling: no rows, arithmetic or epilogue).  With the source
    # matrix largely L2 resident this, not the HBM copy bandwidth, is the floor of the aggregation kernel.
    if rank == 0:
        def probe_us(width, transpose):
            Hp = torch.randn((g.n, width), device=dev).to(torch.bfloat16)
            ev = []
            with torch.cuda.stream(stream):
                for it in range(8):
                    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    a.record(stream)
                    ctx.op_gather_ceiling(Hp, transpose=transpose)
                    b.record(stream)
                    ev.append((a, b))
            stream.synchronize()
            return 1e3 * statistics.median(a.elapsed_time(b) for a, b in ev[3:])

        # forward launches walk the CSR, the adjoint launch the transposed structure (layer 1 has no adjoint)
        shapes = [(dims[k], False) for k in range(len(dims) - 1)] + [(dims[k], True) for k in range(1, len(dims) - 1)]
        if all(f * 2 in (128, 256, 512) for f, _ in shapes):
            floor_us = sum(probe_us(f, tr) for f, tr in shapes)
            agg_us_per_step = 1e3 * agg_ms / agg_steps
            roofline["gather_ceiling"] = {"floor_us_per_step": floor_us, "aggregation_us_per_step": agg_us_per_step,
                                          "frac": floor_us / agg_us_per_step if agg_us_per_step > 0 else None,
                                          "note": "time of lp_op_gather_ceiling over the same index streams and row widths "
                                                  "divided by the aggregation time of a step"}

    # ---- breakdown of a few more steps, outside the timed region
    breakdown = None
    if args.breakdown or rank == 0:
        ctx.profile_begin()
        nbk = min(50, args.steps)
        with torch.cuda.stream(stream):
            for i in range(nbk):
                one_step(args.warmup + args.steps + i, args.warmup + args.steps + i + 1)
        bp = ctx.profile_end()
        breakdown = {k: {"us_per_step": 1e3 * d["ms"] / nbk, "GBps": (d["bytes"] / (d["ms"] * 1e-3) / 1e9) if d["ms"] > 0 else None,
                         "frac_of_hbm_peak": (d["bytes"] / (d["ms"] * 1e-3) / 1e9 / hbm_peak) if d["ms"] > 0 else None,
                         "TFLOPs": (d["flops"] / (d["ms"] * 1e-3) / 1e12) if d["ms"] > 0 else None} for k, d in bp.items() if d["spans"]}
        if args.breakdown and rank == 0:
            print(json.dumps({"breakdown_per_step": breakdown}, indent=1), file=sys.stderr)

    # ---- end to end: pinned host batch -> device, negatives, step, gradient average, update, loss -> host, every step
    e2e = None
    if not args.no_e2e:
        hu = torch.from_numpy(pos[0]).pin_memory()
        hv = torch.from_numpy(pos[1]).pin_memory()
        loss_h = torch.zeros(1).pin_memory()
        n_e2e = max(50, min(args.steps, 200))  # at least 50 steps: the first ones still warm the pinned-copy path up
        t_base = args.warmup + args.steps + 100
        du_stage = torch.empty(B, dtype=torch.int32, device=dev)
        dv_stage = torch.empty(B, dtype=torch.int32, device=dev)

        def host_step(i):
            b = batch_for(i, rank, world, nb)
            lo = b * B
            if world == 1:  # the library's host-buffer entry point does all of it in one call
                ctx.train_step_host(p, hu[lo:lo + B], hv[lo:lo + B], K_NEG, seed=SEED, step=i, edge_index_base=lo, adam_m=m, adam_v=v,
                                    adam_t=i + 1, loss_host=loss_h)
                return
            # data parallel: the gradient average of Algorithm 1 sits between the step and the update
            with torch.cuda.stream(stream):
                du_stage.copy_(hu[lo:lo + B], non_blocking=True)
                dv_stage.copy_(hv[lo:lo + B], non_blocking=True)
                ctx._ck(lib.lp_sample_negatives(ctx.h, C.c_uint64(SEED), C.c_uint64(i), C.c_int32(K_NEG), C.c_int32(0), C.c_void_p(du_stage.data_ptr()),
                                                C.c_int64(B), C.c_int64(lo), None, C.c_void_p(neg.data_ptr())))
                ctx.train_step(p, du_stage, dv_stage, None, neg, K_NEG, loss, grads, seed=SEED, step=i)
                scale = sync_gradients(grads, world, dist)
                ctx.adam_step(p, m, v, grads, i + 1, grad_scale=scale)
                loss_h.copy_(loss, non_blocking=True)
            stream.synchronize()

        for i in range(3):
            host_step(t_base + i)
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record(stream)
        for i in range(n_e2e):
            host_step(t_base + 3 + i)
        f1.record(stream)
        stream.synchronize()
        e2e_ms = max(f0.elapsed_time(f1), 1e3 * (time.perf_counter() - t0))
        if world > 1:
            t = torch.tensor([e2e_ms], device=dev, dtype=torch.float64)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            e2e_ms = float(t.item())
        e2e = {"value": n_e2e * edges_per_step / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": 2 * B * 4, "d2h_bytes_per_step": 4,
               "steps": n_e2e, "note": ("lp_train_step_host: pinned host batch -> device, negatives, step, Adam, loss -> host" if world == 1 else
                                        "per rank: pinned host batch -> device, negatives, step, all-reduce of the gradient, Adam, loss -> host")}

    # ---- the same kernel where HBM binds it, and the other configurations (rank 0, one GPU)
    hbm_roofline = other = None
    ctx.close()
    if rank == 0 and world == 1 and not args.no_extras and args.scale == 1.0:
        try:
            hbm_roofline = bench_hbm_roofline(torch, pkg, wl, dev, hbm_peak, peak_kind)
        except Exception as ex:
            hbm_roofline = {"failed": str(ex)}
        try:
            other = bench_other_configs(torch, pkg, wl, dev)
        except Exception as ex:
            other = {"failed": str(ex)}

    # ---- CPU baseline: the oracle on the host cores, rank 0 at N = 1 only
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        try:
            cpu = oracle_baseline(g, X, params, dims, pos, B, args.cpu_baseline_steps)
        except Exception as ex:  # the baseline must never take the GPU result down with it
            cpu = {"value": None, "unit": UNIT, "cores": cpu_cores(), "kind": "oracle", "sample": f"failed: {ex}"}

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
                "ms_per_step": elapsed_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
                "data": "synthetic",
                "config": {"workload": WORKLOAD, "graph": "Chung-Lu power law, exponent 2.1, mean degree 20", "nodes": g.n, "entries": g.nnz,
                           "model": "2-layer GraphSAGE-mean 128-256-256, " + ("3-layer MLP predictor (256)" if pred_hidden else "dot-product predictor"), "batch_pos": B, "neg_per_pos": K_NEG,
                           "scale": args.scale, "cache_input_aggregation": bool(args.cache_input_agg), "parallelism": f"dp{world}" if world > 1 else "single GPU",
                           "l2": "no flush: the step streams ~1 GB of activations per pass, several times the 126 MB L2"},
                "clocks": clocks, "gpu_launches": int(launches), "loss_last": loss_value, "roofline": roofline, "hbm_roofline": hbm_roofline,
                "cpu_baseline": cpu, "e2e": e2e, "breakdown_us_per_step": breakdown, "configs": other}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
