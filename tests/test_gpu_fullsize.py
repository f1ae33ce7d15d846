"""Parity at full size, in the launch configurations the benchmark times.

  config 2: 200,000 nodes, 3.93 M stored entries, 2-layer SAGE-mean 128-256-256, one batch of 65,536 positives +
            65,536 negatives (BF16 and FP32)
  config 3: 235,000 nodes, 2.21 M weighted entries, 3-layer GCN, every training edge a positive in one step
            (1.105 M + 1.105 M scored edges; BF16 and FP32)
  config 4: 2.9 M nodes, 30 M directed entries, fan-outs 15/10/5, 65,536 positives: the sampled computational graph
            bit for bit at full size (the oracle's samplers are cheap there), the whole step at scale 0.1
            (290,000 nodes, about half a minute of oracle time; at full size the FP64 oracle would hold tens of GB)
  config 5: 1 M nodes, 15.8 M entries, 8 partitions; the global graph sparsified and the workers' views built on the
            GPU (structures bit for bit against the oracle); at full size the BF16 steps of two partitions with local
            and of one with global negatives against the oracle (an oracle step on 1 M nodes takes about 25 s, so not all
            sixteen), and the 8-way accumulated gradient against the sum of the 8 separate gradients; at scale 0.1 every
            partition's step in both modes and the accumulated gradient against the oracle's average over the 8 workers

The oracle computes whole steps here (tens of seconds each on the host cores)."""
import numpy as np
import pytest

import oracle
import workloads as wl
from helpers import assert_relu_decisions_agree, rel_l2

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu
DEV = "cuda:0"
TOL = {"fp32": 1e-5, "bf16": 2e-2}


@pytest.fixture(scope="module")
def pkg():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import __graft_entry__ as ge
    ge.build()
    import paper_2506_20818_b200 as p
    return p


@pytest.fixture(scope="module")
def config2():
    g, X, params, pos, cfg = wl.make_config("c2_chunglu_sage2")
    B = 65536
    lo = 7 * B  # the eighth batch of the epoch, as bench.py would slice it
    u, v = pos[0][lo:lo + B].copy(), pos[1][lo:lo + B].copy()
    return g, X, params, cfg["dims"], u, v, lo


def t32(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


@pytest.mark.parametrize("prec", ["bf16", "fp32"])
def test_config2_full_size_step(pkg, config2, prec):
    g, X, params, dims, u, v, lo = config2
    B = len(u)
    ctx = pkg.Context(0)
    ctx.load_graph(g.n, g.rowptr, g.col, g.w, X)
    ctx.set_model("sage", dims, prec=prec, max_batch=B, max_k=1)  # bench.py's configuration
    du, dv = t32(u), t32(v)
    seed, step = 1234, 17
    _, nd = ctx.sample_negatives(seed, step, 1, du, edge_index_base=lo)
    p = t32(params)
    loss = torch.zeros(1, device=DEV)
    grads = torch.zeros(ctx.n_params, device=DEV)
    ctx.train_step(p, du, dv, None, nd, 1, loss, grads, seed=seed, step=step)
    torch.cuda.synchronize()
    ons, ond, oex = oracle.sample_negatives(g.n, g.rowptr, g.col, u, seed, step, 1, edge_index_base=lo)
    assert np.array_equal(nd.cpu().numpy(), ond) and ctx.stats().negatives_exhausted == oex
    H1 = ctx.embeddings(1).cpu().numpy()
    ref = oracle.train_step(g, X, params, "sage", dims, u, v, ons, ond, relu_ties=[H1 > 0], rounding=prec)
    assert_relu_decisions_agree(ref["cache"], [H1 > 0], None, f"config 2 full size {prec}")
    err = {"loss": abs(loss.item() - ref["loss"]) / abs(ref["loss"]),
           "H1": rel_l2(H1, ref["cache"]["H"][1]),
           "H2": rel_l2(ctx.embeddings(2).cpu().numpy(), ref["cache"]["H"][2]),
           "dHK": rel_l2(ctx.output_gradient().cpu().numpy(), ref["dHK"]),
           "grads": rel_l2(grads.cpu().numpy(), ref["grads"])}
    gg, off = grads.cpu().numpy(), 0
    for li in range(2):
        nw = 2 * dims[li] * dims[li + 1]
        err[f"dW{li}"] = rel_l2(gg[off:off + nw], ref["grads"][off:off + nw])
        err[f"db{li}"] = rel_l2(gg[off + nw:off + nw + dims[li + 1]], ref["grads"][off + nw:off + nw + dims[li + 1]])
        off += nw + dims[li + 1]
    bad = {k: e for k, e in err.items() if not e < TOL[prec]}
    assert not bad, f"outside {TOL[prec]}: {bad} (all {err})"
    # structure of the loaded graph, bit-exact at full size
    colptr, rowidx, perm = ctx.get_structure()
    ocp, ori, ope = oracle.csc_transpose(g.n, g.rowptr, g.col)
    assert np.array_equal(colptr.cpu().numpy(), ocp) and np.array_equal(rowidx.cpu().numpy(), ori) and np.array_equal(perm.cpu().numpy(), ope)
    ctx.close()


def test_config4_sampled_large(pkg):
    g, X, params, pos, cfg = wl.make_config("c4_citation_sage3_sampled", scale=0.1)
    dims, fanout = cfg["dims"], cfg["fanout"]
    B = 6554
    sel = np.sort(np.random.default_rng(4).choice(len(pos[0]), B, replace=False))
    u, v = pos[0][sel].copy(), pos[1][sel].copy()
    ctx = pkg.Context(0)
    ctx.load_graph(g.n, g.rowptr, g.col, None, X)
    ctx.set_model("sage", dims, prec="bf16", fanout=fanout, max_batch=B, max_k=1)
    du, dv = t32(u), t32(v)
    seed, step = 99, 5
    _, nd = ctx.sample_negatives(seed, step, 1, du)
    loss = torch.zeros(1, device=DEV)
    grads = torch.zeros(ctx.n_params, device=DEV)
    ctx.train_step(t32(params), du, dv, None, nd, 1, loss, grads, seed=seed, step=step)
    torch.cuda.synchronize()
    ons, ond, _ = oracle.sample_negatives(g.n, g.rowptr, g.col, u, seed, step, 1)
    assert np.array_equal(nd.cpu().numpy(), ond)
    fr, blks = oracle.build_blocks(g.n, g.rowptr, g.col, np.concatenate([u, v, ond]), fanout, seed, step)
    st = ctx.stats()
    assert [int(st.block_nodes[h]) for h in range(3)] == [len(f) for f in fr[:3]]
    assert [int(st.block_edges[h]) for h in range(3)] == [len(b[1]) for b in blks]
    for h in range(0, 4):
        f_, ptr_, col_ = ctx.block(h)
        if h < 3:
            assert np.array_equal(f_.cpu().numpy(), fr[h])
        if h >= 1:
            assert np.array_equal(ptr_.cpu().numpy(), blks[h - 1][0]) and np.array_equal(col_.cpu().numpy(), blks[h - 1][1])
    ref = oracle.train_step(g, X, params, "sage", dims, u, v, ons, ond, blocks=(fr, blks))
    err = {"loss": abs(loss.item() - ref["loss"]) / abs(ref["loss"]),
           "HK": rel_l2(ctx.embeddings(3, rows=len(fr[0])).cpu().numpy(), ref["cache"]["H"][3][fr[0]]),
           "grads": rel_l2(grads.cpu().numpy(), ref["grads"])}
    bad = {k: e for k, e in err.items() if not e < TOL["bf16"]}
    assert not bad, f"outside tolerance: {bad}"
    ctx.close()


# ------------------------------------------------------------------------------------------ config 3
def check_step(ctx, ref, loss, grads, arch, dims, tol, extra=None):
    err = {"loss": abs(loss.item() - ref["loss"]) / abs(ref["loss"]), "grads": rel_l2(grads.cpu().numpy(), ref["grads"])}
    K = len(dims) - 1
    gg, off = grads.cpu().numpy(), 0
    for li in range(K):
        nw = (2 if arch == "sage" else 1) * dims[li] * dims[li + 1]
        err[f"dW{li}"] = rel_l2(gg[off:off + nw], ref["grads"][off:off + nw])
        err[f"db{li}"] = rel_l2(gg[off + nw:off + nw + dims[li + 1]], ref["grads"][off + nw:off + nw + dims[li + 1]])
        off += nw + dims[li + 1]
    err.update(extra or {})
    bad = {k: e for k, e in err.items() if not e < tol}
    assert not bad, f"outside {tol}: {bad} (all {err})"
    return err


@pytest.mark.parametrize("prec", ["bf16", "fp32"])
def test_config3_full_size_step(pkg, prec):
    g, X, params, pos, cfg = wl.make_config("c3_coauthor_gcn3")
    assert g.n == 235000 and g.w is not None and g.w.max() == 5.0
    dims = cfg["dims"]
    u, v = pos
    B = len(u)  # every training edge is a positive of the one step: 1.105 M positives + as many negatives
    assert B > 1_000_000
    ctx = pkg.Context(0)
    ctx.load_graph(g.n, g.rowptr, g.col, g.w, X)
    ctx.set_model("gcn", dims, prec=prec, max_batch=B, max_k=1)
    du, dv = t32(u), t32(v)
    seed, step = 77, 3
    _, nd = ctx.sample_negatives(seed, step, 1, du)
    loss, grads = torch.zeros(1, device=DEV), torch.zeros(ctx.n_params, device=DEV)
    ctx.train_step(t32(params), du, dv, None, nd, 1, loss, grads, seed=seed, step=step)
    torch.cuda.synchronize()
    ons, ond, oex = oracle.sample_negatives(g.n, g.rowptr, g.col, u, seed, step, 1)
    assert np.array_equal(nd.cpu().numpy(), ond) and ctx.stats().negatives_exhausted == oex
    masks = [ctx.embeddings(layer).cpu().numpy() > 0 for layer in (1, 2)]
    ref = oracle.train_step(g, X, params, "gcn", dims, u, v, ons, ond, relu_ties=masks, rounding=prec)
    assert_relu_decisions_agree(ref["cache"], masks, None, f"config 3 full size {prec}")
    extra = {f"H{l}": rel_l2(ctx.embeddings(l).cpu().numpy(), ref["cache"]["H"][l]) for l in (1, 2, 3)}
    extra["dHK"] = rel_l2(ctx.output_gradient().cpu().numpy(), ref["dHK"])
    check_step(ctx, ref, loss, grads, "gcn", dims, TOL[prec], extra)
    ctx.close()


# ------------------------------------------------------------------------------------------ config 4
def test_config4_full_size_blocks(pkg):
    g, X, params, pos, cfg = wl.make_config("c4_citation_sage3_sampled")
    assert g.n == 2_900_000 and g.nnz > 29_900_000
    dims, fanout = cfg["dims"], cfg["fanout"]
    B = 65536
    sel = np.sort(np.random.default_rng(4).choice(len(pos[0]), B, replace=False))
    u, v = pos[0][sel].copy(), pos[1][sel].copy()
    ctx = pkg.Context(0)
    ctx.load_graph(g.n, g.rowptr, g.col, None, X)
    ctx.set_model("sage", dims, prec="bf16", fanout=fanout, max_batch=B, max_k=1)
    du, dv = t32(u), t32(v)
    seed, step = 99, 5
    _, nd = ctx.sample_negatives(seed, step, 1, du)
    loss, grads = torch.zeros(1, device=DEV), torch.zeros(ctx.n_params, device=DEV)
    ctx.train_step(t32(params), du, dv, None, nd, 1, loss, grads, seed=seed, step=step)
    torch.cuda.synchronize()
    ons, ond, _ = oracle.sample_negatives(g.n, g.rowptr, g.col, u, seed, step, 1)
    assert np.array_equal(nd.cpu().numpy(), ond)
    fr, blks = oracle.build_blocks(g.n, g.rowptr, g.col, np.concatenate([u, v, ond]), fanout, seed, step)
    st = ctx.stats()
    assert [int(st.block_nodes[h]) for h in range(3)] == [len(f) for f in fr[:3]]
    assert [int(st.block_edges[h]) for h in range(3)] == [len(b[1]) for b in blks]
    assert len(fr[2]) > 2_000_000  # the 3-hop neighbourhood of a batch covers most of the graph
    for h in range(0, 4):
        f_, ptr_, col_ = ctx.block(h)
        if h < 3:
            assert np.array_equal(f_.cpu().numpy(), fr[h])
        if h >= 1:
            assert np.array_equal(ptr_.cpu().numpy(), blks[h - 1][0]) and np.array_equal(col_.cpu().numpy(), blks[h - 1][1])
    # what holds at any size: a finite positive loss (untrained embeddings are not normalised, so it can be far above
    # ln 2), finite gradients, and a second run that repeats the first bit for bit
    assert np.isfinite(loss.item()) and 0.1 < loss.item() < 1e4
    g1 = grads.clone()
    assert torch.isfinite(g1).all() and float(g1.abs().max()) > 0
    l2 = torch.zeros(1, device=DEV)
    ctx.train_step(t32(params), du, dv, None, nd, 1, l2, grads, seed=seed, step=step)
    torch.cuda.synchronize()
    assert torch.equal(grads, g1) and torch.equal(l2, loss)
    ctx.close()


# ------------------------------------------------------------------------------------------ config 5
def _views(g, part, i, sp, negatives):
    """Oracle-side graph, candidate set and positives of worker i (config 5: own rows node-induced; foreign rows empty
    for local negatives, taken from the sparsified global graph for global negatives)."""
    mode = 0 if negatives == "local" else 1
    rp, col, stats = oracle.worker_view(g.n, g.rowptr, g.col, part, i, keep_cross_edges=False, foreign_mode=mode, sparsified=sp)
    view = wl.Graph(n=g.n, rowptr=rp, col=col)
    own = np.nonzero(part == i)[0].astype(np.int32)
    cand = own if negatives == "local" else None
    # positives: the partition's own undirected edges, each once (u < v), in row order
    rows = np.repeat(np.arange(g.n, dtype=np.int64), np.diff(g.rowptr))
    keep = (part[rows] == i) & (part[g.col] == i) & (g.col > rows)
    return view, cand, (rows[keep].astype(np.int32), g.col[keep].astype(np.int32)), stats


def _gpu_view_step(pkg, ctxG, dpart, X_dev, X, g, part, i, sp, negatives, params, dims, prec, B, acc=None, check_structure=False):
    """Worker i's step on the view that the GPU builds from the global context; returns (loss, grads, view inputs)."""
    view, cand, (pu, pv), ostats = _views(g, part, i, sp, negatives) if check_structure else (None, None, (None, None), None)
    rp, col, stats = ctxG.worker_view(dpart, i, keep_cross_edges=False, foreign_mode=0 if negatives == "local" else 1)
    if check_structure:
        assert np.array_equal(rp.cpu().numpy(), view.rowptr) and np.array_equal(col.cpu().numpy(), view.col) and stats == ostats
    else:  # positives without the oracle's view: the same rule on the host
        rows = np.repeat(np.arange(g.n, dtype=np.int64), np.diff(g.rowptr))
        keep = (part[rows] == i) & (part[g.col] == i) & (g.col > rows)
        pu, pv = rows[keep].astype(np.int32), g.col[keep].astype(np.int32)
        cand = np.nonzero(part == i)[0].astype(np.int32) if negatives == "local" else None
    pu, pv = pu[:B].copy(), pv[:B].copy()
    ctx = pkg.Context(0)
    ctx.load_graph(g.n, rp, col, None, X_dev, on_device=True)
    ctx.set_model("sage", dims, prec=prec, max_batch=len(pu), max_k=1)
    if cand is not None:
        ctx.set_candidates(t32(cand))
    du, dv = t32(pu), t32(pv)
    seed, step = 11, i
    _, nd = ctx.sample_negatives(seed, step, 1, du)
    loss = torch.zeros(1, device=DEV)
    grads = acc if acc is not None else torch.zeros(ctx.n_params, device=DEV)
    ctx.train_step(t32(params), du, dv, None, nd, 1, loss, grads, seed=seed, step=step, accumulate=acc is not None)
    torch.cuda.synchronize()
    return ctx, loss, grads, (view, cand, pu, pv, nd, seed, step)


@pytest.mark.parametrize("scale,p_check", [(1.0, {"local": [0], "global": [5]}), (0.1, {"local": list(range(8)), "global": list(range(8))})])
def test_config5_gpu_built_views(pkg, scale, p_check):
    g, X, params, pos, cfg = wl.make_config("c5_partitioned_sage2", scale=scale)
    dims, p, alpha, prec, B = cfg["dims"], cfg["partitions"], cfg["alpha"], "bf16", 65536
    assert p == 8 and (scale < 1.0 or g.n == 1_000_000)
    part = wl.random_partition(g.n, p, seed=5)
    ctxG = pkg.Context(0)
    ctxG.load_graph(g.n, g.rowptr, g.col, None, X)
    srp, scol, sw = ctxG.sparsify(alpha, 5)
    orp, ocol, ow = oracle.sparsified_graph(g.n, g.rowptr, g.col, alpha, 5)
    assert np.array_equal(srp.cpu().numpy(), orp) and np.array_equal(scol.cpu().numpy(), ocol)
    assert np.max(np.abs(sw.cpu().numpy() - ow) / ow) < 1e-6
    sp = (orp, ocol)
    dpart, X_dev = t32(part), t32(X)
    for negatives in ("local", "global"):
        ora = {}
        for i in p_check[negatives]:
            ctx, loss, grads, (view, cand, pu, pv, nd, seed, step) = _gpu_view_step(pkg, ctxG, dpart, X_dev, X, g, part, i, sp, negatives, params, dims,
                                                                                   prec, B, check_structure=True)
            ons, ond, _ = oracle.sample_negatives(view.n, view.rowptr, view.col, pu, seed, step, 1, cand=cand)
            assert np.array_equal(nd.cpu().numpy(), ond)
            H1 = ctx.embeddings(1).cpu().numpy() > 0
            ref = oracle.train_step(view, X, params, "sage", dims, pu, pv, ons, ond, relu_ties=[H1], rounding=prec)
            assert_relu_decisions_agree(ref["cache"], [H1], None, f"config 5 scale {scale} worker {i} {negatives}")
            check_step(ctx, ref, loss, grads, "sage", dims, TOL[prec], {"dHK": rel_l2(ctx.output_gradient().cpu().numpy(), ref["dHK"])})
            ora[i] = ref["grads"]
            ctx.close()
        # gradient synchronisation of Algorithm 1: the 8 workers' gradients accumulated on the device in partition order
        acc = torch.zeros(len(params), device=DEV)
        separate = np.zeros(len(params), dtype=np.float64)
        for i in range(p):
            ctx, _, _, _ = _gpu_view_step(pkg, ctxG, dpart, X_dev, X, g, part, i, sp, negatives, params, dims, prec, B, acc=acc)
            ctx.close()
            ctx, _, gi, _ = _gpu_view_step(pkg, ctxG, dpart, X_dev, X, g, part, i, sp, negatives, params, dims, prec, B)
            separate += gi.double().cpu().numpy()
            ctx.close()
        assert rel_l2(acc.cpu().numpy(), separate) < 1e-6  # the accumulate flag adds, in FP32, exactly what a separate step returns
        if len(ora) == p:
            avg = oracle.average_gradients([ora[i] for i in range(p)])
            assert rel_l2(acc.cpu().numpy() / p, avg) < TOL[prec]
    ctxG.close()


def test_config5_full_size_local_partitions_as_own_graphs(pkg):
    # Local negatives never leave the partition, so a worker can hold its induced subgraph as a graph of its own (about
    # 125,000 of the 1 M nodes, renumbered in ascending id order) -- the form the benchmark times.  Every partition's BF16 step
    # against the oracle on the same subgraph, and the 8-way accumulated gradient against the oracle's average (Algorithm 1).
    g, X, params, pos, cfg = wl.make_config("c5_partitioned_sage2")
    dims, p, prec, B = cfg["dims"], cfg["partitions"], "bf16", 65536
    part = wl.random_partition(g.n, p, seed=5)
    rows = np.repeat(np.arange(g.n, dtype=np.int64), np.diff(g.rowptr))
    prow, pcol, upper = part[rows], part[g.col], g.col > rows
    acc = torch.zeros(len(params), device=DEV)
    ora = []
    for i in range(p):
        own = np.nonzero(part == i)[0]
        new_id = np.full(g.n, -1, dtype=np.int64)
        new_id[own] = np.arange(own.shape[0])
        inside = (prow == i) & (pcol == i)
        sub = wl.csr_from_edges(own.shape[0], new_id[rows[inside]], new_id[g.col[inside]])
        Xs = np.ascontiguousarray(X[own])
        keep = inside & upper
        pu, pv = new_id[rows[keep]].astype(np.int32)[:B].copy(), new_id[g.col[keep]].astype(np.int32)[:B].copy()
        ctx = pkg.Context(0)
        ctx.load_graph(sub.n, sub.rowptr, sub.col, None, Xs)
        ctx.set_model("sage", dims, prec=prec, max_batch=len(pu), max_k=1)
        du, dv = t32(pu), t32(pv)
        seed, step = 11, i
        _, nd = ctx.sample_negatives(seed, step, 1, du)
        loss, grads = torch.zeros(1, device=DEV), torch.zeros(ctx.n_params, device=DEV)
        ctx.train_step(t32(params), du, dv, None, nd, 1, loss, grads, seed=seed, step=step)
        ctx.train_step(t32(params), du, dv, None, nd, 1, loss, acc, seed=seed, step=step, accumulate=True)
        torch.cuda.synchronize()
        ons, ond, _ = oracle.sample_negatives(sub.n, sub.rowptr, sub.col, pu, seed, step, 1)
        assert np.array_equal(nd.cpu().numpy(), ond)
        # the same negatives as a draw among the partition's nodes in the 1 M-node numbering (candidate set = own nodes)
        if i == 0:
            view = wl.induced_subgraph(g, part == i)
            _, gnd, _ = oracle.sample_negatives(g.n, view.rowptr, view.col, own[pu].astype(np.int32), seed, step, 1, cand=own.astype(np.int32))
            assert np.array_equal(own[ond], gnd)
        H1 = ctx.embeddings(1).cpu().numpy() > 0
        ref = oracle.train_step(sub, Xs, params, "sage", dims, pu, pv, ons, ond, relu_ties=[H1], rounding=prec)
        assert_relu_decisions_agree(ref["cache"], [H1], None, f"config 5 partition {i} as its own graph")
        check_step(ctx, ref, loss, grads, "sage", dims, TOL[prec], {"dHK": rel_l2(ctx.output_gradient().cpu().numpy(), ref["dHK"])})
        ora.append(ref["grads"])
        ctx.close()
    assert rel_l2(acc.cpu().numpy() / p, oracle.average_gradients(ora)) < TOL[prec]
