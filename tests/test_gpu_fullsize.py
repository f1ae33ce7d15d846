"""Parity at the benchmark's full size and launch configuration (config 2: 200,000 nodes, 3.93 M stored
entries, 2-layer SAGE-mean 128-256-256, one batch of 65,536 positives + 65,536 negatives), and a larger
sampled case of config 4.  The oracle computes the whole step (a few seconds on the host cores)."""
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
    g, X, params, pos, cfg = wl.make_config("c4_citation_sage3_sampled", scale=0.05)
    dims, fanout = cfg["dims"], cfg["fanout"]
    B = 3277
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
