"""GPU parity: the CUDA library (through the C ABI) against the CPU oracle on the same seeded inputs.

Tolerances (per tensor, relative L2): 1e-5 on the FP32 path, 2e-2 on the BF16 path; integer
results (negatives, transposed structure, sampled blocks) bit-exact.
"""
import numpy as np
import pytest

import oracle
import workloads as wl
from helpers import assert_relu_decisions_agree, rel_l2

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

TOL = {"fp32": 1e-5, "bf16": 2e-2}
DEV = "cuda:0"


@pytest.fixture(scope="module")
def pkg():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import __graft_entry__ as ge
    ge.build()
    import paper_2506_20818_b200 as p
    return p


def make_ctx(pkg, g, X):
    ctx = pkg.Context(0)
    ctx.load_graph(g.n, g.rowptr, g.col, g.w, X)
    return ctx


def t32(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


# ------------------------------------------------------------------------------------------ structure
@pytest.mark.parametrize("maker", [
    lambda: wl.citation_directed(5000, 60000, 2.2, seed=1),
    lambda: wl.chung_lu(30000, 12.0, 2.1, seed=2),
    lambda: wl.erdos_renyi(300, 299, seed=3),
    lambda: wl.Graph(n=7, rowptr=np.zeros(8, dtype=np.int64), col=np.zeros(0, dtype=np.int32)),
])
def test_transposed_structure_bit_exact(pkg, maker):
    g = maker()
    ctx = make_ctx(pkg, g, wl.node_features(g.n, 8, 0))
    colptr, rowidx, perm = ctx.get_structure()
    torch.cuda.synchronize()
    ocp, ori, ope = oracle.csc_transpose(g.n, g.rowptr, g.col)
    assert np.array_equal(colptr.cpu().numpy(), ocp)
    assert np.array_equal(rowidx.cpu().numpy(), ori)
    assert np.array_equal(perm.cpu().numpy(), ope)
    ctx.close()


def test_bad_graphs_are_rejected(pkg):
    ctx = pkg.Context(0)
    X = wl.node_features(4, 8, 0)
    bad = [
        (np.array([0, 1, 3, 3, 3]), np.array([1, 0, 9], dtype=np.int32)),       # column out of range
        (np.array([0, 2, 1, 3, 3]), np.array([1, 2, 0], dtype=np.int32)),       # rowptr decreasing
        (np.array([0, 2, 3, 3, 3]), np.array([2, 1, 0], dtype=np.int32)),       # columns not ascending
        (np.array([0, 2, 3, 3, 3]), np.array([1, 1, 0], dtype=np.int32)),       # duplicate column
        (np.array([1, 2, 3, 3, 3]), np.array([1, 2, 0], dtype=np.int32)),       # rowptr[0] != 0
        (np.array([0, 1, 2, 2, 2]), np.array([1, 2, 0], dtype=np.int32)),       # rowptr[n] != nnz
    ]
    for rp, col in bad:
        with pytest.raises(pkg.LpError) as ei:
            ctx.load_graph(4, rp.astype(np.int64), col, None, X)
        assert ei.value.status == -1
    with pytest.raises(pkg.LpError) as ei:  # wrong call order
        ctx.set_model("gcn", [8, 8], max_batch=4)
    assert ei.value.status == -2
    with pytest.raises(pkg.LpError):        # feature width not a multiple of 8
        ctx.load_graph(4, np.array([0, 0, 0, 0, 0], dtype=np.int64), np.zeros(0, dtype=np.int32), None, wl.node_features(4, 6, 0))
    # the context is still usable
    g = wl.erdos_renyi(50, 100, seed=0)
    ctx.load_graph(g.n, g.rowptr, g.col, None, wl.node_features(g.n, 8, 0))
    with pytest.raises(pkg.LpError):
        ctx.set_model("gcn", [16, 8], max_batch=4)  # dims[0] != f
    with pytest.raises(pkg.LpError):
        ctx.set_model("gcn", [8, 8, 8], fanout=[3, 0], max_batch=4)  # fanouts must be all zero or all positive
    with pytest.raises(pkg.LpError):
        ctx.set_model("sage", [8, 8], fanout=[33], max_batch=4)  # above the largest supported fan-out
    ctx.close()


# ------------------------------------------------------------------------------------------ aggregation
@pytest.mark.parametrize("F", [8, 64, 128, 256, 264, 512])
@pytest.mark.parametrize("arch", ["gcn", "sage"])
def test_aggregate_fp32(pkg, arch, F):
    g = wl.coauthor_weighted(3000, 12000, seed=1) if arch == "gcn" else wl.citation_directed(3000, 40000, 2.2, seed=1)
    ctx = make_ctx(pkg, g, wl.node_features(g.n, 8, 0))
    H = np.random.default_rng(F).standard_normal((g.n, F)).astype(np.float32)
    for transpose in (False, True):
        out = ctx.op_aggregate(arch, t32(H), transpose=transpose).cpu().numpy()
        mode = "gcn" if arch == "gcn" else "mean"
        ref = (oracle.aggregate_backward if transpose else oracle.aggregate)(mode, g.n, g.rowptr, g.col, g.w if arch == "gcn" else None, H)
        assert rel_l2(out, ref) < 1e-6
        assert np.max(np.abs(out - ref)) < 1e-5 * max(1.0, np.abs(ref).max())
    ctx.close()


@pytest.mark.parametrize("F", [64, 128, 256])
def test_aggregate_bf16(pkg, F):
    g = wl.chung_lu(20000, 20.0, 2.1, seed=4)
    ctx = make_ctx(pkg, g, wl.node_features(g.n, 8, 0))
    Hb = torch.from_numpy(np.random.default_rng(1).standard_normal((g.n, F)).astype(np.float32)).to(DEV).to(torch.bfloat16)
    Hq = Hb.float().cpu().numpy()  # the oracle sees exactly the BF16-rounded inputs
    for arch in ("gcn", "sage"):
        for transpose in (False, True):
            out = ctx.op_aggregate(arch, Hb, transpose=transpose).float().cpu().numpy()
            mode = "gcn" if arch == "gcn" else "mean"
            ref = (oracle.aggregate_backward if transpose else oracle.aggregate)(mode, g.n, g.rowptr, g.col, None, Hq)
            assert rel_l2(out, ref) < 4e-3  # output rounding to BF16: 2^-9 relative per element
    ctx.close()


@pytest.mark.parametrize("F", [32, 128])
def test_aggregate_piece_and_group_boundaries(pkg, F):
    # the static structures are walked in padded form: rows cut into pieces of 128 entries and groups of four.  This
    # directed graph has a row of every length around those boundaries (0..9, 127..130, 255..258, 511..514, 1000), in
    # scattered positions with empty rows between them and at both ends; mean and its adjoint against the oracle, FP32
    # (one piece per row, pieces combined, pads in the last group, the all-pad group of an empty row)
    lengths = list(range(0, 10)) + [127, 128, 129, 130, 255, 256, 257, 258, 511, 512, 513, 514, 1000]
    n = 1200
    rng = np.random.default_rng(F)
    rows = rng.permutation(np.arange(3, n - 3))[: len(lengths)]
    dst, src = [], []
    for r, d in zip(rows, lengths):
        cand = np.delete(np.arange(n), r)
        dst.append(np.full(d, r))
        src.append(rng.choice(cand, size=d, replace=False))
    g = wl.csr_from_edges(n, np.concatenate(dst), np.concatenate(src))
    assert np.array_equal(np.sort(np.diff(g.rowptr)[rows]), np.sort(lengths)) and g.rowptr[3] == 0
    ctx = make_ctx(pkg, g, wl.node_features(n, 8, 0))
    H = rng.standard_normal((n, F)).astype(np.float32)
    for transpose in (False, True):
        out = ctx.op_aggregate("sage", t32(H), transpose=transpose).cpu().numpy()
        ref = (oracle.aggregate_backward if transpose else oracle.aggregate)("mean", n, g.rowptr, g.col, None, H)
        assert rel_l2(out, ref) < 1e-6
        assert np.max(np.abs(out - ref)) < 1e-5 * max(1.0, np.abs(ref).max())
        if not transpose:
            assert not out[np.diff(g.rowptr) == 0].any()  # empty rows are written, as zeros
    Hb = t32(H).to(torch.bfloat16)
    outb = ctx.op_aggregate("sage", Hb).float().cpu().numpy()
    refb = oracle.aggregate("mean", n, g.rowptr, g.col, None, Hb.float().cpu().numpy())
    assert rel_l2(outb, refb) < 4e-3
    ctx.close()
    # the same lengths as COLUMNS (the graph with every entry reversed), with per-entry coefficients: the GCN operator and
    # its adjoint, so that the padded transposed structure meets the boundaries too
    gt = wl.csr_from_edges(n, np.concatenate(src), np.concatenate(dst))
    ctx = make_ctx(pkg, gt, wl.node_features(n, 8, 0))
    for transpose in (False, True):
        out = ctx.op_aggregate("gcn", t32(H), transpose=transpose).cpu().numpy()
        ref = (oracle.aggregate_backward if transpose else oracle.aggregate)("gcn", n, gt.rowptr, gt.col, None, H)
        assert rel_l2(out, ref) < 1e-6
        assert np.max(np.abs(out - ref)) < 1e-5 * max(1.0, np.abs(ref).max())
    ctx.close()


@pytest.mark.parametrize("words", [32, 64, 128])
def test_gather_ceiling_folds_are_exact(pkg, words):
    # the measurement kernel behind the roofline figures does the gathers it claims: XOR folds of runs of 64 entries,
    # an integer result, checked against numpy on a graph whose entry count leaves a ragged last run
    g = wl.chung_lu(5000, 12.0, 2.1, seed=9)
    assert g.nnz % 64 != 0
    ctx = make_ctx(pkg, g, wl.node_features(g.n, 8, 0))
    H = np.random.default_rng(2).integers(-2**31, 2**31 - 1, size=(g.n, words), dtype=np.int64).astype(np.int32)
    _, rowidx, _ = ctx.get_structure()
    for transpose, idx in ((False, g.col), (True, rowidx.cpu().numpy())):
        folds = ctx.op_gather_ceiling(t32(H), transpose=transpose).cpu().numpy()
        ref = np.bitwise_xor.reduceat(H[idx], np.arange(0, g.nnz, 64), axis=0)
        assert folds.shape == ref.shape and np.array_equal(folds, ref)
    ctx.close()


# ------------------------------------------------------------------------------------------ dense transforms
@pytest.mark.parametrize("M,K,N", [(1000, 64, 64), (3333, 256, 256), (517, 512, 256), (129, 128, 264), (1, 8, 8)])
def test_linear_and_weight_grad_fp32(pkg, M, K, N):
    g = wl.erdos_renyi(50, 100, seed=0)
    ctx = make_ctx(pkg, g, wl.node_features(g.n, 8, 0))
    rng = np.random.default_rng(M)
    A = rng.standard_normal((M, K)).astype(np.float32)
    W = (rng.standard_normal((K, N)) / np.sqrt(K)).astype(np.float32)
    b = rng.standard_normal(N).astype(np.float32)
    ref = A.astype(np.float64) @ W.astype(np.float64) + b
    out = ctx.op_linear(t32(A), t32(W), t32(b), relu=False).cpu().numpy()
    assert rel_l2(out, ref) < 1e-6
    out = ctx.op_linear(t32(A), t32(np.ascontiguousarray(W.T)), t32(b), relu=True, trans_b=True).cpu().numpy()
    assert rel_l2(out, np.maximum(ref, 0)) < 1e-6
    dZ = rng.standard_normal((M, N)).astype(np.float32)
    dW = ctx.op_weight_grad(t32(A), t32(dZ)).cpu().numpy()
    assert rel_l2(dW, A.astype(np.float64).T @ dZ.astype(np.float64)) < 1e-6
    ctx.close()


@pytest.mark.parametrize("M,K,N", [(1000, 64, 64), (4099, 256, 256), (70000, 512, 256), (300, 128, 256), (131, 256, 128), (5, 256, 512),
                                   (8192, 256, 256), (20001, 256, 512), (33000, 512, 512), (9000, 128, 128), (50000, 64, 256)])
def test_linear_and_weight_grad_bf16(pkg, M, K, N):
    g = wl.erdos_renyi(50, 100, seed=0)
    ctx = make_ctx(pkg, g, wl.node_features(g.n, 8, 0))
    rng = np.random.default_rng(M + K)
    A = torch.from_numpy(rng.standard_normal((M, K)).astype(np.float32)).to(DEV).to(torch.bfloat16)
    W = torch.from_numpy((rng.standard_normal((K, N)) / np.sqrt(K)).astype(np.float32)).to(DEV).to(torch.bfloat16)
    b = rng.standard_normal(N).astype(np.float32)
    Aq, Wq = A.float().cpu().numpy().astype(np.float64), W.float().cpu().numpy().astype(np.float64)
    ref = Aq @ Wq + b
    out = ctx.op_linear(A, W, t32(b), relu=False).float().cpu().numpy()
    assert rel_l2(out, ref) < 4e-3
    out = ctx.op_linear(A, W.t().contiguous(), t32(b), relu=True, trans_b=True).float().cpu().numpy()
    assert rel_l2(out, np.maximum(ref, 0)) < 4e-3
    dZ = torch.from_numpy(rng.standard_normal((M, N)).astype(np.float32)).to(DEV).to(torch.bfloat16)
    dW = ctx.op_weight_grad(A, dZ).cpu().numpy()
    assert rel_l2(dW, Aq.T @ dZ.float().cpu().numpy().astype(np.float64)) < 1e-4  # FP32 accumulation of exact products
    ctx.close()


# ------------------------------------------------------------------------------------------ negatives
def test_negatives_bit_exact(pkg):
    g = wl.chung_lu(20000, 16.0, 2.1, seed=7)
    ctx = make_ctx(pkg, g, wl.node_features(g.n, 8, 0))
    u, v = wl.undirected_edge_list(g)
    du = t32(u)
    seed, step = (0xABCD << 32) | 77, (1 << 33) + 5
    for k in (1, 3):
        _, nd = ctx.sample_negatives(seed, step, k, du)
        _, ond, oex = oracle.sample_negatives(g.n, g.rowptr, g.col, u, seed, step, k)
        assert np.array_equal(nd.cpu().numpy(), ond)
        assert ctx.stats().negatives_exhausted == oex
    # batch-split invariance through edge_index_base, ragged last batch
    _, full = ctx.sample_negatives(seed, step, 1, du)
    lo, hi = 65536, min(len(u), 65536 + 4097)
    _, part = ctx.sample_negatives(seed, step, 1, du[lo:hi].contiguous(), edge_index_base=lo)
    assert torch.equal(part, full[lo:hi])
    # partition-local candidates, global pairs
    cand = np.arange(3, g.n, 8, dtype=np.int32)
    ctx.set_candidates(t32(cand))
    ns, nd = ctx.sample_negatives(seed, step, 2, du, mode=pkg.LP_NEG_GLOBAL_PAIR)
    ons, ond, _ = oracle.sample_negatives(g.n, g.rowptr, g.col, u, seed, step, 2, mode="global_pair", cand=cand)
    assert np.array_equal(ns.cpu().numpy(), ons) and np.array_equal(nd.cpu().numpy(), ond)
    _, nd = ctx.sample_negatives(seed, step, 1, du)
    assert np.array_equal(nd.cpu().numpy(), oracle.sample_negatives(g.n, g.rowptr, g.col, u, seed, step, 1, cand=cand)[1])
    ctx.set_candidates(None)
    with pytest.raises(pkg.LpError):
        ctx.set_candidates(t32(np.array([1, g.n], dtype=np.int32)))
    # rejection switched off through the model description
    ctx.set_model("sage", [8, 8], reject_edges=False, max_batch=len(u), max_k=1)
    _, nd = ctx.sample_negatives(seed, step, 1, du)
    assert np.array_equal(nd.cpu().numpy(), oracle.sample_negatives(g.n, g.rowptr, g.col, u, seed, step, 1, reject_edges=False)[1])
    ctx.close()


def test_negatives_exhaustion_counter(pkg):
    n = 8
    full = wl.csr_from_edges(n, *np.array([(a, b) for a in range(n) for b in range(n) if a != b]).T)
    ctx = make_ctx(pkg, full, wl.node_features(n, 8, 0))
    src = np.arange(n, dtype=np.int32)
    _, nd = ctx.sample_negatives(1, 0, 2, t32(src))
    _, ond, oex = oracle.sample_negatives(n, full.rowptr, full.col, src, 1, 0, 2)
    assert oex == 2 * n and ctx.stats().negatives_exhausted == oex
    assert np.array_equal(nd.cpu().numpy(), ond)
    ctx.close()


# ------------------------------------------------------------------------------------------ full step
def run_step(pkg, g, X, params, arch, dims, prec, pos, k=1, seed=5, step=0, fanout=None, cand=None, check_layers=True, adopt=True):
    """One training step both ways; returns a dict of relative errors and the raw results.
    adopt = False: the oracle takes every ReLU decision by itself (the caller has made sure that no pre-activation
    lies inside a rounding window) and the implementation's decisions must equal them everywhere."""
    u, v = pos
    ctx = make_ctx(pkg, g, X)
    ctx.set_model(arch, dims, prec=prec, fanout=fanout, max_batch=len(u), max_k=max(k, 1))
    if cand is not None:
        ctx.set_candidates(t32(cand))
    du, dv = t32(u), t32(v)
    nd = None
    if k > 0:
        _, nd = ctx.sample_negatives(seed, step, k, du)
    p = t32(params)
    loss = torch.zeros(1, device=DEV)
    grads = torch.full((ctx.n_params,), 7.0, device=DEV)  # must be overwritten
    ctx.train_step(p, du, dv, None, nd, k, loss, grads, seed=seed, step=step)
    torch.cuda.synchronize()
    K = len(dims) - 1
    if k > 0:
        ons, ond, _ = oracle.sample_negatives(g.n, g.rowptr, g.col, u, seed, step, k, cand=cand)
        assert np.array_equal(nd.cpu().numpy(), ond)
    else:
        ons, ond = np.zeros(0, dtype=np.int32), np.zeros(0, dtype=np.int32)
    blocks = None
    if fanout:
        seeds = np.concatenate([u, v, ond])
        blocks = oracle.build_blocks(g.n, g.rowptr, g.col, seeds, fanout, seed, step)
    # ReLU decisions: where a pre-activation is zero up to the rounding of the path (the oracle's window, derived from
    # the unit roundoffs of the FP32 or BF16 arithmetic) the oracle adopts the GPU's decision; outside the window the GPU's
    # decisions must equal the oracle's own, bit for bit.
    ties, rows_per_layer = None, None
    if K > 1:
        ties = []
        if fanout:
            rows_per_layer = [blocks[0][K - layer] for layer in range(1, K)]
        for layer in range(1, K):
            if fanout:
                full = np.zeros((g.n, dims[layer]), dtype=bool)
                rows_l = rows_per_layer[layer - 1]
                full[rows_l] = ctx.embeddings(layer, rows=len(rows_l)).cpu().numpy() > 0
                ties.append(full)
            else:
                ties.append(ctx.embeddings(layer).cpu().numpy() > 0)
    ref = oracle.train_step(g, X, params, arch, dims, u, v, ons, ond, blocks=blocks, relu_ties=ties if adopt else None, rounding=prec)
    if K > 1:
        inside, _ = assert_relu_decisions_agree(ref["cache"], ties, rows_per_layer, f"{arch}/{prec}")
        if not adopt:
            assert inside == 0 and ref["cache"]["ties"] == 0
    err = {"loss": abs(loss.item() - ref["loss"]) / abs(ref["loss"]),
           "grads": rel_l2(grads.cpu().numpy(), ref["grads"])}
    if fanout:
        fr, blks = blocks
        st = ctx.stats()
        assert [int(st.block_nodes[h]) for h in range(K)] == [len(f) for f in fr[:K]]
        assert [int(st.block_edges[h]) for h in range(K)] == [len(b[1]) for b in blks]
        for h in range(0, K + 1):
            f_, ptr_, col_ = ctx.block(h)
            if h < K:
                assert np.array_equal(f_.cpu().numpy(), fr[h])
            if h >= 1:
                assert np.array_equal(ptr_.cpu().numpy(), blks[h - 1][0])
                assert np.array_equal(col_.cpu().numpy(), blks[h - 1][1])
        rows = fr[0]
        HK = ctx.embeddings(K, rows=len(rows)).cpu().numpy()
        err["HK"] = rel_l2(HK, ref["cache"]["H"][K][rows])
        err["dHK"] = rel_l2(ctx.output_gradient(rows=len(rows)).cpu().numpy(), ref["dHK"][rows])
        if check_layers:
            for layer in range(1, K):
                rows_l = fr[K - layer]
                Hl = ctx.embeddings(layer, rows=len(rows_l)).cpu().numpy()
                err[f"H{layer}"] = rel_l2(Hl, ref["cache"]["H"][layer][rows_l])
    else:
        for layer in range(1, K + 1):
            err[f"H{layer}"] = rel_l2(ctx.embeddings(layer).cpu().numpy(), ref["cache"]["H"][layer])
        err["dHK"] = rel_l2(ctx.output_gradient().cpu().numpy(), ref["dHK"])
    # per-layer gradient blocks (a small block must not hide behind a large one)
    off = 0
    for li in range(K):
        kin = dims[li] * (2 if arch == "sage" else 1)
        nw = kin * dims[li + 1]
        gg = grads.cpu().numpy()
        err[f"dW{li}"] = rel_l2(gg[off:off + nw], ref["grads"][off:off + nw])
        err[f"db{li}"] = rel_l2(gg[off + nw:off + nw + dims[li + 1]], ref["grads"][off + nw:off + nw + dims[li + 1]])
        off += nw + dims[li + 1]
    launches = ctx.stats().kernel_launches
    ctx.close()
    return err, ref, launches


def assert_within(err, tol):
    bad = {k: v for k, v in err.items() if not (v < tol)}
    assert not bad, f"outside tolerance {tol}: {bad} (all: {err})"


def test_config1_tiny_er_gcn_fp32(pkg):
    g, X, params, pos, cfg = wl.make_config("c1_tiny_er_gcn2")
    err, _, launches = run_step(pkg, g, X, params, "gcn", cfg["dims"], "fp32", pos)
    assert_within(err, TOL["fp32"])
    assert launches > 10


@pytest.mark.parametrize("prec", ["fp32", "bf16"])
def test_config2_chunglu_sage(pkg, prec):
    g, X, params, pos, cfg = wl.make_config("c2_chunglu_sage2", scale=0.05)
    B = 4099  # one ragged batch of positives, full-graph encoder
    sel = np.random.default_rng(0).choice(len(pos[0]), B, replace=False)
    err, _, _ = run_step(pkg, g, X, params, "sage", cfg["dims"], prec, (pos[0][sel], pos[1][sel]))
    assert_within(err, TOL[prec])


@pytest.mark.parametrize("dims", [[64, 128, 128, 64], [64, 64, 128, 128]])
def test_sage3_one_pass_on_the_pair_kernel(pkg, dims):
    # Three SAGE layers over 9,001 nodes (35 row tiles of 256 and a ragged one) in BF16: every transform runs on pairs of
    # SMs, and each layer whose output is not wider than its input takes its input gradient as aggregate-then-transform (the
    # adjoint aggregation of dZ beside dZ, one transform over both halves, the ReLU mask from the forward pass's sign
    # bits).  First shape: both upper layers, chained through the two operand buffers; second shape: the top layer only (the
    # middle layer widens 64 -> 128 and keeps transform-then-aggregate), so the two forms of the input gradient follow one another.
    g = wl.chung_lu(9001, 14.0, 2.1, seed=21)
    X = wl.node_features(g.n, dims[0], 3)
    params = wl.glorot_params("sage", dims, 5, 0.05)
    u, v = wl.undirected_edge_list(g)
    sel = np.random.default_rng(1).choice(len(u), 5000, replace=False)
    err, _, _ = run_step(pkg, g, X, params, "sage", dims, "bf16", (u[sel], v[sel]))
    assert_within(err, TOL["bf16"])


@pytest.mark.parametrize("prec", ["fp32", "bf16"])
def test_config3_coauthor_gcn3_weighted(pkg, prec):
    g, X, params, pos, cfg = wl.make_config("c3_coauthor_gcn3", scale=0.04)
    assert g.w is not None and g.w.max() > 1
    err, _, _ = run_step(pkg, g, X, params, "gcn", cfg["dims"], prec, pos)
    assert_within(err, TOL[prec])


@pytest.mark.parametrize("arch,prec", [("gcn", "fp32"), ("gcn", "bf16"), ("sage", "fp32"), ("sage", "bf16")])
def test_step_parity_without_adopted_relu_decisions(pkg, arch, prec):
    # A 3-layer step in which the oracle takes EVERY ReLU decision itself.  The biases of the two hidden layers are set to
    # +-6 standard deviations of the layer's pre-activations (alternating by unit), so that -- as the oracle alone
    # establishes -- no pre-activation lies inside a rounding window; the GPU's decisions must then equal the oracle's on
    # every unit, and the gradients are compared without anything taken from the code under test.
    g = wl.erdos_renyi(3000, 24000, seed=12)
    dims = [64, 128, 128, 64]
    X = wl.node_features(g.n, 64, 2)
    params = wl.glorot_params(arch, dims, 3, 0.0)
    P = oracle.split_params(arch, dims, params)  # views into params
    for k in (0, 1):
        Z = oracle.forward(g, X, params, arch, dims)["Z"][k]
        P[k]["b"][:] = 6.0 * np.sqrt(np.mean(Z * Z)) * np.where(np.arange(dims[k + 1]) % 2 == 0, 1.0, -1.0)
    own = oracle.forward(g, X, params, arch, dims, rounding=prec)
    assert own["n_near"] == 0 and all(0.3 < a.mean() < 0.7 for a in own["own_active"])
    u, v = wl.undirected_edge_list(g)
    err, _, _ = run_step(pkg, g, X, params, arch, dims, prec, (u[:6000].copy(), v[:6000].copy()), adopt=False)
    assert_within(err, TOL[prec])


@pytest.mark.parametrize("prec", ["fp32", "bf16"])
def test_config4_citation_sage3_sampled(pkg, prec):
    g, X, params, pos, cfg = wl.make_config("c4_citation_sage3_sampled", scale=0.004)
    sel = np.random.default_rng(1).choice(len(pos[0]), 700, replace=False)
    err, _, _ = run_step(pkg, g, X, params, "sage", cfg["dims"], prec, (pos[0][sel], pos[1][sel]), fanout=cfg["fanout"], step=3)
    assert_within(err, TOL[prec])


def test_sampled_two_layer_and_one_layer(pkg):
    g = wl.citation_directed(4000, 60000, 2.2, seed=9)
    X = wl.node_features(g.n, 64, 1)
    rows = np.repeat(np.arange(g.n, dtype=np.int32), np.diff(g.rowptr))
    sel = np.random.default_rng(2).choice(g.nnz, 300, replace=False)
    pos = (g.col[sel].copy(), rows[sel].copy())
    for dims, fan in (([64, 64, 64], [4, 3]), ([64, 128], [6])):
        params = wl.glorot_params("sage", dims, 2, 0.05)
        err, _, _ = run_step(pkg, g, X, params, "sage", dims, "fp32", pos, fanout=fan, k=2)
        assert_within(err, TOL["fp32"])


@pytest.mark.parametrize("prec", ["fp32", "bf16"])
def test_sampled_gcn_minibatch(pkg, prec):
    # mini-batch training of the weighted 3-layer GCN configuration with the fan-outs 25 / 10 / 5 of Section IV
    g, X, params, pos, cfg = wl.make_config("c3_coauthor_gcn3", scale=0.04)
    sel = np.random.default_rng(3).choice(len(pos[0]), 256, replace=False)
    err, _, _ = run_step(pkg, g, X, params, "gcn", cfg["dims"], prec, (pos[0][sel], pos[1][sel]), fanout=[25, 10, 5], step=2)
    assert_within(err, TOL[prec])


@pytest.mark.parametrize("prec", ["fp32", "bf16"])
def test_sampled_sage_minibatch_fanout_25_10(pkg, prec):
    g, X, params, pos, cfg = wl.make_config("c2_chunglu_sage2", scale=0.05)
    sel = np.random.default_rng(4).choice(len(pos[0]), 1024, replace=False)
    err, _, _ = run_step(pkg, g, X, params, "sage", cfg["dims"], prec, (pos[0][sel], pos[1][sel]), fanout=[25, 10], step=1)
    assert_within(err, TOL[prec])


def test_sampled_gcn_full_fanout_matches_full_graph_step(pkg):
    # every degree below the fan-out: the sampled GCN step is the full-graph step on the seeds' neighbourhood
    g = wl.erdos_renyi(400, 1200, seed=5)
    assert np.diff(g.rowptr).max() <= 32
    dims = [16, 24, 8]
    X = wl.node_features(g.n, 16, 1)
    params = wl.glorot_params("gcn", dims, 2, 0.05)
    u, v = wl.undirected_edge_list(g)
    pos = (u[:64].astype(np.int32), v[:64].astype(np.int32))
    ctx = pkg.Context(0)
    ctx.load_graph(g.n, g.rowptr, g.col, g.w, X)
    out = {}
    for name, fan in (("full", None), ("sampled", [32, 32])):
        ctx.set_model("gcn", dims, prec="fp32", fanout=fan, max_batch=64, max_k=1)
        du, dv = t32(pos[0]), t32(pos[1])
        _, nd = ctx.sample_negatives(3, 0, 1, du)
        p = t32(params)
        grads = torch.zeros_like(p)
        loss = torch.zeros(1, device="cuda:0")
        ctx.train_step(p, du, dv, None, nd, 1, loss, grads, seed=3, step=0)
        out[name] = (loss.item(), grads.cpu().numpy())
    ctx.close()
    assert abs(out["full"][0] - out["sampled"][0]) <= 1e-6 * abs(out["full"][0])
    assert rel_l2(out["sampled"][1], out["full"][1]) < 1e-5


def test_step_edge_cases(pkg):
    # graph without edges, k = 0, a single positive, self pair as a positive
    n = 40
    g = wl.Graph(n=n, rowptr=np.zeros(n + 1, dtype=np.int64), col=np.zeros(0, dtype=np.int32))
    X = wl.node_features(n, 16, 0)
    for arch in ("gcn", "sage"):
        dims = [16, 24, 8]
        params = wl.glorot_params(arch, dims, 1, 0.1)
        err, _, _ = run_step(pkg, g, X, params, arch, dims, "fp32", (np.array([3], dtype=np.int32), np.array([3], dtype=np.int32)), k=0)
        assert_within(err, TOL["fp32"])
    g = wl.erdos_renyi(64, 200, seed=1)
    X = wl.node_features(g.n, 16, 0)
    u, v = wl.undirected_edge_list(g)
    u = np.concatenate([u, [5, 5]]).astype(np.int32)  # duplicates and a self pair
    v = np.concatenate([v, [5, 9]]).astype(np.int32)
    params = wl.glorot_params("sage", [16, 8], 1, 0.1)
    err, _, _ = run_step(pkg, g, X, params, "sage", [16, 8], "fp32", (u, v), k=4)
    assert_within(err, TOL["fp32"])


def test_closed_form_ln2_and_determinism(pkg):
    g, X, params, pos, cfg = wl.make_config("c1_tiny_er_gcn2")
    ctx = make_ctx(pkg, g, X)
    ctx.set_model("gcn", cfg["dims"], max_batch=len(pos[0]), max_k=1)
    du, dv = t32(pos[0]), t32(pos[1])
    _, nd = ctx.sample_negatives(1, 0, 1, du)
    loss = torch.zeros(1, device=DEV)
    grads = torch.zeros(ctx.n_params, device=DEV)
    ctx.train_step(torch.zeros(ctx.n_params, device=DEV), du, dv, None, nd, 1, loss, grads)
    assert abs(loss.item() - np.log(2.0)) < 1e-6  # zero weights: every score is 0
    # no float atomics anywhere: two runs are identical bit for bit; accumulate doubles the gradient
    p = t32(params)
    g1 = torch.zeros(ctx.n_params, device=DEV)
    g2 = torch.zeros(ctx.n_params, device=DEV)
    l1, l2 = torch.zeros(1, device=DEV), torch.zeros(1, device=DEV)
    ctx.train_step(p, du, dv, None, nd, 1, l1, g1)
    ctx.train_step(p, du, dv, None, nd, 1, l2, g2)
    assert torch.equal(g1, g2) and torch.equal(l1, l2)
    ctx.train_step(p, du, dv, None, nd, 1, l2, g2, accumulate=True)
    assert torch.allclose(g2, 2 * g1, rtol=1e-6, atol=0)
    ctx.close()


def test_bad_ids_are_reported_not_faulted(pkg):
    g = wl.erdos_renyi(100, 300, seed=0)
    ctx = make_ctx(pkg, g, wl.node_features(g.n, 8, 0))
    ctx.set_model("sage", [8, 8], max_batch=16, max_k=1)
    u = t32(np.array([1, 2, 100000], dtype=np.int32))
    v = t32(np.array([3, -4, 5], dtype=np.int32))
    loss = torch.zeros(1, device=DEV)
    grads = torch.zeros(ctx.n_params, device=DEV)
    ctx.train_step(torch.zeros(ctx.n_params, device=DEV), u, v, None, v, 1, loss, grads)
    with pytest.raises(pkg.LpError) as ei:
        ctx.stats()
    assert ei.value.status == -1
    ctx.stats()  # reported once; the context keeps working
    ctx.close()


# ------------------------------------------------------------------------------------------ optimiser, scoring
def test_adam_and_sgd(pkg):
    g = wl.erdos_renyi(50, 100, seed=0)
    ctx = make_ctx(pkg, g, wl.node_features(g.n, 64, 0))
    npar = ctx.set_model("sage", [64, 64, 64], max_batch=8)
    rng = np.random.default_rng(0)
    p0 = rng.standard_normal(npar).astype(np.float32)
    p, m, v = t32(p0), torch.zeros(npar, device=DEV), torch.zeros(npar, device=DEV)
    op, om, ov = p0.astype(np.float64), np.zeros(npar), np.zeros(npar)
    for t in range(1, 6):
        gr = (rng.standard_normal(npar) * 10.0 ** rng.integers(-4, 2, npar)).astype(np.float32)
        ctx.adam_step(p, m, v, t32(gr), t, grad_scale=0.125)
        op, om, ov = oracle.adam_step(op, om, ov, 0.125 * gr.astype(np.float64), t)
    assert rel_l2(p.cpu().numpy(), op) < 1e-6
    assert rel_l2((p.cpu().numpy() - p0), (op - p0)) < 1e-4  # the update itself, not just the weights
    assert rel_l2(m.cpu().numpy(), om) < 1e-6 and rel_l2(v.cpu().numpy(), ov) < 1e-6
    q = t32(p0)
    ctx.adam_step(q, None, None, t32(gr), 1, grad_scale=0.5, lr=0.1)
    assert rel_l2(q.cpu().numpy(), p0 - 0.1 * 0.5 * gr.astype(np.float64)) < 1e-6
    ctx.close()


@pytest.mark.parametrize("arch,prec", [("gcn", "fp32"), ("sage", "bf16")])
def test_score(pkg, arch, prec):
    g = wl.chung_lu(5000, 10.0, 2.1, seed=3)
    dims = [64, 128, 64]
    X = wl.node_features(g.n, 64, 3)
    params = wl.glorot_params(arch, dims, 3, 0.05)
    ctx = make_ctx(pkg, g, X)
    ctx.set_model(arch, dims, prec=prec, max_batch=1024)
    u, v = wl.undirected_edge_list(g)
    s1 = ctx.score(t32(params), t32(u), t32(v)).cpu().numpy()
    s2 = ctx.score(t32(params), t32(v), t32(u)).cpu().numpy()
    ref = oracle.score(g, X, params, arch, dims, u, v)
    assert rel_l2(s1, ref) < TOL[prec]
    assert np.array_equal(s1, s2) or rel_l2(s1, s2) < 1e-6  # undirected scores are symmetric
    ctx.close()


def test_score_keeps_embeddings_between_calls(pkg):
    # an evaluation pass scores positives and negatives in batches (Section IV): the encoder runs once, later calls
    # with the same weights only score; an update of the weights (or an explicit invalidation) runs it again
    g = wl.chung_lu(5000, 10.0, 2.1, seed=3)
    dims = [64, 128, 64]
    X = wl.node_features(g.n, 64, 3)
    params = wl.glorot_params("sage", dims, 3, 0.05)
    ctx = make_ctx(pkg, g, X)
    ctx.set_model("sage", dims, prec="fp32", max_batch=1024)
    u, v = wl.undirected_edge_list(g)
    du, dv, p = t32(u), t32(v), t32(params)
    half = len(u) // 2
    n0 = ctx.stats().kernel_launches
    s_a = ctx.score(p, du[:half].contiguous(), dv[:half].contiguous())
    n1 = ctx.stats().kernel_launches
    s_b = ctx.score(p, du[half:].contiguous(), dv[half:].contiguous())
    n2 = ctx.stats().kernel_launches
    assert n1 - n0 > 3 and n2 - n1 == 1  # encoder + scoring, then scoring alone
    ref = oracle.score(g, X, params, "sage", dims, u, v)
    assert rel_l2(torch.cat([s_a, s_b]).cpu().numpy(), ref) < TOL["fp32"]
    # another parameter vector, an optimiser step, an explicit invalidation: each runs the encoder again
    p2 = p.clone()
    ctx.score(p2, du, dv)
    n3 = ctx.stats().kernel_launches
    assert n3 - n2 == n1 - n0
    m, vv, grads = torch.zeros_like(p2), torch.zeros_like(p2), torch.ones_like(p2)
    ctx.adam_step(p2, m, vv, grads, 1)
    n4 = ctx.stats().kernel_launches
    s_new = ctx.score(p2, du, dv)
    n5 = ctx.stats().kernel_launches
    assert n5 - n4 == n1 - n0
    assert rel_l2(s_new.cpu().numpy(), oracle.score(g, X, p2.cpu().numpy(), "sage", dims, u, v)) < TOL["fp32"]
    p2.mul_(0.5)  # weights changed behind the library's back: the caller says so
    ctx.invalidate_embeddings()
    s_half = ctx.score(p2, du, dv)
    assert ctx.stats().kernel_launches - n5 == n1 - n0
    assert rel_l2(s_half.cpu().numpy(), oracle.score(g, X, p2.cpu().numpy(), "sage", dims, u, v)) < TOL["fp32"]
    # a training step leaves the embeddings of its weights behind as well
    ctx.set_model("sage", dims, prec="fp32", max_batch=len(u), max_k=1)
    _, nd = ctx.sample_negatives(1, 0, 1, du)
    loss, grads = torch.zeros(1, device=DEV), torch.zeros(ctx.n_params, device=DEV)
    ctx.train_step(p, du, dv, None, nd, 1, loss, grads)
    n6 = ctx.stats().kernel_launches
    s_c = ctx.score(p, du, dv)
    assert ctx.stats().kernel_launches - n6 == 1
    assert rel_l2(s_c.cpu().numpy(), ref) < TOL["fp32"]
    ctx.close()


@pytest.mark.parametrize("M", [100, 4096])
def test_bounded_wait_expires_cleanly(pkg, M):
    # failure detection of the tensor-core kernels, exercised without any fault: the next launch is told to expect 16
    # bytes more than its copies deliver, so every copy lands but the barrier never completes; with the limit at 2 ms
    # every wait gives up, the kernel frees its tensor memory and returns, the call reports LP_ETIMEOUT once, and the
    # context (tensor memory included) works as before.  M = 100 takes the one-tile kernel, M = 4096 the persistent one.
    g = wl.erdos_renyi(50, 100, seed=0)
    ctx = make_ctx(pkg, g, wl.node_features(g.n, 8, 0))
    rng = np.random.default_rng(M)
    A = torch.from_numpy(rng.standard_normal((M, 256)).astype(np.float32)).to(DEV).to(torch.bfloat16)
    W = torch.from_numpy((rng.standard_normal((256, 128)) / 16).astype(np.float32)).to(DEV).to(torch.bfloat16)
    ref = A.float().cpu().numpy().astype(np.float64) @ W.float().cpu().numpy().astype(np.float64)
    assert rel_l2(ctx.op_linear(A, W).float().cpu().numpy(), ref) < 4e-3
    ctx.set_wait_limit(2_000_000, overdeclare_bytes=16)
    with pytest.raises(pkg.LpError) as ei:
        ctx.op_linear(A, W)
    assert ei.value.status == -6 and "wait" in str(ei.value)
    ctx.stats()  # reported once
    for _ in range(3):  # the self-test was consumed by that launch; tensor memory was released (these launches need all of it again)
        assert rel_l2(ctx.op_linear(A, W).float().cpu().numpy(), ref) < 4e-3
    ctx.set_wait_limit(2_000_000_000)
    with pytest.raises(pkg.LpError):
        ctx.set_wait_limit(10)
    ctx.close()


# ------------------------------------------------------------------------------------------ emulated workers (config 5)
def test_config5_partitions_local_vs_global(pkg):
    g, X, params, pos, cfg = wl.make_config("c5_partitioned_sage2", scale=0.01)
    dims, p = cfg["dims"], 4
    part = wl.random_partition(g.n, p, seed=5)
    srp, scol, sw = oracle.sparsified_graph(g.n, g.rowptr, g.col, cfg["alpha"], seed=5)
    sparse = wl.Graph(n=g.n, rowptr=srp, col=scol, w=sw)
    for negatives in ("local", "global"):
        gpu_acc = None
        ora = []
        for i in range(p):
            mask = part == i
            own = wl.induced_subgraph(g, mask)
            if negatives == "local":
                view, cand = own, np.nonzero(mask)[0].astype(np.int32)
            else:  # own rows from the partition, foreign rows from the sparsified global graph
                rows = np.repeat(np.arange(g.n), np.diff(sparse.rowptr))
                keep = ~mask[rows]
                o_rows = np.repeat(np.arange(g.n), np.diff(own.rowptr))
                view = wl.csr_from_edges(g.n, np.concatenate([o_rows, rows[keep]]), np.concatenate([own.col, sparse.col[keep]]).astype(np.int64))
                cand = None
            pu, pv = wl.undirected_edge_list(own)
            err, ref, _ = run_step(pkg, view, X, params, "sage", dims, "fp32", (pu, pv), seed=11, step=i, cand=cand)
            assert_within(err, TOL["fp32"])
            ora.append(ref["grads"])
        avg = oracle.average_gradients(ora)
        # accumulate on the device in partition order, then one Adam step with grad_scale = 1/p
        ctx = None
        acc = torch.zeros(len(params), device=DEV)
        for i in range(p):
            mask = part == i
            own = wl.induced_subgraph(g, mask)
            if negatives == "local":
                view, cand = own, np.nonzero(mask)[0].astype(np.int32)
            else:
                rows = np.repeat(np.arange(g.n), np.diff(sparse.rowptr))
                keep = ~mask[rows]
                o_rows = np.repeat(np.arange(g.n), np.diff(own.rowptr))
                view = wl.csr_from_edges(g.n, np.concatenate([o_rows, rows[keep]]), np.concatenate([own.col, sparse.col[keep]]).astype(np.int64))
                cand = None
            pu, pv = wl.undirected_edge_list(own)
            ctx = make_ctx(pkg, view, X)
            ctx.set_model("sage", dims, prec="fp32", max_batch=len(pu), max_k=1)
            if cand is not None:
                ctx.set_candidates(t32(cand))
            du, dv = t32(pu), t32(pv)
            _, nd = ctx.sample_negatives(11, i, 1, du)
            loss = torch.zeros(1, device=DEV)
            ctx.train_step(t32(params), du, dv, None, nd, 1, loss, acc, accumulate=True)
            torch.cuda.synchronize()
            if i < p - 1:
                ctx.close()
        assert rel_l2(acc.cpu().numpy() / p, avg) < TOL["fp32"]
        pt, m, v = t32(params), torch.zeros(len(params), device=DEV), torch.zeros(len(params), device=DEV)
        ctx.adam_step(pt, m, v, acc, 1, grad_scale=1.0 / p)
        op, _, _ = oracle.adam_step(params, np.zeros(len(params)), np.zeros(len(params)), avg, 1)
        assert rel_l2(pt.cpu().numpy() - params, op - params) < 1e-3
        ctx.close()


def test_host_buffer_step_matches_device_step(pkg):
    g, X, params, pos, cfg = wl.make_config("c2_chunglu_sage2", scale=0.02)
    dims = cfg["dims"]
    B = 2000
    u, v = pos[0][:B].copy(), pos[1][:B].copy()
    ctx = make_ctx(pkg, g, X)
    ctx.set_model("sage", dims, prec="bf16", max_batch=B, max_k=1)
    p = t32(params)
    loss_h = np.zeros(1, dtype=np.float32)
    grads_h = np.zeros(ctx.n_params, dtype=np.float32)
    ctx.train_step_host(p, u, v, 1, seed=3, step=2, edge_index_base=10, loss_host=loss_h, grads_host=grads_h)
    du, dv = t32(u), t32(v)
    _, nd = ctx.sample_negatives(3, 2, 1, du, edge_index_base=10)
    loss = torch.zeros(1, device=DEV)
    grads = torch.zeros(ctx.n_params, device=DEV)
    ctx.train_step(p, du, dv, None, nd, 1, loss, grads, seed=3, step=2)
    assert loss.item() == loss_h[0] and np.array_equal(grads.cpu().numpy(), grads_h)
    # with the optimiser folded in: parameters move exactly as a separate lp_adam_step would move them
    m, vv = torch.zeros_like(p), torch.zeros_like(p)
    p2, m2, v2 = p.clone(), torch.zeros_like(p), torch.zeros_like(p)
    ctx.train_step_host(p, u, v, 1, seed=3, step=2, edge_index_base=10, adam_m=m, adam_v=vv, adam_t=1, loss_host=loss_h)
    ctx.adam_step(p2, m2, v2, grads, 1)
    assert torch.equal(p, p2)
    ctx.close()


# ------------------------------------------------------------------------------------------ sparsifier (Algorithm 1)
@pytest.mark.parametrize("alpha", [0.05, 0.2, 1.5])
def test_sparsifier_matches_oracle(pkg, alpha):
    g = wl.chung_lu(30000, 16.0, 2.1, seed=8)
    assert (np.diff(g.rowptr) == 0).any()  # isolated nodes are skipped by the node draw
    ctx = make_ctx(pkg, g, wl.node_features(g.n, 8, 0))
    seed = (3 << 40) + 17
    rp, col, w = ctx.sparsify(alpha, seed)
    torch.cuda.synchronize()
    orp, ocol, ow = oracle.sparsified_graph(g.n, g.rowptr, g.col, alpha, seed)
    assert np.array_equal(rp.cpu().numpy(), orp) and np.array_equal(col.cpu().numpy(), ocol)  # structure bit-exact
    assert np.max(np.abs(w.cpu().numpy() - ow) / ow) < 1e-6
    # the sparsified graph can be loaded and trained on (it is symmetric with ascending columns)
    ctx2 = pkg.Context(0)
    ctx2.load_graph(g.n, rp.cpu().numpy(), col.cpu().numpy(), w.cpu().numpy(), wl.node_features(g.n, 8, 0))
    ctx2.close()
    ctx.close()


def test_sparsifier_rejects_directed_graph(pkg):
    g = wl.citation_directed(2000, 20000, 2.2, seed=1)
    ctx = make_ctx(pkg, g, wl.node_features(g.n, 8, 0))
    with pytest.raises(pkg.LpError) as ei:
        ctx.sparsify(0.5, 1)
    assert ei.value.status == -1
    with pytest.raises(pkg.LpError):
        ctx.sparsify(0.0, 1)
    ctx.close()


def test_step_on_a_caller_stream_matches_default_stream(pkg):
    g, X, params, pos, cfg = wl.make_config("c2_chunglu_sage2", scale=0.02)
    dims = cfg["dims"]
    u, v = pos[0][:3000].copy(), pos[1][:3000].copy()
    results = []
    for stream in (None, torch.cuda.Stream(device=DEV)):
        ctx = pkg.Context(0, stream=stream)
        cm = torch.cuda.stream(stream) if stream is not None else torch.cuda.stream(torch.cuda.current_stream())
        with cm:
            ctx.load_graph(g.n, g.rowptr, g.col, g.w, X)
            ctx.set_model("sage", dims, prec="bf16", max_batch=len(u), max_k=1)
            du, dv, p = t32(u), t32(v), t32(params)
            _, nd = ctx.sample_negatives(3, 1, 1, du)
            loss = torch.zeros(1, device=DEV)
            grads = torch.zeros(ctx.n_params, device=DEV)
            if stream is not None:
                stream.wait_stream(torch.cuda.default_stream())
            ctx.train_step(p, du, dv, None, nd, 1, loss, grads)
            (stream or torch.cuda.current_stream()).synchronize()
        results.append((loss.clone(), grads.clone(), nd.clone()))
        ctx.close()
    assert torch.equal(results[0][2], results[1][2])
    assert torch.equal(results[0][0], results[1][0]) and torch.equal(results[0][1], results[1][1])


def test_profiler_times_every_nth_step_and_leaves_results_alone(pkg):
    # per-category event timing: every step, then every 4th step of 8 (2 steps x 3 aggregation launches of a 2-layer SAGE
    # model: two forward, one adjoint), and the timed steps give the same bits as untimed ones
    g, X, params, pos, cfg = wl.make_config("c2_chunglu_sage2", scale=0.02)
    u, v = pos[0][:2000].copy(), pos[1][:2000].copy()
    ctx = make_ctx(pkg, g, X)
    ctx.set_model("sage", cfg["dims"], prec="bf16", max_batch=len(u), max_k=1)
    du, dv, p = t32(u), t32(v), t32(params)
    _, nd = ctx.sample_negatives(3, 1, 1, du)
    loss, grads = torch.zeros(1, device=DEV), torch.zeros(ctx.n_params, device=DEV)

    def steps(n):
        out = []
        for _ in range(n):
            ctx.train_step(p, du, dv, None, nd, 1, loss, grads)
            out.append((loss.clone(), grads.clone()))
        return out

    plain = steps(1)[0]
    ctx.profile_begin(["agg_fwd", "agg_bwd", "score"])
    timed = steps(8)
    prof = ctx.profile_end()
    assert prof["agg_fwd"]["spans"] == 16 and prof["agg_bwd"]["spans"] == 8 and prof["score"]["spans"] == 8
    assert prof["agg_fwd"]["ms"] > 0 and prof["agg_fwd"]["bytes"] > 0 and prof["gemm_fwd"]["spans"] == 0
    ctx.profile_sample_every(4)
    ctx.profile_begin(["agg_fwd", "agg_bwd"])
    timed += steps(8)
    prof = ctx.profile_end()
    assert prof["agg_fwd"]["spans"] == 4 and prof["agg_bwd"]["spans"] == 2
    ctx.profile_sample_every(1)
    with pytest.raises(pkg.LpError):
        ctx.profile_sample_every(0)
    for l, gr in timed:
        assert torch.equal(l, plain[0]) and torch.equal(gr, plain[1])
    ctx.close()


@pytest.mark.parametrize("arch", ["gcn", "sage"])
def test_cached_input_aggregation_gives_identical_steps(pkg, arch):
    g, X, params, pos, cfg = wl.make_config("c3_coauthor_gcn3", scale=0.02)
    dims = [128, 64, 64]
    params = wl.glorot_params(arch, dims, 1, 0.05)
    u, v = pos[0][:2000].copy(), pos[1][:2000].copy()
    out = []
    for cache in (False, True):
        ctx = make_ctx(pkg, g, X)
        ctx.set_model(arch, dims, prec="bf16", max_batch=len(u), max_k=1, cache_input_aggregation=cache)
        du, dv, p = t32(u), t32(v), t32(params)
        m, vv = torch.zeros_like(p), torch.zeros_like(p)
        loss, grads = torch.zeros(1, device=DEV), torch.zeros(ctx.n_params, device=DEV)
        for step in range(3):  # the weights change between steps; the cached aggregate must not
            _, nd = ctx.sample_negatives(9, step, 1, du)
            ctx.train_step(p, du, dv, None, nd, 1, loss, grads)
            ctx.adam_step(p, m, vv, grads, step + 1)
        torch.cuda.synchronize()
        out.append((loss.clone(), grads.clone(), p.clone()))
        ctx.close()
    assert all(torch.equal(a, b) for a, b in zip(out[0], out[1]))
    ctx = make_ctx(pkg, wl.citation_directed(500, 4000, 2.2, seed=1), wl.node_features(500, 64, 0))
    with pytest.raises(pkg.LpError):
        ctx.set_model("sage", [64, 64], fanout=[3], max_batch=8, cache_input_aggregation=True)
    ctx.close()


# ------------------------------------------------------------------------------------------ worker views (Section III)
def test_worker_views_match_oracle(pkg):
    g = wl.chung_lu(20000, 14.0, 2.1, seed=6)
    part = wl.random_partition(g.n, 4, seed=3)
    ctx = make_ctx(pkg, g, wl.node_features(g.n, 8, 0))
    dpart = t32(part)
    with pytest.raises(pkg.LpError) as ei:
        ctx.worker_view(dpart, 0, True, 1)  # sparsified rows requested before lp_sparsify
    assert ei.value.status == -2
    srp, scol, _ = ctx.sparsify(0.2, 9)
    sp = (srp.cpu().numpy(), scol.cpu().numpy())
    for worker in (0, 3):
        for keep_cross, mode in ((True, 1), (True, 2), (True, 0), (False, 0)):  # SpLPG, SpLPG+, SpLPG-, SpLPG--
            rp, col, st = ctx.worker_view(dpart, worker, keep_cross, mode)
            orp, ocol, ost = oracle.worker_view(g.n, g.rowptr, g.col, part, worker, keep_cross, mode, sparsified=sp)
            assert np.array_equal(rp.cpu().numpy(), orp) and np.array_equal(col.cpu().numpy(), ocol) and st == ost
    # the sparsified sharing moves far fewer foreign entries than complete sharing (the method's point)
    _, _, s1 = ctx.worker_view(dpart, 0, True, 1)
    _, _, s2 = ctx.worker_view(dpart, 0, True, 2)
    assert s1["foreign_entries"] < 0.45 * s2["foreign_entries"]
    ctx.close()


# ------------------------------------------------------------------------------------------ MLP edge predictor, Hits@K
@pytest.mark.parametrize("arch,prec,fanout", [("sage", "fp32", None), ("gcn", "fp32", None), ("sage", "bf16", None), ("sage", "fp32", [4, 3])])
def test_mlp_predictor_step(pkg, arch, prec, fanout):
    if fanout:
        g = wl.citation_directed(5000, 60000, 2.2, seed=5)
        rows = np.repeat(np.arange(g.n, dtype=np.int32), np.diff(g.rowptr))
        sel = np.random.default_rng(3).choice(g.nnz, 900, replace=False)
        u, v = g.col[sel].copy(), rows[sel].copy()
    else:
        # (the BF16 case is large enough for the transforms to run on pairs of SMs, so the top layer takes its input gradient
        # as aggregate-then-transform behind the two-operand gradient gather)
        g = wl.chung_lu(9001 if prec == "bf16" else 6000, 14.0, 2.1, seed=5)
        pu, pv = wl.undirected_edge_list(g)
        sel = np.random.default_rng(3).choice(len(pu), 2500, replace=False)
        u, v = pu[sel].copy(), pv[sel].copy()
    dims, Hp, k = [64, 128, 64], 128, 2
    X = wl.node_features(g.n, 64, 1)
    params = wl.glorot_params(arch, dims, 2, bias_scale=0.05, pred_hidden=Hp)
    ctx = make_ctx(pkg, g, X)
    assert ctx.set_model(arch, dims, prec=prec, fanout=fanout, max_batch=len(u), max_k=k, pred_hidden=Hp) == len(params)
    du, dv, p = t32(u), t32(v), t32(params)
    seed, step = 21, 4
    _, nd = ctx.sample_negatives(seed, step, k, du)
    loss, grads = torch.zeros(1, device=DEV), torch.full((len(params),), 3.0, device=DEV)
    ctx.train_step(p, du, dv, None, nd, k, loss, grads, seed=seed, step=step)
    torch.cuda.synchronize()
    ons, ond, _ = oracle.sample_negatives(g.n, g.rowptr, g.col, u, seed, step, k)
    assert np.array_equal(nd.cpu().numpy(), ond)
    blocks = oracle.build_blocks(g.n, g.rowptr, g.col, np.concatenate([u, v, ond]), fanout, seed, step) if fanout else None
    rows0 = blocks[0][0] if fanout else np.arange(g.n)
    ties = None
    if not fanout:
        ties = [ctx.embeddings(1).cpu().numpy() > 0]
    E = len(u) * (1 + k)
    pred_ties = [ctx.predictor_activations(1, E).cpu().numpy() > 0, ctx.predictor_activations(2, E).cpu().numpy() > 0]
    ref = oracle.train_step(g, X, params, arch, dims, u, v, ons, ond, blocks=blocks, relu_ties=ties, rounding=prec, pred_hidden=Hp,
                            pred_ties=pred_ties)
    # outside the rounding windows the GPU's ReLU decisions equal the oracle's own (encoder and predictor)
    if ties is not None:
        assert_relu_decisions_agree(ref["cache"], ties, None, f"{arch}/{prec} encoder")
    assert_relu_decisions_agree(ref["pred_cache"], pred_ties, None, f"{arch}/{prec} predictor")
    n_enc = oracle.encoder_param_count(arch, dims)
    gg = grads.cpu().numpy()
    err = {"loss": abs(loss.item() - ref["loss"]) / abs(ref["loss"]),
           "HK": rel_l2(ctx.embeddings(2, rows=len(rows0)).cpu().numpy(), ref["cache"]["H"][2][rows0]),
           "dHK": rel_l2(ctx.output_gradient(rows=len(rows0)).cpu().numpy(), ref["dHK"][rows0]),
           "enc_grads": rel_l2(gg[:n_enc], ref["grads"][:n_enc]),
           "pred_grads": rel_l2(gg[n_enc:], ref["grads"][n_enc:])}
    D = dims[-1]
    o = n_enc
    for name, size in (("W0", D * Hp), ("b0", Hp), ("W1", Hp * Hp), ("b1", Hp), ("w2", Hp), ("b2", 1)):
        err["d" + name] = rel_l2(gg[o:o + size], ref["grads"][o:o + size])
        o += size
    tol = TOL[prec]
    bad = {kk: e for kk, e in err.items() if not e < tol}
    assert not bad, f"outside {tol}: {bad} (all {err})"
    # scores through lp_score agree with the oracle's predictor
    s_gpu = ctx.score(p, du, dv, seed=seed, step=step).cpu().numpy()
    s_ref = oracle.score(g, X, params, arch, dims, u, v, blocks=oracle.build_blocks(g.n, g.rowptr, g.col, np.concatenate([u, v]), fanout, seed, step) if fanout else None, pred_hidden=Hp)
    assert rel_l2(s_gpu, s_ref) < (2e-2 if prec == "bf16" else 1e-5)
    ctx.close()


def test_hits_at_k(pkg):
    g = wl.erdos_renyi(50, 100, seed=0)
    ctx = make_ctx(pkg, g, wl.node_features(g.n, 8, 0))
    rng = np.random.default_rng(0)
    pos = rng.standard_normal(5000).astype(np.float32)
    neg = np.concatenate([rng.standard_normal(300000), [0.0, -0.0, 1.5, 1.5]]).astype(np.float32)
    for k in (1, 100, 5000, len(neg)):
        assert ctx.hits_at_k(t32(pos), t32(neg), k) == oracle.hits_at_k(pos, neg, k)
    assert ctx.hits_at_k(t32(pos), t32(neg[:50]), 100) == 1.0
    small_pos, small_neg = np.array([2.0, 0.0, -0.0], dtype=np.float32), np.array([1.0, 2.0, 3.0, 0.0], dtype=np.float32)
    assert ctx.hits_at_k(t32(small_pos), t32(small_neg), 3) == oracle.hits_at_k(small_pos, small_neg, 3)
    ctx.close()
