"""Pins for the CPU oracle: closed forms, dense brute force, finite differences, published
known-answer vectors and invariants.  None of these re-use the oracle's own formulas."""
import math
import os

import numpy as np
import pytest

import oracle
from oracle import model as omodel
from oracle import sparse as osparse
import workloads as wl
from helpers import (dense_adjacency, dense_forward, dense_gcn_operator, dense_loss,
                     dense_mean_operator, rel_l2)

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ------------------------------------------------------------------ Philox
def np_philox(c0, c1, c2, c3, k0, k1):
    """Independent vectorised Philox4x32-10 on uint64 lanes (from the published definition)."""
    c0, c1, c2, c3 = (np.asarray(x, dtype=np.uint64) for x in (c0, c1, c2, c3))
    k0, k1 = np.uint64(k0), np.uint64(k1)
    mask = np.uint64(0xFFFFFFFF)
    for _ in range(10):
        p0 = np.uint64(0xD2511F53) * c0
        p1 = np.uint64(0xCD9E8D57) * c2
        c0, c1, c2, c3 = ((p1 >> np.uint64(32)) ^ c1 ^ k0) & mask, p1 & mask, \
                         ((p0 >> np.uint64(32)) ^ c3 ^ k1) & mask, p0 & mask
        k0 = (k0 + np.uint64(0x9E3779B9)) & mask
        k1 = (k1 + np.uint64(0xBB67AE85)) & mask
    return c0, c1, c2, c3


def test_philox_known_answers():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) if l.strip() and l[0] != "#"]
    assert len(rows) == 3
    for r in rows:
        v = [int(x, 16) for x in r]
        out = oracle.philox4x32_10(v[0:4], v[4:6])
        assert out.tolist() == v[6:10]


def test_philox_constants_closed_form():
    # Weyl increments are the fractional parts of the golden ratio and sqrt(3), scaled by 2^32
    assert int((math.sqrt(5.0) - 1.0) / 2.0 * 2 ** 32) == 0x9E3779B9
    assert int((math.sqrt(3.0) - 1.0) * 2 ** 32) == 0xBB67AE85
    a = oracle.philox4x32_10([5, 6, 7, 8], [9, 10])
    b = [int(x[()]) for x in np_philox(5, 6, 7, 8, 9, 10)]
    assert a.tolist() == b


# ------------------------------------------------------------------ structure
def test_csc_transpose_bruteforce_and_involution():
    g = wl.citation_directed(60, 400, 2.2, seed=11)
    colptr, rowidx, perm = oracle.csc_transpose(g.n, g.rowptr, g.col)
    A = dense_adjacency(g)
    # brute force: transposed row c lists the v with A[v, c] != 0 ascending
    exp_rows = [np.nonzero(A[:, c])[0] for c in range(g.n)]
    assert colptr.tolist() == np.concatenate([[0], np.cumsum([len(r) for r in exp_rows])]).tolist()
    assert rowidx.tolist() == np.concatenate(exp_rows).tolist()
    assert sorted(perm.tolist()) == list(range(g.nnz))
    rows = np.repeat(np.arange(g.n), np.diff(g.rowptr))
    assert np.array_equal(rows[perm], rowidx) and np.array_equal(g.col[perm], np.repeat(np.arange(g.n), np.diff(colptr)))
    # transpose of the transpose is the original
    rp2, ci2, _ = oracle.csc_transpose(g.n, colptr, rowidx)
    assert np.array_equal(rp2, g.rowptr) and np.array_equal(ci2, g.col)
    # degrees
    assert np.array_equal(np.diff(colptr), (A != 0).sum(axis=0))


def test_csc_transpose_rejects_bad_input():
    with pytest.raises(ValueError):
        oracle.csc_transpose(3, np.array([0, 1, 2, 3]), np.array([0, 5, 1]))
    with pytest.raises(ValueError):
        oracle.csc_transpose(3, np.array([0, 2, 1, 3]), np.array([0, 1, 1]))


# ------------------------------------------------------------------ aggregation
@pytest.mark.parametrize("weighted", [False, True])
def test_gcn_aggregate_dense_bruteforce(weighted):
    g = wl.coauthor_weighted(50, 160, seed=5) if weighted else wl.erdos_renyi(50, 150, seed=5)
    H = np.random.default_rng(0).standard_normal((g.n, 7))
    S = dense_gcn_operator(g)
    M = oracle.aggregate("gcn", g.n, g.rowptr, g.col, g.w, H)
    assert np.allclose(M, S @ H, rtol=1e-12, atol=1e-13)
    # invariants of the renormalised adjacency: symmetric, and sqrt(d~) is a fixed vector
    dt = oracle.gcn_degree(g.n, g.rowptr, g.w)
    assert np.allclose(dt, 1 + dense_adjacency(g).sum(axis=1))
    assert np.allclose(S, S.T)
    fixed = oracle.aggregate("gcn", g.n, g.rowptr, g.col, g.w, np.sqrt(dt)[:, None])
    assert np.allclose(fixed[:, 0], np.sqrt(dt), rtol=1e-12)
    # backward is multiplication by the transposed operator
    dM = np.random.default_rng(1).standard_normal((g.n, 5))
    assert np.allclose(oracle.aggregate_backward("gcn", g.n, g.rowptr, g.col, g.w, dM), S.T @ dM, atol=1e-13)


def test_mean_aggregate_dense_bruteforce_directed():
    g = wl.citation_directed(70, 200, 2.2, seed=3)
    H = np.random.default_rng(0).standard_normal((g.n, 6))
    S = dense_mean_operator(g)
    M = oracle.aggregate("mean", g.n, g.rowptr, g.col, None, H)
    assert np.allclose(M, S @ H, atol=1e-13)
    deg = np.diff(g.rowptr)
    assert (deg == 0).any(), "want an isolated row in this case"
    assert np.all(M[deg == 0] == 0)
    # rows of the mean operator sum to one: constants are preserved where deg > 0
    ones = oracle.aggregate("mean", g.n, g.rowptr, g.col, None, np.full((g.n, 2), 3.5))
    assert np.allclose(ones[deg > 0], 3.5)
    dM = np.random.default_rng(1).standard_normal((g.n, 4))
    assert np.allclose(oracle.aggregate_backward("mean", g.n, g.rowptr, g.col, None, dM), S.T @ dM, atol=1e-13)


def test_empty_graph_reduces_to_mlp():
    n, dims = 9, [4, 5, 3]
    g = wl.Graph(n=n, rowptr=np.zeros(n + 1, dtype=np.int64), col=np.zeros(0, dtype=np.int32))
    X = wl.node_features(n, 4, 0)
    for arch in ("gcn", "sage"):
        p = wl.glorot_params(arch, dims, 1, bias_scale=0.3)
        HK = oracle.forward(g, X, p, arch, dims)["H"][2]
        P = oracle.split_params(arch, dims, p.astype(np.float64))
        W1 = P[0]["W"] if arch == "gcn" else P[0]["W_self"]
        W2 = P[1]["W"] if arch == "gcn" else P[1]["W_self"]
        ref = np.maximum(X.astype(np.float64) @ W1 + P[0]["b"], 0) @ W2 + P[1]["b"]
        assert np.allclose(HK, ref, atol=1e-13)


# ------------------------------------------------------------------ encoder forward
@pytest.mark.parametrize("arch,dims", [("gcn", [6, 8, 5]), ("sage", [6, 8, 5]), ("gcn", [6, 7, 7, 4]), ("sage", [5, 6, 6, 3])])
def test_forward_dense_bruteforce(arch, dims):
    g = wl.coauthor_weighted(48, 140, seed=2) if arch == "gcn" else wl.citation_directed(48, 300, 2.2, seed=2)
    X = wl.node_features(g.n, dims[0], 1)
    p = wl.glorot_params(arch, dims, 3, bias_scale=0.2)
    HK = oracle.forward(g, X, p, arch, dims)["H"][len(dims) - 1]
    ref, _ = dense_forward(g, X, p, arch, dims)
    assert np.allclose(HK, ref, rtol=1e-11, atol=1e-12)


# ------------------------------------------------------------------ loss
def test_loss_closed_forms():
    g = wl.erdos_renyi(40, 100, seed=1)
    dims = [4, 6, 5]
    X = wl.node_features(g.n, 4, 0)
    u, v = wl.undirected_edge_list(g)
    ns, nd, _ = oracle.sample_negatives(g.n, g.rowptr, g.col, u, seed=1, step=0)
    zero = np.zeros(wl.model_dims_param_count("gcn", dims), dtype=np.float32)
    out = oracle.train_step(g, X, zero, "gcn", dims, u, v, ns, nd)
    N = 2 * len(u)
    assert abs(out["loss"] - math.log(2.0)) < 1e-15
    assert np.allclose(out["g"][: len(u)], -0.5 / N) and np.allclose(out["g"][len(u):], 0.5 / N)
    # symmetry of the undirected score
    p = wl.glorot_params("gcn", dims, 3, 0.1)
    assert np.allclose(oracle.score(g, X, p, "gcn", dims, u, v), oracle.score(g, X, p, "gcn", dims, v, u), rtol=1e-14)


def test_bce_stability_against_extended_precision():
    from decimal import Decimal, getcontext
    getcontext().prec = 60
    s = np.array([-800.0, -40.0, -3.0, -1e-9, 0.0, 1e-9, 2.5, 37.0, 745.0])
    for y in (0.0, 1.0):
        ell, d = oracle.bce_with_logits(s, np.full_like(s, y))
        for si, li, di in zip(s, ell, d):
            sig = Decimal(1) / (Decimal(1) + (-Decimal(float(si))).exp())
            ref = -(sig.ln()) if y == 1.0 else -((Decimal(1) - sig).ln()) if sig != 1 else None
            if y == 0.0:  # -log(1 - sigma(s)) = log(1 + e^s)
                ref = (Decimal(1) + Decimal(float(si)).exp()).ln()
            assert abs(float(ref) - li) <= 1e-14 * max(1.0, abs(float(ref)))
            assert abs(float(sig) - y - di) <= 1e-15


# ------------------------------------------------------------------ backward
@pytest.mark.parametrize("arch,dims", [("gcn", [3, 4, 3]), ("sage", [3, 4, 3]), ("gcn", [3, 4, 4, 2]), ("sage", [3, 3, 4, 2])])
def test_backward_finite_differences(arch, dims):
    g = wl.coauthor_weighted(24, 60, seed=4) if arch == "gcn" else wl.citation_directed(24, 110, 2.2, seed=4)
    X = wl.node_features(g.n, dims[0], 2)
    p = wl.glorot_params(arch, dims, 5, bias_scale=0.3).astype(np.float64)
    rng = np.random.default_rng(0)
    src = rng.integers(0, g.n, 40).astype(np.int32)
    dst = rng.integers(0, g.n, 40).astype(np.int32)
    dst[:3] = src[:3]  # self pairs exercise the u == v branch
    nsrc, ndst = src[:20], rng.integers(0, g.n, 20).astype(np.int32)
    y = np.concatenate([np.ones(40), np.zeros(20)])
    out = oracle.train_step(g, X, p, arch, dims, src, dst, nsrc, ndst)
    s_all, d_all = np.concatenate([src, nsrc]), np.concatenate([dst, ndst])
    assert abs(out["loss"] - dense_loss(g, X, p, arch, dims, s_all, d_all, y)) < 1e-13
    h = 1e-6
    fd = np.zeros_like(p)
    for i in range(p.shape[0]):
        pp, pm = p.copy(), p.copy()
        pp[i] += h
        pm[i] -= h
        fd[i] = (dense_loss(g, X, pp, arch, dims, s_all, d_all, y) - dense_loss(g, X, pm, arch, dims, s_all, d_all, y)) / (2 * h)
    assert rel_l2(out["grads"], fd) < 1e-7
    assert np.max(np.abs(out["grads"] - fd)) < 1e-8
    # gradient with respect to the input features (goes through every aggregation backward)
    dX = omodel.input_gradient(g, X, p, arch, dims, src, dst, nsrc, ndst)
    Xd = X.astype(np.float64)
    for (r, c) in [(0, 0), (5, 1), (g.n - 1, 2), (11, 0)]:
        xp, xm = Xd.copy(), Xd.copy()
        xp[r, c] += h
        xm[r, c] -= h
        num = (dense_loss(g, xp, p, arch, dims, s_all, d_all, y) - dense_loss(g, xm, p, arch, dims, s_all, d_all, y)) / (2 * h)
        assert abs(num - dX[r, c]) < 1e-8


def test_gradient_averaging_identical_workers():
    g = wl.erdos_renyi(30, 80, seed=9)
    dims = [4, 5, 4]
    X = wl.node_features(g.n, 4, 1)
    p = wl.glorot_params("sage", dims, 1, 0.1)
    u, v = wl.undirected_edge_list(g)
    ns, nd, _ = oracle.sample_negatives(g.n, g.rowptr, g.col, u, seed=3, step=0)
    g1 = oracle.train_step(g, X, p, "sage", dims, u, v, ns, nd)["grads"]
    assert np.allclose(oracle.average_gradients([g1] * 8), g1, rtol=1e-15)
    assert np.allclose(oracle.average_gradients([g1, 3 * g1]), 2 * g1, rtol=1e-15)


# ------------------------------------------------------------------ Adam
def test_adam_closed_forms():
    rng = np.random.default_rng(0)
    p0, g1, g2 = rng.standard_normal(50), rng.standard_normal(50), rng.standard_normal(50)
    lr, eps = 1e-3, 1e-8
    p1, m1, v1 = oracle.adam_step(p0, np.zeros(50), np.zeros(50), g1, t=1, lr=lr, eps=eps)
    # first step: bias correction gives m^ = g, v^ = g^2
    assert np.allclose(p1, p0 - lr * g1 / (np.abs(g1) + eps), rtol=1e-12, atol=1e-15)
    p2, m2, v2 = oracle.adam_step(p1, m1, v1, g2, t=2, lr=lr, eps=eps)
    mh = (0.9 * 0.1 * g1 + 0.1 * g2) / (1 - 0.81)
    vh = (0.999 * 0.001 * g1 ** 2 + 0.001 * g2 ** 2) / (1 - 0.999 ** 2)
    assert np.allclose(p2, p1 - lr * mh / (np.sqrt(vh) + eps), rtol=1e-12, atol=1e-15)


# ------------------------------------------------------------------ negative sampler
def test_negative_sampler_properties():
    g = wl.chung_lu(3000, 12.0, 2.1, seed=7)
    u, v = wl.undirected_edge_list(g)
    ns, nd, exhausted = oracle.sample_negatives(g.n, g.rowptr, g.col, u, seed=42, step=3, k=2)
    assert exhausted == 0
    assert np.array_equal(ns, np.repeat(u, 2))  # per-source: the source is kept
    A = set(zip(np.repeat(np.arange(g.n), np.diff(g.rowptr)).tolist(), g.col.tolist()))
    assert all(a != b and (b, a) not in A for a, b in zip(ns.tolist(), nd.tolist()))
    # batch-split invariance: the draw depends on the global edge index only
    lo = 1000
    ns2, nd2, _ = oracle.sample_negatives(g.n, g.rowptr, g.col, u[lo:lo + 500], seed=42, step=3, k=2, edge_index_base=lo)
    assert np.array_equal(nd2, nd[2 * lo: 2 * (lo + 500)])
    # different step or seed -> different draws
    assert not np.array_equal(nd, oracle.sample_negatives(g.n, g.rowptr, g.col, u, seed=42, step=4, k=2)[1])
    assert not np.array_equal(nd, oracle.sample_negatives(g.n, g.rowptr, g.col, u, seed=43, step=3, k=2)[1])


def test_negative_sampler_matches_independent_philox_and_is_uniform():
    g = wl.erdos_renyi(500, 1500, seed=1)
    B = 40000
    src = np.zeros(B, dtype=np.int32)
    seed, step = (7 << 32) | 12345, 9
    _, nd, _ = oracle.sample_negatives(g.n, g.rowptr, g.col, src, seed=seed, step=step, k=1, reject_edges=False)
    j = np.arange(B, dtype=np.uint64)
    x = np_philox(j & np.uint64(0xFFFFFFFF), j >> np.uint64(32), np.full(B, step, dtype=np.uint64),
                  np.full(B, 1, dtype=np.uint64), seed & 0xFFFFFFFF, seed >> 32)[0]
    assert np.array_equal(nd.astype(np.uint64), (x * np.uint64(g.n)) >> np.uint64(32))
    counts = np.bincount(nd, minlength=g.n)
    chi2 = ((counts - B / g.n) ** 2 / (B / g.n)).sum()
    assert chi2 < 499 + 5 * math.sqrt(2 * 499)  # 5 sigma of chi-square with n-1 degrees of freedom


def test_negative_sampler_candidates_and_global_pairs():
    g = wl.erdos_renyi(400, 1200, seed=2)
    cand = np.arange(0, 400, 4, dtype=np.int32)  # a "partition"
    u, _ = wl.undirected_edge_list(g)
    _, nd, _ = oracle.sample_negatives(g.n, g.rowptr, g.col, u, seed=5, step=0, cand=cand)
    assert np.isin(nd, cand).all()
    ns, nd, _ = oracle.sample_negatives(g.n, g.rowptr, g.col, u, seed=5, step=0, mode="global_pair", cand=cand)
    assert np.isin(nd, cand).all() and np.isin(ns, cand).all() and (ns != nd).all()
    assert len(np.unique(ns)) > 50
    # exhausted attempts are reported: a complete graph has no valid per-source negative
    n = 6
    full = wl.csr_from_edges(n, *np.array([(a, b) for a in range(n) for b in range(n) if a != b]).T)
    _, _, ex = oracle.sample_negatives(n, full.rowptr, full.col, np.arange(n, dtype=np.int32), seed=1, step=0, max_attempts=4)
    assert ex == n


def _np_draw(j, step, tag, kk, attempt, seed):
    """Word 0 of the Philox block for positive j: counter (lo(j), hi(j), lo(step), tag | kk << 8 | attempt << 16)."""
    j = np.asarray(j, dtype=np.uint64)
    w3 = np.full(j.shape, tag | (kk << 8) | (attempt << 16), dtype=np.uint64)
    return np_philox(j & np.uint64(0xFFFFFFFF), j >> np.uint64(32), np.full(j.shape, step & 0xFFFFFFFF, dtype=np.uint64), w3,
                     seed & 0xFFFFFFFF, seed >> 32)[0]


@pytest.mark.parametrize("mode", ["per_source", "global_pair"])
def test_negative_sampler_retry_draws_match_independent_philox(mode):
    # a dense graph, so that most first draws are rejected: the redraws (attempt in bits 16.., negative index in bits
    # 8..), the source draw of the global-pair mode (tag 2) and the exhaustion count are rebuilt here from the
    # independent Philox and a Python set of the edges; base and step beyond 2^32 exercise the high / low words
    n = 48
    rng = np.random.default_rng(7)
    A = rng.random((n, n)) < 0.55
    np.fill_diagonal(A, False)
    dst_e, src_e = np.nonzero(A)  # row = destination, column = in-neighbour
    g = wl.csr_from_edges(n, dst_e, src_e)
    edges = set(zip(src_e.tolist(), dst_e.tolist()))  # (source, destination)
    cand = np.arange(1, n, 2, dtype=np.int32) if mode == "global_pair" else None
    space = n if cand is None else len(cand)
    B, k, attempts = 1500, 3, 3
    base, step, seed = (5 << 32) + 123, (9 << 32) + 77, (0xDEADBEEF << 32) | 0x1234567
    pos_src = rng.integers(0, n, B).astype(np.int32)
    ns, nd, ex = oracle.sample_negatives(n, g.rowptr, g.col, pos_src, seed, step, k, mode=mode, cand=cand, max_attempts=attempts,
                                         edge_index_base=base)
    j = np.arange(B, dtype=np.uint64) + np.uint64(base)
    exp_s, exp_d = np.zeros((B, k), dtype=np.int64), np.zeros((B, k), dtype=np.int64)
    exhausted = 0
    for kk in range(k):
        done = np.zeros(B, dtype=bool)
        for a in range(attempts):
            pick = (_np_draw(j, step, 1, kk, a, seed) * np.uint64(space)) >> np.uint64(32)
            d = pick.astype(np.int64) if cand is None else cand[pick.astype(np.int64)].astype(np.int64)
            if mode == "per_source":
                sft = pos_src.astype(np.int64)
            else:
                pick2 = (_np_draw(j, step, 2, kk, a, seed) * np.uint64(space)) >> np.uint64(32)
                sft = cand[pick2.astype(np.int64)].astype(np.int64)
            ok = np.array([x != y and (x, y) not in edges for x, y in zip(sft.tolist(), d.tolist())])
            upd = ~done  # a positive keeps redrawing until a draw is accepted; the last draw stays
            exp_s[upd, kk], exp_d[upd, kk] = sft[upd], d[upd]
            done |= upd & ok
        exhausted += int((~done).sum())
    assert np.array_equal(nd, exp_d.ravel()) and np.array_equal(ns, exp_s.ravel())
    assert ex == exhausted and 0 < exhausted < B * k
    first = (_np_draw(j, step, 1, 0, 0, seed) * np.uint64(space)) >> np.uint64(32)
    first = first.astype(np.int64) if cand is None else cand[first.astype(np.int64)].astype(np.int64)
    assert (first != exp_d[:, 0]).mean() > 0.3  # the redraws really happened


def test_neighbor_sampler_matches_independent_floyd_with_philox():
    # rows longer than the fan-out: Floyd's subset algorithm over row positions with draw i of node v at hop h taken
    # from counter (v, i, lo(step), 3 | h << 8), rebuilt from the independent Philox
    g = wl.citation_directed(1500, 40000, 2.2, seed=4)
    frontier = np.unique(np.random.default_rng(1).integers(0, g.n, 400)).astype(np.int32)
    fanout, hop, step, seed = 7, 2, (3 << 32) + 11, (21 << 32) | 5
    ptr, cols = oracle.sample_neighbors(g.rowptr, g.col, frontier, fanout, seed, step, hop)
    longer = 0
    for i, v in enumerate(frontier.tolist()):
        row = g.col[g.rowptr[v]:g.rowptr[v + 1]]
        d = len(row)
        if d <= fanout:
            exp = row
        else:
            longer += 1
            chosen = []
            for q in range(fanout):
                jq = d - fanout + q
                x = int(np_philox(v, q, step & 0xFFFFFFFF, 3 | (hop << 8), seed & 0xFFFFFFFF, seed >> 32)[0])
                t = (x * (jq + 1)) >> 32
                chosen.append(jq if t in chosen else t)
            exp = row[np.sort(np.array(chosen))]
        assert np.array_equal(cols[ptr[i]:ptr[i + 1]], exp)
    assert longer > 50


# ------------------------------------------------------------------ neighbour sampler
def test_neighbor_sampler_properties_and_uniformity():
    g = wl.citation_directed(2000, 40000, 2.2, seed=8)
    frontier = np.unique(np.random.default_rng(0).integers(0, g.n, 600)).astype(np.int32)
    ptr, cols = oracle.sample_neighbors(g.rowptr, g.col, frontier, fanout=5, seed=3, step=1, hop=2)
    deg = np.diff(g.rowptr)[frontier]
    assert np.array_equal(np.diff(ptr), np.minimum(deg, 5))
    for i, v in enumerate(frontier):
        row = g.col[g.rowptr[v]:g.rowptr[v + 1]]
        pick = cols[ptr[i]:ptr[i + 1]]
        assert np.all(np.diff(pick) > 0) and np.isin(pick, row).all()
    # uniform over the C(5,2) = 10 subsets of a 5-neighbour row, over many steps
    star = wl.csr_from_edges(6, np.zeros(5, dtype=np.int64), np.arange(1, 6))
    seen = {}
    T = 20000
    for step in range(T):
        _, c = oracle.sample_neighbors(star.rowptr, star.col, np.array([0], dtype=np.int32), 2, seed=11, step=step, hop=1)
        seen[tuple(c.tolist())] = seen.get(tuple(c.tolist()), 0) + 1
    assert len(seen) == 10
    chi2 = sum((c - T / 10) ** 2 / (T / 10) for c in seen.values())
    assert chi2 < 9 + 5 * math.sqrt(18)


def test_blocks_and_sampled_forward_bruteforce():
    g = wl.citation_directed(120, 1500, 2.2, seed=6)
    dims = [4, 5, 5, 3]
    X = wl.node_features(g.n, 4, 0)
    p = wl.glorot_params("sage", dims, 2, 0.2)
    seeds = np.array([3, 17, 17, 40, 99], dtype=np.int32)
    fr, blks = oracle.build_blocks(g.n, g.rowptr, g.col, seeds, [3, 2, 2], seed=5, step=0)
    assert fr[0].tolist() == [3, 17, 40, 99]
    for h in range(3):
        assert np.all(np.diff(fr[h + 1]) > 0) and np.isin(fr[h], fr[h + 1]).all() and np.isin(blks[h][1], fr[h + 1]).all()
    HK = oracle.forward(g, X, p, "sage", dims, blocks=(fr, blks))["H"][3]
    # brute force: per layer a dense mean operator made from that hop's sampled rows
    H = X.astype(np.float64)
    P = oracle.split_params("sage", dims, p.astype(np.float64))
    for l in range(1, 4):
        h = 3 - l + 1
        ptr, cols = blks[h - 1]
        S = np.zeros((g.n, g.n))
        for i, v in enumerate(fr[h - 1]):
            nb = cols[ptr[i]:ptr[i + 1]]
            if len(nb):
                S[v, nb] = 1.0 / len(nb)
        Z = H @ P[l - 1]["W_self"] + (S @ H) @ P[l - 1]["W_neigh"] + P[l - 1]["b"]
        Hn = np.maximum(Z, 0) if l < 3 else Z
        keep = np.zeros(g.n, dtype=bool)
        keep[fr[h - 1]] = True
        H = np.where(keep[:, None], Hn, 0.0)
    assert np.allclose(HK, H, atol=1e-13)
    assert np.all(HK[np.setdiff1d(np.arange(g.n), fr[0])] == 0)


# ------------------------------------------------------------------ sparsifier (Algorithm 1, Theorems 1-2)
def test_sparsifier_probabilities_and_weights():
    g = wl.chung_lu(400, 10.0, 2.1, seed=3)
    deg = np.diff(g.rowptr).astype(np.float64)
    u, v = wl.undirected_edge_list(g)
    npr = (deg > 0).sum()
    pe = (1 / deg[u] + 1 / deg[v]) / npr
    assert abs(pe.sum() - 1.0) < 1e-12  # the degree-based probabilities are normalised by n'
    alpha = 0.2
    L = int(alpha * len(u))
    rows = np.repeat(np.arange(g.n), np.diff(g.rowptr))
    upper = g.col > rows
    acc = np.zeros(len(u))
    hits = np.zeros(len(u))
    T = 300
    for s in range(T):
        w = oracle.sparsify(g.n, g.rowptr, g.col, alpha, seed=s)
        wu = w[upper]
        # symmetric output, every kept weight is a positive multiple of 1 / (L p_e)
        colptr, rowidx, perm = oracle.csc_transpose(g.n, g.rowptr, g.col)
        assert np.array_equal(w[perm], w)
        mult = wu * L * pe
        assert np.allclose(mult, np.round(mult), atol=1e-9)
        assert int(np.round(mult).sum()) == L  # exactly L draws
        assert (wu > 0).sum() <= L
        acc += wu
        hits += np.round(mult)
    # E[w~_e] = 1 (Theorem 1 weights): check the average over edges and over seeds
    assert abs(acc.mean() / T - 1.0) < 0.02
    # empirical draw frequencies follow p_e (chi-square over edges pooled in 20 probability bins)
    order = np.argsort(pe)
    bins = np.array_split(order, 20)
    obs = np.array([hits[b].sum() for b in bins])
    exp = np.array([pe[b].sum() for b in bins]) * T * L
    chi2 = ((obs - exp) ** 2 / exp).sum()
    assert chi2 < 19 + 5 * math.sqrt(38)
    # removed fraction for alpha = 0.2 is "about 80 %" (Section IV): distinct kept edges in (0.15, 0.2] |E|
    kept = (oracle.sparsify(g.n, g.rowptr, g.col, alpha, seed=1)[upper] > 0).mean()
    expected_kept = (1 - (1 - pe) ** L).sum() / len(u)
    assert 0.14 < kept <= 0.2 and abs(kept - expected_kept) < 0.02


def test_effective_resistance_bounds_on_tiny_graph():
    # Theorem 2: (1/2)(1/d_u + 1/d_v) <= r_(u,v) <= (1/gamma)(1/d_u + 1/d_v), r from Eq. 3
    g = wl.erdos_renyi(40, 160, seed=2)
    A = dense_adjacency(g)
    d = A.sum(axis=1)
    assert (d > 0).all()
    Lp = np.linalg.pinv(np.diag(d) - A)
    Lsym = np.eye(g.n) - A / np.sqrt(np.outer(d, d))
    gamma = np.sort(np.linalg.eigvalsh(Lsym))[1]
    u, v = wl.undirected_edge_list(g)
    r = Lp[u, u] + Lp[v, v] - 2 * Lp[u, v]
    approx = 1 / d[u] + 1 / d[v]
    assert np.all(r >= 0.5 * approx - 1e-12) and np.all(r <= approx / gamma + 1e-12)


def test_sparsified_graph_csr():
    g = wl.erdos_renyi(200, 900, seed=4)
    rp, cc, w = oracle.sparsified_graph(g.n, g.rowptr, g.col, 0.2, seed=0)
    assert rp[-1] == len(cc) == len(w) and (w > 0).all()
    for v in range(g.n):
        assert np.all(np.diff(cc[rp[v]:rp[v + 1]]) > 0)
        assert np.isin(cc[rp[v]:rp[v + 1]], g.col[g.rowptr[v]:g.rowptr[v + 1]]).all()


def test_sampled_step_backward_finite_differences():
    g = wl.citation_directed(60, 700, 2.2, seed=6)
    dims = [3, 4, 3]
    X = wl.node_features(g.n, 3, 0).astype(np.float64)
    p = wl.glorot_params("sage", dims, 2, 0.2).astype(np.float64)
    src = np.array([1, 5, 9, 30], dtype=np.int32)
    dst = np.array([2, 7, 9, 41], dtype=np.int32)
    nsrc, ndst = src.copy(), np.array([50, 3, 22, 8], dtype=np.int32)
    seeds = np.concatenate([src, dst, ndst])
    fr, blks = oracle.build_blocks(g.n, g.rowptr, g.col, seeds, [3, 2], seed=1, step=7)
    out = oracle.train_step(g, X, p, "sage", dims, src, dst, nsrc, ndst, blocks=(fr, blks))
    ops = []
    for l in range(1, 3):
        h = 2 - l + 1
        ptr, cols = blks[h - 1]
        S = np.zeros((g.n, g.n))
        for i, v in enumerate(fr[h - 1]):
            nb = cols[ptr[i]:ptr[i + 1]]
            if len(nb):
                S[v, nb] = 1.0 / len(nb)
        ops.append(S)
    s_all, d_all = np.concatenate([src, nsrc]), np.concatenate([dst, ndst])
    y = np.concatenate([np.ones(4), np.zeros(4)])

    def bf_loss(pp):
        P = oracle.split_params("sage", dims, pp)
        H1 = np.maximum(X @ P[0]["W_self"] + (ops[0] @ X) @ P[0]["W_neigh"] + P[0]["b"], 0)
        keep = np.zeros(g.n, dtype=bool)
        keep[fr[1]] = True
        H1 = np.where(keep[:, None], H1, 0.0)
        H2 = H1 @ P[1]["W_self"] + (ops[1] @ H1) @ P[1]["W_neigh"] + P[1]["b"]
        s = (H2[s_all] * H2[d_all]).sum(axis=1)
        return float(np.mean(y * np.logaddexp(0, -s) + (1 - y) * np.logaddexp(0, s)))

    assert abs(bf_loss(p) - out["loss"]) < 1e-13
    fd = np.zeros_like(p)
    for i in range(p.shape[0]):
        pp, pm = p.copy(), p.copy()
        pp[i] += 1e-6
        pm[i] -= 1e-6
        fd[i] = (bf_loss(pp) - bf_loss(pm)) / 2e-6
    assert rel_l2(out["grads"], fd) < 1e-7


def _dense_sampled_gcn_operator(g, frontier, ptr, cols):
    """Dense operator of one sampled GCN hop, written from the definition: self term 1 / d~_v, sampled entries
    w_vu / sqrt(d~_v d~_u) * |N(v)| / |S(v)|, degrees of the full graph."""
    A = dense_adjacency(g)
    dt = 1.0 + A.sum(axis=1)
    S = np.zeros((g.n, g.n))
    for i, v in enumerate(frontier):
        nb = cols[ptr[i]:ptr[i + 1]]
        deg = int(g.rowptr[v + 1] - g.rowptr[v])
        S[v, v] += 1.0 / dt[v]
        for u in nb:
            S[v, u] += A[v, u] / math.sqrt(dt[v] * dt[u]) * deg / len(nb)
    return S


def test_sampled_gcn_with_full_fanout_equals_full_graph_training():
    # a fan-out at least as large as every degree samples every neighbour: the sampled step must then give
    # the loss and the parameter gradients of full-graph training (pinned elsewhere against dense operators)
    g = wl.coauthor_weighted(70, 260, seed=4)
    fan = int(np.diff(g.rowptr).max())
    dims = [4, 5, 3]
    X = wl.node_features(g.n, 4, 0).astype(np.float64)
    p = wl.glorot_params("gcn", dims, 3, 0.2).astype(np.float64)
    src = np.array([1, 5, 9, 30], dtype=np.int32)
    dst = np.array([2, 7, 9, 41], dtype=np.int32)
    nsrc, ndst = src.copy(), np.array([50, 3, 22, 8], dtype=np.int32)
    blocks = oracle.build_blocks(g.n, g.rowptr, g.col, np.concatenate([src, dst, ndst]), [fan, fan], seed=1, step=0)
    a = oracle.train_step(g, X, p, "gcn", dims, src, dst, nsrc, ndst, blocks=blocks)
    b = oracle.train_step(g, X, p, "gcn", dims, src, dst, nsrc, ndst)
    assert abs(a["loss"] - b["loss"]) < 1e-12
    assert rel_l2(a["grads"], b["grads"]) < 1e-6  # float32 rounding of the per-entry ratio-times-weight only


def test_sampled_gcn_forward_bruteforce_and_unbiased():
    g = wl.coauthor_weighted(90, 700, seed=8)
    assert g.w is not None and np.diff(g.rowptr).max() > 6
    dims = [4, 5, 3]
    X = wl.node_features(g.n, 4, 0).astype(np.float64)
    p = wl.glorot_params("gcn", dims, 2, 0.2).astype(np.float64)
    P = oracle.split_params("gcn", dims, p)
    seeds = np.array([3, 17, 40, 77], dtype=np.int32)
    fr, blks = oracle.build_blocks(g.n, g.rowptr, g.col, seeds, [3, 2], seed=5, step=0)
    HK = oracle.forward(g, X, p, "gcn", dims, blocks=(fr, blks))["H"][2]
    H = X
    for l in (1, 2):
        h = 2 - l + 1
        S = _dense_sampled_gcn_operator(g, fr[h - 1], *blks[h - 1])
        Z = (S @ H) @ P[l - 1]["W"] + P[l - 1]["b"]
        Hn = np.maximum(Z, 0) if l < 2 else Z
        keep = np.zeros(g.n, dtype=bool)
        keep[fr[h - 1]] = True
        H = np.where(keep[:, None], Hn, 0.0)
    assert rel_l2(HK, H) < 1e-6
    # the sampled operator averages to the full one over many independent samples
    v = int(np.argmax(np.diff(g.rowptr)))
    full = dense_gcn_operator(g)[v]
    acc = np.zeros(g.n)
    T = 3000
    for step in range(T):
        fr1, blk1 = oracle.build_blocks(g.n, g.rowptr, g.col, np.array([v], dtype=np.int32), [3], seed=9, step=step)
        acc += _dense_sampled_gcn_operator(g, fr1[0], *blk1[0])[v]
    nz = full > 0
    assert np.abs(acc[nz] / T - full[nz]).max() < 0.12 * full[nz].max()
    assert np.abs(acc[~nz]).max() == 0.0


def test_sampled_gcn_step_backward_finite_differences():
    g = wl.coauthor_weighted(60, 300, seed=6)
    dims = [3, 4, 3]
    X = wl.node_features(g.n, 3, 0).astype(np.float64)
    p = wl.glorot_params("gcn", dims, 2, 0.2).astype(np.float64)
    src = np.array([1, 5, 9, 30], dtype=np.int32)
    dst = np.array([2, 7, 9, 41], dtype=np.int32)
    nsrc, ndst = src.copy(), np.array([50, 3, 22, 8], dtype=np.int32)
    fr, blks = oracle.build_blocks(g.n, g.rowptr, g.col, np.concatenate([src, dst, ndst]), [3, 2], seed=1, step=7)
    out = oracle.train_step(g, X, p, "gcn", dims, src, dst, nsrc, ndst, blocks=(fr, blks))
    ops = [_dense_sampled_gcn_operator(g, fr[2 - l], *blks[2 - l]) for l in (1, 2)]
    s_all, d_all = np.concatenate([src, nsrc]), np.concatenate([dst, ndst])
    y = np.concatenate([np.ones(4), np.zeros(4)])

    def bf_loss(pp):
        P = oracle.split_params("gcn", dims, pp)
        H1 = np.maximum((ops[0] @ X) @ P[0]["W"] + P[0]["b"], 0)
        keep = np.zeros(g.n, dtype=bool)
        keep[fr[1]] = True
        H1 = np.where(keep[:, None], H1, 0.0)
        H2 = (ops[1] @ H1) @ P[1]["W"] + P[1]["b"]
        s = (H2[s_all] * H2[d_all]).sum(axis=1)
        return float(np.mean(y * np.logaddexp(0, -s) + (1 - y) * np.logaddexp(0, s)))

    assert abs(bf_loss(p) - out["loss"]) < 1e-7
    fd = np.zeros_like(p)
    for i in range(p.shape[0]):
        pp, pm = p.copy(), p.copy()
        pp[i] += 1e-6
        pm[i] -= 1e-6
        fd[i] = (bf_loss(pp) - bf_loss(pm)) / 2e-6
    assert rel_l2(out["grads"], fd) < 1e-5


def test_relu_tie_window_only_touches_near_zero_units():
    g = wl.erdos_renyi(60, 200, seed=3)
    dims = [6, 8, 4]
    X = wl.node_features(g.n, 6, 0)
    p = wl.glorot_params("gcn", dims, 1, 0.2)
    base = oracle.forward(g, X, p, "gcn", dims)
    Z = base["Z"][0]
    flipped = ~(Z > 0)  # decisions that are all wrong
    wide = dict(omodel.ROUNDING["bf16"], u_store=2.0 ** -4, u_w=2.0 ** -4, u_in=2.0 ** -4)  # a coarse arithmetic: a window that holds some units
    out = oracle.forward(g, X, p, "gcn", dims, relu_ties=[flipped], rounding=wide)
    near = out["near"][0]
    assert 0 < near.sum() < near.size // 2
    assert np.array_equal(near, np.abs(Z) <= out["window"][0])
    assert out["ties"] == int(near.sum()) == out["n_near"]
    assert np.array_equal(out["active"][0][~near], (Z > 0)[~near])  # untouched outside the window
    assert np.array_equal(out["active"][0][near], flipped[near])
    assert np.array_equal(out["own_active"][0], Z > 0)
    # no rounding model: nothing is adopted and nothing else changes; with a model but no decisions given, the oracle's own stand
    assert oracle.forward(g, X, p, "gcn", dims, relu_ties=[flipped])["ties"] == 0
    own = oracle.forward(g, X, p, "gcn", dims, rounding=wide)
    assert own["ties"] == 0 and np.array_equal(own["active"][0], Z > 0) and np.array_equal(own["H"][2], base["H"][2])
    # the window scales with the unit roundoff and vanishes for exact arithmetic
    exact = {k: 0.0 for k in wide}
    assert oracle.forward(g, X, p, "gcn", dims, relu_ties=[flipped], rounding=exact)["n_near"] == int((Z == 0).sum())


def _round_bf16(x):
    """Round-to-nearest-even to 8 significand bits, on the bit pattern (independent of any library conversion)."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    return ((b + (((b >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF))) & np.uint32(0xFFFF0000)).view(np.float32)


@pytest.mark.parametrize("arch", ["sage", "gcn"])
@pytest.mark.parametrize("path", ["bf16", "fp32"])
def test_rounding_window_bounds_an_emulated_low_precision_path(arch, path):
    # The ReLU window comes from a first-order model of the rounding of the arithmetic under test.  Pin it against an
    # emulation of that arithmetic written here in numpy (inputs, weights and stored activations rounded to BF16 or
    # FP32, FP32 aggregation and matrix product): every pre-activation of the emulation lies inside the oracle's
    # window around the FP64 value, and the modelled standard deviation is the right size (not vacuous).
    g = wl.chung_lu(3000, 14.0, 2.1, seed=3) if arch == "sage" else wl.coauthor_weighted(3000, 12000, seed=1)
    dims = [64, 128, 128, 64]
    X = wl.node_features(g.n, 64, 1)
    p = wl.glorot_params(arch, dims, 2, 0.05)
    n_sigma = 6.0
    c = oracle.forward(g, X, p, arch, dims, rounding=path, final_variance=True, n_sigma=n_sigma)
    P = omodel.split_params(arch, dims, p.astype(np.float64))
    rnd = _round_bf16 if path == "bf16" else (lambda x: np.asarray(x, dtype=np.float32))
    deg = np.diff(g.rowptr)
    rows = np.repeat(np.arange(g.n), deg)
    H = rnd(X)
    for k in range(3):
        if arch == "sage":
            M = np.zeros((g.n, H.shape[1]), dtype=np.float32)
            np.add.at(M, rows, H[g.col])
            inv = np.where(deg > 0, np.float32(1) / np.maximum(deg, 1).astype(np.float32), np.float32(0)).astype(np.float32)
            A = np.concatenate([H, rnd(M * inv[:, None])], axis=1)
            W = np.concatenate([P[k]["W_self"], P[k]["W_neigh"]], axis=0)
        else:
            dt = (1.0 + np.bincount(rows, weights=g.w, minlength=g.n)).astype(np.float32)
            coef = (g.w / np.sqrt(dt[rows] * dt[g.col])).astype(np.float32)
            M = (H / dt[:, None]).astype(np.float32)
            np.add.at(M, rows, coef[:, None] * H[g.col])
            A, W = rnd(M), P[k]["W"]
        Z = (A.astype(np.float32) @ rnd(W).astype(np.float32) + P[k]["b"].astype(np.float32)).astype(np.float32)
        if k < 2:
            err, win = np.abs(Z - c["Z"][k]), c["window"][k]
            assert (err <= win).all(), f"layer {k}: {(err / win).max()} windows"
            ratio = np.sqrt(np.mean((err / (win / n_sigma)) ** 2))  # emulated error over modelled standard deviation, RMS
            assert (0.4 < ratio < 1.2) if path == "bf16" else (0.02 < ratio < 1.2), ratio
            # the emulation's own decisions agree with the oracle's outside the window
            assert np.array_equal((Z > 0)[~c["near"][k]], c["own_active"][k][~c["near"][k]])
            H = rnd(np.maximum(Z, 0))
        else:
            err = np.abs(rnd(Z) - c["H"][3])
            assert (err <= n_sigma * np.sqrt(c["var_HK"])).all()
    frac = np.mean([m.mean() for m in c["near"]])
    assert frac < (0.04 if path == "bf16" else 1e-3)  # how many units the window holds on this input


def test_worker_view_bruteforce():
    g = wl.chung_lu(300, 8.0, 2.1, seed=4)
    part = wl.random_partition(g.n, 3, seed=1)
    sp = oracle.sparsified_graph(g.n, g.rowptr, g.col, 0.3, seed=2)
    for keep_cross in (True, False):
        for mode in (0, 1, 2):
            ptr, col, st = oracle.worker_view(g.n, g.rowptr, g.col, part, 1, keep_cross, mode, sparsified=sp[:2])
            own = foreign = frows = 0
            for v in range(g.n):  # row by row, straight from the definition
                if part[v] == 1:
                    exp = [u for u in g.col[g.rowptr[v]:g.rowptr[v + 1]] if keep_cross or part[u] == 1]
                    own += len(exp)
                elif mode == 1:
                    exp = list(sp[1][sp[0][v]:sp[0][v + 1]])
                elif mode == 2:
                    exp = list(g.col[g.rowptr[v]:g.rowptr[v + 1]])
                else:
                    exp = []
                if part[v] != 1:
                    foreign += len(exp)
                    frows += 1 if exp else 0
                assert col[ptr[v]:ptr[v + 1]].tolist() == exp
            assert st == {"own_entries": own, "foreign_entries": foreign, "foreign_rows": frows, "own_nodes": int((part == 1).sum())}


# ------------------------------------------------------------------ MLP edge predictor, Hits@K
def _dense_mlp_loss(g, X, p, arch, dims, Hp, src, dst, y):
    """Loss with the 3-layer MLP predictor written independently of the oracle (dense operators)."""
    n_enc = wl.model_dims_param_count(arch, dims)
    H, _ = dense_forward(g, X, p[:n_enc], arch, dims)
    t, D = p[n_enc:], dims[-1]
    o = 0
    W0 = t[o:o + D * Hp].reshape(D, Hp); o += D * Hp
    b0 = t[o:o + Hp]; o += Hp
    W1 = t[o:o + Hp * Hp].reshape(Hp, Hp); o += Hp * Hp
    b1 = t[o:o + Hp]; o += Hp
    w2 = t[o:o + Hp]; o += Hp
    b2 = t[o]
    z = H[src] * H[dst]
    s = np.maximum(np.maximum(z @ W0 + b0, 0) @ W1 + b1, 0) @ w2 + b2
    return float(np.mean(y * np.logaddexp(0.0, -s) + (1 - y) * np.logaddexp(0.0, s))), s


@pytest.mark.parametrize("arch", ["gcn", "sage"])
def test_mlp_predictor_forward_and_finite_differences(arch):
    g = wl.erdos_renyi(26, 70, seed=4)
    dims, Hp = [3, 4, 3], 5
    X = wl.node_features(g.n, 3, 2)
    p = wl.glorot_params(arch, dims, 5, bias_scale=0.3, pred_hidden=Hp).astype(np.float64)
    assert p.shape[0] == wl.model_dims_param_count(arch, dims, Hp)
    rng = np.random.default_rng(1)
    src = rng.integers(0, g.n, 30).astype(np.int32)
    dst = rng.integers(0, g.n, 30).astype(np.int32)
    dst[:2] = src[:2]
    nsrc, ndst = src[:15], rng.integers(0, g.n, 15).astype(np.int32)
    s_all, d_all = np.concatenate([src, nsrc]), np.concatenate([dst, ndst])
    y = np.concatenate([np.ones(30), np.zeros(15)])
    out = oracle.train_step(g, X, p, arch, dims, src, dst, nsrc, ndst, pred_hidden=Hp)
    ref_loss, ref_s = _dense_mlp_loss(g, X, p, arch, dims, Hp, s_all, d_all, y)
    assert abs(out["loss"] - ref_loss) < 1e-13 and np.allclose(out["scores"], ref_s, atol=1e-13)
    assert np.allclose(oracle.score(g, X, p, arch, dims, s_all, d_all, pred_hidden=Hp), ref_s, atol=1e-13)
    fd = np.zeros_like(p)
    for i in range(p.shape[0]):
        pp, pm = p.copy(), p.copy()
        pp[i] += 1e-6
        pm[i] -= 1e-6
        fd[i] = (_dense_mlp_loss(g, X, pp, arch, dims, Hp, s_all, d_all, y)[0] - _dense_mlp_loss(g, X, pm, arch, dims, Hp, s_all, d_all, y)[0]) / 2e-6
    assert rel_l2(out["grads"], fd) < 1e-7 and np.max(np.abs(out["grads"] - fd)) < 1e-8
    n_enc = wl.model_dims_param_count(arch, dims)
    assert np.linalg.norm(out["grads"][n_enc:]) > 0 and np.linalg.norm(out["grads"][:n_enc]) > 0


def test_hits_at_k_definition():
    rng = np.random.default_rng(0)
    pos, neg = rng.standard_normal(200), rng.standard_normal(1000)
    for k in (1, 10, 100, 1000):
        brute = np.mean([(neg >= p_).sum() < k for p_ in pos])  # fewer than k negatives score at least as high
        assert abs(oracle.hits_at_k(pos, neg, k) - brute) < 1e-15
    assert oracle.hits_at_k(pos, neg, 1001) == 1.0                 # fewer negatives than K
    assert oracle.hits_at_k(np.array([5.0, 6.0]), np.array([1.0, 2.0, 3.0]), 1) == 1.0
    assert oracle.hits_at_k(np.array([2.5, 0.0]), np.array([1.0, 2.0, 3.0]), 2) == 0.5
    assert oracle.hits_at_k(np.array([2.0]), np.array([1.0, 2.0, 3.0]), 2) == 0.0  # ties do not count as hits
