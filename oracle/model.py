"""FP64 oracle of the encoder, predictor, loss, gradient and optimiser.

TEST INFRASTRUCTURE ONLY -- see oracle/__init__.py.  Dense algebra is numpy matmul in
float64; aggregation and samplers come from oracle/sparse.py.  The backward pass is
written out by hand from the chain rule (no autograd).
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import numpy as np

from . import sparse


def split_params(arch: str, dims: Sequence[int], params: np.ndarray):
    """Views into the flat parameter vector.  Per layer k (input F_k, output F_{k+1}):
    gcn : W [F_k, F_{k+1}] row-major, then b [F_{k+1}]
    sage: W_self [F_k, F_{k+1}], W_neigh [F_k, F_{k+1}], then b [F_{k+1}]."""
    out, o = [], 0
    for k in range(len(dims) - 1):
        fi, fo = dims[k], dims[k + 1]
        layer = {}
        if arch == "sage":
            layer["W_self"] = params[o:o + fi * fo].reshape(fi, fo); o += fi * fo
            layer["W_neigh"] = params[o:o + fi * fo].reshape(fi, fo); o += fi * fo
        else:
            layer["W"] = params[o:o + fi * fo].reshape(fi, fo); o += fi * fo
        layer["b"] = params[o:o + fo]; o += fo
        out.append(layer)
    assert o == params.shape[0], "parameter vector has the wrong length"
    return out


def encoder_param_count(arch: str, dims: Sequence[int]) -> int:
    return sum((2 if arch == "sage" else 1) * dims[k] * dims[k + 1] + dims[k + 1] for k in range(len(dims) - 1))


def split_predictor(D: int, Hp: int, tail: np.ndarray):
    """Views into the predictor part of the flat parameter vector: W0[D,Hp], b0[Hp], W1[Hp,Hp], b1[Hp], w2[Hp], b2[1]."""
    o = 0
    out = {}
    for name, shape in (("W0", (D, Hp)), ("b0", (Hp,)), ("W1", (Hp, Hp)), ("b1", (Hp,)), ("w2", (Hp,)), ("b2", (1,))):
        size = int(np.prod(shape))
        out[name] = tail[o:o + size].reshape(shape)
        o += size
    assert o == tail.shape[0], "predictor parameters have the wrong length"
    return out


def mlp_predictor_forward(HK, src, dst, pred, ties=None, rounding=None, var_HK=None, n_sigma: float = 6.0):
    """EdgePredictor of Eq. 2 as the 3-layer MLP of the paper's experiments (Section IV) on the Hadamard
    product of the two embeddings: z0 = h_u * h_v; p1 = ReLU(z0 W0 + b0); p2 = ReLU(p1 W1 + b1);
    s = p2 . w2 + b2.  ties = (active1, active2) decisions of the implementation under test, adopted only
    inside the rounding window of the pre-activation (see forward()); var_HK is the rounding-error variance
    of H^(K) that forward() returns under the same rounding model."""
    r = rounding_model(rounding)
    z0 = HK[src] * HK[dst]
    out = {"z0": z0, "ties": 0, "n_near": 0, "near": [], "own_active": [], "window": [], "Z": []}
    V = None
    if r is not None:
        vk = np.zeros_like(HK) if var_HK is None else var_HK
        V = HK[dst] ** 2 * vk[src] + HK[src] ** 2 * vk[dst] + (r["u_store"] * z0) ** 2 / 3.0
    A = z0
    for li, (Wn, bn) in enumerate((("W0", "b0"), ("W1", "b1"))):
        a = A @ pred[Wn] + pred[bn]
        active = a > 0.0
        given = None if ties is None else ties[li]
        if r is not None:
            var = _dense_error_variance([(A, V, pred[Wn])], pred[bn], r)
            active, near, win, flipped = _relu_decisions(a, var, given, n_sigma)
            out["ties"] += flipped
            out["n_near"] += int(near.sum())
            out["near"].append(near)
            out["window"].append(win)
            V = np.where(active, var + (r["u_store"] * a) ** 2 / 3.0, 0.0)
        out["own_active"].append(a > 0.0)
        out["Z"].append(a)
        A = np.where(active, a, 0.0)
        out["p%d" % (li + 1)] = A
        out["active%d" % (li + 1)] = active
    s = out["p2"] @ pred["w2"] + pred["b2"][0]
    return s, out


def mlp_predictor_backward(HK, src, dst, pred, cache, gs):
    """Chain rule through the MLP predictor: returns (gradient dict, dL/dH^(K))."""
    G = {}
    G["w2"] = cache["p2"].T @ gs
    G["b2"] = np.array([gs.sum()])
    dp2 = np.outer(gs, pred["w2"]) * cache["active2"]
    G["W1"] = cache["p1"].T @ dp2
    G["b1"] = dp2.sum(axis=0)
    dp1 = (dp2 @ pred["W1"].T) * cache["active1"]
    G["W0"] = cache["z0"].T @ dp1
    G["b0"] = dp1.sum(axis=0)
    dz0 = dp1 @ pred["W0"].T
    dH = np.zeros_like(HK)
    np.add.at(dH, src, dz0 * HK[dst])
    np.add.at(dH, dst, dz0 * HK[src])
    return G, dH


def _block_as_global_csr(n: int, frontier: np.ndarray, ptr: np.ndarray, cols: np.ndarray):
    counts = np.zeros(n, dtype=np.int64)
    counts[frontier] = np.diff(ptr)
    rowptr = np.zeros(n + 1, dtype=np.int64)
    np.cumsum(counts, out=rowptr[1:])
    return rowptr, cols


def _sampled_gcn_weights(g, frontier: np.ndarray, ptr: np.ndarray, cols: np.ndarray) -> np.ndarray:
    """Per-entry weights of a sampled block for the GCN aggregation: the weight the entry has in
    the loaded graph, times |N(v)| / |S(v)| for its destination v -- every neighbour is drawn
    with probability |S(v)| / |N(v)|, so the sampled sum estimates the full neighbour sum
    without bias.  The normalisation 1 / sqrt(d~_v d~_u) keeps the degrees of the full graph."""
    w = np.zeros(cols.shape[0], dtype=np.float64)
    for i, v in enumerate(frontier):
        lo, hi = int(ptr[i]), int(ptr[i + 1])
        if hi == lo:
            continue
        r0, r1 = int(g.rowptr[v]), int(g.rowptr[v + 1])
        pos = r0 + np.searchsorted(g.col[r0:r1], cols[lo:hi])
        assert np.array_equal(g.col[pos], cols[lo:hi])
        full = np.ones(hi - lo) if g.w is None else g.w[pos].astype(np.float64)
        w[lo:hi] = full * ((r1 - r0) / (hi - lo))
    return w.astype(np.float32)  # the aggregation routine takes float32 weights; the ratio of two small integers times a
    #                              float32 weight is rounded once here


def _layer_graphs(g, n_layers: int, blocks, arch: str = "sage"):
    """Per layer l = 1..K: (rowptr, col, w, active_rows or None, dtilde or None).
    Full-graph training uses the loaded graph at every layer.  With a sampled computational
    graph, layer l works on hop h = K - l + 1: rows F_{h-1} aggregate their sampled neighbours
    (mean over the sample; GCN: rescaled sample with the full graph's degrees, self term exact)."""
    if blocks is None:
        return [(g.rowptr, g.col, g.w, None, None)] * n_layers
    frontiers, blks = blocks
    dt = sparse.gcn_degree(g.n, g.rowptr, g.w) if arch == "gcn" else None
    out = []
    for l in range(1, n_layers + 1):
        h = n_layers - l + 1
        ptr, cols = blks[h - 1]
        rp, cc = _block_as_global_csr(g.n, frontiers[h - 1], ptr, cols)
        w = _sampled_gcn_weights(g, frontiers[h - 1], ptr, cols) if arch == "gcn" else None
        out.append((rp, cc, w, frontiers[h - 1], dt))
    return out


# Unit roundoffs of the two arithmetic paths a checked implementation may take (first-order rounding-error
# model; the unit roundoff of round-to-nearest with p significand bits is 2^-p: 2^-8 for BF16, 2^-24 for FP32):
#   u_in    rounding of the input features X when they are stored          (BF16 path: X is converted)
#   u_store rounding of every stored activation (aggregates, embeddings)
#   u_w     rounding of the weights before the dense transform             (BF16 path: W is converted)
#   u_acc   one addition of the dense transform's accumulator; the tensor-core accumulator is credited with
#           two bits less than FP32 because its additions need not round to nearest
#   u_coef  one FP32 operation on an aggregation coefficient (1/deg, w / sqrt(d~ d~))
ROUNDING = {
    "fp32": {"u_in": 0.0, "u_store": 2.0 ** -24, "u_w": 0.0, "u_acc": 2.0 ** -24, "u_coef": 2.0 ** -24},
    "bf16": {"u_in": 2.0 ** -8, "u_store": 2.0 ** -8, "u_w": 2.0 ** -8, "u_acc": 2.0 ** -22, "u_coef": 2.0 ** -24},
}


def rounding_model(rounding):
    """None, the name of a path in ROUNDING, or a dict with the same keys."""
    if rounding is None:
        return None
    return ROUNDING[rounding] if isinstance(rounding, str) else rounding


def _dense_error_variance(parts, b, r):
    """Variance of the rounding error of Z = sum_i A_i W_i + b computed in finite precision with ONE accumulator
    (parts = [(A_i, VA_i, W_i), ...]), to first order, with every rounding taken as an independent error uniform in
    +-u|x| (variance (u x)^2 / 3):
      errors already in A (variance VA) and the rounding of W pass through the product;
      each of the K additions of the accumulator rounds a partial sum that is at most sum_j |A_j W_j| + |b|."""
    prop, S, K = 0.0, np.abs(b), 0
    for A, VA, W in parts:
        prop = prop + (VA + (r["u_w"] ** 2 / 3.0) * A * A) @ (W * W)
        S = S + np.abs(A) @ np.abs(W)
        K += A.shape[1]
    return prop + K * (r["u_acc"] * S) ** 2 / 3.0


def _aggregate_error_variance(mode, n, rp, cc, w, dt, H, VH, M, r):
    """The same for M = AGG(H): the errors of H pass through with the squared coefficients; the coefficients
    carry three FP32 roundings; the FP32 accumulator rounds deg partial sums bounded by AGG(|H|); the
    result is rounded once more when it is stored."""
    deg = np.diff(rp).astype(np.float64)
    if mode == "gcn":
        w32 = np.ones(cc.shape[0], dtype=np.float32) if w is None else np.asarray(w, dtype=np.float32)
        d1 = sparse.gcn_degree(n, rp, w32) if dt is None else np.asarray(dt, dtype=np.float64)
        prop = sparse.aggregate("gcn", n, rp, cc, (w32.astype(np.float64) ** 2).astype(np.float32), VH, d1 * d1)
        absum = sparse.aggregate("gcn", n, rp, cc, w32, np.abs(H), d1)
        terms = deg + 1.0
    else:
        prop = sparse.aggregate("mean", n, rp, cc, None, VH) / np.maximum(deg, 1.0)[:, None]
        absum = sparse.aggregate("mean", n, rp, cc, None, np.abs(H))
        terms = deg
    return (prop + (3.0 * r["u_coef"] * absum) ** 2 / 3.0 + terms[:, None] * (2.0 ** -24 * absum) ** 2 / 3.0
            + (r["u_store"] * M) ** 2 / 3.0)


def _relu_decisions(Z, var, given, n_sigma, rows=None):
    """The oracle's own decisions Z > 0, and the units whose pre-activation lies within n_sigma standard
    deviations of the modelled rounding error of zero (the window): only there may the decisions `given`
    by the implementation under test replace the oracle's own.  Returns (active, near, window, adopted
    decisions that differ)."""
    own = Z > 0.0
    win = n_sigma * np.sqrt(var)
    near = np.abs(Z) <= win
    if rows is not None:  # rows outside the frontier are not computed at all: nothing to adopt there
        inside = np.zeros(Z.shape[0], dtype=bool)
        inside[rows] = True
        near &= inside[:, None]
    if given is None:
        return own, near, win, 0
    flipped = int((near & (own != given)).sum())
    return np.where(near, given, own), near, win, flipped


def forward(g, X: np.ndarray, params: np.ndarray, arch: str, dims: Sequence[int], blocks=None, relu_ties=None,
            rounding=None, n_sigma: float = 6.0, final_variance: bool = False):
    """K-layer encoder (Eq. 1).  Layer k: A = AGG(H^(k-1)) [gcn] or [H^(k-1) | mean] [sage];
    Z = A W + b; H^(k) = ReLU(Z) for k < K and Z for k = K.  Returns the per-layer cache.

    ReLU turns a floating-point value into a yes/no decision (is the unit active?).  When a
    pre-activation is zero up to the rounding of the arithmetic under test, that arithmetic and
    FP64 may decide differently although both are right.  With `rounding` (a key of ROUNDING or a
    dict of unit roundoffs) the oracle propagates a first-order model of that arithmetic's rounding
    error through the layers (variances of independent roundings) and marks the units with
    |Z| <= n_sigma * sigma(Z) -- cache["near"][k], cache["window"][k].  relu_ties[k] (bool [n, F_{k+1}],
    the decisions of the implementation under test) is adopted ONLY on those units; everywhere else
    the oracle decides by itself (cache["own_active"][k] holds its own decision on every unit, so a
    test can demand equality outside the window).  cache["ties"] counts the adopted decisions that
    differ from the oracle's own, cache["n_near"] the units inside the windows."""
    K = len(dims) - 1
    P = split_params(arch, dims, np.asarray(params, dtype=np.float64))
    H = np.asarray(X, dtype=np.float64)
    r = rounding_model(rounding)
    cache = {"H": [H], "M": [], "Z": [], "active": [], "own_active": [], "near": [], "window": [], "ties": 0, "n_near": 0,
             "var_HK": None, "graphs": _layer_graphs(g, K, blocks, arch)}
    mode = "gcn" if arch == "gcn" else "mean"
    VH = (r["u_in"] * H) ** 2 / 3.0 if r is not None else None
    for k in range(K):
        rp, cc, w, act, dt = cache["graphs"][k]
        M = sparse.aggregate(mode, g.n, rp, cc, w if arch == "gcn" else None, H, dt)
        if arch == "gcn":
            Z = M @ P[k]["W"] + P[k]["b"]
        else:
            Z = H @ P[k]["W_self"] + M @ P[k]["W_neigh"] + P[k]["b"]
        var = None
        if r is not None and (k < K - 1 or final_variance):
            VM = _aggregate_error_variance(mode, g.n, rp, cc, w if arch == "gcn" else None, dt, H, VH, M, r)
            if arch == "gcn":
                var = _dense_error_variance([(M, VM, P[k]["W"])], P[k]["b"], r)
            else:
                var = _dense_error_variance([(H, VH, P[k]["W_self"]), (M, VM, P[k]["W_neigh"])], P[k]["b"], r)
        if k < K - 1:
            active = Z > 0.0
            cache["own_active"].append(active)
            if r is not None:
                given = None if relu_ties is None else relu_ties[k]
                active, near, win, flipped = _relu_decisions(Z, var, given, n_sigma, act)
                cache["ties"] += flipped
                cache["n_near"] += int(near.sum())
                cache["near"].append(near)
                cache["window"].append(win)
            cache["active"].append(active)
            Hn = np.where(active, Z, 0.0)
            if r is not None:
                VH = np.where(active, var + (r["u_store"] * Z) ** 2 / 3.0, 0.0)
        else:
            Hn = Z
            if var is not None:
                cache["var_HK"] = var + (r["u_store"] * Z) ** 2 / 3.0
        if act is not None:  # rows outside the frontier are not part of the computational graph
            keep = np.zeros(g.n, dtype=bool)
            keep[act] = True
            Z = np.where(keep[:, None], Z, 0.0)
            Hn = np.where(keep[:, None], Hn, 0.0)
        cache["M"].append(M)
        cache["Z"].append(Z)
        cache["H"].append(Hn)
        H = Hn
    return cache


def edge_dot(HK: np.ndarray, src: np.ndarray, dst: np.ndarray, chunk: int = 65536) -> np.ndarray:
    """s_e = <h_src(e), h_dst(e)> (Eq. 2 with the dot product), one edge at a time; the edges are taken in slices so that
    the two gathered row blocks stay small whatever the number of scored edges (no sum is split or reordered)."""
    out = np.empty(src.shape[0], dtype=np.float64)
    for lo in range(0, src.shape[0], chunk):
        out[lo:lo + chunk] = np.einsum("ij,ij->i", HK[src[lo:lo + chunk]], HK[dst[lo:lo + chunk]])
    return out


def bce_with_logits(s: np.ndarray, y: np.ndarray):
    """Per-edge binary cross-entropy of label y and probability sigmoid(s), in the
    overflow-free form  max(s,0) - s*y + log(1 + exp(-|s|)), and d/ds = sigmoid(s) - y."""
    ell = np.maximum(s, 0.0) - s * y + np.log1p(np.exp(-np.abs(s)))
    sig = np.where(s >= 0, 1.0 / (1.0 + np.exp(-np.abs(s))), np.exp(-np.abs(s)) / (1.0 + np.exp(-np.abs(s))))
    return ell, sig - y


def train_step(g, X, params, arch, dims, pos_src, pos_dst, neg_src, neg_dst, blocks=None, relu_ties=None, rounding=None,
               pred_hidden: int = 0, pred_ties=None, n_sigma: float = 6.0):
    """One training step of Algorithm 1 for one worker: scores of Eq. 2 (dot product) for
    positives (label 1) and negatives (label 0), loss L = (1/N) sum ell with N = |P| + |N|,
    and the gradient with respect to every parameter in the flat layout."""
    K = len(dims) - 1
    params = np.asarray(params, dtype=np.float64)
    n_enc = encoder_param_count(arch, dims)
    enc_params = params[:n_enc]
    P = split_params(arch, dims, enc_params)
    cache = forward(g, X, enc_params, arch, dims, blocks, relu_ties, rounding, n_sigma, final_variance=pred_hidden > 0)
    HK = cache["H"][K]
    src = np.concatenate([pos_src, neg_src]).astype(np.int32)
    dst = np.concatenate([pos_dst, neg_dst]).astype(np.int32)
    y = np.concatenate([np.ones(len(pos_src)), np.zeros(len(neg_src))])
    pred = pcache = None
    if pred_hidden > 0:
        pred = split_predictor(dims[K], pred_hidden, params[n_enc:])
        s, pcache = mlp_predictor_forward(HK, src, dst, pred, pred_ties, rounding, cache["var_HK"], n_sigma)
    else:
        s = edge_dot(HK, src, dst)
    ell, dls = bce_with_logits(s, y)
    N = s.shape[0]
    loss = ell.sum() / N
    gs = dls / N
    grads_full = np.zeros(params.shape[0], dtype=np.float64)
    if pred_hidden > 0:
        PG, dH = mlp_predictor_backward(HK, src, dst, pred, pcache, gs)
        GP = split_predictor(dims[K], pred_hidden, grads_full[n_enc:])
        for name in GP:
            GP[name][...] = PG[name]
    else:
        dH = sparse.edge_grad(HK, src, dst, gs)
    dHK = dH

    grads = grads_full
    G = split_params(arch, dims, grads[:n_enc])
    mode = "gcn" if arch == "gcn" else "mean"
    for k in range(K - 1, -1, -1):
        rp, cc, w, act, dt = cache["graphs"][k]
        dZ = dH if k == K - 1 else dH * cache["active"][k]
        if act is not None:
            keep = np.zeros(g.n, dtype=bool)
            keep[act] = True
            dZ = np.where(keep[:, None], dZ, 0.0)
        Hprev, M = cache["H"][k], cache["M"][k]
        G[k]["b"][:] = dZ.sum(axis=0)
        if arch == "gcn":
            G[k]["W"][:] = M.T @ dZ
            dM = dZ @ P[k]["W"].T
            dH = sparse.aggregate_backward(mode, g.n, rp, cc, w, dM, dt) if k > 0 else None
        else:
            G[k]["W_self"][:] = Hprev.T @ dZ
            G[k]["W_neigh"][:] = M.T @ dZ
            if k > 0:
                dH = dZ @ P[k]["W_self"].T + sparse.aggregate_backward(mode, g.n, rp, cc, None, dZ @ P[k]["W_neigh"].T)
    return {"loss": loss, "grads": grads, "scores": s, "g": gs, "dHK": dHK,
            "cache": cache, "src": src, "dst": dst, "pred_cache": pcache}


def input_gradient(g, X, params, arch, dims, pos_src, pos_dst, neg_src, neg_dst):
    """dL/dX (not needed for training; used by the finite-difference pin of the backward
    pass through the first layer's aggregation)."""
    K = len(dims) - 1
    P = split_params(arch, dims, np.asarray(params, dtype=np.float64))
    cache = forward(g, X, params, arch, dims)
    HK = cache["H"][K]
    src = np.concatenate([pos_src, neg_src]).astype(np.int32)
    dst = np.concatenate([pos_dst, neg_dst]).astype(np.int32)
    y = np.concatenate([np.ones(len(pos_src)), np.zeros(len(neg_src))])
    s = edge_dot(HK, src, dst)
    _, dls = bce_with_logits(s, y)
    dH = sparse.edge_grad(HK, src, dst, dls / s.shape[0])
    mode = "gcn" if arch == "gcn" else "mean"
    for k in range(K - 1, -1, -1):
        dZ = dH if k == K - 1 else dH * (cache["Z"][k] > 0.0)
        if arch == "gcn":
            dH = sparse.aggregate_backward(mode, g.n, g.rowptr, g.col, g.w, dZ @ P[k]["W"].T)
        else:
            dH = dZ @ P[k]["W_self"].T + sparse.aggregate_backward(mode, g.n, g.rowptr, g.col, None,
                                                                   dZ @ P[k]["W_neigh"].T)
    return dH


def score(g, X, params, arch, dims, src, dst, blocks=None, pred_hidden: int = 0) -> np.ndarray:
    """Edge scores of Eq. 2: <h_u^(K), h_v^(K)> (dot product) or the MLP predictor's output."""
    params = np.asarray(params, dtype=np.float64)
    n_enc = encoder_param_count(arch, dims)
    HK = forward(g, X, params[:n_enc], arch, dims, blocks)["H"][len(dims) - 1]
    if pred_hidden > 0:
        pred = split_predictor(dims[-1], pred_hidden, params[n_enc:])
        return mlp_predictor_forward(HK, np.asarray(src), np.asarray(dst), pred)[0]
    return edge_dot(HK, np.asarray(src), np.asarray(dst))


def hits_at_k(pos_scores, neg_scores, k: int) -> float:
    """Hits@K (Section IV's accuracy metric): the fraction of positive scores that are strictly greater
    than the K-th largest negative score (1.0 when there are fewer than K negatives)."""
    pos = np.asarray(pos_scores, dtype=np.float64)
    neg = np.asarray(neg_scores, dtype=np.float64)
    if neg.shape[0] < k:
        return 1.0
    kth = np.sort(neg)[-k]
    return float((pos > kth).mean())


def average_gradients(grads_per_worker: List[np.ndarray]) -> np.ndarray:
    """Gradient synchronisation of Algorithm 1: (1/p) * sum over the p workers."""
    acc = np.zeros_like(np.asarray(grads_per_worker[0], dtype=np.float64))
    for gi in grads_per_worker:
        acc = acc + np.asarray(gi, dtype=np.float64)
    return acc / len(grads_per_worker)


def adam_step(params, m, v, grads, t: int, lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8):
    """Adam (the optimiser of the paper's experiments, lr 1e-3) with bias correction,
    no weight decay.  t counts from 1.  Returns new (params, m, v) in float64."""
    params = np.asarray(params, dtype=np.float64)
    g = np.asarray(grads, dtype=np.float64)
    m = beta1 * np.asarray(m, dtype=np.float64) + (1.0 - beta1) * g
    v = beta2 * np.asarray(v, dtype=np.float64) + (1.0 - beta2) * g * g
    mhat = m / (1.0 - beta1 ** t)
    vhat = v / (1.0 - beta2 ** t)
    return params - lr * mhat / (np.sqrt(vhat) + eps), m, v
