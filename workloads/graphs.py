"""Seeded graph / feature / parameter generators (numpy only).

Shapes follow the paper's workloads (Table I: citation-, co-authorship- and
protein-association-scale graphs with 58..128-d features) but every record is
synthetic: the public datasets themselves are not used anywhere.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, Optional, Tuple

import numpy as np


@dataclass
class Graph:
    """CSR by destination: row v lists the in-neighbours of v (sorted, unique)."""

    n: int
    rowptr: np.ndarray  # int64 [n+1]
    col: np.ndarray  # int32 [nnz]
    w: Optional[np.ndarray] = None  # float32 [nnz] or None (all ones)
    directed: bool = False
    meta: Dict = field(default_factory=dict)

    @property
    def nnz(self) -> int:
        return int(self.col.shape[0])


def csr_from_edges(n: int, dst: np.ndarray, src: np.ndarray, w: Optional[np.ndarray] = None, presorted: bool = False) -> Graph:
    """Build CSR (rows = dst, cols = src) from a list of distinct directed entries
    (presorted: the list is already ordered by (dst, src), so the sort is skipped)."""
    dst = np.asarray(dst, dtype=np.int64)
    src = np.asarray(src, dtype=np.int64)
    if presorted:
        order = slice(None)
    else:
        order = np.lexsort((src, dst))
        dst, src = dst[order], src[order]
    counts = np.bincount(dst, minlength=n).astype(np.int64)
    rowptr = np.zeros(n + 1, dtype=np.int64)
    np.cumsum(counts, out=rowptr[1:])
    ww = None if w is None else np.ascontiguousarray(np.asarray(w, dtype=np.float32)[order])
    return Graph(n=n, rowptr=rowptr, col=np.ascontiguousarray(src.astype(np.int32)), w=ww)


def _symmetrise(n: int, a: np.ndarray, b: np.ndarray, w: Optional[np.ndarray] = None) -> Graph:
    """Undirected edge list {a,b} (distinct, a != b) -> symmetric CSR."""
    dst = np.concatenate([a, b])
    src = np.concatenate([b, a])
    ww = None if w is None else np.concatenate([w, w])
    g = csr_from_edges(n, dst, src, ww)
    g.directed = False
    return g


def undirected_edge_list(g: Graph) -> Tuple[np.ndarray, np.ndarray]:
    """Each undirected edge of a symmetric CSR once, as (u, v) with u < v, in row order."""
    rows = np.repeat(np.arange(g.n, dtype=np.int64), np.diff(g.rowptr))
    keep = g.col.astype(np.int64) > rows  # (v=row, u=col) with u > v  -> pair (row, col)
    return rows[keep].astype(np.int32), g.col[keep].astype(np.int32)


def _dedupe_pairs(n: int, a: np.ndarray, b: np.ndarray):
    """Drop self pairs, order each pair (lo, hi), return unique keys and multiplicities."""
    keep = a != b
    a, b = a[keep], b[keep]
    lo = np.minimum(a, b).astype(np.int64)
    hi = np.maximum(a, b).astype(np.int64)
    key = lo * n + hi
    ukey, first, mult = np.unique(key, return_index=True, return_counts=True)
    return ukey, first, mult


def erdos_renyi(n: int, m: int, seed: int) -> Graph:
    """G(n, m): exactly m distinct undirected edges, uniform, no self-loops."""
    rng = np.random.Generator(np.random.PCG64(seed))
    have = np.zeros(0, dtype=np.int64)
    while have.shape[0] < m:
        need = m - have.shape[0]
        a = rng.integers(0, n, size=int(need * 1.2) + 16)
        b = rng.integers(0, n, size=a.shape[0])
        keep = a != b
        lo = np.minimum(a, b)[keep].astype(np.int64)
        hi = np.maximum(a, b)[keep].astype(np.int64)
        key = lo * n + hi
        # keep first occurrences in draw order so the result depends on the seed only
        allk = np.concatenate([have, key])
        _, first = np.unique(allk, return_index=True)
        allk = allk[np.sort(first)]
        have = allk[:m]
    g = _symmetrise(n, (have // n), (have % n))
    g.meta = {"family": "erdos_renyi", "seed": seed, "undirected_edges": m}
    return g


def _power_law_weights(n: int, gamma: float, mean_deg: float) -> np.ndarray:
    """Expected degrees w_i ~ (i + i0)^(-1/(gamma-1)), scaled to the mean, capped at sqrt(sum w)."""
    i0 = 10.0
    w = (np.arange(n, dtype=np.float64) + i0) ** (-1.0 / (gamma - 1.0))
    w *= mean_deg * n / w.sum()
    for _ in range(8):  # cap + rescale until stable
        cap = np.sqrt(w.sum())
        w = np.minimum(w, cap)
        w *= mean_deg * n / w.sum()
    return w


def _draw_weighted(rng, cdf: np.ndarray, size: int) -> np.ndarray:
    return np.searchsorted(cdf, rng.random(size) * cdf[-1], side="right").clip(0, cdf.shape[0] - 1)


def chung_lu(n: int, mean_deg: float, gamma: float, seed: int, shuffle_ids: bool = True) -> Graph:
    """Chung-Lu power-law graph: m = n*mean_deg/2 endpoint pairs drawn proportional to w_i*w_j,
    self-loops dropped, duplicates merged (so the edge count is slightly below m)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    w = _power_law_weights(n, gamma, mean_deg)
    cdf = np.cumsum(w)
    m = int(round(n * mean_deg / 2.0))
    a = _draw_weighted(rng, cdf, m)
    b = _draw_weighted(rng, cdf, m)
    if shuffle_ids:  # hubs should not sit at the low ids
        relabel = rng.permutation(n)
        a, b = relabel[a], relabel[b]
    ukey, _, _ = _dedupe_pairs(n, a, b)
    g = _symmetrise(n, ukey // n, ukey % n)
    g.meta = {"family": "chung_lu", "seed": seed, "gamma": gamma, "mean_deg": mean_deg,
              "undirected_edges": int(ukey.shape[0])}
    return g


def coauthor_weighted(n: int, m_distinct: int, seed: int, gamma: float = 2.3) -> Graph:
    """Power-law graph with about m_distinct distinct undirected edges; each edge carries an
    integer weight in 1..5 (truncated geometric, ratio 1/2) standing for repeated co-authorship."""
    rng = np.random.Generator(np.random.PCG64(seed))
    mean_deg = 2.0 * m_distinct / n
    w = _power_law_weights(n, gamma, mean_deg * 1.03)
    cdf = np.cumsum(w)
    m = int(round(n * mean_deg * 1.03 / 2.0))
    a = _draw_weighted(rng, cdf, m)
    b = _draw_weighted(rng, cdf, m)
    relabel = rng.permutation(n)
    a, b = relabel[a], relabel[b]
    ukey, _, _ = _dedupe_pairs(n, a, b)
    if ukey.shape[0] > m_distinct:
        ukey = np.sort(rng.choice(ukey, size=m_distinct, replace=False))
    p = 0.5 ** np.arange(1, 6)
    p /= p.sum()
    mult = rng.choice(np.arange(1, 6), size=ukey.shape[0], p=p).astype(np.float32)
    g = _symmetrise(n, ukey // n, ukey % n, mult)
    g.meta = {"family": "coauthor_weighted", "seed": seed, "undirected_edges": int(ukey.shape[0])}
    return g


def citation_directed(n: int, m: int, gamma_in: float, seed: int) -> Graph:
    """Directed graph: destination drawn proportional to a power-law in-weight, source uniform.
    Entry (v <- u) is stored in row v.  Duplicates and self-loops dropped."""
    rng = np.random.Generator(np.random.PCG64(seed))
    w = _power_law_weights(n, gamma_in, m / n)
    cdf = np.cumsum(w)
    relabel = rng.permutation(n)
    dst = relabel[_draw_weighted(rng, cdf, m)].astype(np.int64)
    src = rng.integers(0, n, size=m).astype(np.int64)
    keep = dst != src
    key = np.sort(dst[keep] * n + src[keep])  # ascending (dst, src); duplicates are neighbours
    key = key[np.concatenate([[True], key[1:] != key[:-1]])]
    g = csr_from_edges(n, key // n, key % n, presorted=True)
    g.directed = True
    g.meta = {"family": "citation_directed", "seed": seed, "gamma_in": gamma_in, "entries": g.nnz}
    return g


def node_features(n: int, f: int, seed: int) -> np.ndarray:
    """X[n, f] float32 ~ N(0, 1), row-major (row v = x_v)."""
    rng = np.random.Generator(np.random.PCG64(seed + 7919))
    return rng.standard_normal((n, f), dtype=np.float32)


def model_dims_param_count(arch: str, dims, pred_hidden: int = 0) -> int:
    """Flat parameter layout: per layer W_self? / W then bias.
    gcn : W[in,out] row-major, b[out]
    sage: W_self[in,out], W_neigh[in,out] (both row-major), b[out]
    With an MLP edge predictor (pred_hidden > 0) three more layers follow the encoder:
    W0[D, Hp], b0[Hp], W1[Hp, Hp], b1[Hp], w2[Hp], b2[1]  (D = dims[-1], Hp = pred_hidden)."""
    total = 0
    for k in range(len(dims) - 1):
        fi, fo = dims[k], dims[k + 1]
        total += (2 if arch == "sage" else 1) * fi * fo + fo
    if pred_hidden > 0:
        D, Hp = dims[-1], pred_hidden
        total += D * Hp + Hp + Hp * Hp + Hp + Hp + 1
    return total


def glorot_params(arch: str, dims, seed: int, bias_scale: float = 0.0, pred_hidden: int = 0) -> np.ndarray:
    """Glorot-uniform weights in the flat layout; biases zero unless bias_scale > 0
    (non-zero biases make parity tests sensitive to the bias path)."""
    rng = np.random.Generator(np.random.PCG64(seed + 104729))
    parts = []
    for k in range(len(dims) - 1):
        fi, fo = dims[k], dims[k + 1]
        lim = np.sqrt(6.0 / (fi + fo))
        for _ in range(2 if arch == "sage" else 1):
            parts.append(rng.uniform(-lim, lim, size=fi * fo).astype(np.float32))
        parts.append((bias_scale * rng.standard_normal(fo)).astype(np.float32))
    if pred_hidden > 0:
        for fi, fo in ((dims[-1], pred_hidden), (pred_hidden, pred_hidden), (pred_hidden, 1)):
            lim = np.sqrt(6.0 / (fi + fo))
            parts.append(rng.uniform(-lim, lim, size=fi * fo).astype(np.float32))
            parts.append((bias_scale * rng.standard_normal(fo)).astype(np.float32))
    return np.concatenate(parts)


def edge_split(g: Graph, fractions, seed: int):
    """Random split of the undirected edges of a symmetric graph.  Returns a list of
    (u, v, w) triples, one per fraction, with u < v."""
    rng = np.random.Generator(np.random.PCG64(seed + 15485863))
    rows = np.repeat(np.arange(g.n, dtype=np.int64), np.diff(g.rowptr))
    keep = g.col.astype(np.int64) > rows
    u, v = rows[keep], g.col[keep].astype(np.int64)
    w = None if g.w is None else g.w[keep]
    perm = rng.permutation(u.shape[0])
    cuts = np.floor(np.cumsum(fractions) * u.shape[0]).astype(np.int64)
    cuts[-1] = u.shape[0]
    out, lo = [], 0
    for hi in cuts:
        idx = np.sort(perm[lo:hi])
        out.append((u[idx], v[idx], None if w is None else w[idx]))
        lo = hi
    return out


def graph_from_undirected(n: int, u, v, w=None) -> Graph:
    return _symmetrise(n, np.asarray(u, dtype=np.int64), np.asarray(v, dtype=np.int64), w)


def random_partition(n: int, p: int, seed: int) -> np.ndarray:
    """Independent uniform node -> partition assignment (int32 [n])."""
    rng = np.random.Generator(np.random.PCG64(seed + 32452843))
    return rng.integers(0, p, size=n).astype(np.int32)


def induced_subgraph(g: Graph, mask: np.ndarray) -> Graph:
    """Keep entries whose row and column are both in the node mask; node ids unchanged
    (nodes outside the mask become isolated rows)."""
    rows = np.repeat(np.arange(g.n, dtype=np.int64), np.diff(g.rowptr))
    keep = mask[rows] & mask[g.col]
    sub = csr_from_edges(g.n, rows[keep], g.col[keep].astype(np.int64), None if g.w is None else g.w[keep])
    sub.directed = g.directed
    return sub


# ----------------------------------------------------------------------------------------
# The five workload configurations (scale < 1 shrinks node and edge counts proportionally;
# tests use scaled copies that the CPU oracle finishes in seconds).
# ----------------------------------------------------------------------------------------
CONFIGS = {
    "c1_tiny_er_gcn2": dict(arch="gcn", dims=[64, 64, 64], prec="fp32", n=2000, batch=None),
    "c2_chunglu_sage2": dict(arch="sage", dims=[128, 256, 256], prec="bf16", n=200_000, batch=65536),
    "c3_coauthor_gcn3": dict(arch="gcn", dims=[128, 256, 256, 256], prec="fp32", n=235_000, batch=None),
    "c4_citation_sage3_sampled": dict(arch="sage", dims=[128, 256, 256, 256], prec="bf16", n=2_900_000,
                                      batch=65536, fanout=[15, 10, 5]),
    "c5_partitioned_sage2": dict(arch="sage", dims=[128, 256, 256], prec="bf16", n=1_000_000, batch=65536,
                                 partitions=8, alpha=0.2),
}


def make_config(name: str, scale: float = 1.0):
    """Return (graph, X, params, positives(u,v), info) for a named configuration."""
    cfg = dict(CONFIGS[name])
    n = max(64, int(round(cfg["n"] * scale)))
    arch, dims = cfg["arch"], cfg["dims"]
    if name == "c1_tiny_er_gcn2":
        g = erdos_renyi(n, 10 * n, seed=0)
        pos = undirected_edge_list(g)
        seed = 0
    elif name == "c2_chunglu_sage2":
        g = chung_lu(n, 20.0, 2.1, seed=2)
        pos = undirected_edge_list(g)
        seed = 2
    elif name == "c3_coauthor_gcn3":
        full = coauthor_weighted(n, int(round(1_300_000 * n / 235_000)), seed=3)
        train, _val, _test = edge_split(full, [0.85, 0.10, 0.05], seed=3)
        g = graph_from_undirected(n, train[0], train[1], train[2])
        g.meta = dict(full.meta, split="85/10/5", undirected_edges=int(train[0].shape[0]))
        pos = (train[0].astype(np.int32), train[1].astype(np.int32))
        seed = 3
    elif name == "c4_citation_sage3_sampled":
        g = citation_directed(n, int(round(30_000_000 * n / 2_900_000)), 2.2, seed=4)
        rows = np.repeat(np.arange(g.n, dtype=np.int32), np.diff(g.rowptr))
        pos = (g.col.copy(), rows)  # (source u, destination v) for every stored entry v <- u
        seed = 4
    elif name == "c5_partitioned_sage2":
        g = chung_lu(n, 16.0, 2.1, seed=5)
        pos = undirected_edge_list(g)
        seed = 5
    else:
        raise KeyError(name)
    X = node_features(g.n, dims[0], seed)
    params = glorot_params(arch, dims, seed, bias_scale=0.05)
    cfg.update(n=g.n, nnz=g.nnz, seed=seed, scale=scale)
    return g, X, params, pos, cfg
