"""ctypes wrappers over oracle/lp_oracle.c (sparse and integer parts of the oracle).

TEST INFRASTRUCTURE ONLY -- see oracle/__init__.py.
"""
from __future__ import annotations

import ctypes as C
from typing import List, Optional, Tuple

import numpy as np

from .build import lib


def _p(a: Optional[np.ndarray], ty):
    if a is None:
        return None
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(C.POINTER(ty))


def _i64(a):
    return np.ascontiguousarray(a, dtype=np.int64)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def philox4x32_10(ctr, key) -> np.ndarray:
    """Philox4x32-10 block function: 4 counter words, 2 key words -> 4 output words."""
    c = np.ascontiguousarray(ctr, dtype=np.uint32)
    k = np.ascontiguousarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    lib().orc_philox4x32_10(_p(c, C.c_uint32), _p(k, C.c_uint32), _p(out, C.c_uint32))
    return out


def csc_transpose(n: int, rowptr, col) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Stable transpose of a CSR: (colptr[n+1], rowidx[nnz], perm[nnz])."""
    rowptr, col = _i64(rowptr), _i32(col)
    nnz = int(col.shape[0])
    colptr = np.zeros(n + 1, dtype=np.int64)
    rowidx = np.zeros(nnz, dtype=np.int32)
    perm = np.zeros(nnz, dtype=np.int64)
    f = lib().orc_csc_transpose
    f.restype = C.c_int
    rc = f(C.c_int64(n), C.c_int64(nnz), _p(rowptr, C.c_int64), _p(col, C.c_int32),
           _p(colptr, C.c_int64), _p(rowidx, C.c_int32), _p(perm, C.c_int64))
    if rc != 0:
        raise ValueError("invalid CSR")
    return colptr, rowidx, perm


def gcn_degree(n: int, rowptr, w) -> np.ndarray:
    """d~_v = 1 + sum_u w_vu (self-loop of weight 1 added to every node)."""
    rowptr = _i64(rowptr)
    w = None if w is None else np.ascontiguousarray(w, dtype=np.float32)
    out = np.zeros(n, dtype=np.float64)
    lib().orc_gcn_degree(C.c_int64(n), _p(rowptr, C.c_int64), _p(w, C.c_float), _p(out, C.c_double))
    return out


_MODE = {"gcn": 0, "mean": 1, "sage": 1}


def aggregate(mode: str, n: int, rowptr, col, w, H: np.ndarray, dtilde=None) -> np.ndarray:
    """AGG of Eq. 1 over every row: 'gcn' (renormalised adjacency) or 'mean'.
    dtilde: the GCN degrees to normalise with; by default those of the structure given
    (a sampled block passes the degrees of the full graph)."""
    rowptr, col = _i64(rowptr), _i32(col)
    w = None if w is None else np.ascontiguousarray(w, dtype=np.float32)
    H = np.ascontiguousarray(H, dtype=np.float64)
    F = H.shape[1]
    dt = None
    if _MODE[mode] == 0:
        dt = gcn_degree(n, rowptr, w) if dtilde is None else np.ascontiguousarray(dtilde, dtype=np.float64)
    M = np.zeros((n, F), dtype=np.float64)
    lib().orc_aggregate(C.c_int(_MODE[mode]), C.c_int64(n), _p(rowptr, C.c_int64), _p(col, C.c_int32),
                        _p(w, C.c_float), _p(dt, C.c_double), _p(H, C.c_double), C.c_int64(F), _p(M, C.c_double))
    return M


def aggregate_backward(mode: str, n: int, rowptr, col, w, dM: np.ndarray, dtilde=None) -> np.ndarray:
    """Gradient of AGG with respect to its input embeddings (scatter form)."""
    rowptr, col = _i64(rowptr), _i32(col)
    w = None if w is None else np.ascontiguousarray(w, dtype=np.float32)
    dM = np.ascontiguousarray(dM, dtype=np.float64)
    F = dM.shape[1]
    dt = None
    if _MODE[mode] == 0:
        dt = gcn_degree(n, rowptr, w) if dtilde is None else np.ascontiguousarray(dtilde, dtype=np.float64)
    dH = np.zeros((n, F), dtype=np.float64)
    lib().orc_aggregate_backward(C.c_int(_MODE[mode]), C.c_int64(n), _p(rowptr, C.c_int64), _p(col, C.c_int32),
                                 _p(w, C.c_float), _p(dt, C.c_double), _p(dM, C.c_double), C.c_int64(F),
                                 _p(dH, C.c_double))
    return dH


def sample_negatives(n: int, rowptr, col, pos_src, seed: int, step: int, k: int = 1, mode: str = "per_source",
                     cand=None, reject_edges: bool = True, max_attempts: int = 8, edge_index_base: int = 0):
    """Uniform negatives.  Returns (neg_src[B*k], neg_dst[B*k], n_exhausted)."""
    rowptr, col, pos_src = _i64(rowptr), _i32(col), _i32(pos_src)
    B = int(pos_src.shape[0])
    cand = None if cand is None else _i32(cand)
    neg_src = np.zeros(B * k, dtype=np.int32)
    neg_dst = np.zeros(B * k, dtype=np.int32)
    exhausted = C.c_int64(0)
    lib().orc_sample_negatives(
        C.c_int64(n), _p(rowptr, C.c_int64), _p(col, C.c_int32), _p(cand, C.c_int32),
        C.c_int64(0 if cand is None else cand.shape[0]), C.c_uint64(seed), C.c_uint64(step), C.c_int32(k),
        C.c_int32(0 if mode == "per_source" else 1), C.c_int32(int(reject_edges)), C.c_int32(max_attempts),
        _p(pos_src, C.c_int32), C.c_int64(B), C.c_int64(edge_index_base),
        _p(neg_src, C.c_int32), _p(neg_dst, C.c_int32), C.byref(exhausted))
    return neg_src, neg_dst, int(exhausted.value)


def edge_grad(H: np.ndarray, src, dst, g: np.ndarray) -> np.ndarray:
    """dL/dH^(K) from per-edge score gradients g (dot-product predictor)."""
    H = np.ascontiguousarray(H, dtype=np.float64)
    src, dst = _i32(src), _i32(dst)
    g = np.ascontiguousarray(g, dtype=np.float64)
    dH = np.zeros_like(H)
    lib().orc_edge_grad(C.c_int64(H.shape[0]), C.c_int64(H.shape[1]), _p(H, C.c_double), C.c_int64(src.shape[0]),
                        _p(src, C.c_int32), _p(dst, C.c_int32), _p(g, C.c_double), _p(dH, C.c_double))
    return dH


def sample_neighbors(rowptr, col, frontier, fanout: int, seed: int, step: int, hop: int):
    """One hop of node-wise neighbour sampling: (ptr[len(frontier)+1], cols global ids)."""
    rowptr, col, frontier = _i64(rowptr), _i32(col), _i32(frontier)
    nf = int(frontier.shape[0])
    out_ptr = np.zeros(nf + 1, dtype=np.int64)
    out_col = np.zeros(max(1, nf * fanout), dtype=np.int32)
    lib().orc_sample_neighbors(_p(rowptr, C.c_int64), _p(col, C.c_int32), C.c_uint64(seed), C.c_uint64(step),
                               C.c_int32(hop), C.c_int32(fanout), _p(frontier, C.c_int32), C.c_int64(nf),
                               _p(out_ptr, C.c_int64), _p(out_col, C.c_int32))
    return out_ptr, out_col[: out_ptr[-1]].copy()


def build_blocks(n: int, rowptr, col, seeds, fanouts: List[int], seed: int, step: int):
    """Computational graph of a batch (Section II-B): hop h = 1..K samples fanouts[h-1]
    in-neighbours of every node of frontier F_{h-1}; F_h = sorted-unique(F_{h-1} u sampled);
    F_0 = sorted-unique(seeds).  Returns (frontiers [F_0..F_K], blocks) where blocks[h-1] =
    (ptr over F_{h-1}, cols as global ids)."""
    frontiers = [np.unique(np.asarray(seeds, dtype=np.int32))]
    blocks = []
    for h, fan in enumerate(fanouts, start=1):
        ptr, cols = sample_neighbors(rowptr, col, frontiers[-1], fan, seed, step, h)
        blocks.append((ptr, cols))
        frontiers.append(np.unique(np.concatenate([frontiers[-1], cols])).astype(np.int32))
    return frontiers, blocks


def sparsify(n: int, rowptr, col, alpha: float, seed: int) -> np.ndarray:
    """Algorithm 1, sparsification block, with L = floor(alpha * |E|) draws (|E| = number
    of undirected edges).  Returns the accumulated weight of every stored entry (0 = dropped)."""
    rowptr, col = _i64(rowptr), _i32(col)
    nnz = int(col.shape[0])
    L = int(np.floor(alpha * (nnz // 2)))
    wsum = np.zeros(nnz, dtype=np.float64)
    lib().orc_sparsify(C.c_int64(n), _p(rowptr, C.c_int64), _p(col, C.c_int32), C.c_uint64(seed), C.c_int64(L),
                       _p(wsum, C.c_double))
    return wsum


def sparsified_graph(n: int, rowptr, col, alpha: float, seed: int):
    """The sparsified graph as CSR (rowptr, col, w float32): entries with non-zero weight."""
    rowptr = _i64(rowptr)
    wsum = sparsify(n, rowptr, col, alpha, seed)
    keep = wsum > 0
    rows = np.repeat(np.arange(n, dtype=np.int64), np.diff(rowptr))
    counts = np.bincount(rows[keep], minlength=n)
    new_ptr = np.zeros(n + 1, dtype=np.int64)
    np.cumsum(counts, out=new_ptr[1:])
    return new_ptr, _i32(col)[keep].copy(), wsum[keep].astype(np.float32)


def worker_view(n: int, rowptr, col, part, worker: int, keep_cross_edges: bool = True, foreign_mode: int = 1, sparsified=None):
    """Graph that one worker trains on (Section III; Algorithm 1's use of G^i and the shared sparsified
    subgraphs): own rows (part[v] == worker) keep every neighbour (full-neighbour partition) or only
    neighbours of the same partition (node-induced subgraph); foreign rows are empty (foreign_mode 0), taken
    from the sparsified graph `sparsified = (rowptr, col)` (1) or kept in full (2).
    Returns (rowptr int64, col int32, stats)."""
    rowptr, col = _i64(rowptr), _i32(col)
    part = np.asarray(part)
    rows = np.repeat(np.arange(n, dtype=np.int64), np.diff(rowptr))
    own_row = part[rows] == worker
    keep = own_row if keep_cross_edges else (own_row & (part[col] == worker))
    out_rows, out_cols = [rows[keep]], [col[keep].astype(np.int64)]
    own_entries = int(keep.sum())
    foreign_entries = 0
    foreign_rows = 0
    if foreign_mode == 1:
        sp_ptr, sp_col = _i64(sparsified[0]), _i32(sparsified[1])
        srows = np.repeat(np.arange(n, dtype=np.int64), np.diff(sp_ptr))
        f = part[srows] != worker
        out_rows.append(srows[f]); out_cols.append(sp_col[f].astype(np.int64))
        foreign_entries = int(f.sum()); foreign_rows = int(np.unique(srows[f]).shape[0])
    elif foreign_mode == 2:
        f = ~own_row
        out_rows.append(rows[f]); out_cols.append(col[f].astype(np.int64))
        foreign_entries = int(f.sum()); foreign_rows = int(np.unique(rows[f]).shape[0])
    r = np.concatenate(out_rows); c = np.concatenate(out_cols)
    order = np.lexsort((c, r))
    r, c = r[order], c[order]
    ptr = np.zeros(n + 1, dtype=np.int64)
    np.cumsum(np.bincount(r, minlength=n), out=ptr[1:])
    stats = {"own_entries": own_entries, "foreign_entries": foreign_entries, "foreign_rows": foreign_rows,
             "own_nodes": int((part == worker).sum())}
    return ptr, c.astype(np.int32), stats
