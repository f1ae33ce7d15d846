"""Independent dense brute-force restatements used to pin the oracle (numpy, FP64, n <= a few hundred)
and small utilities shared by the tests.  Nothing here is used by the library or by the oracle."""
import numpy as np


def dense_adjacency(g):
    """A[v, u] = weight of stored entry (v <- u)."""
    A = np.zeros((g.n, g.n))
    for v in range(g.n):
        for e in range(g.rowptr[v], g.rowptr[v + 1]):
            A[v, g.col[e]] += 1.0 if g.w is None else float(g.w[e])
    return A


def dense_gcn_operator(g):
    At = dense_adjacency(g) + np.eye(g.n)
    d = At.sum(axis=1)
    return At / np.sqrt(np.outer(d, d))


def dense_mean_operator(g):
    A = (dense_adjacency(g) > 0).astype(np.float64)
    deg = A.sum(axis=1)
    S = np.zeros_like(A)
    nzr = deg > 0
    S[nzr] = A[nzr] / deg[nzr, None]
    return S


def dense_forward(g, X, params, arch, dims, op=None):
    """Encoder with a dense aggregation operator; returns H^(K) and the list of pre-activations."""
    S = op if op is not None else (dense_gcn_operator(g) if arch == "gcn" else dense_mean_operator(g))
    H = np.asarray(X, dtype=np.float64)
    o, Zs = 0, []
    p = np.asarray(params, dtype=np.float64)
    K = len(dims) - 1
    for k in range(K):
        fi, fo = dims[k], dims[k + 1]
        if arch == "sage":
            Ws = p[o:o + fi * fo].reshape(fi, fo); o += fi * fo
            Wn = p[o:o + fi * fo].reshape(fi, fo); o += fi * fo
            b = p[o:o + fo]; o += fo
            Z = H @ Ws + (S @ H) @ Wn + b
        else:
            W = p[o:o + fi * fo].reshape(fi, fo); o += fi * fo
            b = p[o:o + fo]; o += fo
            Z = (S @ H) @ W + b
        Zs.append(Z)
        H = np.maximum(Z, 0) if k < K - 1 else Z
    return H, Zs


def dense_loss(g, X, params, arch, dims, src, dst, y):
    H, _ = dense_forward(g, X, params, arch, dims)
    s = (H[src] * H[dst]).sum(axis=1)
    # -[y log sigma(s) + (1-y) log(1 - sigma(s))] written with logaddexp
    return float(np.mean(y * np.logaddexp(0.0, -s) + (1 - y) * np.logaddexp(0.0, s)))


def rel_l2(a, b):
    a = np.asarray(a, dtype=np.float64).ravel()
    b = np.asarray(b, dtype=np.float64).ravel()
    den = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / den) if den > 0 else float(np.linalg.norm(a - b))
