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


def assert_relu_decisions_agree(cache, gpu_masks, rows_per_layer=None, label=""):
    """ReLU is the one place where floating point decides a yes/no.  `cache` is the oracle's forward cache computed
    with a rounding model: outside the rounding window of a pre-activation the decision is unique, so the decisions of
    the implementation under test (`gpu_masks[k]`, bool [n, F]) must equal the oracle's OWN decisions there, bit for
    bit; inside the window either decision is valid.  The number of units inside the window is bounded by what a window
    of that width can hold: a pre-activation with standard deviation s has density at most 0.4 / s at zero, so a unit
    falls within +-w of zero with probability about 0.8 w / s (twice that, plus 16, is allowed).
    Returns (units inside the windows, adopted decisions that differ from the oracle's own)."""
    inside = differ = 0
    for k, gm in enumerate(gpu_masks):
        own, near, win, Z = cache["own_active"][k], cache["near"][k], cache["window"][k], cache["Z"][k]
        if rows_per_layer is not None:
            r = rows_per_layer[k]
            gm, own, near, win, Z = gm[r], own[r], near[r], win[r], Z[r]
        wrong = (gm != own) & ~near
        assert not wrong.any(), f"{label} layer {k + 1}: {int(wrong.sum())} ReLU decisions differ outside the rounding window"
        s = np.sqrt(np.mean(Z * Z))
        capacity = 16 + 2.0 * float(np.minimum(1.0, 0.8 * win / s).sum()) if s > 0 else 16
        assert near.sum() <= capacity, f"{label} layer {k + 1}: {int(near.sum())} units inside the window, a window of this width holds {capacity:.0f}"
        inside += int(near.sum())
        differ += int((near & (gm != own)).sum())
    print(f"{label} ReLU windows: {inside} units inside, {differ} decisions adopted from the implementation under test")
    return inside, differ
