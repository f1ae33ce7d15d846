"""Thin ctypes binding of the C ABI in include/lp.h.

Argument marshalling only: every step of the path runs inside liblp_b200.so.  torch is used
for device memory and streams.  There is no CPU fall-back: if the library is missing or no
B200 is present, calls raise.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "liblp_b200.so")

LP_OK = 0
LP_GCN, LP_SAGE_MEAN = 0, 1
LP_FP32, LP_BF16 = 0, 1
LP_NEG_PER_SOURCE, LP_NEG_GLOBAL_PAIR = 0, 1
LP_MAX_LAYERS = 4

STATUS_NAMES = {0: "LP_OK", -1: "LP_EINVAL", -2: "LP_ESTATE", -3: "LP_ENOMEM", -4: "LP_ECUDA",
                -5: "LP_EUNSUPPORTED", -6: "LP_ETIMEOUT"}

EXPORTS = [
    "lp_create", "lp_destroy", "lp_last_error", "lp_load_graph", "lp_get_structure", "lp_set_model",
    "lp_param_count", "lp_set_candidates", "lp_sample_negatives", "lp_train_step", "lp_train_step_host",
    "lp_adam_step", "lp_score", "lp_get_embeddings", "lp_get_output_gradient", "lp_get_block",
    "lp_get_stats", "lp_op_aggregate", "lp_op_gather_ceiling", "lp_op_linear", "lp_op_weight_grad", "lp_profile_begin", "lp_profile_end", "lp_profile_sample_every",
    "lp_weight_grad_static", "lp_sparsify", "lp_get_sparsified",
    "lp_worker_view", "lp_get_worker_view", "lp_hits_at_k", "lp_get_predictor_activations",
    "lp_invalidate_embeddings", "lp_set_wait_limit",
]

PROF_CATEGORIES = ["agg_fwd", "agg_bwd", "gemm_fwd", "gemm_dgrad", "gemm_wgrad", "score", "incidence", "scatter",
                   "negatives", "blocks", "adam"]


class LpError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{STATUS_NAMES.get(status, status)}: {message}")
        self.status = status


class ModelDesc(C.Structure):
    _fields_ = [("arch", C.c_int32), ("n_layers", C.c_int32), ("dims", C.c_int32 * (LP_MAX_LAYERS + 1)),
                ("prec", C.c_int32), ("fanout", C.c_int32 * LP_MAX_LAYERS), ("reject_edges", C.c_int32),
                ("max_attempts", C.c_int32), ("cache_input_aggregation", C.c_int32), ("predictor", C.c_int32),
                ("pred_hidden", C.c_int32)]


class Stats(C.Structure):
    _fields_ = [("negatives_exhausted", C.c_int64), ("block_nodes", C.c_int64 * (LP_MAX_LAYERS + 1)),
                ("block_edges", C.c_int64 * LP_MAX_LAYERS), ("workspace_bytes", C.c_int64),
                ("kernel_launches", C.c_int64)]


class ViewStats(C.Structure):
    _fields_ = [("own_entries", C.c_int64), ("foreign_entries", C.c_int64), ("foreign_rows", C.c_int64), ("own_nodes", C.c_int64)]


class Profile(C.Structure):
    _fields_ = [("ms", C.c_double * 11), ("bytes", C.c_double * 11), ("flops", C.c_double * 11), ("spans", C.c_int64 * 11)]


_lib = None


def load_library() -> C.CDLL:
    """dlopen the in-tree library (raises if it has not been built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise FileNotFoundError(f"{_LIB_PATH} is missing: build it with paper_2506_20818_b200.build.build()")
        lib = C.CDLL(_LIB_PATH)
        lib.lp_last_error.restype = C.c_char_p
        lib.lp_last_error.argtypes = [C.c_void_p]
        lib.lp_destroy.restype = None
        lib.lp_destroy.argtypes = [C.c_void_p]
        for name in EXPORTS:
            if name not in ("lp_last_error", "lp_destroy"):
                getattr(lib, name).restype = C.c_int
        _lib = lib
    return _lib


def _ptr(t):
    """Device (or host) address of a torch tensor / numpy array, or None."""
    if t is None:
        return None
    if hasattr(t, "data_ptr"):
        assert t.is_contiguous()
        return C.c_void_p(t.data_ptr())
    assert t.flags["C_CONTIGUOUS"]
    return C.c_void_p(t.ctypes.data)


class Context:
    """One lp_ctx: one graph, one model, one CUDA stream."""

    def __init__(self, device: int = 0, stream=None):
        import torch

        self._torch = torch
        self.lib = load_library()
        self.device = device
        self.stream = stream if stream is not None else torch.cuda.current_stream(device)
        h = C.c_void_p()
        st = self.lib.lp_create(C.byref(h), C.c_int32(device), C.c_void_p(self.stream.cuda_stream))
        if st != LP_OK:
            raise LpError(st, self.lib.lp_last_error(None).decode())
        self.h = h
        self.n = self.nnz = self.f = 0
        self.n_params = 0
        self.desc: Optional[ModelDesc] = None

    def close(self):
        if getattr(self, "h", None):
            self.lib.lp_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _ck(self, st: int):
        if st != LP_OK:
            raise LpError(st, self.lib.lp_last_error(self.h).decode())

    # ---- graph
    def load_graph(self, n, rowptr, col, w, X, on_device: bool = False):
        """rowptr int64 [n+1], col int32 [nnz], w float32 [nnz] or None, X float32 [n, f]
        (numpy / CPU tensors, or CUDA tensors with on_device=True)."""
        nnz = int(col.shape[0])
        f = int(X.shape[1])
        self._ck(self.lib.lp_load_graph(self.h, C.c_int64(n), C.c_int64(nnz), _ptr(rowptr), _ptr(col), _ptr(w), _ptr(X),
                                        C.c_int32(f), C.c_int32(1 if on_device else 0)))
        self.n, self.nnz, self.f = int(n), nnz, f

    def get_structure(self):
        t = self._torch
        dev = f"cuda:{self.device}"
        colptr = t.empty(self.n + 1, dtype=t.int64, device=dev)
        rowidx = t.empty(max(self.nnz, 1), dtype=t.int32, device=dev)
        perm = t.empty(max(self.nnz, 1), dtype=t.int64, device=dev)
        self._ck(self.lib.lp_get_structure(self.h, _ptr(colptr), _ptr(rowidx), _ptr(perm)))
        return colptr, rowidx[: self.nnz], perm[: self.nnz]

    def sparsify(self, alpha: float, seed: int):
        """Algorithm 1's sparsification of the loaded (symmetric) graph: (rowptr int64, col int32, w float32) on the device."""
        t = self._torch
        dev = f"cuda:{self.device}"
        nnz = C.c_int64()
        self._ck(self.lib.lp_sparsify(self.h, C.c_double(alpha), C.c_uint64(seed), C.byref(nnz)))
        k = int(nnz.value)
        rowptr = t.empty(self.n + 1, dtype=t.int64, device=dev)
        col = t.empty(max(k, 1), dtype=t.int32, device=dev)
        w = t.empty(max(k, 1), dtype=t.float32, device=dev)
        self._ck(self.lib.lp_get_sparsified(self.h, _ptr(rowptr), _ptr(col), _ptr(w)))
        return rowptr, col[:k], w[:k]

    def worker_view(self, part, worker: int, keep_cross_edges: bool = True, foreign_mode: int = 1):
        """Graph that `worker` trains on (Section III): (rowptr int64, col int32, stats dict) on the device.
        foreign_mode 0 = no sharing, 1 = sparsified rows of the last sparsify(), 2 = full rows."""
        t = self._torch
        dev = f"cuda:{self.device}"
        nnz, st = C.c_int64(), ViewStats()
        self._ck(self.lib.lp_worker_view(self.h, _ptr(part), C.c_int32(worker), C.c_int32(int(keep_cross_edges)), C.c_int32(foreign_mode),
                                         C.byref(nnz), C.byref(st)))
        k = int(nnz.value)
        rowptr = t.empty(self.n + 1, dtype=t.int64, device=dev)
        col = t.empty(max(k, 1), dtype=t.int32, device=dev)
        self._ck(self.lib.lp_get_worker_view(self.h, _ptr(rowptr), _ptr(col)))
        return rowptr, col[:k], {"own_entries": st.own_entries, "foreign_entries": st.foreign_entries,
                                 "foreign_rows": st.foreign_rows, "own_nodes": st.own_nodes}

    # ---- model
    def set_model(self, arch: str, dims: Sequence[int], prec: str = "fp32", fanout: Optional[Sequence[int]] = None,
                  reject_edges: bool = True, max_attempts: int = 8, max_batch: int = 65536, max_k: int = 1,
                  cache_input_aggregation: bool = False, pred_hidden: int = 0):
        """pred_hidden = 0: dot-product predictor; > 0: 3-layer MLP predictor with that hidden width."""
        d = ModelDesc()
        d.arch = LP_GCN if arch == "gcn" else LP_SAGE_MEAN
        d.n_layers = len(dims) - 1
        for i, v in enumerate(dims):
            d.dims[i] = int(v)
        d.prec = LP_BF16 if prec == "bf16" else LP_FP32
        for i, v in enumerate(fanout or []):
            d.fanout[i] = int(v)
        d.reject_edges = int(bool(reject_edges))
        d.max_attempts = int(max_attempts)
        d.cache_input_aggregation = int(bool(cache_input_aggregation))
        d.predictor = 1 if pred_hidden > 0 else 0
        d.pred_hidden = int(pred_hidden)
        self._ck(self.lib.lp_set_model(self.h, C.byref(d), C.c_int64(max_batch), C.c_int32(max_k)))
        np_ = C.c_int64()
        self._ck(self.lib.lp_param_count(self.h, C.byref(np_)))
        self.n_params = int(np_.value)
        self.desc = d
        self.dims = list(dims)
        self.K = len(dims) - 1
        return self.n_params

    # ---- sampling
    def set_candidates(self, cand):
        self._ck(self.lib.lp_set_candidates(self.h, _ptr(cand), C.c_int64(0 if cand is None else cand.numel())))

    def sample_negatives(self, seed: int, step: int, k: int, pos_src, mode: int = LP_NEG_PER_SOURCE, edge_index_base: int = 0,
                         want_src: bool = False):
        t = self._torch
        B = int(pos_src.numel())
        neg_dst = t.empty(B * k, dtype=t.int32, device=pos_src.device)
        neg_src = t.empty(B * k, dtype=t.int32, device=pos_src.device) if (want_src or mode == LP_NEG_GLOBAL_PAIR) else None
        self._ck(self.lib.lp_sample_negatives(self.h, C.c_uint64(seed), C.c_uint64(step), C.c_int32(k), C.c_int32(mode), _ptr(pos_src),
                                              C.c_int64(B), C.c_int64(edge_index_base), _ptr(neg_src), _ptr(neg_dst)))
        return neg_src, neg_dst

    # ---- step
    def train_step(self, params, pos_src, pos_dst, neg_src, neg_dst, k: int, loss, grads, seed: int = 0, step: int = 0,
                   accumulate: bool = False):
        self._ck(self.lib.lp_train_step(self.h, _ptr(params), _ptr(pos_src), _ptr(pos_dst), C.c_int64(pos_src.numel()), _ptr(neg_src),
                                        _ptr(neg_dst), C.c_int32(k), C.c_uint64(seed), C.c_uint64(step), _ptr(loss), _ptr(grads),
                                        C.c_int32(int(accumulate))))

    def train_step_host(self, params, pos_src_host, pos_dst_host, k: int, seed: int, step: int, edge_index_base: int = 0,
                        adam_m=None, adam_v=None, adam_t: int = 1, loss_host=None, grads_host=None):
        self._ck(self.lib.lp_train_step_host(self.h, _ptr(params), _ptr(pos_src_host), _ptr(pos_dst_host), C.c_int64(pos_src_host.shape[0]),
                                             C.c_int32(k), C.c_uint64(seed), C.c_uint64(step), C.c_int64(edge_index_base), _ptr(adam_m),
                                             _ptr(adam_v), C.c_int64(adam_t), _ptr(loss_host), _ptr(grads_host)))

    def adam_step(self, params, m, v, grads, t: int, grad_scale: float = 1.0, lr: float = 1e-3, beta1: float = 0.9, beta2: float = 0.999,
                  eps: float = 1e-8):
        self._ck(self.lib.lp_adam_step(self.h, _ptr(params), _ptr(m), _ptr(v), _ptr(grads), C.c_double(grad_scale), C.c_double(lr),
                                       C.c_double(beta1), C.c_double(beta2), C.c_double(eps), C.c_int64(t)))

    def score(self, params, src, dst, seed: int = 0, step: int = 0):
        t = self._torch
        out = t.empty(src.numel(), dtype=t.float32, device=src.device)
        self._ck(self.lib.lp_score(self.h, _ptr(params), _ptr(src), _ptr(dst), C.c_int64(src.numel()), C.c_uint64(seed), C.c_uint64(step),
                                   _ptr(out)))
        return out

    def invalidate_embeddings(self):
        """Tell the library that the weights changed outside its own calls (see lp_score)."""
        self._ck(self.lib.lp_invalidate_embeddings(self.h))

    def set_wait_limit(self, limit_ns: int, overdeclare_bytes: int = 0):
        """Bound of the device-side waits of the tensor-core kernels; overdeclare_bytes > 0 makes the next such
        launch run into that bound (self-test of the LP_ETIMEOUT path)."""
        self._ck(self.lib.lp_set_wait_limit(self.h, C.c_uint64(limit_ns), C.c_int32(overdeclare_bytes)))

    def hits_at_k(self, pos_scores, neg_scores, k: int) -> float:
        """Hits@K of device score vectors (float32)."""
        out = C.c_double()
        self._ck(self.lib.lp_hits_at_k(self.h, _ptr(pos_scores), C.c_int64(pos_scores.numel()), _ptr(neg_scores), C.c_int64(neg_scores.numel()),
                                       C.c_int64(k), C.byref(out)))
        return float(out.value)

    # ---- inspection
    def stats(self) -> Stats:
        s = Stats()
        self._ck(self.lib.lp_get_stats(self.h, C.byref(s)))
        return s

    def embeddings(self, layer: int, rows: Optional[int] = None):
        t = self._torch
        rows = self.n if rows is None else rows
        out = t.empty((rows, self.dims[layer]), dtype=t.float32, device=f"cuda:{self.device}")
        self._ck(self.lib.lp_get_embeddings(self.h, C.c_int32(layer), _ptr(out)))
        return out

    def predictor_activations(self, layer: int, E: int):
        t = self._torch
        out = t.empty((E, int(self.desc.pred_hidden)), dtype=t.float32, device=f"cuda:{self.device}")
        self._ck(self.lib.lp_get_predictor_activations(self.h, C.c_int32(layer), C.c_int64(E), _ptr(out)))
        return out

    def output_gradient(self, rows: Optional[int] = None):
        t = self._torch
        rows = self.n if rows is None else rows
        out = t.empty((rows, self.dims[-1]), dtype=t.float32, device=f"cuda:{self.device}")
        self._ck(self.lib.lp_get_output_gradient(self.h, _ptr(out)))
        return out

    def block(self, hop: int):
        """(frontier F_hop or None for the outermost hop, blk_ptr, blk_col) of the last sampled step."""
        t = self._torch
        dev = f"cuda:{self.device}"
        s = self.stats()
        frontier = None
        if hop < self.K:
            frontier = t.empty(int(s.block_nodes[hop]), dtype=t.int32, device=dev)
        ptr = col = None
        if hop >= 1:
            ptr = t.empty(int(s.block_nodes[hop - 1]) + 1, dtype=t.int64, device=dev)
            col = t.empty(max(int(s.block_edges[hop - 1]), 1), dtype=t.int32, device=dev)
        self._ck(self.lib.lp_get_block(self.h, C.c_int32(hop), _ptr(frontier), _ptr(ptr), _ptr(col)))
        if col is not None:
            col = col[: int(s.block_edges[hop - 1])]
        return frontier, ptr, col

    # ---- per-kernel timing
    def profile_begin(self, categories=None):
        mask = 0
        for c in (categories if categories is not None else PROF_CATEGORIES):
            mask |= 1 << PROF_CATEGORIES.index(c)
        self._ck(self.lib.lp_profile_begin(self.h, C.c_uint32(mask)))

    def profile_sample_every(self, n: int):
        self._ck(self.lib.lp_profile_sample_every(self.h, C.c_uint32(n)))

    def profile_end(self):
        p = Profile()
        self._ck(self.lib.lp_profile_end(self.h, C.byref(p)))
        return {name: {"ms": p.ms[i], "bytes": p.bytes[i], "flops": p.flops[i], "spans": int(p.spans[i])}
                for i, name in enumerate(PROF_CATEGORIES)}

    # ---- single operators
    def op_aggregate(self, arch: str, H, transpose: bool = False):
        t = self._torch
        M = t.empty_like(H)
        self._ck(self.lib.lp_op_aggregate(self.h, C.c_int32(LP_GCN if arch == "gcn" else LP_SAGE_MEAN), C.c_int32(int(transpose)),
                                          C.c_int32(int(H.dtype == t.bfloat16)), _ptr(H), C.c_int32(H.shape[1]), _ptr(M)))
        return M

    def op_gather_ceiling(self, H, transpose: bool = False):
        """XOR folds of the rows of H named by every run of 64 stored entries (see lp_op_gather_ceiling)."""
        t = self._torch
        row_bytes = H.shape[1] * H.element_size()
        runs = (self.nnz + 63) // 64
        folds = t.empty((runs, row_bytes // 4), dtype=t.int32, device=H.device)
        self._ck(self.lib.lp_op_gather_ceiling(self.h, C.c_int32(int(transpose)), _ptr(H), C.c_int32(row_bytes), _ptr(folds)))
        return folds

    def op_linear(self, A, B, bias=None, relu: bool = False, trans_b: bool = False):
        t = self._torch
        M, K = A.shape
        N = B.shape[0] if trans_b else B.shape[1]
        Cout = t.empty((M, N), dtype=A.dtype, device=A.device)
        prec = LP_BF16 if A.dtype == t.bfloat16 else LP_FP32
        self._ck(self.lib.lp_op_linear(self.h, C.c_int32(prec), C.c_int64(M), C.c_int32(N), C.c_int32(K), _ptr(A), _ptr(B),
                                       C.c_int32(int(trans_b)), _ptr(bias), C.c_int32(int(relu)), _ptr(Cout)))
        return Cout

    def op_weight_grad(self, A, dZ):
        t = self._torch
        M, K = A.shape
        N = dZ.shape[1]
        dW = t.empty((K, N), dtype=t.float32, device=A.device)
        prec = LP_BF16 if A.dtype == t.bfloat16 else LP_FP32
        self._ck(self.lib.lp_op_weight_grad(self.h, C.c_int32(prec), C.c_int64(M), C.c_int32(N), C.c_int32(K), _ptr(A), _ptr(dZ), _ptr(dW)))
        return dW


def weight_grad_static(A, dZ, stream=None):
    """dW = A^T dZ (float32 CUDA tensors) through the allocation-free entry point.  The output
    tensor is allocated HERE, by torch, before the call: the library call itself allocates nothing.
    For callers that cannot allocate at call time (allocator-free loops, pre-pooled memory)."""
    import torch

    lib = load_library()
    M, K = A.shape
    N = dZ.shape[1]
    dW = torch.empty((K, N), dtype=torch.float32, device=A.device)
    st = stream if stream is not None else torch.cuda.current_stream(A.device)
    rc = lib.lp_weight_grad_static(C.c_int32(A.device.index or 0), C.c_void_p(st.cuda_stream), C.c_int64(M), C.c_int32(N), C.c_int32(K),
                                   _ptr(A), _ptr(dZ), _ptr(dW))
    if rc != LP_OK:
        raise LpError(rc, lib.lp_last_error(None).decode())
    return dW
