/*
 * lp.h -- C ABI of the B200 link-prediction GNN training step.
 *
 * One context trains on one graph on one GPU.  The step is the body of the per-batch loop
 * of Algorithm 1 for one worker: sample negatives, run the K-layer encoder (Eq. 1), score
 * every positive and negative edge with the dot product (Eq. 2), take the mean binary
 * cross-entropy over N = |P| + |N| edges, back-propagate, and update the weights.
 *
 * General rules
 *   - Every function returns an lp_status; nothing throws, aborts or traps.  After a
 *     failure lp_last_error(ctx) holds a one-line description.
 *   - Unless stated otherwise, array arguments are DEVICE pointers owned by the caller
 *     (in practice torch tensors); the library reads or writes them on the context's
 *     stream and never frees them.  The library owns only its internal workspace
 *     (transposed graph, activations, sampled blocks), allocated with cudaMalloc at
 *     lp_load_graph / lp_set_model and released by lp_destroy.
 *   - All work is enqueued on the stream given to lp_create.  Calls that return a value
 *     to the host (or take host buffers) synchronise that stream; the others do not.
 *   - Graph convention: CSR rows are destination nodes v; the columns of row v are the
 *     in-neighbours u in N(v) whose embeddings v aggregates (Eq. 1), strictly ascending
 *     (no duplicates).  A positive sample (u, v) is an entry u in row v (Section II-B).
 *   - Parameters, gradients and Adam moments are flat float32 vectors.  Layer k
 *     (k = 0..K-1, input width dims[k], output width dims[k+1]) occupies, in order:
 *        GCN       : W      [dims[k], dims[k+1]] row-major, b [dims[k+1]]
 *        SAGE-mean : W_self [dims[k], dims[k+1]], W_neigh [dims[k], dims[k+1]], b [dims[k+1]]
 */
#ifndef LP_H_
#define LP_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct lp_ctx lp_ctx; /* opaque */

typedef enum {
    LP_OK = 0,
    LP_EINVAL = -1,       /* bad argument (null pointer, size, malformed CSR, id out of range) */
    LP_ESTATE = -2,       /* call out of order (e.g. train step before lp_set_model)          */
    LP_ENOMEM = -3,       /* device or host allocation failed                                 */
    LP_ECUDA = -4,        /* a CUDA call or kernel reported an error                          */
    LP_EUNSUPPORTED = -5, /* valid request that this build does not implement                 */
    LP_ETIMEOUT = -6      /* a bounded device-side wait expired; the context stays usable     */
} lp_status;

typedef enum { LP_GCN = 0, LP_SAGE_MEAN = 1 } lp_arch;
typedef enum { LP_FP32 = 0, LP_BF16 = 1 } lp_prec;
typedef enum { LP_NEG_PER_SOURCE = 0, LP_NEG_GLOBAL_PAIR = 1 } lp_neg_mode;
/* Edge predictor of Eq. 2: the dot product <h_u, h_v>, or the 3-layer MLP of the paper's experiments
 * (Section IV) on the element-wise product: z0 = h_u * h_v; p1 = ReLU(z0 W0 + b0); p2 = ReLU(p1 W1 + b1);
 * s = p2 . w2 + b2.  Its parameters follow the encoder's in the flat vector:
 * W0[D, Hp] row-major, b0[Hp], W1[Hp, Hp], b1[Hp], w2[Hp], b2[1]  (D = dims[K]). */
typedef enum { LP_PRED_DOT = 0, LP_PRED_MLP = 1 } lp_predictor;

#define LP_MAX_LAYERS 4

/* Model description (Section IV hyperparameters: 2-3 layers, hidden width 256, per-hop
 * fanouts).  dims = {input, hidden.., output}; every width must be a multiple of 8 (FP32)
 * or of 64 (BF16 tensor-core path).  fanout[h] is the number of in-neighbours sampled at hop
 * h+1 (hop 1 feeds the LAST layer); all zeros = full-graph training (every node aggregates
 * its full neighbour list).  Over a sample S(v) of N(v), LP_SAGE_MEAN takes the mean of the sample;
 * LP_GCN keeps the coefficients and degrees of the loaded graph, multiplies the sampled entries of v
 * by |N(v)| / |S(v)| (an unbiased estimate of the full sum) and keeps the self term exact. */
typedef struct {
    int32_t arch;                    /* lp_arch */
    int32_t n_layers;                /* K, 1..LP_MAX_LAYERS */
    int32_t dims[LP_MAX_LAYERS + 1];
    int32_t prec;                    /* lp_prec: storage of activations and GEMM operand type */
    int32_t fanout[LP_MAX_LAYERS];
    int32_t reject_edges;            /* negatives: redraw self pairs and true edges */
    int32_t max_attempts;            /* draws per negative when reject_edges (1..255) */
    int32_t cache_input_aggregation; /* full-graph models only: AGG(X) of the first layer does not depend on the
                                        weights, so compute it in the first step and reuse it afterwards (off = 0:
                                        every step recomputes it) */
    int32_t predictor;               /* lp_predictor: edge predictor of Eq. 2 */
    int32_t pred_hidden;             /* LP_PRED_MLP: hidden width Hp (multiple of 8, or of 64 in BF16; <= 512) */
} lp_model_desc;

typedef struct {
    int64_t negatives_exhausted;     /* negatives kept although every attempt was rejected (last lp_sample_negatives) */
    int64_t block_nodes[LP_MAX_LAYERS + 1]; /* frontier sizes |F_0|..|F_K| of the last sampled step */
    int64_t block_edges[LP_MAX_LAYERS];     /* sampled entries per hop of the last sampled step */
    int64_t workspace_bytes;         /* device memory owned by the context */
    int64_t kernel_launches;         /* kernels launched by this context since lp_create */
} lp_stats;

/* ---- life cycle ------------------------------------------------------------------- */

/* Create a context on CUDA device `device`; `cuda_stream` is a cudaStream_t (NULL = the
 * legacy default stream).  *out receives the context (NULL on failure). */
lp_status lp_create(lp_ctx **out, int32_t device, void *cuda_stream);

/* Release everything the context owns.  NULL is accepted. */
void lp_destroy(lp_ctx *ctx);

/* Last error text of this context (or of lp_create when ctx is NULL).  Never NULL. */
const char *lp_last_error(const lp_ctx *ctx);

/* ---- graph G = (V, E, X), Section II-A --------------------------------------------- */

/* Load the graph the worker trains on and its node features.
 *   n, nnz      : nodes and stored directed entries (nnz < 2^31)
 *   rowptr[n+1] : int64, rowptr[0] = 0, non-decreasing, rowptr[n] = nnz
 *   col[nnz]    : int32 in [0, n), strictly ascending inside a row
 *   w[nnz]      : float32 edge weights or NULL (= all 1).  GCN uses them in A~ = A + I;
 *                 SAGE-mean ignores them (unweighted mean over the stored neighbours)
 *   X[n, f]     : float32 row-major, row v = x_v
 *   ptrs_on_device : 0 = the four arrays are HOST memory, 1 = DEVICE memory
 * The arrays are copied (the caller may free them afterwards).  The call validates the CSR
 * (LP_EINVAL on any violation), builds the transposed structure used by the backward pass
 * (entries of a transposed row ordered by original row), the degree normalisations
 * (GCN: d~_v = 1 + sum_u w_vu; SAGE: 1/|N(v)|), a BF16 copy of X, and a padded copy of the graph and
 * of its transpose for the aggregation kernel (rows in groups of four entries: about 8.6 bytes per
 * stored entry and structure, a little more where rows are short; lp_get_stats reports the total).
 * Synchronises. */
lp_status lp_load_graph(lp_ctx *ctx, int64_t n, int64_t nnz, const int64_t *rowptr, const int32_t *col,
                        const float *w, const float *X, int32_t f, int32_t ptrs_on_device);

/* Transposed structure built by lp_load_graph, for bit-exact checks (device outputs):
 * colptr[n+1] int64, rowidx[nnz] int32, perm[nnz] int64 (perm[t] = index of the original
 * entry that transposed entry t came from).  Any of the three may be NULL. */
lp_status lp_get_structure(lp_ctx *ctx, int64_t *colptr, int32_t *rowidx, int64_t *perm);

/* ---- graph sparsification, Algorithm 1 (sparsification block), Theorems 1 and 2 -------- */

/* Sparsify the loaded graph (which must be symmetric: every stored entry has its mirror) by the
 * degree-based approximation of effective resistance: L = floor(alpha * |E|) draws with
 * replacement (|E| = nnz / 2 undirected edges), edge {u, v} drawn with probability
 * p = (1/d_u + 1/d_v) / n' (n' = number of non-isolated nodes), each draw adding 1 / (L p) to the
 * weight of its edge; edges never drawn are removed, all nodes are kept.  Draw l picks
 * u = nz[floor(x0 n' / 2^32)] among the non-isolated nodes (ascending) and then the neighbour at
 * position floor(x1 d_u / 2^32) of u's row, with (x0, x1) = words 0 and 1 of
 * philox(counter = (lo32(l), hi32(l), 0, 4), key = (lo32(seed), hi32(seed))).
 * The result stays inside the context until the next lp_sparsify / lp_load_graph; *nnz_out receives
 * its number of stored entries (both orientations).  Synchronises.
 * LP_EINVAL when alpha is not in (0, 1e6] or the graph is not symmetric. */
lp_status lp_sparsify(lp_ctx *ctx, double alpha, uint64_t seed, int64_t *nnz_out);

/* Copy the last sparsified graph out (DEVICE arrays): rowptr[n+1] int64, col[nnz_out] int32
 * ascending inside a row, w[nnz_out] float32 accumulated weights.  Any pointer may be NULL. */
lp_status lp_get_sparsified(lp_ctx *ctx, int64_t *rowptr, int32_t *col, float *w);

/* ---- worker view, Section III (data sharing for negative sampling) ----------------------- */

typedef struct {
    int64_t own_entries;     /* stored entries of the worker's own rows                                   */
    int64_t foreign_entries; /* stored entries of the other partitions' rows: the graph data shared with   */
    int64_t foreign_rows;    /*   this worker, and the number of foreign rows that carry any               */
    int64_t own_nodes;       /* |V^i|                                                                      */
} lp_view_stats;

/* Build the graph that worker `worker` trains on from the loaded (global) graph and a node -> partition
 * assignment part[n] (DEVICE int32):
 *   rows of the worker's own nodes: their list in the loaded graph -- every neighbour when
 *     keep_cross_edges != 0 (the full-neighbour partitions of the method), else only neighbours in the
 *     same partition (node-induced subgraph);
 *   rows of other partitions' nodes, foreign_mode 0: empty (no data sharing, local negatives only);
 *     1: their lists in the last lp_sparsify result (the method: sparsified subgraphs shared for global
 *     negatives); 2: their full lists (complete data sharing).
 * The four variants compared in the paper's ablation are (keep_cross, foreign_mode) = (1, 1), (1, 2),
 * (1, 0) and (0, 0).  The result stays in the context; *nnz_out receives its entry count and *stats (may be
 * NULL) the sizes from which the shared graph data volume follows.  Synchronises.
 * LP_ESTATE when foreign_mode is 1 and lp_sparsify has not been called. */
lp_status lp_worker_view(lp_ctx *ctx, const int32_t *part, int32_t worker, int32_t keep_cross_edges, int32_t foreign_mode, int64_t *nnz_out,
                         lp_view_stats *stats);

/* Copy the last worker view out (DEVICE arrays): rowptr[n+1] int64, col[nnz_out] int32 ascending per row. */
lp_status lp_get_worker_view(lp_ctx *ctx, int64_t *rowptr, int32_t *col);

/* ---- model -------------------------------------------------------------------------- */

/* Fix the encoder (Eq. 1) and allocate the activation workspace.  `max_batch` bounds the
 * number of positives per later call and `max_k` the negatives per positive. */
lp_status lp_set_model(lp_ctx *ctx, const lp_model_desc *desc, int64_t max_batch, int32_t max_k);

/* Length of the flat parameter vector of the model set by lp_set_model. */
lp_status lp_param_count(const lp_ctx *ctx, int64_t *n_params);

/* ---- negative sampling, Sections II-B and III ---------------------------------------- */

/* Candidate set for negative endpoints: the worker's own partition V^i (local negatives)
 * or NULL / n_cand = 0 for the entire node set (global negatives).  cand is a DEVICE array
 * of node ids; it is copied. */
lp_status lp_set_candidates(lp_ctx *ctx, const int32_t *cand, int64_t n_cand);

/* Draw k negatives per positive with Philox4x32-10.  For the positive with global index
 * j = edge_index_base + position, negative kk and attempt a the 32 random bits are word 0
 * of philox(counter = (lo32(j), hi32(j), lo32(step), tag | kk<<8 | a<<16), key = (lo32(seed),
 * hi32(seed))), tag = 1 for destinations and 2 for sources, and the endpoint is
 * cand[floor(bits * |cand| / 2^32)].  LP_NEG_PER_SOURCE keeps the positive's source and
 * draws the destination; LP_NEG_GLOBAL_PAIR draws both (neg_src required).  With
 * reject_edges (model description) a self pair or an edge of the loaded graph is redrawn,
 * at most max_attempts draws; the last draw is kept and counted in lp_stats.
 *   pos_src[B]     : device, sources of the positives (ignored in global-pair mode)
 *   neg_src[B*k]   : device output or NULL (per-source mode: pos_src repeated k times)
 *   neg_dst[B*k]   : device output, negative kk of positive j at index j*k + kk
 * Does not synchronise. */
lp_status lp_sample_negatives(lp_ctx *ctx, uint64_t seed, uint64_t step, int32_t k, int32_t mode,
                              const int32_t *pos_src, int64_t B, int64_t edge_index_base,
                              int32_t *neg_src, int32_t *neg_dst);

/* ---- training step, Algorithm 1 (per-batch body) -------------------------------------- */

/* Forward, loss and gradient for one batch.
 *   params[n_params]  : device float32, current weights W
 *   pos_src/pos_dst[B]: device int32, positives (label 1)
 *   neg_src[B*k]      : device int32 or NULL (= source of positive j for its k negatives)
 *   neg_dst[B*k]      : device int32, negatives (label 0); k may be 0
 *   seed, step        : Philox key / step counter of the neighbour sampler (used only when
 *                       the model has non-zero fanouts)
 *   loss              : device float32 scalar, L = (1/N) sum_e ell(s_e, y_e), N = B(1+k)
 *   grads[n_params]   : device float32, dL/dW; overwritten, or added to when accumulate != 0
 *                       (gradient accumulation over emulated workers)
 * The gradient with respect to the embeddings is summed per node in 64-bit fixed point (order-free, hence
 * reproducible bit for bit) at a resolution of 2^-32 relative to |h| / N (2^-(50 - ceil(log2 N)) for N above
 * 2^18); embeddings must stay below 4096 in magnitude for that sum not to saturate, and a NaN embedding
 * contributes 0 to it.
 * Node ids are checked on the device: an id outside [0, n) is clamped into range (so no
 * access ever leaves the arrays), the results of that call are then meaningless, and the
 * next synchronising call (lp_get_stats, lp_train_step_host) returns LP_EINVAL once.
 * Does not synchronise. */
lp_status lp_train_step(lp_ctx *ctx, const float *params, const int32_t *pos_src, const int32_t *pos_dst, int64_t B,
                        const int32_t *neg_src, const int32_t *neg_dst, int32_t k, uint64_t seed, uint64_t step,
                        float *loss, float *grads, int32_t accumulate);

/* The same step for callers whose data lives in HOST memory: copies the B positives to the
 * device, draws k per-source negatives (as lp_sample_negatives with edge_index_base),
 * runs lp_train_step, optionally applies lp_adam_step to the DEVICE parameter vector
 * (when adam_m/adam_v are non-NULL device arrays; hyper-parameters lr 1e-3, betas 0.9 /
 * 0.999, eps 1e-8, step count adam_t), and copies the loss (and, if grads_host is not NULL,
 * the gradient) back.  pos_src_host, pos_dst_host, loss_host, grads_host are HOST pointers;
 * params, adam_m, adam_v are DEVICE pointers.  Synchronises. */
lp_status lp_train_step_host(lp_ctx *ctx, float *params, const int32_t *pos_src_host, const int32_t *pos_dst_host,
                             int64_t B, int32_t k, uint64_t seed, uint64_t step, int64_t edge_index_base,
                             float *adam_m, float *adam_v, int64_t adam_t, float *loss_host, float *grads_host);

/* Gradient synchronisation and update (Algorithm 1: average over p workers, then update;
 * Section IV: Adam, lr 1e-3).  g = grad_scale * grads (grad_scale = 1/p);
 * m = b1 m + (1-b1) g;  v = b2 v + (1-b2) g^2;
 * params -= lr * (m / (1 - b1^t)) / (sqrt(v / (1 - b2^t)) + eps).   t counts from 1.
 * With adam_m == NULL the plain rule W <- W - lr * g of Algorithm 1 is applied.
 * All arrays are device float32 [n_params].  The scalar hyper-parameters are doubles so that
 * 1 - beta and the bias corrections are formed exactly on the host before being rounded to
 * float32 for the kernel.  Does not synchronise. */
lp_status lp_adam_step(lp_ctx *ctx, float *params, float *adam_m, float *adam_v, const float *grads, double grad_scale,
                       double lr, double beta1, double beta2, double eps, int64_t t);

/* ---- inference, Eq. 2 ------------------------------------------------------------------- */

/* scores[E] = <h_u^(K), h_v^(K)> (or the MLP predictor's output) for the E pairs (src, dst) under the
 * weights `params` (sampled models draw neighbours with seed/step as in lp_train_step).  Device
 * arrays.  Does not synchronise.
 * Full-graph models keep H^(K) between calls: an evaluation pass that scores validation positives and
 * negatives in batches (Section IV) runs the encoder once.  The kept embeddings are used when the call
 * passes the same `params` pointer as the forward pass that produced them (an lp_score or lp_train_step
 * of this context) and no lp_adam_step / lp_train_step_host of this context has updated weights since.
 * A caller that changes the weights behind that pointer by other means must call
 * lp_invalidate_embeddings before scoring. */
lp_status lp_score(lp_ctx *ctx, const float *params, const int32_t *src, const int32_t *dst, int64_t E,
                   uint64_t seed, uint64_t step, float *scores);

/* Forget the embeddings kept for lp_score (see there).  Never fails on a valid context. */
lp_status lp_invalidate_embeddings(lp_ctx *ctx);

/* Hits@K (the accuracy metric of Section IV): the fraction of the n_pos positive scores that are
 * strictly greater than the K-th largest of the n_neg negative scores (1 when n_neg < K).  Scores are
 * DEVICE float32 arrays (as written by lp_score); *hits is a HOST double.  Allocates temporary device
 * memory and synchronises. */
lp_status lp_hits_at_k(lp_ctx *ctx, const float *pos_scores, int64_t n_pos, const float *neg_scores, int64_t n_neg, int64_t K, double *hits);

/* ---- inspection (parity checks) ---------------------------------------------------------- */

/* Embeddings H^(layer) of the last forward pass as float32, layer in 1..K.  For full-graph
 * models `out` is [n, dims[layer]].  For sampled models `out` is [|F_{K-layer}|, dims[layer]],
 * row i belonging to node frontier[i] of that frontier (see lp_get_block).  Device output. */
lp_status lp_get_embeddings(lp_ctx *ctx, int32_t layer, float *out);

/* Hidden activations of the MLP predictor in the last lp_train_step or lp_score: layer 1 (p1) or 2 (p2)
 * as float32 [E, pred_hidden], one row per scored edge (positives, then negatives).  Device output. */
lp_status lp_get_predictor_activations(lp_ctx *ctx, int32_t layer, int64_t E, float *out);

/* Gradient of the loss with respect to H^(K) from the last lp_train_step, float32, same row
 * indexing as lp_get_embeddings(K).  Device output. */
lp_status lp_get_output_gradient(lp_ctx *ctx, float *out);

/* Sampled computational graph of the last step (Section II-B), hop in 1..K:
 *   frontier[|F_hop|]      : int32 global ids of F_hop, ascending (pass hop = 0 for the seeds F_0)
 *   blk_ptr[|F_{hop-1}|+1] : int64 offsets per destination of F_{hop-1}
 *   blk_col[entries]       : int32 sampled in-neighbours as GLOBAL ids, ascending per row
 * Sizes come from lp_get_stats.  Any pointer may be NULL.  Device outputs. */
lp_status lp_get_block(lp_ctx *ctx, int32_t hop, int32_t *frontier, int64_t *blk_ptr, int32_t *blk_col);

/* Counters.  Synchronises the stream.  Returns LP_EINVAL (once) when an earlier step was
 * given a node id outside [0, n), and LP_ETIMEOUT (once) when a bounded wait inside a
 * tensor-core kernel of an earlier call expired. */
lp_status lp_get_stats(lp_ctx *ctx, lp_stats *out);

/* (No counterpart in the paper: failure detection of the library itself.)
 * Every device-side wait of the tensor-core kernels (on a shared-memory barrier that a bulk copy or a matrix
 * instruction completes) is bounded: when it has lasted limit_ns the kernel records which wait gave up, releases
 * its tensor memory and returns; the next synchronising call returns LP_ETIMEOUT once and the context stays
 * usable.  limit_ns (default 2e9, allowed 1e3 .. 6e10) sets that bound for later launches of this context.
 * overdeclare_bytes (normally 0; a multiple of 16, at most 65536) is a self-test of that path: the NEXT tensor-core
 * launch announces that many bytes more than it copies on its first barrier, so every copy lands but the barrier
 * never completes and the waits run into the limit.  Nothing faults and nothing is left running. */
lp_status lp_set_wait_limit(lp_ctx *ctx, uint64_t limit_ns, int32_t overdeclare_bytes);

/* ---- per-kernel timing (roofline measurement) ------------------------------------------------ */

/* Kernel categories of the step. */
enum {
    LP_PROF_AGG_FWD = 0,   /* neighbour aggregation, forward (Eq. 1 AGG)                    */
    LP_PROF_AGG_BWD = 1,   /* its adjoint over the transposed structure                     */
    LP_PROF_GEMM_FWD = 2,  /* dense transform Z = A W + b (Eq. 1 UPDATE)                    */
    LP_PROF_GEMM_DGRAD = 3,/* dA = dZ W^T, or dH = [dZ | A^T dZ] [W_self^T ; W_neigh^T]         */
    LP_PROF_GEMM_WGRAD = 4,/* dW = A^T dZ and db                                            */
    LP_PROF_SCORE = 5,     /* edge scores, loss partials, per-edge gradients (Eq. 2, Alg. 1) */
    LP_PROF_INCIDENCE = 6, /* grouping the scored edges by node; final loss reduction        */
    LP_PROF_SCATTER = 7,   /* dL/dH^(K) gathered per node                                   */
    LP_PROF_NEGATIVES = 8, /* negative sampling                                             */
    LP_PROF_BLOCKS = 9,    /* neighbour sampling and block construction                     */
    LP_PROF_ADAM = 10,     /* optimiser                                                     */
    LP_PROF_CATEGORIES = 11
};

typedef struct {
    double ms[LP_PROF_CATEGORIES];      /* device time between CUDA events on the context's stream      */
    double bytes[LP_PROF_CATEGORIES];   /* algorithmic bytes of the timed launches (gather convention:  */
                                        /* every stored entry reads its source row once, nothing cached) */
    double flops[LP_PROF_CATEGORIES];   /* algorithmic floating-point operations                        */
    int64_t spans[LP_PROF_CATEGORIES];  /* number of timed spans                                        */
} lp_profile;

/* Start timing the categories selected by `category_mask` (bit c = category c) with CUDA events
 * recorded on the context's stream around the corresponding launches of every later call.
 * A mask of 0 switches timing off.  Event records cost about a microsecond each. */
lp_status lp_profile_begin(lp_ctx *ctx, uint32_t category_mask);

/* Stop timing, synchronise the stream and return the sums per category since lp_profile_begin. */
lp_status lp_profile_end(lp_ctx *ctx, lp_profile *out);

/* Time only the launches of every n-th call of lp_train_step / lp_train_step_host (n >= 1; 1, the default,
 * times every call).  An event record between two kernels keeps the second from being made resident while
 * the first still runs, so timed steps run a few percent slower than untimed ones: sampling keeps the timed
 * launches representative while the whole run stays close to its untimed speed.  The setting lasts until it
 * is changed.  LP_EINVAL when n is 0. */
lp_status lp_profile_sample_every(lp_ctx *ctx, uint32_t n);

/* ---- single operators (used by the parity tests and the roofline benchmark) -------------- */

/* AGG of Eq. 1 on the loaded graph, float32 in / float32 out (bf16 = 0) or BF16 in / BF16 out
 * given as raw 16-bit words (bf16 = 1):
 *   transpose = 0 : M[v] = AGG over N(v)        transpose = 1 : the adjoint, dH = AGG^T dM
 *   arch LP_GCN: renormalised adjacency with self-loops; LP_SAGE_MEAN: mean over N(v).
 * H and M are [n, F] row-major device arrays; F a multiple of 8, F <= 512. */
lp_status lp_op_aggregate(lp_ctx *ctx, int32_t arch, int32_t transpose, int32_t bf16, const void *H, int32_t F, void *M);

/* (No counterpart in the paper: a measurement aid for the roofline of lp_op_aggregate.)
 * Bare gather over the loaded graph's index stream: the stored entries (column indices of the CSR, or the row
 * indices of its transpose when transpose = 1) are cut into runs of 64 consecutive entries; for every run the rows
 * H[index] (row_bytes bytes each, row-major, n rows) are loaded and folded with bitwise XOR, and folds receives
 * ceil(nnz / 64) rows of row_bytes bytes.  No row structure, arithmetic or epilogue: the time of this call is the
 * floor for any kernel that gathers these rows in this order, whether they come from L2 or from HBM.
 *   H, folds : DEVICE, 16-byte aligned, caller-owned; row_bytes in {128, 256, 512}.  Does not synchronise. */
lp_status lp_op_gather_ceiling(lp_ctx *ctx, int32_t transpose, const void *H, int32_t row_bytes, void *folds);

/* Dense transform C[M, N] = A[M, K] * B + bias, optional ReLU; B is [K, N] row-major
 * (trans_b = 0) or [N, K] row-major (trans_b = 1).  prec LP_FP32: float32 everywhere;
 * LP_BF16: A, B, C are BF16 words, bias float32, FP32 accumulation on the tensor cores. */
lp_status lp_op_linear(lp_ctx *ctx, int32_t prec, int64_t M, int32_t N, int32_t K, const void *A, const void *B,
                       int32_t trans_b, const float *bias, int32_t relu, void *C);

/* Weight gradient dW[K, N] = A[M, K]^T * dZ[M, N] (float32 output, fixed reduction order). */
lp_status lp_op_weight_grad(lp_ctx *ctx, int32_t prec, int64_t M, int32_t N, int32_t K, const void *A, const void *dZ,
                            float *dW);

/* ---- allocation-free variant ---------------------------------------------------------------- */

/* (No counterpart in the paper: this entry point exists for the callers described below.)
 * Weight gradient dW[K, N] = A[M, K]^T * dZ[M, N] in float32, the same result as
 * lp_op_weight_grad(LP_FP32) up to the order of the row-split summation, for callers that cannot
 * allocate device memory when they need it: latency-critical loops that forbid allocator calls
 * because those take driver locks and may synchronise the device, processes that handed all
 * device memory to a pool at start-up, and code sections in which the CUDA runtime itself
 * refuses to allocate.  It needs no context and calls no cudaMalloc, cudaFree or any allocating routine:
 * the partial sums of the split-row reduction live in a fixed 8 MiB array inside the library
 * (every GPU that uses the library holds that array until the process exits).
 *   device, cuda_stream : device index (made current by the call) and cudaStream_t (NULL = default)
 *   A[M, K], dZ[M, N], dW[K, N] : DEVICE float32, row-major, caller-owned; dW is overwritten
 * Limit: K * N <= 2^21 (2,097,152); larger requests return LP_EINVAL with a message available
 * from lp_last_error(NULL) (that message is kept per host thread).  M is unbounded.
 * The first call on each device looks up the device address of the fixed array; make that first
 * call before starting any stream capture.  All calls on a device share the array and it keeps
 * the previous call's contents (each call overwrites what it reads, so nothing needs clearing):
 * two calls whose kernels overlap on the GPU (different streams, no ordering) race on it and
 * must be serialised by the caller.  Does not synchronise. */
lp_status lp_weight_grad_static(int32_t device, void *cuda_stream, int64_t M, int32_t N, int32_t K, const float *A, const float *dZ,
                                float *dW);

#ifdef __cplusplus
}
#endif
#endif /* LP_H_ */
