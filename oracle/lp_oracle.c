/*
 * CPU oracle for the link-prediction GNN training step -- TEST INFRASTRUCTURE ONLY.
 *
 * Plain, slow, obviously-correct C (FP64 arithmetic, integer-exact samplers) for the
 * sparse / integer parts of the step; the dense algebra and the orchestration of the
 * layers live in oracle/model.py (numpy, FP64).  Nothing here is shared with the CUDA
 * library: no headers, no tables, no helpers.  Only tests, the smoke check and the CPU
 * baseline leg of the benchmark may call it.
 *
 * Conventions: CSR rows are destination nodes v, the columns of row v are the
 * in-neighbours u in N(v) (Eq. 1), sorted ascending.  Dense matrices are row-major
 * [n, F] doubles (row v = h_v).
 *
 * Each function names the passage of the paper it follows.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------------------
 * Philox4x32-10 (Salmon, Moraes, Dror, Shaw, "Parallel random numbers: as easy as
 * 1, 2, 3", SC'11).  The paper only says negatives and neighbours are drawn "uniformly
 * at random" (Section II-B); the counter-based generator makes every draw a pure
 * function of (seed, global edge index, step, ...), independent of batching.
 * ---------------------------------------------------------------------------------- */
void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;   /* round multipliers          */
    const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;   /* Weyl key increments        */
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int r = 0; r < 10; ++r) {
        uint64_t p0 = (uint64_t)M0 * c0;
        uint64_t p1 = (uint64_t)M1 * c2;
        uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
        uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n1 = lo1;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        uint32_t n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += W0; k1 += W1;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* uniform integer in [0, c) from 32 random bits: floor(x * c / 2^32) */
static uint32_t mulhi32(uint32_t x, uint32_t c) { return (uint32_t)(((uint64_t)x * (uint64_t)c) >> 32); }

/* draw tags (low byte of counter word 3) */
enum { TAG_NEG_DST = 1, TAG_NEG_SRC = 2, TAG_NBR = 3, TAG_SPARS = 4 };

/* ------------------------------------------------------------------------------------
 * Structure: transpose of the CSR (Section II-A graph G = (V, E, X); the transpose is
 * what backpropagation through the aggregation of Eq. 1 walks).  Entries of a transposed
 * row are ordered by original row ascending; perm[t] = index of the original entry.
 * Returns 0, or -1 when the input is not a valid CSR.
 * ---------------------------------------------------------------------------------- */
int orc_csc_transpose(int64_t n, int64_t nnz, const int64_t *rowptr, const int32_t *col,
                      int64_t *colptr, int32_t *rowidx, int64_t *perm)
{
    if (rowptr[0] != 0 || rowptr[n] != nnz) return -1;
    for (int64_t c = 0; c <= n; ++c) colptr[c] = 0;
    for (int64_t v = 0; v < n; ++v) {
        if (rowptr[v + 1] < rowptr[v]) return -1;
        for (int64_t e = rowptr[v]; e < rowptr[v + 1]; ++e) {
            if (col[e] < 0 || col[e] >= n) return -1;
            colptr[col[e] + 1] += 1;
        }
    }
    for (int64_t c = 0; c < n; ++c) colptr[c + 1] += colptr[c];
    int64_t *fill = (int64_t *)malloc(sizeof(int64_t) * (size_t)(n > 0 ? n : 1));
    for (int64_t c = 0; c < n; ++c) fill[c] = colptr[c];
    for (int64_t v = 0; v < n; ++v)
        for (int64_t e = rowptr[v]; e < rowptr[v + 1]; ++e) {
            int64_t t = fill[col[e]]++;
            rowidx[t] = (int32_t)v;
            perm[t] = e;
        }
    free(fill);
    return 0;
}

/* ------------------------------------------------------------------------------------
 * GCN normalisation (the paper names GCN only, Section IV hyperparameters; the formula
 * is Kipf & Welling's renormalised adjacency): A~ = A + I, d~_v = 1 + sum_u w_vu.
 * ---------------------------------------------------------------------------------- */
void orc_gcn_degree(int64_t n, const int64_t *rowptr, const float *w, double *dtilde)
{
    for (int64_t v = 0; v < n; ++v) {
        double d = 1.0;
        for (int64_t e = rowptr[v]; e < rowptr[v + 1]; ++e) d += w ? (double)w[e] : 1.0;
        dtilde[v] = d;
    }
}

/* ------------------------------------------------------------------------------------
 * AGG of Eq. 1.
 *   mode 0 (GCN) : M[v] = h_v / d~_v + sum_{u in N(v)} w_vu / sqrt(d~_v d~_u) * h_u
 *   mode 1 (mean): M[v] = (1/|N(v)|) sum_{u in N(v)} h_u     (0 when N(v) is empty)
 * ---------------------------------------------------------------------------------- */
void orc_aggregate(int mode, int64_t n, const int64_t *rowptr, const int32_t *col, const float *w,
                   const double *dtilde, const double *H, int64_t F, double *M)
{
#pragma omp parallel for schedule(dynamic, 64)
    for (int64_t v = 0; v < n; ++v) {
        double *m = M + v * F;
        for (int64_t d = 0; d < F; ++d) m[d] = 0.0;
        int64_t deg = rowptr[v + 1] - rowptr[v];
        if (mode == 0) {
            for (int64_t d = 0; d < F; ++d) m[d] = H[v * F + d] / dtilde[v];
            for (int64_t e = rowptr[v]; e < rowptr[v + 1]; ++e) {
                int64_t u = col[e];
                double a = (w ? (double)w[e] : 1.0) / sqrt(dtilde[v] * dtilde[u]);
                for (int64_t d = 0; d < F; ++d) m[d] += a * H[u * F + d];
            }
        } else if (deg > 0) {
            for (int64_t e = rowptr[v]; e < rowptr[v + 1]; ++e) {
                int64_t u = col[e];
                for (int64_t d = 0; d < F; ++d) m[d] += H[u * F + d];
            }
            for (int64_t d = 0; d < F; ++d) m[d] /= (double)deg;
        }
    }
}

/* ------------------------------------------------------------------------------------
 * Backpropagation through AGG (the gradient step of Algorithm 1, "Compute the gradient"):
 * dH[u] += coefficient(v,u) * dM[v] for every stored entry, written as the scatter that
 * the chain rule gives directly -- no transposed structure is used here, so this checks
 * the transposed-CSR path of the CUDA library independently.  Serial on purpose.
 * ---------------------------------------------------------------------------------- */
void orc_aggregate_backward(int mode, int64_t n, const int64_t *rowptr, const int32_t *col, const float *w,
                            const double *dtilde, const double *dM, int64_t F, double *dH)
{
    for (int64_t i = 0; i < n * F; ++i) dH[i] = 0.0;
    for (int64_t v = 0; v < n; ++v) {
        int64_t deg = rowptr[v + 1] - rowptr[v];
        const double *g = dM + v * F;
        if (mode == 0) {
            for (int64_t d = 0; d < F; ++d) dH[v * F + d] += g[d] / dtilde[v];
            for (int64_t e = rowptr[v]; e < rowptr[v + 1]; ++e) {
                int64_t u = col[e];
                double a = (w ? (double)w[e] : 1.0) / sqrt(dtilde[v] * dtilde[u]);
                for (int64_t d = 0; d < F; ++d) dH[u * F + d] += a * g[d];
            }
        } else if (deg > 0) {
            for (int64_t e = rowptr[v]; e < rowptr[v + 1]; ++e) {
                int64_t u = col[e];
                for (int64_t d = 0; d < F; ++d) dH[u * F + d] += g[d] / (double)deg;
            }
        }
    }
}

/* is (src -> dst) an edge of the loaded graph?  Row dst holds the in-neighbours of dst. */
static int is_edge(const int64_t *rowptr, const int32_t *col, int32_t src, int32_t dst)
{
    int64_t lo = rowptr[dst], hi = rowptr[dst + 1];
    while (lo < hi) {
        int64_t mid = lo + (hi - lo) / 2;
        if (col[mid] < src) lo = mid + 1; else hi = mid;
    }
    return lo < rowptr[dst + 1] && col[lo] == src;
}

/* ------------------------------------------------------------------------------------
 * Negative sampling (Section II-B: negatives are pairs (u,v), u != v, (u,v) not in E;
 * 'per-source' keeps the source of each positive and draws the destination uniformly,
 * 'global' draws both ends; Section III: the candidate set is the worker's partition
 * (local negatives) or the entire node set (global negatives)).
 *
 * Draw for positive with global index j = edge_index_base + position, negative kk,
 * attempt a:  x = philox(ctr = (lo(j), hi(j), lo(step), tag | kk<<8 | a<<16),
 *                        key = (lo(seed), hi(seed)))[0];  id = cand[floor(x*|cand|/2^32)].
 * With reject_edges, a draw that is a self pair or an edge of the loaded graph is redrawn
 * with a+1, at most max_attempts draws; the last draw is kept regardless (counted in
 * *n_exhausted).  mode 0 = per-source, mode 1 = global pair.
 * ---------------------------------------------------------------------------------- */
void orc_sample_negatives(int64_t n, const int64_t *rowptr, const int32_t *col,
                          const int32_t *cand, int64_t n_cand,
                          uint64_t seed, uint64_t step, int32_t k, int32_t mode,
                          int32_t reject_edges, int32_t max_attempts,
                          const int32_t *pos_src, int64_t B, int64_t edge_index_base,
                          int32_t *neg_src, int32_t *neg_dst, int64_t *n_exhausted)
{
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t space = (uint32_t)(cand ? n_cand : n);
    int64_t exhausted = 0;
    if (max_attempts < 1) max_attempts = 1;
    for (int64_t j = 0; j < B; ++j) {
        uint64_t gj = (uint64_t)(edge_index_base + j);
        for (int32_t kk = 0; kk < k; ++kk) {
            int32_t s = 0, d = 0, ok = 0;
            for (int32_t a = 0; a < max_attempts && !ok; ++a) {
                uint32_t ctr[4] = { (uint32_t)gj, (uint32_t)(gj >> 32), (uint32_t)step,
                                    (uint32_t)TAG_NEG_DST | ((uint32_t)kk << 8) | ((uint32_t)a << 16) };
                uint32_t r[4];
                orc_philox4x32_10(ctr, key, r);
                uint32_t pick = mulhi32(r[0], space);
                d = cand ? cand[pick] : (int32_t)pick;
                if (mode == 0) {
                    s = pos_src[j];
                } else {
                    ctr[3] = (uint32_t)TAG_NEG_SRC | ((uint32_t)kk << 8) | ((uint32_t)a << 16);
                    orc_philox4x32_10(ctr, key, r);
                    pick = mulhi32(r[0], space);
                    s = cand ? cand[pick] : (int32_t)pick;
                }
                ok = !reject_edges || (s != d && !is_edge(rowptr, col, s, d));
            }
            if (!ok) exhausted++;
            if (neg_src) neg_src[j * k + kk] = s;
            neg_dst[j * k + kk] = d;
        }
    }
    if (n_exhausted) *n_exhausted = exhausted;
}

/* ------------------------------------------------------------------------------------
 * Edge predictor gradient (Eq. 2 with the dot product, then the chain rule):
 * s = <h_u, h_v>  =>  dL/dh_u += g * h_v,  dL/dh_v += g * h_u   (both apply when u == v).
 * ---------------------------------------------------------------------------------- */
void orc_edge_grad(int64_t n, int64_t D, const double *H, int64_t E, const int32_t *src, const int32_t *dst,
                   const double *g, double *dH)
{
    for (int64_t i = 0; i < n * D; ++i) dH[i] = 0.0;
    for (int64_t e = 0; e < E; ++e) {
        int64_t u = src[e], v = dst[e];
        for (int64_t d = 0; d < D; ++d) {
            double hu = H[u * D + d], hv = H[v * D + d];
            dH[u * D + d] += g[e] * hv;
            dH[v * D + d] += g[e] * hu;
        }
    }
}

/* ------------------------------------------------------------------------------------
 * Node-wise neighbour sampling for one hop (Section II-B "constructs a computational
 * graph"; Section IV: a fixed number of neighbours per hop).  For a frontier node v with
 * in-degree d: all neighbours when d <= fanout, otherwise `fanout` distinct positions of
 * its row chosen by Floyd's subset algorithm:  for i = 0..fanout-1, j = d - fanout + i,
 * t = floor(x_i (j+1) / 2^32) with x_i = philox(ctr = (v, i, lo(step), tag | hop<<8))[0];
 * take t unless already taken, else take j.  Chosen positions are emitted ascending.
 * out_ptr has n_front+1 entries, out_col (global ids) must hold n_front*fanout entries.
 * ---------------------------------------------------------------------------------- */
static int cmp_i64(const void *a, const void *b)
{
    int64_t x = *(const int64_t *)a, y = *(const int64_t *)b;
    return (x > y) - (x < y);
}

void orc_sample_neighbors(const int64_t *rowptr, const int32_t *col, uint64_t seed, uint64_t step, int32_t hop,
                          int32_t fanout, const int32_t *frontier, int64_t n_front,
                          int64_t *out_ptr, int32_t *out_col)
{
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    int64_t *pos = (int64_t *)malloc(sizeof(int64_t) * (size_t)(fanout > 0 ? fanout : 1));
    int64_t w = 0;
    out_ptr[0] = 0;
    for (int64_t i = 0; i < n_front; ++i) {
        int64_t v = frontier[i];
        int64_t d = rowptr[v + 1] - rowptr[v];
        if (d <= fanout) {
            for (int64_t e = rowptr[v]; e < rowptr[v + 1]; ++e) out_col[w++] = col[e];
        } else {
            for (int32_t q = 0; q < fanout; ++q) {
                int64_t j = d - fanout + q;
                uint32_t ctr[4] = { (uint32_t)v, (uint32_t)q, (uint32_t)step,
                                    (uint32_t)TAG_NBR | ((uint32_t)hop << 8) };
                uint32_t r[4];
                orc_philox4x32_10(ctr, key, r);
                int64_t t = (int64_t)mulhi32(r[0], (uint32_t)(j + 1));
                int taken = 0;
                for (int32_t z = 0; z < q; ++z) if (pos[z] == t) taken = 1;
                pos[q] = taken ? j : t;
            }
            qsort(pos, (size_t)fanout, sizeof(int64_t), cmp_i64);
            for (int32_t q = 0; q < fanout; ++q) out_col[w++] = col[rowptr[v] + pos[q]];
        }
        out_ptr[i + 1] = w;
    }
    free(pos);
}

/* ------------------------------------------------------------------------------------
 * Degree-based effective-resistance sparsification (Algorithm 1, sparsification block;
 * Theorems 1 and 2): L draws with replacement, edge {u,v} drawn with probability
 * p = (1/d_u + 1/d_v) / n'  (n' = number of non-isolated nodes = sum over edges of
 * 1/d_u + 1/d_v), each draw adding 1/(L p) to the weight of its edge.
 * A draw is made by choosing a non-isolated node u uniformly (nz[floor(x0 n'/2^32)]) and
 * then one of its neighbours uniformly (row(u)[floor(x1 d_u/2^32)]): the unordered edge
 * {u,v} is hit with probability (1/n')(1/d_u) + (1/n')(1/d_v) = p.  (x0, x1) are words 0
 * and 1 of philox(ctr = (lo(l), hi(l), 0, tag), key = seed) for draw l = 0..L-1.
 * Output: for every stored entry e of the symmetric input CSR, wsum[e] = accumulated
 * weight of its undirected edge (0 = edge not kept); both orientations get the same value.
 * ---------------------------------------------------------------------------------- */
void orc_sparsify(int64_t n, const int64_t *rowptr, const int32_t *col, uint64_t seed, int64_t L, double *wsum)
{
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    int64_t nnz = rowptr[n];
    for (int64_t e = 0; e < nnz; ++e) wsum[e] = 0.0;
    int32_t *nz = (int32_t *)malloc(sizeof(int32_t) * (size_t)(n > 0 ? n : 1));
    int64_t np = 0;
    for (int64_t v = 0; v < n; ++v) if (rowptr[v + 1] > rowptr[v]) nz[np++] = (int32_t)v;
    for (int64_t l = 0; l < L && np > 0; ++l) {
        uint32_t ctr[4] = { (uint32_t)l, (uint32_t)((uint64_t)l >> 32), 0u, (uint32_t)TAG_SPARS };
        uint32_t r[4];
        orc_philox4x32_10(ctr, key, r);
        int64_t u = nz[mulhi32(r[0], (uint32_t)np)];
        int64_t du = rowptr[u + 1] - rowptr[u];
        int64_t e = rowptr[u] + (int64_t)mulhi32(r[1], (uint32_t)du);
        int64_t v = col[e];
        int64_t dv = rowptr[v + 1] - rowptr[v];
        double p = (1.0 / (double)du + 1.0 / (double)dv) / (double)np;
        double add = 1.0 / ((double)L * p);
        /* mirrored entry: u in row v */
        int64_t lo = rowptr[v], hi = rowptr[v + 1];
        while (lo < hi) { int64_t mid = lo + (hi - lo) / 2; if (col[mid] < u) lo = mid + 1; else hi = mid; }
        wsum[e] += add;
        wsum[lo] += add;
    }
    free(nz);
}
