// Counter-based samplers: uniform negatives (Section II-B: per-source and global; Section III:
// partition-local or global candidate set) and node-wise neighbour sampling for the
// computational graph of a batch.  All integer work; every draw is a pure function of
// (seed, step, global edge or node id, draw index), so results do not depend on batching or
// on the launch shape.
#pragma once
#include "common.cuh"
#include "scan_sort.cuh"

// Philox4x32-10 block function (Salmon et al., SC'11): 10 rounds of two 32x32->64 multiplies.
LP_DEVINL uint4 philox4x32_10(uint4 ctr, uint2 key)
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, ctr.x), lo0 = 0xD2511F53u * ctr.x;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, ctr.z), lo1 = 0xCD9E8D57u * ctr.z;
        ctr = make_uint4(hi1 ^ ctr.y ^ key.x, lo1, hi0 ^ ctr.w ^ key.y, lo0);
        key.x += 0x9E3779B9u;
        key.y += 0xBB67AE85u;
    }
    return ctr;
}

enum : uint32_t { DRAW_NEG_DST = 1, DRAW_NEG_SRC = 2, DRAW_NEIGHBOR = 3, DRAW_SPARSIFY = 4 };

// Is (src -> dst) stored in the graph?  Row dst lists the in-neighbours of dst, ascending.
LP_DEVINL bool csr_has_entry(const int *__restrict__ rowptr, const int *__restrict__ col, int src, int dst)
{
    int lo = rowptr[dst], hi = rowptr[dst + 1];
    const int end = hi;
    while (lo < hi) {
        const int mid = lo + ((hi - lo) >> 1);
        if (col[mid] < src) lo = mid + 1; else hi = mid;
    }
    return lo < end && col[lo] == src;
}

// one thread per (positive j, negative kk)
__global__ void sample_negatives_kernel(int n, const int *__restrict__ rowptr, const int *__restrict__ col,
                                        const int *__restrict__ cand, uint32_t n_space, uint2 key, uint32_t step_lo, int k, int mode,
                                        int reject, int max_attempts, const int *__restrict__ pos_src, int64_t B, int64_t base,
                                        int *__restrict__ neg_src, int *__restrict__ neg_dst, unsigned long long *__restrict__ exhausted,
                                        unsigned long long *__restrict__ exhausted_next)
{
    LP_DEP_ENTER();
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t == 0) *exhausted_next = 0ull;  // the counter of the next call (the counters are used in turn, so no call needs a memset)
    if (t >= B * k) return;
    const int64_t j = t / k;
    const uint32_t kk = (uint32_t)(t - j * k);
    const uint64_t gj = (uint64_t)(base + j);
    int s = 0, d = 0;
    bool ok = false;
    for (int a = 0; a < max_attempts && !ok; ++a) {
        const uint32_t w3 = (kk << 8) | ((uint32_t)a << 16);
        uint32_t x = philox4x32_10(make_uint4((uint32_t)gj, (uint32_t)(gj >> 32), step_lo, DRAW_NEG_DST | w3), key).x;
        uint32_t pick = __umulhi(x, n_space);
        d = cand ? min(max(cand[pick], 0), n - 1) : (int)pick;
        if (mode == LP_NEG_PER_SOURCE) {
            s = pos_src[j];
        } else {
            x = philox4x32_10(make_uint4((uint32_t)gj, (uint32_t)(gj >> 32), step_lo, DRAW_NEG_SRC | w3), key).x;
            pick = __umulhi(x, n_space);
            s = cand ? min(max(cand[pick], 0), n - 1) : (int)pick;
        }
        ok = !reject || (s != d && !csr_has_entry(rowptr, col, s, d));
    }
    if (!ok) atomicAdd(exhausted, 1ull);
    if (neg_src) neg_src[t] = s;
    neg_dst[t] = d;
}

// ------------------------------------------------------------------------------------------
// neighbour sampling: hop h from frontier F_{h-1} (sorted global ids)
// ------------------------------------------------------------------------------------------
constexpr int MAX_FANOUT = 32;

// counts[i] = min(deg(frontier[i]), fanout)
__global__ void nbr_count_kernel(const int *__restrict__ rowptr, const int *__restrict__ frontier, const int *__restrict__ n_front_dev,
                                 int fanout, int *__restrict__ counts, int max_front)
{
    LP_DEP_ENTER();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= max_front) return;
    const int nf = *n_front_dev;
    if (i >= nf) { counts[i] = 0; return; }
    const int v = frontier[i];
    counts[i] = min(rowptr[v + 1] - rowptr[v], fanout);
}

// Floyd's subset algorithm: for q = 0..fanout-1, j = d - fanout + q, t uniform in [0, j];
// take t unless already taken, else j.  Positions are emitted in ascending order.
// One group of G lanes (8, 16 or 32, at least the fan-out) per frontier row: lane q evaluates draw q (the
// draws are independent counter-based numbers), the "already taken" decisions are resolved in order
// with one ballot per draw, and every lane finds the rank of its position among the (distinct)
// positions of the row.
template <int G>
__global__ void nbr_sample_kernel(const int *__restrict__ rowptr, const int *__restrict__ col, const int *__restrict__ frontier,
                                  const int *__restrict__ n_front_dev, int fanout, uint2 key, uint32_t step_lo, uint32_t hop,
                                  const int *__restrict__ blk_ptr, int *__restrict__ blk_col_global, int *__restrict__ blk_row,
                                  unsigned char *__restrict__ mark, int *__restrict__ blk_eid)
{
    LP_DEP_ENTER();
    const unsigned lane = threadIdx.x & 31;
    const int gl = threadIdx.x % G;  // lane inside the group
    const unsigned gmask = (G == 32) ? 0xffffffffu : (((1u << G) - 1u) << (lane & ~(unsigned)(G - 1)));
    const int64_t i64 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) / G;
    if (i64 >= *n_front_dev) return;  // uniform over the group
    const int i = (int)i64;
    const int v = frontier[i];
    const int r0 = rowptr[v], d = rowptr[v + 1] - r0;
    const int out = blk_ptr[i];
    if (d <= fanout) {
        for (int e = gl; e < d; e += G) {
            const int u = col[r0 + e];
            blk_col_global[out + e] = u;
            blk_row[out + e] = i;
            if (blk_eid) blk_eid[out + e] = r0 + e;  // position of the sampled entry in the graph's CSR
            mark[u] = 1;
        }
        return;
    }
    const int j = d - fanout + gl;
    int t = 0;
    if (gl < fanout) {
        const uint32_t x = philox4x32_10(make_uint4((uint32_t)v, (uint32_t)gl, step_lo, DRAW_NEIGHBOR | (hop << 8)), key).x;
        t = (int)__umulhi(x, (uint32_t)(j + 1));
    }
    int mypos = -1;
    for (int q = 0; q < fanout; ++q) {
        const int tq = __shfl_sync(gmask, t, q, G);
        const unsigned taken = __ballot_sync(gmask, gl < q && mypos == tq);
        if (gl == q) mypos = taken ? j : tq;
    }
    int rank = 0;
    for (int z = 0; z < fanout; ++z) rank += __shfl_sync(gmask, mypos, z, G) < mypos ? 1 : 0;
    if (gl < fanout) {
        const int u = col[r0 + mypos];
        blk_col_global[out + rank] = u;
        blk_row[out + rank] = i;
        if (blk_eid) blk_eid[out + rank] = r0 + mypos;
        mark[u] = 1;
    }
}

// GCN over a sampled block: entry e of destination i = frontier position of v keeps the graph's coefficient
// w_vu / sqrt(d~_v d~_u), rescaled by |N(v)| / |S(v)| (every neighbour is kept with probability |S(v)| / |N(v)|, so the
// sampled sum estimates the full one without bias); the self coefficient 1 / d~_v is exact.
__global__ void gcn_block_coef_kernel(const int *__restrict__ rowptr, const int *__restrict__ frontier, const int *__restrict__ blk_ptr,
                                      const int *__restrict__ blk_row, const int *__restrict__ blk_eid, const int *__restrict__ n_entries_dev,
                                      const float *__restrict__ gcn_val, float *__restrict__ blk_val)
{
    LP_DEP_ENTER();
    const int e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= *n_entries_dev) return;
    const int i = blk_row[e];
    const int v = frontier[i];
    const float ratio = (float)(rowptr[v + 1] - rowptr[v]) / (float)(blk_ptr[i + 1] - blk_ptr[i]);
    blk_val[e] = gcn_val[blk_eid[e]] * ratio;
}

// out[i] = table[ids[i]] for i < *count
__global__ void gather_by_id_kernel(const float *__restrict__ table, const int *__restrict__ ids, const int *__restrict__ count_dev, int cap,
                                    float *__restrict__ out)
{
    LP_DEP_ENTER();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < min(*count_dev, cap)) out[i] = table[ids[i]];
}

__global__ void mark_ids_kernel(const int *__restrict__ ids, int64_t m, int n, unsigned char *__restrict__ mark)
{
    LP_DEP_ENTER();
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < m) mark[min(max(ids[i], 0), n - 1)] = 1;
}

__global__ void mark_to_int_kernel(const unsigned char *__restrict__ mark, int n, int *__restrict__ flags)
{
    LP_DEP_ENTER();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) flags[i] = mark[i] ? 1 : 0;
}

// frontier[posmap[v]] = v for marked v (posmap = exclusive scan of the marks): sorted and unique
__global__ void compact_frontier_kernel(const unsigned char *__restrict__ mark, const int *__restrict__ posmap, int n, int *__restrict__ frontier)
{
    LP_DEP_ENTER();
    const int v = blockIdx.x * blockDim.x + threadIdx.x;
    if (v < n && mark[v]) frontier[posmap[v]] = v;
}

// local ids of the sampled columns inside the new frontier
__global__ void relabel_kernel(const int *__restrict__ ids_global, const int *__restrict__ count_dev, int64_t max_count,
                               const int *__restrict__ posmap, int *__restrict__ ids_local)
{
    LP_DEP_ENTER();
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < max_count && i < (int64_t)*count_dev) ids_local[i] = posmap[ids_global[i]];
}

// self_idx[i] = position of destination i (node prev_frontier[i]) inside the new frontier;
// inv_self[that position] = i  (inv_self must be pre-filled with -1)
__global__ void self_index_kernel(const int *__restrict__ prev_frontier, const int *__restrict__ n_prev_dev, const int *__restrict__ posmap,
                                  int *__restrict__ self_idx, int *__restrict__ inv_self)
{
    LP_DEP_ENTER();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= *n_prev_dev) return;
    const int p = posmap[prev_frontier[i]];
    self_idx[i] = p;
    inv_self[p] = i;
}

__global__ void fill_i32_kernel(int *__restrict__ p, int64_t m, int v)
{
    LP_DEP_ENTER();
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < m) p[i] = v;
}

// 1 / |sampled neighbours| per destination row, and the same value per transposed entry
__global__ void inv_degree_kernel(const int *__restrict__ ptr, int n_rows, const int *__restrict__ n_rows_dev, float *__restrict__ inv)
{
    LP_DEP_ENTER();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    const int lim = n_rows_dev ? min(*n_rows_dev, n_rows) : n_rows;
    if (i >= lim) return;
    const int d = ptr[i + 1] - ptr[i];
    inv[i] = d > 0 ? 1.f / (float)d : 0.f;
}

__global__ void gather_f32_kernel(const float *__restrict__ src, const int *__restrict__ idx, int64_t m, float *__restrict__ dst)
{
    LP_DEP_ENTER();
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < m) dst[i] = src[idx[i]];
}
