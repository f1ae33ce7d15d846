// Edge predictor (Eq. 2, dot product), mean binary cross-entropy over N = |P| + |N| edges
// (Algorithm 1) and the per-edge score gradients; plus the batch-edge incidence lists that let
// the gradient with respect to H^(K) be gathered row by row (no float atomics).
#pragma once
#include "common.cuh"
#include "optim.cuh"
#include "scan_sort.cuh"

constexpr int EDGE_THREADS = 256;

// Node ids arrive from the caller in device memory; every consumer clamps them into [0, n_ids) so
// that a bad id can never cause an out-of-range access (check_ids_kernel reports it instead).
LP_DEVINL int clamp_id(int v, int n_ids) { return min(max(v, 0), n_ids - 1); }

__global__ void check_ids_kernel(const int *__restrict__ ids, int64_t m, int n_ids, int *__restrict__ err)
{
    LP_DEP_ENTER();
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < m && (ids[i] < 0 || ids[i] >= n_ids)) atomicOr(err, 1);
}

// the same for the up to four id arrays of a step in one launch (null arrays are skipped)
// First kernel of a step.  Blocks below id_blocks check the step's node ids and clear the incidence-list counters the scoring
// kernel adds into and the two counters of the heavy-row plan of those lists; the blocks behind them (BF16 path) make the
// BF16 copies of the parameter vector that the transforms read (weights_cache_element).
__global__ void check_step_ids_kernel(const int *__restrict__ a, int64_t na, const int *__restrict__ b, int64_t nb, const int *__restrict__ c, int64_t nc,
                                      const int *__restrict__ d, int64_t nd, int n_ids, int *__restrict__ err, int *__restrict__ zero, int64_t n_zero,
                                      int *__restrict__ plan_counts, int id_blocks, const float *__restrict__ w_params, long long w_n, WeightBlocks w_blocks,
                                      bf16 *__restrict__ w_asis, bf16 *__restrict__ w_transposed, bf16 *__restrict__ w_stacked)
{
    LP_DEP_ENTER();
    if ((int)blockIdx.x >= id_blocks) {
        weights_cache_element((long long)(blockIdx.x - id_blocks) * blockDim.x + threadIdx.x, w_params, w_n, w_blocks, w_asis, w_transposed, w_stacked);
        return;
    }
    if (blockIdx.x == 0 && threadIdx.x < 2 && plan_counts) plan_counts[threadIdx.x] = 0;
    for (int64_t z = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; z < n_zero; z += (int64_t)id_blocks * blockDim.x) zero[z] = 0;
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int *p = a;
    if (i >= na) { i -= na; p = b; if (i >= nb) { i -= nb; p = c; if (i >= nc) { i -= nc; p = d; if (i >= nd) return; } } }
    const int v = p[i];
    if (v < 0 || v >= n_ids) atomicOr(err, 1);
}

LP_DEVINL float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// ell(s, y) = max(s, 0) - s*y + log(1 + exp(-|s|));   d ell / d s = sigmoid(s) - y
LP_DEVINL void bce_logits(float s, float y, float &ell, float &dls)
{
    const float e = expf(-fabsf(s));
    ell = fmaxf(s, 0.f) - s * y + log1pf(e);
    const float sig = (s >= 0.f) ? 1.f / (1.f + e) : e / (1.f + e);
    dls = sig - y;
}

// One warp per positive j: loads h_u once, then h_v and the k negative destinations (per-source
// negatives share the source row).  Writes g for the positive and its negatives (already divided
// by N), the raw scores if asked, and one loss partial per block.
//   idmap : optional global id -> row of H (sampled models: position inside the seed frontier)
template <typename T, int NV>
__global__ void __launch_bounds__(EDGE_THREADS)
edge_score_bce_kernel(const T *__restrict__ H, int ldh, int D, int n_ids, const int *__restrict__ idmap, const int *__restrict__ pos_src,
                      const int *__restrict__ pos_dst, int64_t B, const int *__restrict__ neg_src, const int *__restrict__ neg_dst, int k,
                      float inv_N, float *__restrict__ g_pos, float *__restrict__ g_neg, float *__restrict__ s_pos, float *__restrict__ s_neg,
                      float *__restrict__ loss_partials, int *__restrict__ inc_counts = nullptr)
{
    LP_DEP_ENTER();
    constexpr int VN = Vec16<T>::N;
    __shared__ float s_loss[EDGE_THREADS / 32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t j = (int64_t)blockIdx.x * (EDGE_THREADS / 32) + warp;
    const int nchunks = D / VN;
    float loss = 0.f;
    if (j < B) {
        int u = clamp_id(pos_src[j], n_ids), v = clamp_id(pos_dst[j], n_ids);
        if (idmap) { u = idmap[u]; v = idmap[v]; }
        // the first negative row is requested together with h_u and h_v, and each further negative row while
        // the previous one is reduced: one memory round trip per edge instead of two dependent ones
        Vec16<T> nxt[NV];
        int vn_nxt = 0;
        if (k > 0) {
            vn_nxt = clamp_id(neg_dst[j * k], n_ids);
            if (idmap) vn_nxt = idmap[vn_nxt];
#pragma unroll
            for (int i = 0; i < NV; ++i) {
                const int ch = lane + i * 32;
                if (ch < nchunks) nxt[i].load(H + (size_t)vn_nxt * ldh + ch * VN);
            }
        }
        float hu[NV][VN];
        float dot = 0.f;
#pragma unroll
        for (int i = 0; i < NV; ++i) {
            const int ch = lane + i * 32;
            if (ch < nchunks) {
                Vec16<T> a, b;
                a.load(H + (size_t)u * ldh + ch * VN);
                b.load(H + (size_t)v * ldh + ch * VN);
                float fb[VN];
                a.to_float(hu[i]);
                b.to_float(fb);
#pragma unroll
                for (int t = 0; t < VN; ++t) dot = fmaf(hu[i][t], fb[t], dot);
            }
        }
        dot = warp_sum(dot);
        float ell, dls;
        bce_logits(dot, 1.f, ell, dls);
        loss += ell;
        if (lane == 0) {
            g_pos[j] = dls * inv_N;
            if (s_pos) s_pos[j] = dot;
            if (inc_counts) {  // lengths of the per-node incidence lists, counted while the endpoints are at hand
                atomicAdd(&inc_counts[u], 1);
                atomicAdd(&inc_counts[v], 1);
            }
        }
        for (int kk = 0; kk < k; ++kk) {
            const int64_t t = j * k + kk;
            Vec16<T> cur[NV];
#pragma unroll
            for (int i = 0; i < NV; ++i) cur[i] = nxt[i];
            const int vn_cur = vn_nxt;
            if (kk + 1 < k) {
                vn_nxt = clamp_id(neg_dst[t + 1], n_ids);
                if (idmap) vn_nxt = idmap[vn_nxt];
#pragma unroll
                for (int i = 0; i < NV; ++i) {
                    const int ch = lane + i * 32;
                    if (ch < nchunks) nxt[i].load(H + (size_t)vn_nxt * ldh + ch * VN);
                }
            }
            const bool own_src = neg_src != nullptr;
            int un = u;
            if (own_src) { un = clamp_id(neg_src[t], n_ids); if (idmap) un = idmap[un]; }
            float d2 = 0.f;
#pragma unroll
            for (int i = 0; i < NV; ++i) {
                const int ch = lane + i * 32;
                if (ch < nchunks) {
                    float fb[VN];
                    cur[i].to_float(fb);
                    if (own_src && un != u) {
                        Vec16<T> a;
                        a.load(H + (size_t)un * ldh + ch * VN);
                        float fa[VN];
                        a.to_float(fa);
#pragma unroll
                        for (int q = 0; q < VN; ++q) d2 = fmaf(fa[q], fb[q], d2);
                    } else {
#pragma unroll
                        for (int q = 0; q < VN; ++q) d2 = fmaf(hu[i][q], fb[q], d2);
                    }
                }
            }
            d2 = warp_sum(d2);
            bce_logits(d2, 0.f, ell, dls);
            loss += ell;
            if (lane == 0) {
                g_neg[t] = dls * inv_N;
                if (s_neg) s_neg[t] = d2;
                if (inc_counts) {
                    atomicAdd(&inc_counts[un], 1);
                    atomicAdd(&inc_counts[vn_cur], 1);
                }
            }
        }
    }
    if (lane == 0) s_loss[warp] = loss;
    __syncthreads();
    if (threadIdx.x == 0 && loss_partials) {
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < EDGE_THREADS / 32; ++w) s += s_loss[w];
        loss_partials[blockIdx.x] = s;
    }
}

// The common case (one negative per positive that shares the positive's source, rows of at most 32 vectors): a warp
// takes two positives and requests their six rows together before it reduces any, which halves the number of
// dependent memory round trips per scored edge.  The four dot products of the warp are reduced together (lane i of
// every group of four ends up with the sum of value i: 8 shuffles instead of 20) and their losses and gradients are
// evaluated side by side, one score per lane, instead of one after the other on every lane: the kernel is bound by
// instruction issue, not by memory.  A block's loss partial covers 16 positives.
template <typename T>
__global__ void __launch_bounds__(EDGE_THREADS)
edge_score_bce_pair_kernel(const T *__restrict__ H, int ldh, int D, int n_ids, const int *__restrict__ idmap, const int *__restrict__ pos_src,
                           const int *__restrict__ pos_dst, int64_t B, const int *__restrict__ neg_dst, float inv_N, float *__restrict__ g_pos,
                           float *__restrict__ g_neg, float *__restrict__ loss_partials, int *__restrict__ inc_counts)
{
    LP_DEP_ENTER();
    constexpr int VN = Vec16<T>::N;
    constexpr int P = 2;
    __shared__ float s_loss[EDGE_THREADS / 32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t j0 = ((int64_t)blockIdx.x * (EDGE_THREADS / 32) + warp) * P;
    const int nchunks = D / VN;
    const bool active = lane < nchunks;
    const int ch = min(lane, nchunks - 1);
    float loss = 0.f;
    if (j0 < B) {
        int u[P], v[P], vn[P];
        Vec16<T> ru[P], rv[P], rn[P];
#pragma unroll
        for (int p = 0; p < P; ++p) {
            const int64_t j = min(j0 + p, B - 1);  // a missing second positive repeats the first one's loads and writes nothing
            u[p] = clamp_id(pos_src[j], n_ids);
            v[p] = clamp_id(pos_dst[j], n_ids);
            vn[p] = clamp_id(neg_dst[j], n_ids);
            if (idmap) { u[p] = idmap[u[p]]; v[p] = idmap[v[p]]; vn[p] = idmap[vn[p]]; }
        }
#pragma unroll
        for (int p = 0; p < P; ++p) {
            ru[p].load(H + (size_t)u[p] * ldh + ch * VN);
            rv[p].load(H + (size_t)v[p] * ldh + ch * VN);
            rn[p].load(H + (size_t)vn[p] * ldh + ch * VN);
        }
        // d[2p] = <h_u, h_v> and d[2p + 1] = <h_u, h_v'> of positive p, this lane's 16 bytes of each
        float d[4];
#pragma unroll
        for (int p = 0; p < P; ++p) {
            d[2 * p] = active ? dot_vec<T>(ru[p], rv[p], 0.f) : 0.f;
            d[2 * p + 1] = active ? dot_vec<T>(ru[p], rn[p], 0.f) : 0.f;
        }
        // four sums at once: after two exchange steps lane l holds value (l & 3) summed over the lanes l, l ^ 1, l ^ 2, l ^ 3;
        // three butterfly steps over the lanes with equal (l & 3) finish it
        {
            const bool hi1 = (lane & 1) != 0;
            const float a0 = hi1 ? d[0] : d[1], k0 = hi1 ? d[1] : d[0];
            const float a1 = hi1 ? d[2] : d[3], k1 = hi1 ? d[3] : d[2];
            const float e0 = k0 + __shfl_xor_sync(0xffffffffu, a0, 1);  // lanes with bit 0 clear keep values 0 and 2, the others 1 and 3
            const float e1 = k1 + __shfl_xor_sync(0xffffffffu, a1, 1);
            const bool hi2 = (lane & 2) != 0;
            const float give = hi2 ? e0 : e1, keep = hi2 ? e1 : e0;
            float sum = keep + __shfl_xor_sync(0xffffffffu, give, 2);      // lane l: value (l & 1) + 2 * ((l >> 1) & 1)
            sum += __shfl_xor_sync(0xffffffffu, sum, 4);
            sum += __shfl_xor_sync(0xffffffffu, sum, 8);
            sum += __shfl_xor_sync(0xffffffffu, sum, 16);
            // lane l < 4 now evaluates score l: positive p = l >> 1, label 1 for even l (the positive), 0 for odd l (its negative)
            const int p = (lane >> 1) & 1;
            const bool is_pos = (lane & 1) == 0;
            float ell, dls;
            bce_logits(sum, is_pos ? 1.f : 0.f, ell, dls);
            if (lane < 4 && j0 + p < B) {
                loss = ell;
                (is_pos ? g_pos : g_neg)[j0 + p] = dls * inv_N;
            }
        }
        if (lane < P && j0 + lane < B && inc_counts) {  // lane p counts the endpoints of positive p and of its negative
            const int up = lane == 0 ? u[0] : u[1], vp = lane == 0 ? v[0] : v[1], np_ = lane == 0 ? vn[0] : vn[1];
            atomicAdd(&inc_counts[up], 2);  // source of the positive and of its negative
            atomicAdd(&inc_counts[vp], 1);
            atomicAdd(&inc_counts[np_], 1);
        }
        loss += __shfl_xor_sync(0xffffffffu, loss, 1);  // the warp's four losses (the other lanes hold 0)
        loss += __shfl_xor_sync(0xffffffffu, loss, 2);
    }
    if (lane == 0) s_loss[warp] = loss;
    __syncthreads();
    if (threadIdx.x == 0 && loss_partials) {
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < EDGE_THREADS / 32; ++w) s += s_loss[w];
        loss_partials[blockIdx.x] = s;
    }
}

// loss = inv_N * sum of partials by one block of THREADS threads: thread t adds partials t, t + THREADS, ... in double
// (tens of thousands of nearly equal terms), then a fixed binary tree over the threads
template <int THREADS> LP_DEVINL void loss_reduce_block(const float *__restrict__ partials, int64_t m, float inv_N, float *__restrict__ loss)
{
    __shared__ double sh[THREADS];
    double s = 0.0;
    for (int64_t i = threadIdx.x; i < m; i += THREADS) s += (double)partials[i];
    sh[threadIdx.x] = s;
    __syncthreads();
    for (int w = THREADS / 2; w > 0; w >>= 1) {
        if ((int)threadIdx.x < w) sh[threadIdx.x] += sh[threadIdx.x + w];
        __syncthreads();
    }
    if (threadIdx.x == 0) *loss = (float)(sh[0] * (double)inv_N);
}
__global__ void __launch_bounds__(1024) loss_reduce_kernel(const float *__restrict__ partials, int64_t m, float inv_N, float *__restrict__ loss)
{
    LP_DEP_ENTER();
    loss_reduce_block<1024>(partials, m, inv_N, loss);
}

// plain scores for lp_score: one warp per edge
template <typename T, int NV>
__global__ void __launch_bounds__(EDGE_THREADS)
edge_score_kernel(const T *__restrict__ H, int ldh, int D, int n_ids, const int *__restrict__ idmap, const int *__restrict__ src,
                  const int *__restrict__ dst, int64_t E, float *__restrict__ scores)
{
    LP_DEP_ENTER();
    constexpr int VN = Vec16<T>::N;
    const int lane = threadIdx.x & 31;
    const int64_t e = (int64_t)blockIdx.x * (EDGE_THREADS / 32) + (threadIdx.x >> 5);
    if (e >= E) return;
    int u = clamp_id(src[e], n_ids), v = clamp_id(dst[e], n_ids);
    if (idmap) { u = idmap[u]; v = idmap[v]; }
    const int nchunks = D / VN;
    float dot = 0.f;
#pragma unroll
    for (int i = 0; i < NV; ++i) {
        const int ch = lane + i * 32;
        if (ch < nchunks) {
            Vec16<T> a, b;
            a.load(H + (size_t)u * ldh + ch * VN);
            b.load(H + (size_t)v * ldh + ch * VN);
            dot = dot_vec<T>(a, b, dot);
        }
    }
    dot = warp_sum(dot);
    if (lane == 0) scores[e] = dot;
}

// Incidence lists of the scored edges, grouped by node: dL/dH^(K)[v] = sum over incident edges of g_e * h_other.
// Edge slots: positives 0..B-1, negatives B..B+B*k-1; slot e contributes (node src_e, other dst_e) and
// (node dst_e, other src_e).  Counts and slot claims use integer atomics, so the ORDER of a node's entries
// is not reproducible; the gather that consumes the lists therefore sums exactly (64-bit fixed point),
// which makes its result independent of that order and reproducible bit for bit.
LP_DEVINL void incidence_endpoints(int n_ids, const int *idmap, const int *pos_src, const int *pos_dst, int64_t B, const int *neg_src,
                                   const int *neg_dst, int k, int64_t e, int &s, int &d)
{
    if (e < B) {
        s = pos_src[e];
        d = pos_dst[e];
    } else {
        const int64_t t = e - B;
        s = neg_src ? neg_src[t] : pos_src[t / k];
        d = neg_dst[t];
    }
    s = clamp_id(s, n_ids);
    d = clamp_id(d, n_ids);
    if (idmap) { s = idmap[s]; d = idmap[d]; }
}

__global__ void incidence_count_kernel(int n_ids, const int *__restrict__ idmap, const int *__restrict__ pos_src, const int *__restrict__ pos_dst,
                                       int64_t B, const int *__restrict__ neg_src, const int *__restrict__ neg_dst, int k, int *__restrict__ counts)
{
    LP_DEP_ENTER();
    const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= B * (1 + k)) return;
    int s, d;
    incidence_endpoints(n_ids, idmap, pos_src, pos_dst, B, neg_src, neg_dst, k, e, s, d);
    atomicAdd(&counts[s], 1);
    atomicAdd(&counts[d], 1);
}

// cursor[v] starts at the offset of node v's list and is advanced by every claim.  The lanes of a warp that claim
// slots of the same node (batches often hold runs of positives with a common source) make one claim together: the
// lowest of them adds their number to the cursor and every lane takes its rank inside the claimed run.
LP_DEVINL int claim_slot(int *cursor, int node, unsigned active, int lane)
{
    const unsigned peers = __match_any_sync(active, node);
    const int leader = __ffs(peers) - 1;
    int base = 0;
    if (lane == leader) base = atomicAdd(&cursor[node], __popc(peers));
    base = __shfl_sync(peers, base, leader);
    return base + __popc(peers & ((1u << lane) - 1u));
}

// Work that rides along with the list fill in blocks of its own, behind the fill_blocks blocks that fill: the heavy-row plan of
// the lists (it needs only their offsets, which the scan before this launch produced; one thread per row) and the final
// reduction of the loss partials (one block).  plan_rows = 0 / loss = null switch a rider off.
struct FillRiders {
    int fill_blocks = 0;
    const int *plan_rowptr = nullptr;
    int plan_rows = 0;
    HeavyPlan plan;
    const float *loss_partials = nullptr;
    long long n_partials = 0;
    float inv_N = 0.f;
    float *loss = nullptr;
};
static inline unsigned fill_rider_blocks(const FillRiders &x) { return (unsigned)((x.plan_rows + 255) / 256 + (x.loss ? 1 : 0)); }

__global__ void __launch_bounds__(256) incidence_fill_kernel(int n_ids, const int *__restrict__ idmap, const int *__restrict__ pos_src,
                                                             const int *__restrict__ pos_dst, int64_t B, const int *__restrict__ neg_src,
                                                             const int *__restrict__ neg_dst, int k, const float *__restrict__ g_pos,
                                                             const float *__restrict__ g_neg, int *__restrict__ cursor, int *__restrict__ inc_col,
                                                             float *__restrict__ inc_val, int *__restrict__ inc_edge, int *__restrict__ plan_counts,
                                                             const FillRiders x)
{
    LP_DEP_ENTER();
    if (x.fill_blocks > 0 && (int)blockIdx.x >= x.fill_blocks) {
        const int pb = (int)blockIdx.x - x.fill_blocks, plan_blocks = (x.plan_rows + 255) / 256;
        if (pb < plan_blocks) {
            const int r = pb * 256 + (int)threadIdx.x;
            if (r < x.plan_rows) heavy_plan_row(x.plan_rowptr, r, x.plan, nullptr);
        } else if (x.loss) {
            loss_reduce_block<256>(x.loss_partials, x.n_partials, x.inv_N, x.loss);
        }
        return;
    }
    const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e == 0 && plan_counts) { plan_counts[0] = 0; plan_counts[1] = 0; }  // the heavy-row plan of these lists is built by the next launch
    const bool valid = e < B * (1 + k);
    const unsigned active = __ballot_sync(0xffffffffu, valid);
    if (!valid) return;
    const int lane = threadIdx.x & 31;
    int s, d;
    incidence_endpoints(n_ids, idmap, pos_src, pos_dst, B, neg_src, neg_dst, k, e, s, d);
    const float g = g_pos ? (e < B ? g_pos[e] : g_neg[e - B]) : 0.f;
    const int ps = claim_slot(cursor, s, active, lane);
    inc_col[ps] = d;
    const int pd = claim_slot(cursor, d, active, lane);
    inc_col[pd] = s;
    if (inc_val) { inc_val[ps] = g; inc_val[pd] = g; }
    if (inc_edge) { inc_edge[ps] = (int)e; inc_edge[pd] = (int)e; }  // MLP predictor: the entry's edge (row of dL/dz0)
}
