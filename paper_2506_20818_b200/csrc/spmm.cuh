// CSR neighbour aggregation (AGG of Eq. 1, and its adjoint over the transposed structure).
//
//   Y[r, :] = mask_r( init_coef[r] * Init[init_idx[r], :]  +  row_scale[r] * sum_e val[e] * X[col[e], :] )
//
// Two kernels.  spmm_padded_kernel serves the static structures (the loaded graph and its transpose), for which a
// padded copy of the rows is built once at load: it is described above its definition.  spmm_csr_kernel serves
// every structure as it is stored (per-step structures, wide rows, exact sums):
// one group of G lanes (8, 16 or 32) owns a row; every lane gathers 16-byte vectors of the
// source rows (4 floats or 8 bf16) and accumulates in FP32 in entry order.  Rows with more than
// a per-structure threshold of entries (power-law hubs) are cut into items of SPMM_SEG entries; the items run as extra
// blocks of the same grid (so hubs spread over the whole GPU and overlap the light rows), each
// writes an FP32 partial row, and a small second kernel adds a row's partials in item order and
// applies the epilogue.  The summation order is a function of the row length
// only: results are reproducible bit for bit (no atomics anywhere).  Row offsets of the block's
// rows are staged in shared memory with one coalesced load.  Optional parts (null pointers) cost
// a warp-uniform branch:
//   val        : per-entry coefficient (GCN: w_vu / sqrt(d~_v d~_u); batch-edge gradients g_e)
//   row_scale  : per-row factor applied to the neighbour sum (mean: 1/|N(v)|)
//   Init       : extra term (GCN self-loop h_v / d~_v; SAGE backward: gradient of the self path)
//   init_idx   : row of Init to use (-1 = none); null = identity
//   relu_ref   : forward activation; the output is zeroed where relu_ref <= 0 (ReLU backward)
//   self_out   : copy of X[self_idx[r]] written next to the aggregate (sampled SAGE blocks)
#pragma once
#include "common.cuh"
#include "scan_sort.cuh"

// Rows with more than `threshold` entries are cut into segments of SPMM_SEG entries ("items").
// rows[i] / base[i]: heavy row i and the index of its first item; item_row / item_first: for every
// item its row and that row's first item; counts[0] = heavy rows, counts[1] = items.
// partials[item][F] holds the FP32 partial sum of an item.  A plan is either built once for a
// static structure (host_rows >= 0 tells the launcher the counts) or refilled per launch.
struct HeavyPlan {
    int *rows = nullptr, *base = nullptr, *item_row = nullptr, *item_first = nullptr, *counts = nullptr;
    int *nseg = nullptr;                  // optional: items of heavy row i (saves the combine kernel the row-offset round trip)
    float *partials = nullptr;
    int host_rows = -1, host_items = -1;  // -1: unknown on the host (plan built on the device per launch)
    bool counts_zeroed = false;           // per-launch plans: the caller's previous kernel has already cleared `counts`
    bool plan_prebuilt = false;           // per-launch plans: an earlier kernel of the caller has already run heavy_plan_row over the rows
    int threshold = 32;                   // rows with more entries than this are heavy (>= SPMM_HEAVY_MIN)
    int seg = 512;                        // entries per item (SPMM_SEG; SPMM_PIECE for the padded form's own plan)
    // Static structures only: every row again in padded form for spmm_padded_kernel.  A row is cut into pieces of at
    // most SPMM_PIECE entries (one piece unless it is heavy), a piece into groups of four entries (a pad repeats the
    // group's first index, or names row 0 in the all-pad group that an empty row keeps so that its output is written;
    // pad coefficient 0).  pcol / pval hold the groups back to back; grow[g] is -1 inside a piece and
    // (id << 4 | kind << 3 | cnt) for the group that finishes a piece: cnt = real entries of that group (0..4), kind 0:
    // the piece is all of row id, kind 1: the piece belongs to a heavy row and its FP32 partial sum goes to slot id of
    // `partials` (p_rows / p_base / p_counts list the heavy rows and their first slots for the combine kernel).  chunk_start
    // cuts the groups into chunks that begin at piece starts (n_chunks + 1 offsets).
    const int4 *pcol = nullptr;
    const float4 *pval = nullptr;
    const float *pval_src = nullptr;      // the per-entry coefficient array pval was padded from
    const float4 *pval2 = nullptr;        // a second padded coefficient array of the same structure
    const float *pval2_src = nullptr;
    const int *grow = nullptr;
    const int *chunk_start = nullptr;
    int n_chunks = 0;
    int *p_rows = nullptr, *p_base = nullptr, *p_counts = nullptr, *p_nseg = nullptr;
    int p_host_rows = 0;
};

template <typename T> struct SpmmArgs {
    int n_rows = 0;
    const int *n_rows_dev = nullptr;  // optional device-resident row count (<= n_rows)
    const int *rowptr = nullptr;
    const int *col = nullptr;
    const float *val = nullptr;
    const float *row_scale = nullptr;
    const T *X = nullptr;
    int ldx = 0;
    const T *X2 = nullptr;       // optional second operand: entry e contributes X[col[e], :] * X2[col2[e], :] (element-wise)
    int ldx2 = 0;
    const int *col2 = nullptr;
    int F = 0;
    T *Y = nullptr;
    int ldy = 0;
    const T *init = nullptr;
    int ldinit = 0;
    const float *init_coef = nullptr;
    const int *init_idx = nullptr;
    const T *relu_ref = nullptr;
    int ldref = 0;
    const int *self_idx = nullptr;
    T *self_out = nullptr;
    int ldself = 0;
    T *Y2 = nullptr;             // optional second copy of the output, row r multiplied by y2_scale[r] (row-per-group kernel only)
    int ldy2 = 0;
    const float *y2_scale = nullptr;
    int64_t nnz = 0;             // stored entries (host-known upper bound), sizes the heavy-row part of the grid
    // exact (64-bit fixed-point) sums only: every product is multiplied by exact_scale, a power of two chosen by the caller
    // from the magnitude of the coefficients, before it is rounded to an integer; the sum is multiplied by exact_inv = 1 / exact_scale
    float exact_scale = 1099511627776.f, exact_inv = 1.f / 1099511627776.f;  // 2^40
    HeavyPlan heavy;             // heavy rows of this structure: prebuilt (static graph) or scratch to fill per launch
};

constexpr int SPMM_THREADS = 256;

// Accumulator of one output element.  float: FMA in entry order (the result depends on the order of a
// row's entries, which is fixed for every structure built by a stable sort).  long long: each product
// (coefficient already multiplied by the power-of-two scale of SpmmArgs) is rounded once to an integer and
// added as an integer -- exact and therefore independent of the order of the entries; used for lists whose
// entry order is not reproducible (slots claimed with integer atomics), so that their sums still are, bit
// for bit.  With scale 2^s the resolution of a product is 2^-s and the sum of a row must stay below 2^(63-s)
// in magnitude; NaN counts as 0 and larger values saturate, so the caller picks s from the data's range.
template <typename ACC> LP_DEVINL void acc_add(ACC &a, float w, float f);
template <> LP_DEVINL void acc_add<float>(float &a, float w, float f) { a = fmaf(w, f, a); }
template <> LP_DEVINL void acc_add<long long>(long long &a, float w, float f) { a += __float2ll_rn(w * f); }
// acc[0..VN) += w * v for one 16-byte vector.  Unit coefficients on BF16 data into FP32 accumulators use the
// mixed-precision add of sm_100 (add.rn.f32.bf16: the BF16 operand is widened exactly, one rounding, the
// same result as convert-then-add) and so skip the eight conversion instructions per vector.
template <typename T, typename ACC, bool HAS_VAL> LP_DEVINL void acc_add_vec(ACC *acc, float w, const Vec16<T> &v)
{
    constexpr int VN = Vec16<T>::N;
    float f[VN];
    v.to_float(f);
#pragma unroll
    for (int t = 0; t < VN; ++t) acc_add<ACC>(acc[t], w, f[t]);
}
template <> LP_DEVINL void acc_add_vec<bf16, float, false>(float *acc, float, const Vec16<bf16> &v)
{
    const uint32_t x[4] = {v.v.x, v.v.y, v.v.z, v.v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i)
        asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %2;\n\tadd.rn.f32.bf16 %0, lo, %0;\n\tadd.rn.f32.bf16 %1, hi, %1;\n\t}"
            : "+f"(acc[2 * i]), "+f"(acc[2 * i + 1])
            : "r"(x[i]));
}
template <typename ACC> LP_DEVINL float acc_value(ACC a);
template <> LP_DEVINL float acc_value<float>(float a) { return a; }
// one rounding (64-bit integer to FP32, to nearest); the epilogue multiplies by the exact power-of-two 1 / scale
template <> LP_DEVINL float acc_value<long long>(long long a) { return __ll2float_rn(a); }
constexpr int SPMM_HEAVY_MIN = 32;  // smallest heavy-row threshold a plan may use (bounds the item count by nnz / 32).
                                    // A lane group keeps only a few gathers in flight, so a long row handled by one
                                    // group is a long dependent chain: long rows are cut into items instead.
constexpr int SPMM_ITEM_BLOCKS = 1184;  // blocks that walk the item list (grid-stride)
constexpr int SPMM_SEG = 512;    // entries per item (one block: 8 lane groups x 64 entries for 32-lane groups)
constexpr int SPMM_PIECE = 128;  // entries per piece of the padded form; rows with more entries are cut and combined (256: slower by 2 %)
constexpr int SPMM_CHUNK_GROUPS = 16;  // groups of four entries per chunk of the padded form (one lane group walks a chunk)

// acc += sum over entries [e_lo, e_hi) of val[e] * X[col[e], :] for the chunks owned by this lane.
// The group loads up to G (col, val) pairs at once and broadcasts them; U source rows are gathered
// before any is consumed, so each lane keeps U * NV 16-byte loads in flight.  Lanes beyond the row
// width repeat the last chunk (their sums are never stored), which keeps the gathers free of
// per-lane predicates.
template <typename T, int G, int NV, int U, typename ACC, bool HAS_VAL, bool HAS_X2 = false>
LP_DEVINL void spmm_accumulate(const SpmmArgs<T> &a, int e_lo, int e_hi, int gl, unsigned gmask, int nchunks, ACC (&acc)[NV][Vec16<T>::N],
                                bool have_first = false, int first_col = 0, float first_val = 0.f)
{
    constexpr int VN = Vec16<T>::N;
    const float wscale = sizeof(ACC) == 8 ? a.exact_scale : 1.f;  // exact sums: the power-of-two scale rides on the coefficient
    for (int e0 = e_lo; e0 < e_hi; e0 += G) {
        const int my_e = e0 + gl;
        int my_col = first_col;
        float my_val = first_val;
        if (!(have_first && e0 == e_lo)) {  // the first batch of a row may have been prefetched by the caller
            my_col = 0;
            my_val = 0.f;
            if (my_e < e_hi) {
                my_col = __ldg(a.col + my_e);
                if (HAS_VAL) my_val = __ldg(a.val + my_e);
            }
        }
        int my_col2 = 0;
        if (HAS_X2 && my_e < e_hi) my_col2 = __ldg(a.col2 + my_e);
        const int cnt = min(G, e_hi - e0);
        if constexpr (sizeof(ACC) == 8) {
            // exact sums (batch incidence lists): full batches of U, then the rest one by one
            int j = 0;
            for (; j + U <= cnt; j += U) {
                int c[U];
                float w[U];
                Vec16<T> v[U][NV];
#pragma unroll
                for (int q = 0; q < U; ++q) {
                    c[q] = __shfl_sync(gmask, my_col, j + q, G);
                    w[q] = (HAS_VAL ? __shfl_sync(gmask, my_val, j + q, G) : 1.f) * wscale;
                }
#pragma unroll
                for (int q = 0; q < U; ++q)
#pragma unroll
                    for (int i = 0; i < NV; ++i) v[q][i].load(a.X + (size_t)c[q] * a.ldx + min(gl + i * G, nchunks - 1) * VN);
                if (HAS_X2) {
#pragma unroll
                    for (int q = 0; q < U; ++q) {
                        const int c2 = __shfl_sync(gmask, my_col2, j + q, G);
#pragma unroll
                        for (int i = 0; i < NV; ++i) {
                            const int ch = gl + i * G;
                            if (ch < nchunks) {
                                Vec16<T> v2;
                                v2.load(a.X2 + (size_t)c2 * a.ldx2 + ch * VN);
                                float f[VN], f2[VN];
                                v[q][i].to_float(f);
                                v2.to_float(f2);
#pragma unroll
                                for (int t = 0; t < VN; ++t) acc_add<ACC>(acc[i][t], w[q], f[t] * f2[t]);
                            }
                        }
                    }
                } else {
#pragma unroll
                    for (int q = 0; q < U; ++q)
#pragma unroll
                        for (int i = 0; i < NV; ++i) acc_add_vec<T, ACC, HAS_VAL>(acc[i], w[q], v[q][i]);
                }
            }
            for (; j < cnt; ++j) {
                const int c = __shfl_sync(gmask, my_col, j, G);
                const float w = (HAS_VAL ? __shfl_sync(gmask, my_val, j, G) : 1.f) * wscale;
                const int c2 = HAS_X2 ? __shfl_sync(gmask, my_col2, j, G) : 0;
#pragma unroll
                for (int i = 0; i < NV; ++i) {
                    const int ch = gl + i * G;
                    if (HAS_X2 ? ch < nchunks : true) {
                        Vec16<T> v;
                        v.load(a.X + (size_t)c * a.ldx + min(ch, nchunks - 1) * VN);
                        if (HAS_X2) {
                            Vec16<T> v2;
                            v2.load(a.X2 + (size_t)c2 * a.ldx2 + ch * VN);
                            float f[VN], f2[VN];
                            v.to_float(f);
                            v2.to_float(f2);
#pragma unroll
                            for (int t = 0; t < VN; ++t) acc_add<ACC>(acc[i][t], w, f[t] * f2[t]);
                        } else {
                            acc_add_vec<T, ACC, HAS_VAL>(acc[i], w, v);
                        }
                    }
                }
            }
        } else {
            // U source rows are requested together whatever is left of the batch: a short batch (a row of one to three entries,
            // the tail of a longer one) repeats its last entry in the unused slots -- a load that hits L1 -- and leaves the
            // repeats out of the sum, so that it costs one memory round trip instead of one per entry
            for (int j = 0; j < cnt; j += U) {
                int c[U];
                float w[U];
                Vec16<T> v[U][NV];
#pragma unroll
                for (int q = 0; q < U; ++q) {
                    const int src = min(j + q, cnt - 1);
                    c[q] = __shfl_sync(gmask, my_col, src, G);
                    w[q] = (HAS_VAL ? __shfl_sync(gmask, my_val, src, G) : 1.f) * wscale;
                }
#pragma unroll
                for (int q = 0; q < U; ++q)
#pragma unroll
                    for (int i = 0; i < NV; ++i) v[q][i].load(a.X + (size_t)c[q] * a.ldx + min(gl + i * G, nchunks - 1) * VN);
                if (HAS_X2) {
#pragma unroll
                    for (int q = 0; q < U; ++q) {
                        const int c2 = __shfl_sync(gmask, my_col2, min(j + q, cnt - 1), G);
                        if (j + q < cnt) {
#pragma unroll
                            for (int i = 0; i < NV; ++i) {
                                const int ch = gl + i * G;
                                if (ch < nchunks) {
                                    Vec16<T> v2;
                                    v2.load(a.X2 + (size_t)c2 * a.ldx2 + ch * VN);
                                    float f[VN], f2[VN];
                                    v[q][i].to_float(f);
                                    v2.to_float(f2);
#pragma unroll
                                    for (int t = 0; t < VN; ++t) acc_add<ACC>(acc[i][t], w[q], f[t] * f2[t]);
                                }
                            }
                        }
                    }
                } else {
#pragma unroll
                    for (int q = 0; q < U; ++q)
                        if (j + q < cnt) {
#pragma unroll
                            for (int i = 0; i < NV; ++i) acc_add_vec<T, ACC, HAS_VAL>(acc[i], w[q], v[q][i]);
                        }
                }
            }
        }
    }
}

// scale, extra term, ReLU mask, store, optional copy of the self row
template <typename T, int G, int NV, typename ACC>
LP_DEVINL void spmm_epilogue(const SpmmArgs<T> &a, int r, int gl, int nchunks, const ACC (&acc)[NV][Vec16<T>::N])
{
    constexpr int VN = Vec16<T>::N;
    const float scale = (a.row_scale ? __ldg(a.row_scale + r) : 1.f) * (sizeof(ACC) == 8 ? a.exact_inv : 1.f);
    int irow = -1;
    float icoef = 0.f;
    if (a.init) {
        irow = a.init_idx ? __ldg(a.init_idx + r) : r;
        icoef = a.init_coef ? __ldg(a.init_coef + r) : 1.f;
    }
    const int srow = a.self_out ? (a.self_idx ? __ldg(a.self_idx + r) : r) : -1;
#pragma unroll
    for (int i = 0; i < NV; ++i) {
        const int ch = gl + i * G;
        if (ch >= nchunks) continue;
        float o[VN];
#pragma unroll
        for (int t = 0; t < VN; ++t) o[t] = acc_value<ACC>(acc[i][t]) * scale;
        if (irow >= 0) {
            Vec16<T> v;
            v.load_once(a.init + (size_t)irow * a.ldinit + ch * VN);
            float f[VN];
            v.to_float(f);
#pragma unroll
            for (int t = 0; t < VN; ++t) o[t] = fmaf(icoef, f[t], o[t]);
        }
        if (a.relu_ref) {
            Vec16<T> v;
            v.load_once(a.relu_ref + (size_t)r * a.ldref + ch * VN);
            float f[VN];
            v.to_float(f);
#pragma unroll
            for (int t = 0; t < VN; ++t) o[t] = f[t] > 0.f ? o[t] : 0.f;
        }
        Vec16<T> out;
        out.from_float(o);
        out.store_once(a.Y + (size_t)r * a.ldy + ch * VN);
        if (a.Y2) {  // gathered by the next launch: an ordinary store
            const float s2 = __ldg(a.y2_scale + r);
#pragma unroll
            for (int t = 0; t < VN; ++t) o[t] *= s2;
            out.from_float(o);
            out.store(a.Y2 + (size_t)r * a.ldy2 + ch * VN);
        }
        if (srow >= 0) {
            Vec16<T> v;
            v.load(a.X + (size_t)srow * a.ldx + ch * VN);
            v.store(a.self_out + (size_t)r * a.ldself + ch * VN);
        }
    }
}

template <typename T, int G, int NV, int RPG, int U, int MINB, typename ACC, bool HAS_VAL, bool HAS_X2>
__global__ void __launch_bounds__(SPMM_THREADS, MINB) spmm_csr_kernel(const SpmmArgs<T> a, const int light_blocks)
{
    LP_DEP_ENTER();
    constexpr int VN = Vec16<T>::N;
    constexpr int NG = SPMM_THREADS / G;  // lane groups per block
    constexpr int ROWS = NG * RPG;        // rows per block: every group walks RPG rows
    __shared__ int s_ptr[ROWS + 1];
    __shared__ __align__(16) ACC s_part[NG][G * NV * VN];  // partial sums of an item, one per group
    const int n_rows = a.n_rows_dev ? min(*a.n_rows_dev, a.n_rows) : a.n_rows;
    const int g = threadIdx.x / G;   // group inside the block
    const int gl = threadIdx.x % G;  // lane inside the group
    const unsigned lane = threadIdx.x & 31;
    const unsigned gmask = (G == 32) ? 0xffffffffu : (((1u << G) - 1u) << (lane & ~(unsigned)(G - 1)));
    const int nchunks = a.F / VN;  // 16-byte chunks per row

    const int item_blocks = (int)gridDim.x - light_blocks;
    if ((int)blockIdx.x < item_blocks) {
        // ---- heavy item: SPMM_SEG consecutive entries of a hub row, one contiguous piece per lane group,
        // pieces added in group order (fixed), FP32 partial row written for the combine kernel.  The item blocks come
        // FIRST in the grid: they are the longest chains of dependent gathers, so they start before the light rows
        const int n_items = a.heavy.counts[1];
        for (int item = blockIdx.x; item < n_items; item += item_blocks) {
        const int r = a.heavy.item_row[item];
        const int sidx = item - a.heavy.item_first[item];
        const int hb = a.rowptr[r] + sidx * a.heavy.seg, he = min(a.rowptr[r + 1], hb + a.heavy.seg);
        const int piece = ((he - hb + NG - 1) / NG + U - 1) / U * U;
        const int lo = min(he, hb + g * piece), hi = min(he, lo + piece);
        ACC hacc[NV][VN];
#pragma unroll
        for (int q = 0; q < NV; ++q)
#pragma unroll
            for (int j = 0; j < VN; ++j) hacc[q][j] = ACC(0);
        spmm_accumulate<T, G, NV, U, ACC, HAS_VAL, HAS_X2>(a, lo, hi, gl, gmask, nchunks, hacc);
#pragma unroll
        for (int q = 0; q < NV; ++q)
#pragma unroll
            for (int t = 0; t < VN; ++t) s_part[g][(gl + q * G) * VN + t] = hacc[q][t];
        __syncthreads();
        for (int j = threadIdx.x; j < a.F; j += SPMM_THREADS) {
            ACC sum = ACC(0);
            for (int w = 0; w < NG; ++w) sum += s_part[w][j];
            reinterpret_cast<ACC *>(a.heavy.partials)[(size_t)item * a.F + j] = sum;
        }
        __syncthreads();
        }
        return;
    }
    const int row0 = ((int)blockIdx.x - item_blocks) * ROWS;
    if (row0 >= n_rows) return;
    for (int i = threadIdx.x; i <= ROWS; i += SPMM_THREADS) s_ptr[i] = a.rowptr[min(row0 + i, n_rows)];
    __syncthreads();

    ACC acc[NV][VN];
    // ---- light rows: group g walks rows g, g + NG, g + 2 NG, ... of the block.  The (column, coefficient)
    // pairs of the next row are fetched before the current row's gathers are consumed, so a group has
    // its index loads and its feature gathers in flight at the same time.
    int pre_col = 0;
    float pre_val = 0.f;
    {
        const int eb = s_ptr[g], ee = s_ptr[g + 1];
        if (eb + gl < ee && ee - eb <= a.heavy.threshold) {
            pre_col = __ldg(a.col + eb + gl);
            pre_val = HAS_VAL ? __ldg(a.val + eb + gl) : 1.f;
        }
    }
#pragma unroll 1
    for (int it = 0; it < RPG; ++it) {
        const int lr = it * NG + g;
        const int r = row0 + lr;
        const int e_begin = s_ptr[lr], e_end = s_ptr[lr + 1];
        const int cur_col = pre_col;
        const float cur_val = pre_val;
        if (it + 1 < RPG) {
            const int eb = s_ptr[lr + NG], ee = s_ptr[lr + NG + 1];
            pre_col = 0;
            pre_val = 0.f;
            if (eb + gl < ee && ee - eb <= a.heavy.threshold) {
                pre_col = __ldg(a.col + eb + gl);
                pre_val = HAS_VAL ? __ldg(a.val + eb + gl) : 1.f;
            }
        }
        if (r < n_rows && e_end == e_begin && !a.init && !a.self_out) {
            // empty row without an extra term: the output row is zero
            Vec16<T> z;
            float zf[VN];
#pragma unroll
            for (int j = 0; j < VN; ++j) zf[j] = 0.f;
            z.from_float(zf);
#pragma unroll
            for (int i = 0; i < NV; ++i) {
                const int ch = gl + i * G;
                if (ch < nchunks) z.store(a.Y + (size_t)r * a.ldy + ch * VN);
            }
        } else if (r < n_rows && e_end - e_begin <= a.heavy.threshold) {
#pragma unroll
            for (int i = 0; i < NV; ++i)
#pragma unroll
                for (int j = 0; j < VN; ++j) acc[i][j] = ACC(0);
            spmm_accumulate<T, G, NV, U, ACC, HAS_VAL, HAS_X2>(a, e_begin, e_end, gl, gmask, nchunks, acc, !HAS_X2, cur_col, cur_val);
            spmm_epilogue<T, G, NV, ACC>(a, r, gl, nchunks, acc);
        }
    }
}


// ---------------------------------------------------------------------------------------------
// Padded flat form for static structures (one 16-byte vector per lane, FP32 sums, source rows G * MULT vectors apart).
// A lane group streams the groups of one chunk: the four rows a group names are gathered at once and added in entry
// order; when the group finishes a piece, the epilogue runs (only piece of a row) or the FP32 partial row is written
// for the combine kernel (piece of a heavy row), and the sums restart from zero.  A row that is one piece is summed
// in the same order as by the row-per-group kernel and gives the same bits.  Nothing in the inner loop depends on a
// row's length: no tails, no per-entry end tests, the next group's indices are fetched while this group's rows are
// in flight, a short row costs one group instead of a round trip of its own, and hub rows are pieces like any other.
// Only the last group of a piece can hold pads: they repeat an index of the group (a load that hits L1) and are left
// out of the sum by a count the finishing code carries (unit coefficients) or by their zero coefficient.
// ---------------------------------------------------------------------------------------------
// EPI 1: the epilogue is the row scale alone (mean aggregation forward); EPI 2: extra term with unit coefficient and
// ReLU mask and nothing else (adjoint of the mean aggregation).  Both are written out compactly so that the loop keeps
// the register budget of a bare gather; EPI 0 is the general epilogue.
LP_DEVINL void prefetch_l1(const void *p) { asm volatile("prefetch.global.L1 [%0];" ::"l"(p)); }

template <typename T, int G, int MULT, int MINB, bool HAS_VAL, int EPI>
__global__ void __launch_bounds__(SPMM_THREADS, MINB) spmm_padded_kernel(const SpmmArgs<T> a)
{
    LP_DEP_ENTER();
    constexpr int VN = Vec16<T>::N;
    constexpr int NG = SPMM_THREADS / G;
    constexpr unsigned PITCH = (unsigned)(G * VN * MULT);  // elements between source rows
    const int gl = threadIdx.x % G;
    const int nchunks = a.F / VN;
    const int c = blockIdx.x * NG + threadIdx.x / G;
    if (c >= a.heavy.n_chunks) return;
    const int gs = __ldg(a.heavy.chunk_start + c), ge = __ldg(a.heavy.chunk_start + c + 1);
    if (gs >= ge) return;
    const T *xl = a.X + min(gl, nchunks - 1) * VN;  // lanes beyond the row width repeat the last chunk and store nothing
    float acc[1][VN];
#pragma unroll
    for (int t = 0; t < VN; ++t) acc[0][t] = 0.f;
    int4 cn = __ldg(a.heavy.pcol + gs);
    float4 wn = HAS_VAL ? __ldg(a.heavy.pval + gs) : make_float4(1.f, 1.f, 1.f, 1.f);
    int rn = __ldg(a.heavy.grow + gs);
    for (int grp = gs; grp < ge; ++grp) {
        const int4 cc = cn;
        const float4 ww = wn;
        const int rr = rn;
        Vec16<T> v0, v1, v2, v3;
        v0.load(xl + (size_t)(unsigned)cc.x * PITCH);
        v1.load(xl + (size_t)(unsigned)cc.y * PITCH);
        v2.load(xl + (size_t)(unsigned)cc.z * PITCH);
        v3.load(xl + (size_t)(unsigned)cc.w * PITCH);
        if (grp + 1 < ge) {
            cn = __ldg(a.heavy.pcol + grp + 1);
            if (HAS_VAL) wn = __ldg(a.heavy.pval + grp + 1);
            rn = __ldg(a.heavy.grow + grp + 1);
        }
        const int id = rr >> 4;  // row or partial slot finished by this group (when rr != -1)
        if constexpr (EPI != 1) {
            // the row operands of the epilogue (extra term, ReLU reference) are requested when this group finishes a
            // row, before its gathers are waited for, so that the epilogue finds them in L1
            if (rr != -1 && (rr & 8) == 0 && gl < nchunks) {
                if (a.init) prefetch_l1(a.init + (size_t)id * a.ldinit + gl * VN);
                if (a.relu_ref) prefetch_l1(a.relu_ref + (size_t)id * a.ldref + gl * VN);
            }
        }
        if (rr == -1 || (HAS_VAL && (rr & 7) != 0)) {  // inside a piece all four entries are real; with coefficients a pad
                                                        // repeats a real entry of its group under a zero coefficient
            acc_add_vec<T, float, HAS_VAL>(acc[0], ww.x, v0);
            acc_add_vec<T, float, HAS_VAL>(acc[0], ww.y, v1);
            acc_add_vec<T, float, HAS_VAL>(acc[0], ww.z, v2);
            acc_add_vec<T, float, HAS_VAL>(acc[0], ww.w, v3);
        } else if (!HAS_VAL) {  // (with coefficients what is left is the all-pad group of an empty row: nothing to add)
            const int cnt = rr & 7;
            if (cnt > 0) acc_add_vec<T, float, HAS_VAL>(acc[0], ww.x, v0);
            if (cnt > 1) acc_add_vec<T, float, HAS_VAL>(acc[0], ww.y, v1);
            if (cnt > 2) acc_add_vec<T, float, HAS_VAL>(acc[0], ww.z, v2);
            if (cnt > 3) acc_add_vec<T, float, HAS_VAL>(acc[0], ww.w, v3);
        }
        if (rr != -1) {
            if ((rr & 8) == 0) {
                const int row = id;
                if constexpr (EPI == 1) {
                    if (gl < nchunks) {
                        const float scale = a.row_scale ? __ldg(a.row_scale + row) : 1.f;
                        float o[VN];
#pragma unroll
                        for (int t = 0; t < VN; ++t) o[t] = acc[0][t] * scale;
                        Vec16<T> out;
                        out.from_float(o);
                        out.store_once(a.Y + (size_t)row * a.ldy + gl * VN);
                    }
                } else if constexpr (EPI == 2) {
                    if (gl < nchunks) {  // y = relu_ref > 0 ? sum + init : 0 (the general epilogue's arithmetic with scale and coefficient 1)
                        Vec16<T> vi, vr;
                        vi.load_once(a.init + (size_t)row * a.ldinit + gl * VN);
                        vr.load_once(a.relu_ref + (size_t)row * a.ldref + gl * VN);
                        float fi[VN], fr[VN];
                        vi.to_float(fi);
                        vr.to_float(fr);
#pragma unroll
                        for (int t = 0; t < VN; ++t) fi[t] = fr[t] > 0.f ? fmaf(1.f, fi[t], acc[0][t] * 1.f) : 0.f;
                        Vec16<T> out;
                        out.from_float(fi);
                        out.store_once(a.Y + (size_t)row * a.ldy + gl * VN);
                    }
                } else {
                    spmm_epilogue<T, G, 1, float>(a, row, gl, nchunks, acc);
                }
            } else if (gl < nchunks) {
                float *dst = a.heavy.partials + (size_t)id * a.F + gl * VN;
#pragma unroll
                for (int t = 0; t < VN; t += 4) *reinterpret_cast<float4 *>(dst + t) = make_float4(acc[0][t], acc[0][t + 1], acc[0][t + 2], acc[0][t + 3]);
            }
#pragma unroll
            for (int t = 0; t < VN; ++t) acc[0][t] = 0.f;
        }
    }
}

// groups owned by every row of the padded form
LP_DEVINL int padded_row_groups(int d, int threshold)
{
    if (d <= threshold) return max(1, (d + 3) / 4);
    const int rem = d % SPMM_PIECE;
    return (d / SPMM_PIECE) * (SPMM_PIECE / 4) + (rem + 3) / 4;
}
__global__ void padded_count_kernel(const int *__restrict__ rowptr, int n, int threshold, int *__restrict__ ngroups)
{
    LP_DEP_ENTER();
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= n) return;
    ngroups[r] = padded_row_groups(rowptr[r + 1] - rowptr[r], threshold);
}
// chunk starts contributed by row r: every piece of a heavy row opens a chunk; a light row opens one when it is the
// first row, follows a heavy row, or when first_group crosses a multiple of SPMM_CHUNK_GROUPS between rows r - 1 and r
__global__ void padded_chunk_count_kernel(const int *__restrict__ rowptr, const int *__restrict__ first_group, int n, int threshold, int *__restrict__ count)
{
    LP_DEP_ENTER();
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= n) return;
    const int d = rowptr[r + 1] - rowptr[r];
    if (d > threshold) {
        count[r] = (d + SPMM_PIECE - 1) / SPMM_PIECE;
        return;
    }
    const bool opens = r == 0 || rowptr[r] - rowptr[r - 1] > threshold || first_group[r] / SPMM_CHUNK_GROUPS != first_group[r - 1] / SPMM_CHUNK_GROUPS;
    count[r] = opens ? 1 : 0;
}
// one thread per row writes the row's groups, their finishing codes and the chunk offsets it contributes
__global__ void padded_fill_kernel(const int *__restrict__ rowptr, const int *__restrict__ col, const float *__restrict__ val, int n, int threshold,
                                   const int *__restrict__ first_group, const int *__restrict__ chunk_count, const int *__restrict__ chunk_of,
                                   const int *__restrict__ row_base, int *__restrict__ chunk_start, int *__restrict__ pcol, float *__restrict__ pval,
                                   int *__restrict__ grow)
{
    LP_DEP_ENTER();
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= n) return;
    if (r == n - 1) chunk_start[chunk_of[n]] = first_group[n];  // chunk_of[n] = number of chunks, first_group[n] = all groups
    const int b = rowptr[r], d = rowptr[r + 1] - b;
    const bool heavy = d > threshold;
    const int np = heavy ? (d + SPMM_PIECE - 1) / SPMM_PIECE : 1;
    int g = first_group[r];
    if (!heavy && chunk_count[r]) chunk_start[chunk_of[r]] = g;
    for (int s = 0; s < np; ++s) {
        const int lo = s * SPMM_PIECE;
        const int len = heavy ? min(SPMM_PIECE, d - lo) : d;
        const int ng = max(1, (len + 3) / 4);
        if (heavy) chunk_start[chunk_of[r] + s] = g;
        for (int i = 0; i < 4 * ng; ++i) {
            const int first = (i / 4) * 4;  // a pad repeats the first index of its group (row 0 in an all-pad group)
            pcol[4 * (size_t)g + i] = i < len ? col[b + lo + i] : (first < len ? col[b + lo + first] : 0);
            if (pval) pval[4 * (size_t)g + i] = i < len ? val[b + lo + i] : 0.f;
        }
        const int cnt = len - 4 * (ng - 1);  // real entries of the last group: 1..4, 0 for an empty row
        const int code = heavy ? ((row_base[r] + s) << 4 | 8 | cnt) : (r << 4 | cnt);
        for (int j = 0; j < ng; ++j) grow[g + j] = j < ng - 1 ? -1 : code;
        g += ng;
    }
}

// one row of a heavy-row plan: a row above the threshold claims a slot and a run of items
// (row_base, optional: first item of every heavy row, -1 for the others)
LP_DEVINL void heavy_plan_row(const int *__restrict__ rowptr, int r, const HeavyPlan &hp, int *__restrict__ row_base)
{
    const int d = rowptr[r + 1] - rowptr[r];
    if (d <= hp.threshold) {
        if (row_base) row_base[r] = -1;
        return;
    }
    const int nseg = (d + hp.seg - 1) / hp.seg;
    const int i = atomicAdd(&hp.counts[0], 1);
    const int b = atomicAdd(&hp.counts[1], nseg);
    hp.rows[i] = r;
    hp.base[i] = b;
    if (hp.nseg) hp.nseg[i] = nseg;
    if (row_base) row_base[r] = b;
    for (int s = 0; s < nseg; ++s) {
        hp.item_row[b + s] = r;
        hp.item_first[b + s] = b;
    }
}
// one thread per row
__global__ void spmm_heavy_plan_kernel(const int *__restrict__ rowptr, int n_rows, const int *__restrict__ n_rows_dev, HeavyPlan hp,
                                       int *__restrict__ row_base = nullptr)
{
    LP_DEP_ENTER();
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    const int lim = n_rows_dev ? min(*n_rows_dev, n_rows) : n_rows;
    if (r >= lim) return;
    heavy_plan_row(rowptr, r, hp, row_base);
}

// adds the items of every heavy row in item order (fixed) and applies the epilogue; one lane group per row
template <typename T, int G, int NV, typename ACC>
__global__ void __launch_bounds__(SPMM_THREADS) spmm_heavy_combine_kernel(const SpmmArgs<T> a)
{
    LP_DEP_ENTER();
    constexpr int VN = Vec16<T>::N;
    constexpr int NG = SPMM_THREADS / G;
    const int count = a.heavy.counts[0];
    const int g = threadIdx.x / G, gl = threadIdx.x % G;
    const int nchunks = a.F / VN;
    for (int i = blockIdx.x * NG + g; i < count; i += gridDim.x * NG) {
        const int r = a.heavy.rows[i], b = a.heavy.base[i];
        const int nseg = a.heavy.nseg ? a.heavy.nseg[i] : (a.rowptr[r + 1] - a.rowptr[r] + a.heavy.seg - 1) / a.heavy.seg;
        ACC acc[NV][VN];
#pragma unroll
        for (int q = 0; q < NV; ++q)
#pragma unroll
            for (int t = 0; t < VN; ++t) acc[q][t] = ACC(0);
        // a batch of partial rows is fetched before any is added (the additions stay in item order); a batch that reaches
        // past the row's last item fetches nothing there and adds zero, so that a short row is one round trip, not one per item
        int s = 0;
        if constexpr (NV == 1) {
            constexpr int W = sizeof(ACC) == 4 ? 8 : 4;
            if (gl < nchunks) {
                for (; s < nseg; s += W) {
                    ACC tmp[W][VN];
#pragma unroll
                    for (int u = 0; u < W; ++u) {
                        const ACC *p = reinterpret_cast<const ACC *>(a.heavy.partials) + (size_t)(b + s + u) * a.F + gl * VN;
                        const bool in = s + u < nseg;
#pragma unroll
                        for (int t = 0; t < VN; ++t) tmp[u][t] = in ? p[t] : ACC(0);
                    }
#pragma unroll
                    for (int u = 0; u < W; ++u)
#pragma unroll
                        for (int t = 0; t < VN; ++t) acc[0][t] += tmp[u][t];
                }
            }
            s = nseg;
        }
        for (; s < nseg; ++s) {
            const ACC *p = reinterpret_cast<const ACC *>(a.heavy.partials) + (size_t)(b + s) * a.F;
#pragma unroll
            for (int q = 0; q < NV; ++q) {
                const int ch = gl + q * G;
                if (ch < nchunks) {
#pragma unroll
                    for (int t = 0; t < VN; ++t) acc[q][t] += p[ch * VN + t];
                }
            }
        }
        spmm_epilogue<T, G, NV, ACC>(a, r, gl, nchunks, acc);
    }
}

template <typename T, int G, int NV, int RPG, int U, int MINB, typename ACC> static void spmm_launch_cfg(Exec &ex, const SpmmArgs<T> &a)
{
    constexpr int ROWS = (SPMM_THREADS / G) * RPG;
    constexpr int NG = SPMM_THREADS / G;
    const int light_blocks = (int)ceil_div64(a.n_rows, ROWS);
    if (light_blocks == 0) return;
    // static structure with a padded plan and source rows G or 2 G vectors apart: the padded kernel walks every row
    if constexpr (NV == 1 && sizeof(ACC) == 4) {
        const int pitch = a.ldx / Vec16<T>::N;
        if (a.heavy.pcol != nullptr && a.heavy.n_chunks > 0 && !a.X2 && !a.self_out && !a.Y2 && !a.n_rows_dev && !a.init_idx && a.ldx % Vec16<T>::N == 0 &&
            (pitch == G || pitch == 2 * G) &&
            (a.val == nullptr || (a.val == a.heavy.pval_src && a.heavy.pval != nullptr) || (a.val == a.heavy.pval2_src && a.heavy.pval2 != nullptr))) {
            SpmmArgs<T> b = a;
            if (a.val && a.val != a.heavy.pval_src) b.heavy.pval = a.heavy.pval2;
            b.heavy.rows = a.heavy.p_rows;
            b.heavy.base = a.heavy.p_base;
            b.heavy.counts = a.heavy.p_counts;
            b.heavy.nseg = a.heavy.p_nseg;
            b.heavy.seg = SPMM_PIECE;
            const unsigned pgrid = (unsigned)ceil_div64(a.heavy.n_chunks, NG);
            const bool plain = !a.init && !a.relu_ref;
            const bool self_mask = a.init && a.relu_ref && !a.init_coef && !a.row_scale && !a.val;
#define LP_PADDED(MULT_, VAL_) do { \
                if (plain) launch_dep(spmm_padded_kernel<T, G, MULT_, VAL_ ? 5 : 6, VAL_, 1>, dim3(pgrid), dim3(SPMM_THREADS), 0, ex.st, b); \
                else if (self_mask) launch_dep(spmm_padded_kernel<T, G, MULT_, 5, false, 2>, dim3(pgrid), dim3(SPMM_THREADS), 0, ex.st, b); \
                else launch_dep(spmm_padded_kernel<T, G, MULT_, 5, VAL_, 0>, dim3(pgrid), dim3(SPMM_THREADS), 0, ex.st, b); } while (0)
            if (pitch == G) {
                if (a.val) LP_PADDED(1, true); else LP_PADDED(1, false);
            } else {
                if (a.val) LP_PADDED(2, true); else LP_PADDED(2, false);
            }
#undef LP_PADDED
            ex.launches += 1;
            if (a.heavy.p_host_rows > 0) {
                launch_dep(spmm_heavy_combine_kernel<T, G, NV, ACC>, dim3((unsigned)std::min<int64_t>(592, ceil_div64(a.heavy.p_host_rows, NG))), dim3(SPMM_THREADS), 0, ex.st, b);
                ex.launches += 1;
            }
            return;
        }
    }
    int64_t items = a.heavy.host_items;
    if (items < 0) {  // plan unknown on the host: rebuild it on the device, size the grid by the upper bound
        if (!a.heavy.plan_prebuilt) {
            if (!a.heavy.counts_zeroed) cudaMemsetAsync(a.heavy.counts, 0, 2 * sizeof(int), ex.st);
            launch_dep(spmm_heavy_plan_kernel, dim3((unsigned)ceil_div64(a.n_rows, 256)), dim3(256), 0, ex.st, a.rowptr, a.n_rows, a.n_rows_dev, a.heavy, nullptr);
            ex.launches += 1;
        }
        items = a.nnz / SPMM_HEAVY_MIN;  // a heavy row has more than SPMM_HEAVY_MIN entries and at most deg / SPMM_HEAVY_MIN items
    }
    const int item_blocks = (int)std::min<int64_t>(items, SPMM_ITEM_BLOCKS);
    const unsigned grid = (unsigned)(light_blocks + item_blocks);
    bool launched = false;
    if constexpr (sizeof(ACC) == 8) {  // the two-operand form exists for the exact accumulator only
        if (a.X2) {
            launch_dep(spmm_csr_kernel<T, G, NV, RPG, U, MINB, ACC, false, true>, dim3(grid), dim3(SPMM_THREADS), 0, ex.st, a, light_blocks);
            launched = true;
        }
    }
    if (!launched) {
        if (a.val) launch_dep(spmm_csr_kernel<T, G, NV, RPG, U, MINB, ACC, true, false>, dim3(grid), dim3(SPMM_THREADS), 0, ex.st, a, light_blocks);
        else launch_dep(spmm_csr_kernel<T, G, NV, RPG, U, MINB, ACC, false, false>, dim3(grid), dim3(SPMM_THREADS), 0, ex.st, a, light_blocks);
    }
    ex.launches += 1;
    if (a.heavy.host_rows != 0) {
        const int64_t rows_bound = a.heavy.host_rows > 0 ? a.heavy.host_rows : std::max<int64_t>(1, items);
        const unsigned grid = (unsigned)std::min<int64_t>(592, ceil_div64(rows_bound, NG));
        launch_dep(spmm_heavy_combine_kernel<T, G, NV, ACC>, dim3(grid), dim3(SPMM_THREADS), 0, ex.st, a);
        ex.launches += 1;
    }
}

// Launch shape (measured on a 200k-node power-law graph, BF16): with one 16-byte vector per lane, 4 gathers in
// flight per lane at 48 registers (5 blocks per SM) beat 8 gathers at 80 registers (3 blocks) by about 10 %.
template <typename T, int G, int NV, typename ACC> static void spmm_launch_gn(Exec &ex, const SpmmArgs<T> &a)
{
    constexpr bool EXACT = sizeof(ACC) == 8;  // 64-bit accumulators need twice the registers
    if constexpr (NV == 1) spmm_launch_cfg<T, G, NV, 8, 4, EXACT ? 3 : 5, ACC>(ex, a);
    else if constexpr (NV == 2) spmm_launch_cfg<T, G, NV, 8, EXACT ? 2 : 4, 2, ACC>(ex, a);
    else spmm_launch_cfg<T, G, NV, 8, 2, EXACT ? 1 : 2, ACC>(ex, a);
}

// F must be a multiple of the 16-byte vector width and at most 32 * 4 vectors wide.  ACC = float sums a
// row's entries in their stored order; ACC = long long sums exactly (order-free), for lists whose entry
// order is not reproducible.  The item partials then hold 8 bytes per element.
template <typename T, typename ACC = float> static bool spmm_launch(Exec &ex, const SpmmArgs<T> &a)
{
    constexpr int VN = Vec16<T>::N;
    if (a.F <= 0 || a.F % VN != 0 || !a.heavy.counts || !a.heavy.partials) return false;
    if (a.X2 && (sizeof(ACC) != 8 || a.val || !a.col2)) return false;
    const int chunks = a.F / VN;
    if (chunks <= 8) spmm_launch_gn<T, 8, 1, ACC>(ex, a);
    else if (chunks <= 16) spmm_launch_gn<T, 16, 1, ACC>(ex, a);
    else if (chunks <= 32) spmm_launch_gn<T, 32, 1, ACC>(ex, a);
    else if (chunks <= 64) spmm_launch_gn<T, 32, 2, ACC>(ex, a);
    else if (chunks <= 128) {
        // 64-bit partials of 1024 BF16 columns would not fit the static shared memory; widths stop at 512 anyway
        if constexpr (sizeof(ACC) == 8 && sizeof(T) == 2) return false;
        else spmm_launch_gn<T, 32, 4, ACC>(ex, a);
    } else return false;
    return true;
}
