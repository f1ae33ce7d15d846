// CSR neighbour aggregation (AGG of Eq. 1, and its adjoint over the transposed structure).
//
//   Y[r, :] = mask_r( init_coef[r] * Init[init_idx[r], :]  +  row_scale[r] * sum_e val[e] * X[col[e], :] )
//
// One group of G lanes (8, 16 or 32) owns a row; every lane gathers 16-byte vectors of the
// source rows (4 floats or 8 bf16) and accumulates in FP32 in entry order.  Rows with more than
// SPMM_HEAVY entries (power-law hubs) are split into one contiguous segment per lane group of the
// block and the partial sums are added in segment order, so a hub costs one block a few
// microseconds instead of one warp hundreds.  The summation order is a function of the row length
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

template <typename T> struct SpmmArgs {
    int n_rows = 0;
    const int *n_rows_dev = nullptr;  // optional device-resident row count (<= n_rows)
    const int *rowptr = nullptr;
    const int *col = nullptr;
    const float *val = nullptr;
    const float *row_scale = nullptr;
    const T *X = nullptr;
    int ldx = 0;
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
};

constexpr int SPMM_THREADS = 256;
constexpr int SPMM_HEAVY = 256;  // rows with more entries than this are processed by the whole block

// acc += sum over entries [e_lo, e_hi) of val[e] * X[col[e], :] for the chunks owned by this lane.
// The group loads up to G (col, val) pairs at once and broadcasts them; U source rows are gathered
// before any is consumed, so each lane keeps U * NV 16-byte loads in flight.
template <typename T, int G, int NV, int U>
LP_DEVINL void spmm_accumulate(const SpmmArgs<T> &a, int e_lo, int e_hi, int gl, unsigned gmask, int nchunks, float (&acc)[NV][Vec16<T>::N])
{
    constexpr int VN = Vec16<T>::N;
    for (int e0 = e_lo; e0 < e_hi; e0 += G) {
        const int my_e = e0 + gl;
        int my_col = 0;
        float my_val = 0.f;
        if (my_e < e_hi) {
            my_col = __ldg(a.col + my_e);
            my_val = a.val ? __ldg(a.val + my_e) : 1.f;
        }
        const int cnt = min(G, e_hi - e0);
        int j = 0;
        for (; j + U <= cnt; j += U) {
            int c[U];
            float w[U];
            Vec16<T> v[U][NV];
#pragma unroll
            for (int q = 0; q < U; ++q) {
                c[q] = __shfl_sync(gmask, my_col, j + q, G);
                w[q] = __shfl_sync(gmask, my_val, j + q, G);
            }
#pragma unroll
            for (int q = 0; q < U; ++q)
#pragma unroll
                for (int i = 0; i < NV; ++i) {
                    const int ch = gl + i * G;
                    if (ch < nchunks) v[q][i].load(a.X + (size_t)c[q] * a.ldx + ch * VN);
                }
#pragma unroll
            for (int q = 0; q < U; ++q)
#pragma unroll
                for (int i = 0; i < NV; ++i) {
                    const int ch = gl + i * G;
                    if (ch < nchunks) {
                        float f[VN];
                        v[q][i].to_float(f);
#pragma unroll
                        for (int t = 0; t < VN; ++t) acc[i][t] = fmaf(w[q], f[t], acc[i][t]);
                    }
                }
        }
        for (; j < cnt; ++j) {
            const int c = __shfl_sync(gmask, my_col, j, G);
            const float w = __shfl_sync(gmask, my_val, j, G);
#pragma unroll
            for (int i = 0; i < NV; ++i) {
                const int ch = gl + i * G;
                if (ch < nchunks) {
                    Vec16<T> v;
                    v.load(a.X + (size_t)c * a.ldx + ch * VN);
                    float f[VN];
                    v.to_float(f);
#pragma unroll
                    for (int t = 0; t < VN; ++t) acc[i][t] = fmaf(w, f[t], acc[i][t]);
                }
            }
        }
    }
}

// scale, extra term, ReLU mask, store, optional copy of the self row
template <typename T, int G, int NV>
LP_DEVINL void spmm_epilogue(const SpmmArgs<T> &a, int r, int gl, int nchunks, const float (&acc)[NV][Vec16<T>::N])
{
    constexpr int VN = Vec16<T>::N;
    const float scale = a.row_scale ? __ldg(a.row_scale + r) : 1.f;
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
        for (int t = 0; t < VN; ++t) o[t] = acc[i][t] * scale;
        if (irow >= 0) {
            Vec16<T> v;
            v.load(a.init + (size_t)irow * a.ldinit + ch * VN);
            float f[VN];
            v.to_float(f);
#pragma unroll
            for (int t = 0; t < VN; ++t) o[t] = fmaf(icoef, f[t], o[t]);
        }
        if (a.relu_ref) {
            Vec16<T> v;
            v.load(a.relu_ref + (size_t)r * a.ldref + ch * VN);
            float f[VN];
            v.to_float(f);
#pragma unroll
            for (int t = 0; t < VN; ++t) o[t] = f[t] > 0.f ? o[t] : 0.f;
        }
        Vec16<T> out;
        out.from_float(o);
        out.store(a.Y + (size_t)r * a.ldy + ch * VN);
        if (srow >= 0) {
            Vec16<T> v;
            v.load(a.X + (size_t)srow * a.ldx + ch * VN);
            v.store(a.self_out + (size_t)r * a.ldself + ch * VN);
        }
    }
}

template <typename T, int G, int NV>
__global__ void __launch_bounds__(SPMM_THREADS) spmm_csr_kernel(const SpmmArgs<T> a)
{
    constexpr int VN = Vec16<T>::N;
    constexpr int ROWS = SPMM_THREADS / G;  // rows per block = lane groups per block
    constexpr int U = (NV == 1) ? 8 : (NV == 2 ? 4 : 2);
    __shared__ int s_ptr[ROWS + 1];
    __shared__ __align__(16) float s_part[ROWS][G * NV * VN];  // partial sums of a heavy row, one per group
    const int n_rows = a.n_rows_dev ? min(*a.n_rows_dev, a.n_rows) : a.n_rows;
    const int row0 = blockIdx.x * ROWS;
    if (row0 >= n_rows) return;
    if (threadIdx.x <= ROWS) s_ptr[threadIdx.x] = a.rowptr[min(row0 + (int)threadIdx.x, n_rows)];
    __syncthreads();
    const int g = threadIdx.x / G;   // group (row) inside the block
    const int gl = threadIdx.x % G;  // lane inside the group
    const int r = row0 + g;
    const unsigned lane = threadIdx.x & 31;
    const unsigned gmask = (G == 32) ? 0xffffffffu : (((1u << G) - 1u) << (lane & ~(unsigned)(G - 1)));
    const int nchunks = a.F / VN;  // 16-byte chunks per row

    float acc[NV][VN];
    // ---- light rows: one lane group per row, entries in order
    const int e_begin = s_ptr[g], e_end = s_ptr[g + 1];
    if (r < n_rows && e_end - e_begin <= SPMM_HEAVY) {
#pragma unroll
        for (int i = 0; i < NV; ++i)
#pragma unroll
            for (int j = 0; j < VN; ++j) acc[i][j] = 0.f;
        spmm_accumulate<T, G, NV, U>(a, e_begin, e_end, gl, gmask, nchunks, acc);
        spmm_epilogue<T, G, NV>(a, r, gl, nchunks, acc);
    }
    // ---- heavy rows (power-law hubs): every group of the block takes one contiguous segment of the
    // row, the partial sums meet in shared memory and are added in segment order (fixed order, no atomics)
    for (int hr = 0; hr < ROWS; ++hr) {
        const int hb = s_ptr[hr], he = s_ptr[hr + 1];
        if (row0 + hr >= n_rows || he - hb <= SPMM_HEAVY) continue;  // uniform over the block
        const int seg = ((he - hb + ROWS - 1) / ROWS + G - 1) / G * G;
        const int lo = min(he, hb + g * seg), hi = min(he, lo + seg);
#pragma unroll
        for (int i = 0; i < NV; ++i)
#pragma unroll
            for (int j = 0; j < VN; ++j) acc[i][j] = 0.f;
        spmm_accumulate<T, G, NV, U>(a, lo, hi, gl, gmask, nchunks, acc);
#pragma unroll
        for (int i = 0; i < NV; ++i)
#pragma unroll
            for (int t = 0; t < VN; ++t) s_part[g][(gl + i * G) * VN + t] = acc[i][t];
        __syncthreads();
        if (g == 0) {
#pragma unroll
            for (int i = 0; i < NV; ++i)
#pragma unroll
                for (int t = 0; t < VN; ++t) {
                    float s = 0.f;
                    for (int q = 0; q < ROWS; ++q) s += s_part[q][(gl + i * G) * VN + t];
                    acc[i][t] = s;
                }
            spmm_epilogue<T, G, NV>(a, row0 + hr, gl, nchunks, acc);
        }
        __syncthreads();
    }
}

template <typename T, int G, int NV> static void spmm_launch_gn(Exec &ex, const SpmmArgs<T> &a)
{
    constexpr int ROWS = SPMM_THREADS / G;
    const unsigned blocks = (unsigned)ceil_div64(a.n_rows, ROWS);
    if (blocks == 0) return;
    spmm_csr_kernel<T, G, NV><<<blocks, SPMM_THREADS, 0, ex.st>>>(a);
    ex.launches += 1;
}

// F must be a multiple of the 16-byte vector width and at most 32 * 4 vectors wide.
template <typename T> static bool spmm_launch(Exec &ex, const SpmmArgs<T> &a)
{
    constexpr int VN = Vec16<T>::N;
    if (a.F <= 0 || a.F % VN != 0) return false;
    const int chunks = a.F / VN;
    if (chunks <= 8) spmm_launch_gn<T, 8, 1>(ex, a);
    else if (chunks <= 16) spmm_launch_gn<T, 16, 1>(ex, a);
    else if (chunks <= 32) spmm_launch_gn<T, 32, 1>(ex, a);
    else if (chunks <= 64) spmm_launch_gn<T, 32, 2>(ex, a);
    else if (chunks <= 128) spmm_launch_gn<T, 32, 4>(ex, a);
    else return false;
    return true;
}
