// Degree-based effective-resistance sparsification (Algorithm 1, sparsification block; Theorems 1 and 2):
// L draws with replacement, edge {u, v} drawn with probability p = (1/d_u + 1/d_v) / n' (n' = number of
// non-isolated nodes, the normaliser that makes the probabilities sum to one), every draw adding
// 1 / (L p) to the weight of its edge.  A draw picks a non-isolated node uniformly and then one of
// its neighbours uniformly, which hits the unordered edge with exactly that probability.  Draw l
// uses words 0 and 1 of philox(counter = (lo32(l), hi32(l), 0, 4), key = seed).  Hits are counted
// with integer atomics (exact, order-free), so the kept structure is reproducible bit for bit.
#pragma once
#include "common.cuh"
#include "scan_sort.cuh"
#include "sampler.cuh"

__global__ void sp_nonisolated_kernel(const int *__restrict__ rowptr, int n, int *__restrict__ flags)
{
    LP_DEP_ENTER();
    const int v = blockIdx.x * blockDim.x + threadIdx.x;
    if (v < n) flags[v] = rowptr[v + 1] > rowptr[v] ? 1 : 0;
}

__global__ void sp_compact_kernel(const int *__restrict__ rowptr, const int *__restrict__ pos, int n, int *__restrict__ nz)
{
    LP_DEP_ENTER();
    const int v = blockIdx.x * blockDim.x + threadIdx.x;
    if (v < n && rowptr[v + 1] > rowptr[v]) nz[pos[v]] = v;
}

// one thread per draw; err bit 1 = the mirrored entry is missing (the graph is not symmetric)
__global__ void sp_draw_kernel(const int *__restrict__ rowptr, const int *__restrict__ col, const int *__restrict__ nz, uint32_t n_nz, uint2 key,
                               int64_t L, int *__restrict__ hits, int *__restrict__ err)
{
    LP_DEP_ENTER();
    const int64_t l = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (l >= L) return;
    const uint4 r = philox4x32_10(make_uint4((uint32_t)l, (uint32_t)((uint64_t)l >> 32), 0u, DRAW_SPARSIFY), key);
    const int u = nz[__umulhi(r.x, n_nz)];
    const int r0 = rowptr[u], du = rowptr[u + 1] - r0;
    const int e = r0 + (int)__umulhi(r.y, (uint32_t)du);
    const int v = col[e];
    int lo = rowptr[v], hi = rowptr[v + 1];
    const int end = hi;
    while (lo < hi) {
        const int mid = lo + ((hi - lo) >> 1);
        if (col[mid] < u) lo = mid + 1; else hi = mid;
    }
    if (lo >= end || col[lo] != u) { atomicOr(err, 1); return; }
    atomicAdd(&hits[e], 1);
    atomicAdd(&hits[lo], 1);
}

__global__ void sp_keep_flags_kernel(const int *__restrict__ hits, int64_t nnz, int *__restrict__ flags)
{
    LP_DEP_ENTER();
    const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e < nnz) flags[e] = hits[e] > 0 ? 1 : 0;
}

// one thread per row: emits its kept entries in order and the new row offset
__global__ void sp_emit_kernel(const int *__restrict__ rowptr, const int *__restrict__ col, const int *__restrict__ hits, const int *__restrict__ pos,
                               int n, double n_nz, double L, int64_t *__restrict__ out_ptr, int *__restrict__ out_col, float *__restrict__ out_w)
{
    LP_DEP_ENTER();
    const int v = blockIdx.x * blockDim.x + threadIdx.x;
    if (v > n) return;
    if (v == n) { out_ptr[n] = pos[rowptr[n]]; return; }
    const int a = rowptr[v], b = rowptr[v + 1];
    out_ptr[v] = pos[a];
    const double dv = (double)(b - a);
    for (int e = a; e < b; ++e) {
        const int h = hits[e];
        if (h > 0) {
            const int u = col[e];
            const double du = (double)(rowptr[u + 1] - rowptr[u]);
            const double p = (1.0 / du + 1.0 / dv) / n_nz;
            out_col[pos[e]] = u;
            out_w[pos[e]] = (float)((double)h * (1.0 / (L * p)));
        }
    }
}
