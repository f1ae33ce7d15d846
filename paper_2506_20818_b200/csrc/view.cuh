// Worker view of the graph (Section III): the rows of the worker's own partition keep their neighbour
// lists from the loaded graph (every neighbour, or only those inside the partition), the rows of the
// other partitions carry what is shared for negative sampling: nothing, their sparsified lists
// (Algorithm 1) or their full lists.  Integer work only: count, scan, fill.
#pragma once
#include "common.cuh"
#include "scan_sort.cuh"

enum { VIEW_FOREIGN_NONE = 0, VIEW_FOREIGN_SPARSIFIED = 1, VIEW_FOREIGN_FULL = 2 };

// stats: [0] entries of own rows, [1] entries of foreign rows, [2] foreign rows with at least one entry, [3] own nodes
__global__ void view_count_kernel(int n, const int *__restrict__ rowptr, const int *__restrict__ col, const int *__restrict__ part, int worker,
                                  int keep_cross, int foreign_mode, const int64_t *__restrict__ sp_ptr, int *__restrict__ counts,
                                  unsigned long long *__restrict__ stats)
{
    LP_DEP_ENTER();
    const int v = blockIdx.x * blockDim.x + threadIdx.x;
    if (v >= n) return;
    int c = 0;
    if (part[v] == worker) {
        const int a = rowptr[v], b = rowptr[v + 1];
        if (keep_cross) c = b - a;
        else
            for (int e = a; e < b; ++e) c += part[col[e]] == worker ? 1 : 0;
        atomicAdd(&stats[0], (unsigned long long)c);
        atomicAdd(&stats[3], 1ull);
    } else {
        if (foreign_mode == VIEW_FOREIGN_SPARSIFIED) c = (int)(sp_ptr[v + 1] - sp_ptr[v]);
        else if (foreign_mode == VIEW_FOREIGN_FULL) c = rowptr[v + 1] - rowptr[v];
        if (c > 0) {
            atomicAdd(&stats[1], (unsigned long long)c);
            atomicAdd(&stats[2], 1ull);
        }
    }
    counts[v] = c;
}

__global__ void view_fill_kernel(int n, const int *__restrict__ rowptr, const int *__restrict__ col, const int *__restrict__ part, int worker,
                                 int keep_cross, int foreign_mode, const int64_t *__restrict__ sp_ptr, const int *__restrict__ sp_col,
                                 const int *__restrict__ view_ptr, int *__restrict__ view_col)
{
    LP_DEP_ENTER();
    const int v = blockIdx.x * blockDim.x + threadIdx.x;
    if (v >= n) return;
    int o = view_ptr[v];
    if (part[v] == worker) {
        for (int e = rowptr[v]; e < rowptr[v + 1]; ++e) {
            const int u = col[e];
            if (keep_cross || part[u] == worker) view_col[o++] = u;
        }
    } else if (foreign_mode == VIEW_FOREIGN_SPARSIFIED) {
        for (int64_t e = sp_ptr[v]; e < sp_ptr[v + 1]; ++e) view_col[o++] = sp_col[e];
    } else if (foreign_mode == VIEW_FOREIGN_FULL) {
        for (int e = rowptr[v]; e < rowptr[v + 1]; ++e) view_col[o++] = col[e];
    }
}
