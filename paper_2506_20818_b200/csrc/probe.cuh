// Measurement aid: the rate at which this GPU can gather whole source rows by index, with nothing else in the way.
// The aggregation kernels are gather kernels whose source matrix often sits in L2; their fair ceiling is then not
// the HBM copy bandwidth but what a bare gather of the same index stream reaches, which this kernel measures.
#pragma once
#include "common.cuh"
#include "scan_sort.cuh"

constexpr int PROBE_RUN = 64;  // consecutive entries per lane group

// A group of LANES lanes (one 16-byte piece of a row each) takes PROBE_RUN consecutive entries of the index array,
// loads the rows they name with eight loads in flight and folds them with XOR (an exact, order-free integer result
// that the tests can check); out[group][lane] receives the 16-byte fold.  No row structure, no arithmetic, no epilogue.
template <int LANES>
__global__ void __launch_bounds__(256) gather_probe_kernel(const int *__restrict__ col, int64_t nnz, const uint4 *__restrict__ X, int64_t pitch16,
                                                           uint4 *__restrict__ out)
{
    LP_DEP_ENTER();
    const int64_t gid = ((int64_t)blockIdx.x * 256 + threadIdx.x) / LANES;
    const int gl = threadIdx.x % LANES;
    const int64_t e0 = gid * PROBE_RUN;
    if (e0 >= nnz) return;
    const int64_t e1 = min(nnz, e0 + PROBE_RUN);
    uint4 acc = make_uint4(0u, 0u, 0u, 0u);
    for (int64_t e = e0; e < e1; e += 8) {
        int c[8];
        uint4 v[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) c[q] = (e + q < e1) ? __ldg(col + e + q) : -1;
#pragma unroll
        for (int q = 0; q < 8; ++q) v[q] = c[q] >= 0 ? __ldg(X + (size_t)c[q] * pitch16 + gl) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            acc.x ^= v[q].x;
            acc.y ^= v[q].y;
            acc.z ^= v[q].z;
            acc.w ^= v[q].w;
        }
    }
    out[gid * LANES + gl] = acc;
}

// row_bytes must be 128, 256 or 512 (8, 16 or 32 lanes of 16 bytes)
static bool gather_probe_launch(Exec &ex, const int *col, int64_t nnz, const void *X, int row_bytes, void *out)
{
    if (nnz <= 0) return true;
    const int lanes = row_bytes / 16;
    const int64_t groups = ceil_div64(nnz, PROBE_RUN);
    const unsigned blocks = (unsigned)ceil_div64(groups * lanes, 256);
    if (lanes == 32) launch_dep(gather_probe_kernel<32>, dim3(blocks), dim3(256), 0, ex.st, col, nnz, (const uint4 *)X, lanes, (uint4 *)out);
    else if (lanes == 16) launch_dep(gather_probe_kernel<16>, dim3(blocks), dim3(256), 0, ex.st, col, nnz, (const uint4 *)X, lanes, (uint4 *)out);
    else if (lanes == 8) launch_dep(gather_probe_kernel<8>, dim3(blocks), dim3(256), 0, ex.st, col, nnz, (const uint4 *)X, lanes, (uint4 *)out);
    else return false;
    ex.launches += 1;
    return true;
}
