// Weight update (Algorithm 1: average the workers' gradients, then update; Section IV: Adam with
// learning rate 1e-3) and small element-wise helpers.
#pragma once
#include "common.cuh"
#include "scan_sort.cuh"

// g = scale * grad;  m = b1 m + (1-b1) g;  v = b2 v + (1-b2) g^2;
// p -= lr * (m / c1) / (sqrt(v / c2) + eps),  c1 = 1 - b1^t, c2 = 1 - b2^t; 1 - b and 1 / c are formed on the
// host in double (1 - 0.999f would already be off by 1e-5 relative)
__global__ void adam_kernel(float *__restrict__ p, float *__restrict__ m, float *__restrict__ v, const float *__restrict__ grad, int64_t n,
                            float scale, float lr, float b1, float one_minus_b1, float b2, float one_minus_b2, float eps, float inv_c1,
                            float inv_c2)
{
    LP_DEP_ENTER();
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const float g = scale * grad[i];
    const float mi = b1 * m[i] + one_minus_b1 * g;
    const float vi = b2 * v[i] + one_minus_b2 * g * g;
    m[i] = mi;
    v[i] = vi;
    p[i] -= lr * (mi * inv_c1) / (sqrtf(vi * inv_c2) + eps);
}

__global__ void sgd_kernel(float *__restrict__ p, const float *__restrict__ grad, int64_t n, float scale, float lr)
{
    LP_DEP_ENTER();
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) p[i] -= lr * scale * grad[i];
}

template <typename TS, typename TD> __global__ void convert_kernel(const TS *__restrict__ src, TD *__restrict__ dst, int64_t n)
{
    LP_DEP_ENTER();
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) dst[i] = from_f<TD>(to_f<TS>(src[i]));
}

// dst[r, 0:F] (leading dimension ldd) = src[r, 0:F] (leading dimension lds), with conversion
template <typename TS, typename TD>
__global__ void copy_rows_kernel(const TS *__restrict__ src, int64_t lds, TD *__restrict__ dst, int64_t ldd, int64_t rows, int F)
{
    LP_DEP_ENTER();
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= rows * F) return;
    const int64_t r = i / F;
    const int c = (int)(i - r * F);
    dst[r * ldd + c] = from_f<TD>(to_f<TS>(src[r * lds + c]));
}

// W[K, N] row-major float -> Wt[N, K] row-major bf16 (K contiguous) and, optionally, W as bf16
__global__ void weights_to_bf16_kernel(const float *__restrict__ W, int K, int N, bf16 *__restrict__ Wt, bf16 *__restrict__ Wc)
{
    LP_DEP_ENTER();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= K * N) return;
    const int k = i / N, n = i - k * N;
    const bf16 x = __float2bfloat16_rn(W[i]);
    if (Wt) Wt[(size_t)n * K + k] = x;
    if (Wc) Wc[i] = x;
}

// BF16 copies of a whole flat parameter vector in one launch: `asis` element for element, and `transposed` with every
// weight matrix W[Kin, Fo] (row-major, at offset off) stored as its transpose [Fo, Kin] at the same offset (biases are
// copied in place in both).  The forward transforms read the transposed blocks, the input-gradient transforms the others.
// `stacked` (optional): a block with split = Fi > 0 holds W = [W_self ; W_neigh] (2 Fi rows); it is stored as
// [Fi, 2 Fo] with row n = (W_self[n, :] | W_neigh[n, :]), the [N, K] operand of dH = [dZ | A^T dZ] [W_self^T ; W_neigh^T].
struct WeightBlocks {
    int count;
    long long off[8];
    int kin[8], fo[8], split[8];
};
LP_DEVINL void weights_cache_element(long long i, const float *__restrict__ params, long long n, const WeightBlocks &blocks, bf16 *__restrict__ asis,
                                     bf16 *__restrict__ transposed, bf16 *__restrict__ stacked)
{
    if (i >= n) return;
    const bf16 x = __float2bfloat16_rn(params[i]);
    asis[i] = x;
    long long dst = i;
#pragma unroll
    for (int b = 0; b < 8; ++b) {
        if (b < blocks.count) {
            const long long r = i - blocks.off[b];
            if (r >= 0 && r < (long long)blocks.kin[b] * blocks.fo[b]) {
                const int k = (int)(r / blocks.fo[b]), c = (int)(r - (long long)k * blocks.fo[b]);
                dst = blocks.off[b] + (long long)c * blocks.kin[b] + k;
                if (stacked && blocks.split[b] > 0) {
                    const int half = k / blocks.split[b], row = k - half * blocks.split[b];
                    stacked[blocks.off[b] + (long long)row * (2 * blocks.fo[b]) + half * blocks.fo[b] + c] = x;
                }
            }
        }
    }
    transposed[dst] = x;
}
__global__ void weights_cache_kernel(const float *__restrict__ params, long long n, WeightBlocks blocks, bf16 *__restrict__ asis, bf16 *__restrict__ transposed,
                                     bf16 *__restrict__ stacked)
{
    LP_DEP_ENTER();
    weights_cache_element((long long)blockIdx.x * blockDim.x + threadIdx.x, params, n, blocks, asis, transposed, stacked);
}
