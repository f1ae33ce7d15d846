// Dense transforms on the plain FP32 ALUs (validation path, and fall-back shapes of the BF16 path).
//   C[M, N] = epilogue( sum_k A(m, k) * B(k, n) )      accumulation in FP32, k ascending
// Operands may be float or bf16 and may be stored with either index contiguous:
//   A_MCONTIG = false : A(m, k) = A[m * lda + k]      true : A(m, k) = A[k * lda + m]
//   B_NCONTIG = true  : B(k, n) = B[k * ldb + n]      false: B(k, n) = B[n * ldb + k]
// Split-K (gridDim.z > 1) writes FP32 partial tiles that reduce_partials_kernel adds in a
// fixed order, so weight gradients are reproducible bit for bit.
#pragma once
#include "common.cuh"
#include "scan_sort.cuh"

constexpr int SG_BM = 64, SG_BN = 64, SG_BK = 16, SG_THREADS = 256;

template <typename TA, typename TB, typename TC, bool A_MCONTIG, bool B_NCONTIG>
__global__ void __launch_bounds__(SG_THREADS)
gemm_simt_kernel(int64_t M, int N, int64_t K, const TA *__restrict__ A, int64_t lda, const TB *__restrict__ B, int64_t ldb,
                 TC *__restrict__ C, int64_t ldc, const float *__restrict__ bias, int relu, int64_t k_chunk, float *__restrict__ partials,
                 const float *__restrict__ row_scale = nullptr, int scale_col0 = 0)
{
    LP_DEP_ENTER();
    __shared__ __align__(16) float As[SG_BK][SG_BM + 4];
    __shared__ __align__(16) float Bs[SG_BK][SG_BN + 4];
    const int64_t m0 = (int64_t)blockIdx.x * SG_BM;
    const int n0 = blockIdx.y * SG_BN;
    const int64_t k_begin = (int64_t)blockIdx.z * k_chunk;
    const int64_t k_end = min(K, k_begin + k_chunk);
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;  // 16 x 16 threads, 4 x 4 outputs each
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

    for (int64_t k0 = k_begin; k0 < k_end; k0 += SG_BK) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int idx = threadIdx.x + i * SG_THREADS;
            int m, k;
            if (A_MCONTIG) { m = idx % SG_BM; k = idx / SG_BM; } else { k = idx % SG_BK; m = idx / SG_BK; }
            float v = 0.f;
            if (m0 + m < M && k0 + k < k_end)
                v = to_f<TA>(A_MCONTIG ? A[(k0 + k) * lda + (m0 + m)] : A[(m0 + m) * lda + (k0 + k)]);
            As[k][m] = v;
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int idx = threadIdx.x + i * SG_THREADS;
            int n, k;
            if (B_NCONTIG) { n = idx % SG_BN; k = idx / SG_BN; } else { k = idx % SG_BK; n = idx / SG_BK; }
            float v = 0.f;
            if (n0 + n < N && k0 + k < k_end)
                v = to_f<TB>(B_NCONTIG ? B[(k0 + k) * ldb + (n0 + n)] : B[(int64_t)(n0 + n) * ldb + (k0 + k)]);
            Bs[k][n] = v;
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < SG_BK; ++k) {
            const float4 a4 = *reinterpret_cast<const float4 *>(&As[k][ty * 4]);
            const float4 b4 = *reinterpret_cast<const float4 *>(&Bs[k][tx * 4]);
            const float a[4] = {a4.x, a4.y, a4.z, a4.w};
            const float b[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int64_t m = m0 + ty * 4 + i;
        if (m >= M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int n = n0 + tx * 4 + j;
            if (n >= N) continue;
            if (partials) {
                partials[((int64_t)blockIdx.z * M + m) * N + n] = acc[i][j];
            } else {
                float v = acc[i][j] + (bias ? bias[n] : 0.f);
                if (relu) v = fmaxf(v, 0.f);
                if (row_scale && n >= scale_col0) v *= row_scale[m];  // per-row factor on the trailing columns
                C[m * ldc + n] = from_f<TC>(v);
            }
        }
    }
}

// dst[i] = (accumulate ? dst[i] : 0) + sum_z partials[z][i], z ascending
__global__ void reduce_partials_kernel(const float *__restrict__ partials, int64_t count, int splits, float *__restrict__ dst, int accumulate)
{
    LP_DEP_ENTER();
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= count) return;
    float s = 0.f;
    int z = 0;
    for (; z < splits; z += 16) {  // sixteen independent loads in flight (the last batch predicated), added in index order
        float v[16];
#pragma unroll
        for (int q = 0; q < 16; ++q) v[q] = z + q < splits ? __ldg(partials + (int64_t)(z + q) * count + i) : 0.f;
#pragma unroll
        for (int q = 0; q < 16; ++q)
            if (z + q < splits) s += v[q];
    }
    dst[i] = accumulate ? dst[i] + s : s;
}

template <typename TA, typename TB, typename TC, bool A_MCONTIG, bool B_NCONTIG>
static void gemm_simt(Exec &ex, int64_t M, int N, int64_t K, const TA *A, int64_t lda, const TB *B, int64_t ldb, TC *C, int64_t ldc,
                      const float *bias, int relu, const float *row_scale = nullptr, int scale_col0 = 0)
{
    if (M <= 0 || N <= 0) return;
    dim3 grid((unsigned)ceil_div64(M, SG_BM), (unsigned)ceil_div64(N, SG_BN), 1);
    launch_dep(gemm_simt_kernel<TA, TB, TC, A_MCONTIG, B_NCONTIG>, dim3(grid), dim3(SG_THREADS), 0, ex.st, M, N, K, A, lda, B, ldb, C, ldc, bias, relu, K > 0 ? K : 1, nullptr, row_scale, scale_col0);
    ex.launches += 1;
}

constexpr int WG_MAX_SPLITS = 256;
// one split per 256 rows (small graphs still fill the GPU), at most WG_MAX_SPLITS
static int weight_grad_splits(int64_t rows) { return (int)std::max<int64_t>(1, std::min<int64_t>(WG_MAX_SPLITS, ceil_div64(rows, 256))); }

// dW[Kin, N] = A[rows, Kin]^T * dZ[rows, N]; `partials` needs weight_grad_splits(rows) * Kin * N floats.
template <typename T>
static void weight_grad_simt(Exec &ex, int64_t rows, int Kin, int N, const T *A, int64_t lda, const T *dZ, int64_t ldz, float *dW,
                             int accumulate, float *partials)
{
    const int splits = weight_grad_splits(rows);
    int64_t k_chunk = ceil_div64(ceil_div64(rows, splits), SG_BK) * SG_BK;
    if (k_chunk < SG_BK) k_chunk = SG_BK;
    dim3 grid((unsigned)ceil_div64(Kin, SG_BM), (unsigned)ceil_div64(N, SG_BN), (unsigned)splits);
    launch_dep(gemm_simt_kernel<T, T, float, true, true>, dim3(grid), dim3(SG_THREADS), 0, ex.st, Kin, N, rows, A, lda, dZ, ldz, (float *)nullptr, 0, nullptr, 0, k_chunk, partials, nullptr, 0);
    const int64_t count = (int64_t)Kin * N;
    launch_dep(reduce_partials_kernel, dim3((unsigned)ceil_div64(count, 256)), dim3(256), 0, ex.st, partials, count, splits, dW, accumulate);
    ex.launches += 2;
}

// column sums: out[j] = sum_r dZ[r, j] (bias gradient), two deterministic stages.  A block of 256
// threads covers a range of rows with 16-byte loads: thread = (row lane, column vector); the row
// lanes are added in shared memory in lane order, then the blocks' partial rows in block order.
template <typename T>
__global__ void __launch_bounds__(256) colsum_partial_kernel(const T *__restrict__ dZ, int64_t rows, int N, int64_t ldz, int64_t rows_per_block,
                                                             float *__restrict__ partials)
{
    LP_DEP_ENTER();
    constexpr int VN = Vec16<T>::N;
    __shared__ float sh[256 * VN];
    const int nvec = N / VN;           // column vectors per row (<= 256)
    const int lanes_r = 256 / nvec;    // row lanes
    const int c = threadIdx.x % nvec, rl = threadIdx.x / nvec;
    const int64_t r0 = (int64_t)blockIdx.x * rows_per_block, r1 = min(rows, r0 + rows_per_block);
    float acc[VN];
#pragma unroll
    for (int j = 0; j < VN; ++j) acc[j] = 0.f;
    if (rl < lanes_r) {
        int64_t r = r0 + rl;
        for (; r + 7 * (int64_t)lanes_r < r1; r += 8 * (int64_t)lanes_r) {  // eight loads in flight, added in row order
            Vec16<T> v[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) v[q].load(dZ + (r + q * (int64_t)lanes_r) * ldz + c * VN);
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                float f[VN];
                v[q].to_float(f);
#pragma unroll
                for (int j = 0; j < VN; ++j) acc[j] += f[j];
            }
        }
        for (; r < r1; r += lanes_r) {
            Vec16<T> v;
            v.load(dZ + r * ldz + c * VN);
            float f[VN];
            v.to_float(f);
#pragma unroll
            for (int j = 0; j < VN; ++j) acc[j] += f[j];
        }
#pragma unroll
        for (int j = 0; j < VN; ++j) sh[rl * N + c * VN + j] = acc[j];
    }
    __syncthreads();
    for (int j = threadIdx.x; j < N; j += 256) {
        float s = 0.f;
        for (int q = 0; q < lanes_r; ++q) s += sh[q * N + j];
        partials[(int64_t)blockIdx.x * N + j] = s;
    }
}

// dst[j] = (accumulate ? dst[j] : 0) + sum_z partials[z][j] for a SHORT vector (count <= a few hundred) and many
// splits: 32 columns per block, eight groups each add a contiguous range of splits in order, then the
// eight group sums are added in group order (a fixed tree, so the result is reproducible).
__global__ void __launch_bounds__(256) reduce_partials_short_kernel(const float *__restrict__ partials, int count, int splits, float *__restrict__ dst,
                                                                    int accumulate)
{
    LP_DEP_ENTER();
    __shared__ float sh[8][32];
    const int c = blockIdx.x * 32 + (threadIdx.x & 31), g = threadIdx.x >> 5;
    const int per = (splits + 7) / 8;
    const int z0 = g * per, z1 = min(splits, z0 + per);
    float s = 0.f;
    if (c < count)
        for (int z = z0; z < z1; ++z) s += __ldg(partials + (int64_t)z * count + c);
    sh[g][threadIdx.x & 31] = s;
    __syncthreads();
    if (g == 0 && c < count) {
        float t = 0.f;
#pragma unroll
        for (int q = 0; q < 8; ++q) t += sh[q][threadIdx.x];
        dst[c] = accumulate ? dst[c] + t : t;
    }
}

constexpr int CS_MAX_SPLITS = 592;
static int colsum_splits(int64_t rows) { return (int)std::max<int64_t>(1, std::min<int64_t>(CS_MAX_SPLITS, ceil_div64(rows, 64))); }

template <typename T>
static void colsum(Exec &ex, const T *dZ, int64_t rows, int N, int64_t ldz, float *out, int accumulate, float *partials)
{
    const int splits = colsum_splits(rows);
    const int64_t rpb = ceil_div64(rows > 0 ? rows : 1, splits);
    launch_dep(colsum_partial_kernel<T>, dim3(splits), dim3(256), 0, ex.st, dZ, rows, N, ldz, rpb, partials);
    launch_dep(reduce_partials_short_kernel, dim3((unsigned)ceil_div64(N, 32)), dim3(256), 0, ex.st, partials, N, splits, out, accumulate);
    ex.launches += 2;
}
