// MLP edge predictor (Eq. 2 with the 3-layer MLP of the paper's experiments, Section IV):
//   z0 = h_u * h_v (element-wise);  p1 = ReLU(z0 W0 + b0);  p2 = ReLU(p1 W1 + b1);  s = p2 . w2 + b2
// The two wide layers run through the same dense-transform kernels as the encoder; this file
// holds the edge-wise pieces around them, and Hits@K (the accuracy metric of Section IV).
#pragma once
#include "common.cuh"
#include "scan_sort.cuh"
#include "edge.cuh"

// one warp per scored edge: Z0[e, :] = H[src_e, :] * H[dst_e, :]
template <typename T, int NV>
__global__ void __launch_bounds__(EDGE_THREADS)
edge_hadamard_kernel(const T *__restrict__ H, int ldh, int D, int n_ids, const int *__restrict__ idmap, const int *__restrict__ pos_src,
                     const int *__restrict__ pos_dst, int64_t B, const int *__restrict__ neg_src, const int *__restrict__ neg_dst, int k,
                     T *__restrict__ Z0)
{
    LP_DEP_ENTER();
    constexpr int VN = Vec16<T>::N;
    const int lane = threadIdx.x & 31;
    const int64_t e = (int64_t)blockIdx.x * (EDGE_THREADS / 32) + (threadIdx.x >> 5);
    if (e >= B * (1 + k)) return;
    int u, v;
    incidence_endpoints(n_ids, idmap, pos_src, pos_dst, B, neg_src, neg_dst, k, e, u, v);
    const int nchunks = D / VN;
#pragma unroll
    for (int i = 0; i < NV; ++i) {
        const int ch = lane + i * 32;
        if (ch < nchunks) {
            Vec16<T> a, b, o;
            a.load(H + (size_t)u * ldh + ch * VN);
            b.load(H + (size_t)v * ldh + ch * VN);
            float fa[VN], fb[VN];
            a.to_float(fa);
            b.to_float(fb);
#pragma unroll
            for (int t = 0; t < VN; ++t) fa[t] *= fb[t];
            o.from_float(fa);
            o.store(Z0 + (size_t)e * D + ch * VN);
        }
    }
}

// one warp per edge: s[e] = P[e, :] . w + b
template <typename T>
__global__ void __launch_bounds__(EDGE_THREADS)
edge_gemv_kernel(const T *__restrict__ P, int Hp, int64_t E, const float *__restrict__ w, const float *__restrict__ b, float *__restrict__ s)
{
    LP_DEP_ENTER();
    const int lane = threadIdx.x & 31;
    const int64_t e = (int64_t)blockIdx.x * (EDGE_THREADS / 32) + (threadIdx.x >> 5);
    if (e >= E) return;
    float acc = 0.f;
    for (int j = lane; j < Hp; j += 32) acc = fmaf(to_f<T>(P[(size_t)e * Hp + j]), __ldg(w + j), acc);
    acc = warp_sum(acc);
    if (lane == 0) s[e] = acc + __ldg(b);
}

// loss terms and per-edge score gradients from precomputed scores; edges 0..B-1 are positives
__global__ void __launch_bounds__(256)
bce_from_scores_kernel(const float *__restrict__ s, int64_t E, int64_t B, float inv_N, float *__restrict__ g, float *__restrict__ loss_partials)
{
    LP_DEP_ENTER();
    __shared__ float sh[8];
    const int64_t e = (int64_t)blockIdx.x * 256 + threadIdx.x;
    float ell = 0.f;
    if (e < E) {
        float dls;
        bce_logits(s[e], e < B ? 1.f : 0.f, ell, dls);
        g[e] = dls * inv_N;
    }
    ell = warp_sum(ell);
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = ell;
    __syncthreads();
    if (threadIdx.x == 0) {
        float t = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) t += sh[w];
        loss_partials[blockIdx.x] = t;
    }
}

// dP2[e, j] = g_e * w2[j] where p2 > 0, else 0
template <typename T>
__global__ void pred_out_grad_kernel(const T *__restrict__ P2, int Hp, int64_t E, const float *__restrict__ g, const float *__restrict__ w2,
                                     T *__restrict__ dP2)
{
    LP_DEP_ENTER();
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= E * Hp) return;
    const int64_t e = i / Hp;
    const int j = (int)(i - e * Hp);
    dP2[i] = from_f<T>(to_f<T>(P2[i]) > 0.f ? g[e] * __ldg(w2 + j) : 0.f);
}

// partial[block][j] = sum over the block's rows of g_e * P2[e, j]; partial[block][Hp] = sum of g_e  (row order)
template <typename T>
__global__ void __launch_bounds__(256)
pred_last_layer_grad_kernel(const T *__restrict__ P2, int Hp, int64_t E, const float *__restrict__ g, int64_t rows_per_block,
                            float *__restrict__ partials)
{
    LP_DEP_ENTER();
    const int64_t r0 = (int64_t)blockIdx.x * rows_per_block, r1 = min(E, r0 + rows_per_block);
    for (int j = threadIdx.x; j <= Hp; j += 256) {
        float acc = 0.f;
        if (j < Hp)
            for (int64_t r = r0; r < r1; ++r) acc = fmaf(g[r], to_f<T>(P2[(size_t)r * Hp + j]), acc);
        else
            for (int64_t r = r0; r < r1; ++r) acc += g[r];
        partials[(int64_t)blockIdx.x * (Hp + 1) + j] = acc;
    }
}

// x = 0 where the forward activation was not positive (ReLU backward)
template <typename T>
__global__ void relu_mask_kernel(T *__restrict__ x, const T *__restrict__ ref, int64_t count)
{
    LP_DEP_ENTER();
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < count && !(to_f<T>(ref[i]) > 0.f)) x[i] = from_f<T>(0.f);
}

// ---- Hits@K ----------------------------------------------------------------------------------
// order-preserving map float -> uint32 (larger float <=> larger key)
LP_DEVINL uint32_t float_sort_key(float f)
{
    const uint32_t b = __float_as_uint(f + 0.f);  // -0 and +0 share one key
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

__global__ void float_keys_kernel(const float *__restrict__ x, int64_t n, uint32_t *__restrict__ keys, uint32_t *__restrict__ vals)
{
    LP_DEP_ENTER();
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) { keys[i] = float_sort_key(x[i]); vals[i] = (uint32_t)i; }
}

// count positives whose key is strictly greater than sorted_keys[thr_index]
__global__ void count_above_kernel(const float *__restrict__ pos, int64_t n_pos, const uint32_t *__restrict__ sorted_keys, int64_t thr_index,
                                   unsigned long long *__restrict__ count)
{
    LP_DEP_ENTER();
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t thr = sorted_keys[thr_index];
    const bool hit = i < n_pos && float_sort_key(pos[i]) > thr;
    const unsigned m = __ballot_sync(0xffffffffu, hit);
    if ((threadIdx.x & 31) == 0 && m) atomicAdd(count, (unsigned long long)__popc(m));
}
