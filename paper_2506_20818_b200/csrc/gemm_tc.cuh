// Dense transforms of the BF16 path on the 5th-generation tensor cores (tcgen05, sm_100a).
//
//   tc_gemm_kmajor_kernel : C[M, N] = act(A[M, K] * Bt[N, K]^T + bias)       (forward, input gradient)
//   tc_gemm_mnmajor_kernel: P[z][Kin, N] = A[rows_z, Kin]^T * dZ[rows_z, N]   (weight gradient, split over rows)
//
// Both kernels: one CTA owns a 128-row accumulator tile in tensor memory (128 lanes x BN FP32
// columns); operand tiles are brought in by TMA (cp.async.bulk.tensor, 128-byte swizzle, no
// multicast) into a ring of shared-memory stages guarded by full/empty mbarriers; one elected
// thread issues tcgen05.mma (kind::f16, BF16 x BF16 -> FP32) and releases stages with
// tcgen05.commit; all four warps drain the accumulator with tcgen05.ld and apply the epilogue.
// Every mbarrier wait is bounded (two seconds unless the host sets another limit): on expiry the kernel
// records an error word, frees its tensor memory and returns, and the host reports LP_ETIMEOUT.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "scan_sort.cuh"
#include "gemm_simt.cuh"
#include "optim.cuh"

typedef CUresult (*lp_encode_tiled_fn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                       const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                       CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct TcState {
    lp_encode_tiled_fn encode = nullptr;
    int *err_word = nullptr;  // device: 0 = fine, else code of the wait that expired
    bf16 *wbuf = nullptr;     // device scratch: BF16 copy of one layer's weights
    int *host_err = nullptr;  // pinned
    unsigned long long wait_limit_ns = 2000000000ull;  // every mbarrier wait gives up after this long (default two seconds)
    int overdeclare_tx = 0;   // diagnostics: the next launch expects this many bytes more than it copies (consumed by that launch)
};

constexpr int TC_BM = 128;          // accumulator rows (UMMA M)
constexpr int TC_BK = 64;           // K elements per stage: 64 bf16 = one 128-byte swizzle row
constexpr int TC_UMMA_K = 16;       // K per tcgen05.mma for 16-bit operands
constexpr int TC_THREADS = 128;
constexpr int TC_COLSUM_BOXES = 4;  // 64-column boxes of the B tile one CTA may have to add up (BN <= 256)
constexpr int TC_WBUF_ELEMS = 512 * 512;

// ---------------------------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------------------------
LP_DEVINL uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

LP_DEVINL void mbar_init(uint32_t bar, uint32_t count) { asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory"); }
LP_DEVINL void mbar_arrive(uint32_t bar) { asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory"); }
LP_DEVINL void named_barrier_sync(int id, int threads) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory"); }
LP_DEVINL void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
LP_DEVINL bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
LP_DEVINL unsigned long long global_timer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
// bounded wait: false when the time limit was reached
LP_DEVINL bool mbar_wait(uint32_t bar, uint32_t parity, unsigned long long limit_ns)
{
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_timer_ns();
    for (;;) {
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (global_timer_ns() - t0 > limit_ns) return false;
    }
}
LP_DEVINL void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
LP_DEVINL void fence_async_proxy() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

LP_DEVINL void tma_load_2d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int x, int y)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(dst), "l"(map),
                 "r"(bar), "r"(x), "r"(y)
                 : "memory");
}
LP_DEVINL void tma_prefetch_desc(const CUtensorMap *map) { asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory"); }

LP_DEVINL void tmem_alloc(uint32_t smem_dst, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
LP_DEVINL void tmem_dealloc(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
LP_DEVINL void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
LP_DEVINL void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

LP_DEVINL void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
LP_DEVINL void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// 32 lanes x 32 consecutive FP32 columns: thread t of the warp receives lane (32 * (warp % 4) + t).
// tmem_ld_32x32_issue starts the load, tmem_ld_wait makes every issued load's registers valid.
LP_DEVINL void tmem_ld_32x32_issue(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]),
          "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]),
          "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]),
          "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
LP_DEVINL void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

LP_DEVINL void tmem_ld_32x32(uint32_t taddr, float *v)
{
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]),
          "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]),
          "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]),
          "=r"(r[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// Shared-memory matrix descriptor (tcgen05): start address, leading / stride byte offsets in
// 16-byte units, descriptor version 1, 128-byte swizzle.
LP_DEVINL uint64_t make_smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    uint64_t d = 0;
    d |= (uint64_t)((saddr >> 4) & 0x3FFFu);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;  // descriptor version
    d |= (uint64_t)2 << 61;  // SWIZZLE_128B
    return d;
}

// Instruction descriptor, kind::f16: D = FP32, A = B = BF16, M = 128, N = n; *_mn = operand stored MN-major
static __host__ __device__ inline uint32_t make_idesc_bf16(int n, bool a_mn, bool b_mn)
{
    uint32_t d = 0;
    d |= 1u << 4;                      // accumulator format F32
    d |= 1u << 7;                      // A format BF16
    d |= 1u << 10;                     // B format BF16
    d |= (a_mn ? 1u : 0u) << 15;
    d |= (b_mn ? 1u : 0u) << 16;
    d |= (uint32_t)(n >> 3) << 17;
    d |= (uint32_t)(TC_BM >> 4) << 24;
    return d;
}

// ---------------------------------------------------------------------------------------------
// kernel 1: K-major operands.  A tile = 128 rows x 64 K (16 KiB), B tile = BN rows x 64 K.
// ---------------------------------------------------------------------------------------------
struct TcGemmParams {
    int64_t M;
    int N, K;
    int BN;             // accumulator columns of this launch (N tile), multiple of 16, <= 256
    int stages;
    const float *bias;  // [N] or null
    int relu;
    const float *row_scale;  // [M] or null: columns >= scale_col0 of row m are multiplied by row_scale[m]
    int scale_col0;          // (the 1 / |N(v)| of the mean adjoint, folded into the input-gradient transform)
    // pair kernel only.  Sign bits of the output, one 32-bit word per row and 32 columns, word (c / 32) * M + row, column
    // c of the 32 at bit (c / 2) + 16 * (c % 2) (the order in which packed BF16 pairs give them up): mask_out receives
    // "stored BF16 value > 0" (with relu), mask_in zeroes the outputs whose bit is clear (ReLU backward)
    uint32_t *mask_out;
    const uint32_t *mask_in;
    int out_sets;            // pair kernel: 1 or 2 pairs of output staging boxes (a box is refilled once the stores before the latest one or three have read theirs)
    bf16 *C;            // output (BF16) when out_f32 == null
    int64_t ldc;
    float *out_f32;     // FP32 partial output [gridDim.z][M + colsum, N] (weight gradient)
    int colsum;         // weight gradient only: 1 = row M of every partial tile receives the column sums of the B operand
                        // over the split's rows (the bias gradient), taken from the staged tiles by the otherwise idle warps
    int64_t rows;       // weight gradient: reduction length; rows_per_split rows per blockIdx.z
    int64_t rows_per_split;
    int *err;
    unsigned long long wait_ns;  // limit of every mbarrier wait
    int extra_tx;                // diagnostics: bytes added to the first stage's expected transfer so that its wait expires
};

template <bool MN_MAJOR>
__global__ void __launch_bounds__(TC_THREADS) tc_gemm_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB,
                                                             const TcGemmParams p)
{
    LP_DEP_ENTER();
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[8], bar_empty[8], bar_acc;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s, colsum_fail_s;
    __shared__ float colsum_s[8][64];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);  // swizzle atoms need 1024-byte alignment
    const int BN = p.BN;
    const uint32_t a_bytes = TC_BM * TC_BK * 2;  // 16384
    const uint32_t b_bytes = (uint32_t)BN * TC_BK * 2;
    const uint32_t stage_bytes = a_bytes + b_bytes;
    const int S = p.stages;
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < BN) tmem_cols <<= 1;

    // reduction range of this CTA
    int64_t k_begin = 0, k_end = p.K;
    if (MN_MAJOR) {
        k_begin = (int64_t)blockIdx.z * p.rows_per_split;
        k_end = min(p.rows, k_begin + p.rows_per_split);
    }
    const int num_kb = (int)((k_end - k_begin + TC_BK - 1) / TC_BK);
    const int m0 = blockIdx.x * TC_BM;
    const int n0 = blockIdx.y * BN;
    // bias gradient: the 64-column boxes of the B tile are dealt out over the M tiles of the split; warps 2 and 3 add them up
    const int n_boxes = BN / 64;
    const bool do_colsum = MN_MAJOR && p.colsum != 0 && (int)blockIdx.x < n_boxes;
    const int64_t part_rows = p.M + (MN_MAJOR && p.colsum != 0 ? 1 : 0);

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1);
            mbar_init(smem_u32(&bar_empty[s]), do_colsum ? 3 : 1);  // the MMA commit, plus one lane of each summing warp
        }
        mbar_init(smem_u32(&bar_acc), 1);
        abort_s = 0;
        colsum_fail_s = 0;
        fence_barrier_init();
        fence_async_proxy();
        tma_prefetch_desc(&mapA);
        tma_prefetch_desc(&mapB);
    }
    if (warp == 0) {
        __syncwarp();
        tmem_alloc(smem_u32(&tmem_base_s), tmem_cols);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_d = tmem_base_s;

    if (num_kb > 0) {
        if (warp == 0 && lane == 0) {
            // ---- producer: TMA loads into the stage ring
            for (int kb = 0; kb < num_kb; ++kb) {
                const int s = kb % S;
                if (kb >= S && !mbar_wait(smem_u32(&bar_empty[s]), ((kb / S) & 1) ^ 1, p.wait_ns)) {
                    atomicExch(p.err, 1);
                    abort_s = 1;
                    break;
                }
                const uint32_t sa = smem_u32(smem + (size_t)s * stage_bytes), sb = sa + a_bytes;
                const uint32_t bar = smem_u32(&bar_full[s]);
                mbar_expect_tx(bar, stage_bytes + (kb == 0 ? (uint32_t)p.extra_tx : 0u));
                const int kk = (int)(k_begin + (int64_t)kb * TC_BK);
                if (!MN_MAJOR) {
                    tma_load_2d(sa, &mapA, bar, kk, m0);  // box {64 K, 128 rows}
                    tma_load_2d(sb, &mapB, bar, kk, n0);  // box {64 K, BN rows}
                } else {
                    // boxes {64 columns, 64 reduction rows}: 2 for A (128 features), BN / 64 for B
                    for (int c = 0; c < TC_BM / 64; ++c) tma_load_2d(sa + c * 8192, &mapA, bar, m0 + c * 64, kk);
                    for (int c = 0; c < BN / 64; ++c) tma_load_2d(sb + c * 8192, &mapB, bar, n0 + c * 64, kk);
                }
            }
        } else if (warp == 1 && lane == 0) {
            // ---- MMA issuer
            const uint32_t idesc = make_idesc_bf16(BN, MN_MAJOR, MN_MAJOR);
            bool ok = true;
            for (int kb = 0; kb < num_kb && ok; ++kb) {
                const int s = kb % S;
                if (!mbar_wait(smem_u32(&bar_full[s]), (kb / S) & 1, p.wait_ns)) {
                    atomicExch(p.err, 2);
                    abort_s = 1;
                    ok = false;
                    break;
                }
                tc_fence_after();
                const uint32_t sa = smem_u32(smem + (size_t)s * stage_bytes), sb = sa + a_bytes;
#pragma unroll
                for (int k = 0; k < TC_BK / TC_UMMA_K; ++k) {
                    uint64_t da, db;
                    if (!MN_MAJOR) {
                        // K-major, 128-byte swizzle: rows of 128 bytes, 8-row groups 1024 bytes apart;
                        // a K step of 16 elements moves the start by 32 bytes inside the swizzle row
                        da = make_smem_desc(sa + k * 32, 16, 1024);
                        db = make_smem_desc(sb + k * 32, 16, 1024);
                    } else {
                        // MN-major, 128-byte swizzle: 64 MN elements per 128-byte row, 8 K rows per 1024-byte
                        // atom (stride), next 64 MN elements 8192 bytes further (leading); 16 K = 2 atoms
                        da = make_smem_desc(sa + k * 2048, 8192, 1024);
                        db = make_smem_desc(sb + k * 2048, 8192, 1024);
                    }
                    umma_bf16(tmem_d, da, db, idesc, (kb | k) != 0 ? 1u : 0u);
                }
                umma_commit(smem_u32(&bar_empty[s]));  // frees the stage when these MMAs have read it
            }
            if (ok) umma_commit(smem_u32(&bar_acc));   // accumulator complete
        } else if (do_colsum && warp >= 2) {
            // ---- column sums of the B tiles (bias gradient).  A staged B tile is BN / 64 boxes of 64 reduction
            // rows x 128 bytes (64 columns); the 16-byte piece c of row k sits at piece c ^ (k & 7) (128-byte
            // swizzle).  The boxes are dealt out over the CTAs of the split (box b to M tile b mod gridDim.x).
            // Thread t = (rq, c8) adds rows 8 rq .. 8 rq + 7 of every stage for the eight columns of piece c8;
            // the eight row groups are added in order at the end, so the sum is reproducible.
            const int t = threadIdx.x - 64;
            const int c8 = t & 7, rq = t >> 3;
            float acc[TC_COLSUM_BOXES][8];
#pragma unroll
            for (int j = 0; j < TC_COLSUM_BOXES; ++j)
#pragma unroll
                for (int q = 0; q < 8; ++q) acc[j][q] = 0.f;
            bool ok = true;
            for (int kb = 0; kb < num_kb; ++kb) {
                const int s = kb % S;
                ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bar_full[s]), (kb / S) & 1, p.wait_ns));
                if (!ok) {
                    if (lane == 0) atomicExch(p.err, 4);
                    abort_s = 1;
                    break;
                }
                const uint8_t *sb = smem + (size_t)s * stage_bytes + a_bytes + (size_t)rq * 1024;
#pragma unroll
                for (int j = 0; j < TC_COLSUM_BOXES; ++j) {
                    const int b = (int)blockIdx.x + j * (int)gridDim.x;
                    if (b < n_boxes) {
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const uint4 v = *reinterpret_cast<const uint4 *>(sb + (size_t)b * 8192 + i * 128 + ((c8 ^ i) << 4));
                            acc[j][0] += __uint_as_float(v.x << 16);
                            acc[j][1] += __uint_as_float(v.x & 0xffff0000u);
                            acc[j][2] += __uint_as_float(v.y << 16);
                            acc[j][3] += __uint_as_float(v.y & 0xffff0000u);
                            acc[j][4] += __uint_as_float(v.z << 16);
                            acc[j][5] += __uint_as_float(v.z & 0xffff0000u);
                            acc[j][6] += __uint_as_float(v.w << 16);
                            acc[j][7] += __uint_as_float(v.w & 0xffff0000u);
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bar_empty[s]));  // this warp has read the stage
            }
            // both warps take the same path here: `ok` is decided per warp, so exchange it through shared memory
            if (!ok) colsum_fail_s = 1;
            named_barrier_sync(1, 64);
            ok = colsum_fail_s == 0;
#pragma unroll
            for (int j = 0; j < TC_COLSUM_BOXES; ++j) {
                const int b = (int)blockIdx.x + j * (int)gridDim.x;
                if (b < n_boxes) {  // uniform over the 64 threads
#pragma unroll
                    for (int q = 0; q < 8; ++q) colsum_s[rq][c8 * 8 + q] = acc[j][q];
                    named_barrier_sync(1, 64);
                    float r = 0.f;
#pragma unroll
                    for (int g = 0; g < 8; ++g) r += colsum_s[g][t];
                    if (ok) p.out_f32[((int64_t)blockIdx.z * part_rows + p.M) * p.N + n0 + b * 64 + t] = r;
                    named_barrier_sync(1, 64);
                }
            }
        }
        __syncwarp();

        // ---- epilogue: all four warps
        bool ready = mbar_wait(smem_u32(&bar_acc), 0, p.wait_ns);
        if (!ready && lane == 0) atomicExch(p.err, 3);
        ready = ready && (*(volatile int *)&abort_s == 0);
        ready = __all_sync(0xffffffffu, ready);
        tc_fence_after();
        if (ready) {
            const int row_in_tile = warp * 32 + lane;
            const int64_t row = (int64_t)m0 + row_in_tile;
            for (int c0 = 0; c0 < BN; c0 += 32) {
                float v[32];
                tmem_ld_32x32(tmem_d + ((uint32_t)(warp * 32) << 16) + (uint32_t)c0, v);
                if (p.out_f32) {
                    // FP32 partial tile of the weight gradient: [split][row][N]
                    float *dst = p.out_f32 + ((int64_t)blockIdx.z * part_rows + row) * p.N + n0 + c0;
                    if (row < p.M) {
#pragma unroll
                        for (int i = 0; i < 32; i += 4) *reinterpret_cast<float4 *>(dst + i) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
                    }
                } else if (row < p.M) {
                    if (p.bias) {
#pragma unroll
                        for (int i = 0; i < 32; ++i) v[i] += __ldg(p.bias + n0 + c0 + i);
                    }
                    if (p.relu) {
#pragma unroll
                        for (int i = 0; i < 32; ++i) v[i] = fmaxf(v[i], 0.f);
                    }
                    if (p.row_scale && n0 + c0 >= p.scale_col0) {
                        const float rs = __ldg(p.row_scale + row);
#pragma unroll
                        for (int i = 0; i < 32; ++i) v[i] *= rs;
                    }
                    bf16 *dst = p.C + row * p.ldc + n0 + c0;
#pragma unroll
                    for (int i = 0; i < 32; i += 8) {
                        Vec16<bf16> o;
                        o.from_float(v + i);
                        o.store(dst + i);
                    }
                }
            }
        }
    } else if (p.out_f32) {
        // empty reduction range: the partial tile is zero
        const int64_t row = (int64_t)m0 + threadIdx.x;
        if (row < p.M)
            for (int c = 0; c < BN; ++c) p.out_f32[((int64_t)blockIdx.z * part_rows + row) * p.N + n0 + c] = 0.f;
        if (MN_MAJOR && p.colsum != 0 && blockIdx.x == 0)
            for (int c = threadIdx.x; c < BN; c += TC_THREADS) p.out_f32[((int64_t)blockIdx.z * part_rows + p.M) * p.N + n0 + c] = 0.f;
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        __syncwarp();
        tmem_dealloc(tmem_d, tmem_cols);
    }
}

// ---------------------------------------------------------------------------------------------
// kernel 2: persistent K-major transform with the weight slice resident in shared memory.
//
// One CTA per SM.  CTA c owns the N slice (c mod n_slices) of width BN and walks the 128-row tiles
// c / n_slices, c / n_slices + stride, ...  Its slice of Bt (BN x K BF16, at most 128 KiB) is loaded
// once; only A tiles stream through a 4-stage ring.  Two accumulators in tensor memory let the
// epilogue of tile i overlap the MMAs of tile i + 1.  The epilogue (4 warps: tcgen05.ld, bias, ReLU,
// BF16) writes 128-column halves of the tile into a swizzled shared-memory staging area that one
// thread hands to TMA stores (full 128-byte rows instead of 16-byte pieces of 32 different rows per
// store instruction; rows beyond M are clipped by the tensor map).
//   warp 0: TMA producer (one lane)      warp 1: MMA issuer (one lane)      warps 2-9: epilogue
// (two warps per tensor-memory lane quarter, one per 64-column box of the 128-column round; each issues
// both of its 32-column loads before waiting)
// ---------------------------------------------------------------------------------------------
constexpr int TCP_THREADS = 320;       // warp 0 producer, warp 1 MMA issuer, warps 2-9 epilogue
constexpr int TCP_EPI_THREADS = 256;
constexpr int TCP_MAX_STAGES = 8;  // A-tile ring: as many 16 KiB stages as fit beside the weight slice (4..8)
constexpr int TCP_STAGE_OUT_BYTES = 2 * 16384;  // output staging: two boxes of 128 rows x 64 BF16 columns

LP_DEVINL void tma_store_2d(const CUtensorMap *map, uint32_t src, int x, int y)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];" ::"l"(map), "r"(src), "r"(x), "r"(y) : "memory");
}
LP_DEVINL void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
LP_DEVINL void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
LP_DEVINL void tma_store_wait_read_but_one() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }
LP_DEVINL void tma_store_wait_read_but_three() { asm volatile("cp.async.bulk.wait_group.read 3;" ::: "memory"); }
LP_DEVINL void box_barrier() { asm volatile("bar.sync 2, 256;" ::: "memory"); }  // the eight epilogue warps, around one staging box
LP_DEVINL void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
LP_DEVINL void epilogue_barrier() { asm volatile("bar.sync 1, 256;" ::: "memory"); }  // the eight epilogue warps only
LP_DEVINL void group_barrier(int grp) { asm volatile("bar.sync %0, 128;" ::"r"(2 + grp) : "memory"); }  // the four warps of one box group


__global__ void __launch_bounds__(TCP_THREADS, 1) tc_linear_persistent_kernel(const __grid_constant__ CUtensorMap mapA,
                                                                              const __grid_constant__ CUtensorMap mapB,
                                                                              const __grid_constant__ CUtensorMap mapC, const TcGemmParams p)
{
    LP_DEP_ENTER();
    __shared__ float s_bias[256];
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[TCP_MAX_STAGES], bar_empty[TCP_MAX_STAGES], bar_w, bar_acc_full[2], bar_acc_empty[2];
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int BN = p.BN;
    const int KB = p.K / TC_BK;                        // k-blocks per tile
    const uint32_t w_sub_bytes = (uint32_t)BN * 128;   // one k-block of the weight slice: BN rows x 128 B
    uint8_t *smem_w = smem;
    uint8_t *smem_a = smem + (size_t)KB * w_sub_bytes;
    const uint32_t a_bytes = TC_BM * TC_BK * 2;
    const int S = p.stages;
    uint8_t *smem_out = smem_a + (size_t)S * a_bytes;
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < 2 * BN) tmem_cols <<= 1;

    const int n_slices = p.N / BN;
    const int slice = blockIdx.x % n_slices;
    const int n0 = slice * BN;
    const int64_t m_tiles = (p.M + TC_BM - 1) / TC_BM;
    const int64_t first_tile = blockIdx.x / n_slices;
    const int64_t stride = gridDim.x / n_slices;
    const int64_t my_tiles = first_tile < m_tiles ? (m_tiles - first_tile + stride - 1) / stride : 0;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1);
            mbar_init(smem_u32(&bar_empty[s]), 1);
        }
        mbar_init(smem_u32(&bar_w), 1);
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&bar_acc_full[b]), 1);
            mbar_init(smem_u32(&bar_acc_empty[b]), 8);  // one arrival per epilogue warp
        }
        abort_s = 0;
        fence_barrier_init();
        fence_async_proxy();
        tma_prefetch_desc(&mapA);
        tma_prefetch_desc(&mapB);
        tma_prefetch_desc(&mapC);
    }
    if (warp == 0) {
        __syncwarp();
        tmem_alloc(smem_u32(&tmem_base_s), tmem_cols);
    }
    for (int j = threadIdx.x; j < BN; j += TCP_THREADS) s_bias[j] = p.bias ? p.bias[n0 + j] : 0.f;
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;
    volatile int *abort_flag = &abort_s;

    if (my_tiles > 0) {
        if (warp == 0 && lane == 0) {
            // ---- producer
            const uint32_t bw = smem_u32(&bar_w);
            mbar_expect_tx(bw, (uint32_t)KB * w_sub_bytes);
            for (int kb = 0; kb < KB; ++kb) tma_load_2d(smem_u32(smem_w + (size_t)kb * w_sub_bytes), &mapB, bw, kb * TC_BK, n0);
            int64_t it = 0;
            for (int64_t i = 0; i < my_tiles && !*abort_flag; ++i) {
                const int m0 = (int)((first_tile + i * stride) * TC_BM);
                for (int kb = 0; kb < KB; ++kb, ++it) {
                    const int s = (int)(it % S);
                    if (it >= S && !mbar_wait(smem_u32(&bar_empty[s]), (uint32_t)(((it / S) & 1) ^ 1), p.wait_ns)) {
                        atomicExch(p.err, 1);
                        *abort_flag = 1;
                        break;
                    }
                    const uint32_t bar = smem_u32(&bar_full[s]);
                    mbar_expect_tx(bar, a_bytes + (it == 0 ? (uint32_t)p.extra_tx : 0u));
                    tma_load_2d(smem_u32(smem_a + (size_t)s * a_bytes), &mapA, bar, kb * TC_BK, m0);
                }
            }
        } else if (warp == 1 && lane == 0) {
            // ---- MMA issuer
            const uint32_t idesc = make_idesc_bf16(BN, false, false);
            bool ok = mbar_wait(smem_u32(&bar_w), 0, p.wait_ns);
            if (!ok) { atomicExch(p.err, 4); *abort_flag = 1; }
            int64_t it = 0;
            for (int64_t i = 0; i < my_tiles && ok; ++i) {
                const int b = (int)(i & 1);
                if (i >= 2 && !mbar_wait(smem_u32(&bar_acc_empty[b]), (uint32_t)((((i >> 1) - 1) & 1)), p.wait_ns)) {
                    atomicExch(p.err, 5);
                    *abort_flag = 1;
                    break;
                }
                tc_fence_after();
                const uint32_t tmem_d = tmem_base + (uint32_t)(b * BN);
                for (int kb = 0; kb < KB; ++kb, ++it) {
                    const int s = (int)(it % S);
                    if (!mbar_wait(smem_u32(&bar_full[s]), (uint32_t)((it / S) & 1), p.wait_ns)) {
                        atomicExch(p.err, 2);
                        *abort_flag = 1;
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t sa = smem_u32(smem_a + (size_t)s * a_bytes);
                    const uint32_t sb = smem_u32(smem_w + (size_t)kb * w_sub_bytes);
#pragma unroll
                    for (int k = 0; k < TC_BK / TC_UMMA_K; ++k)
                        umma_bf16(tmem_d, make_smem_desc(sa + k * 32, 16, 1024), make_smem_desc(sb + k * 32, 16, 1024), idesc, (kb | k) != 0 ? 1u : 0u);
                    umma_commit(smem_u32(&bar_empty[s]));
                }
                if (ok) umma_commit(smem_u32(&bar_acc_full[b]));
            }
        } else if (warp >= 2) {
            // ---- epilogue: warp w reads the TMEM lanes of quarter (w mod 4); warps 2-5 take the first 64-column
            // box of every 128-column round, warps 6-9 the second
            const int q = warp & 3;
            const int my_box = (warp - 2) >> 2;
            for (int64_t i = 0; i < my_tiles; ++i) {
                const int b = (int)(i & 1);
                bool ready = mbar_wait(smem_u32(&bar_acc_full[b]), (uint32_t)((i >> 1) & 1), p.wait_ns);
                if (!ready && lane == 0) { atomicExch(p.err, 3); *abort_flag = 1; }
                if (!__all_sync(0xffffffffu, ready) && lane == 0) *abort_flag = 1;
                epilogue_barrier();             // the eight warps take the same decision: all continue or all leave
                if (*abort_flag != 0) break;
                tc_fence_after();
                const int m0 = (int)((first_tile + i * stride) * TC_BM);
                const int row_t = q * 32 + lane;  // row inside the tile
                const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(b * BN);
                const bool store_thread = (((warp - 2) & 3) == 0 && lane == 0);  // one per box group (warps 2 and 6)
                const bool row_ok = (int64_t)m0 + row_t < p.M;
                const float rs = (p.row_scale && row_ok) ? __ldg(p.row_scale + m0 + row_t) : 1.f;
                for (int half = 0; half < BN; half += 128) {
                    const int nbox = min(2, (BN - half) / 64);
                    // the two box groups (four warps, one 64-column staging box each) run independently: a group waits
                    // only for its own previous store and synchronises only its own 128 threads
                    if (my_box < nbox) {
                        if (store_thread) tma_store_wait_read();  // this group's previous store has read its staging box
                        group_barrier(my_box);
                        const int cb = half + my_box * 64;
                        uint32_t r[2][32];
                        tmem_ld_32x32_issue(taddr + (uint32_t)cb, r[0]);
                        tmem_ld_32x32_issue(taddr + (uint32_t)(cb + 32), r[1]);
                        tmem_ld_wait();
                        uint8_t *box = smem_out + (size_t)my_box * 16384 + (size_t)row_t * 128;
#pragma unroll
                        for (int h2 = 0; h2 < 2; ++h2) {
                            const int c0 = cb + 32 * h2;
                            float v[32];
#pragma unroll
                            for (int j = 0; j < 32; j += 4) {
                                const float4 bb = *reinterpret_cast<const float4 *>(&s_bias[c0 + j]);
                                v[j] = __uint_as_float(r[h2][j]) + bb.x;
                                v[j + 1] = __uint_as_float(r[h2][j + 1]) + bb.y;
                                v[j + 2] = __uint_as_float(r[h2][j + 2]) + bb.z;
                                v[j + 3] = __uint_as_float(r[h2][j + 3]) + bb.w;
                            }
                            if (p.relu) {
#pragma unroll
                                for (int j = 0; j < 32; ++j) v[j] = fmaxf(v[j], 0.f);
                            }
                            if (p.row_scale && n0 + c0 >= p.scale_col0) {
#pragma unroll
                                for (int j = 0; j < 32; ++j) v[j] *= rs;
                            }
                            // 128-byte swizzle of the staging box: 16-byte chunk index XOR (row mod 8)
                            const int chunk0 = 4 * h2;
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                Vec16<bf16> o;
                                o.from_float(v + 8 * j);
                                *reinterpret_cast<uint4 *>(box + (((chunk0 + j) ^ (row_t & 7)) << 4)) = o.v;
                            }
                        }
                        fence_async_proxy();  // generic-proxy writes -> visible to the TMA engine
                        group_barrier(my_box);
                        if (store_thread) {
                            tma_store_2d(&mapC, smem_u32(smem_out + (size_t)my_box * 16384), n0 + half + my_box * 64, m0);
                            tma_store_commit();
                        }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bar_acc_empty[b]));
            }
        }
    }
    if ((warp == 2 || warp == 6) && lane == 0) tma_store_wait_all();  // output tiles are in global memory before the CTA leaves
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        __syncwarp();
        tmem_dealloc(tmem_base, tmem_cols);
    }
}

// ---------------------------------------------------------------------------------------------
// kernel 3: the persistent transform on PAIRS of SMs (thread-block clusters of two CTAs, tcgen05 cta_group::2).
//
// One tcgen05.mma of the pair multiplies a 256-row tile (128 rows in each CTA's shared memory) by a BN-column weight
// slice of which each CTA holds half (BN / 2 rows of Bt), and leaves 128 rows x BN FP32 columns in each CTA's tensor
// memory.  Against kernel 2 a CTA keeps only half of the weight slice resident, so a slice up to 256 columns wide fits
// for K up to 512 and no operand tile is read by more than one SM.  Roles per CTA as in kernel 2 (warp 0 producer,
// warp 1 MMA issuer, warps 2-9 epilogue); only the issuer of the pair's first CTA (the leader) issues MMAs.
//   operand stages : each producer copies its own 128-row A tile and announces the bytes on the LEADER's full barrier
//                    (two arrivals per phase); the leader's commit releases the stage in both CTAs
//   accumulators   : two per CTA; the leader's commit tells both CTAs' epilogues that one is complete, the eight epilogue
//                    warps of BOTH CTAs arrive on the leader's barrier when they have drained it
//   tensor memory  : allocated and freed by warp 0 of both CTAs (cta_group::2), freed after a cluster barrier
// No bulk copy here is a multicast (every tile is copied by the CTA that consumes it); only the completion signal of the
// MMAs goes to both CTAs.  All waits are bounded.
// ---------------------------------------------------------------------------------------------
LP_DEVINL uint32_t cluster_cta_rank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
LP_DEVINL uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank)  // shared::cluster address of the same location in CTA `rank` of the cluster
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
    return r;
}
LP_DEVINL void cluster_barrier()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
LP_DEVINL void mbar_arrive_remote(uint32_t cluster_addr) { asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory"); }
LP_DEVINL void mbar_expect_tx_remote(uint32_t cluster_addr, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cluster.b64 _, [%0], %1;" ::"r"(cluster_addr), "r"(bytes) : "memory");
}
// tile copy into this CTA's shared memory whose completion is counted on a barrier of either CTA of the pair
LP_DEVINL void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, uint32_t bar_cluster_addr, int x, int y)
{
    asm volatile("cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
                 "l"(map), "r"(bar_cluster_addr), "r"(x), "r"(y)
                 : "memory");
}
LP_DEVINL void tmem_alloc_pair(uint32_t smem_dst, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
LP_DEVINL void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
LP_DEVINL void umma_bf16_pair(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// completion of the pair's earlier MMAs arrives on the barrier at this shared-memory offset in BOTH CTAs of the pair
// (a barrier signal sent to two CTAs; no data is copied)
LP_DEVINL void umma_commit_pair(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar), "h"((uint16_t)3)
                 : "memory");
}
// instruction descriptor of the pair's MMA: 256 rows (128 per CTA), n columns
static __host__ __device__ inline uint32_t make_idesc_bf16_pair(int n)
{
    uint32_t d = 0;
    d |= 1u << 4;                      // accumulator format F32
    d |= 1u << 7;                      // A format BF16
    d |= 1u << 10;                     // B format BF16
    d |= (uint32_t)(n >> 3) << 17;
    d |= (uint32_t)(256 >> 4) << 24;
    return d;
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(TCP_THREADS, 1)
    tc_linear_pair_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB, const __grid_constant__ CUtensorMap mapC,
                          const TcGemmParams p)
{
    LP_DEP_ENTER();
    __shared__ float s_bias[256];
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[TCP_MAX_STAGES], bar_empty[TCP_MAX_STAGES], bar_w, bar_acc_full[2], bar_acc_empty[2];
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_cta_rank();   // 0 = leader of the pair
    const bool leader = rank == 0;
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int BN = p.BN, HB = BN / 2;           // the pair's slice width and this CTA's half of it
    const int KB = p.K / TC_BK;
    const uint32_t w_sub_bytes = (uint32_t)HB * 128;  // one k-block of this CTA's half slice: HB rows x 128 B
    uint8_t *smem_w = smem;
    uint8_t *smem_a = smem + (size_t)KB * w_sub_bytes;
    const uint32_t a_bytes = TC_BM * TC_BK * 2;
    const int S = p.stages;
    uint8_t *smem_out = smem_a + (size_t)S * a_bytes;
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < 2 * BN) tmem_cols <<= 1;

    const int n_slices = p.N / BN;
    const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
    const int slice = pair % n_slices;
    const int n0 = slice * BN;
    const int64_t m_tiles = (p.M + 2 * TC_BM - 1) / (2 * TC_BM);  // tiles of 256 rows
    const int64_t first_tile = pair / n_slices;
    const int64_t stride = n_pairs / n_slices;
    const int64_t my_tiles = first_tile < m_tiles ? (m_tiles - first_tile + stride - 1) / stride : 0;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 2);   // one announcement per CTA of the pair (used in the leader only)
            mbar_init(smem_u32(&bar_empty[s]), 1);
        }
        mbar_init(smem_u32(&bar_w), 2);
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&bar_acc_full[b]), 1);
            mbar_init(smem_u32(&bar_acc_empty[b]), 16);  // eight epilogue warps in each CTA (used in the leader only)
        }
        abort_s = 0;
        fence_barrier_init();
        fence_async_proxy();
        tma_prefetch_desc(&mapA);
        tma_prefetch_desc(&mapB);
        tma_prefetch_desc(&mapC);
    }
    if (warp == 0) {
        __syncwarp();
        tmem_alloc_pair(smem_u32(&tmem_base_s), tmem_cols);
    }
    for (int j = threadIdx.x; j < BN; j += TCP_THREADS) s_bias[j] = p.bias ? p.bias[n0 + j] : 0.f;
    tc_fence_before();
    __syncthreads();
    cluster_barrier();  // both CTAs' barriers are initialised before either announces anything on them
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;
    volatile int *abort_flag = &abort_s;

    if (my_tiles > 0) {
        if (warp == 0 && lane == 0) {
            // ---- producer: this CTA's half of the weight slice, then its 128 rows of every tile
            const uint32_t bw = map_to_cta(smem_u32(&bar_w), 0);
            mbar_expect_tx_remote(bw, (uint32_t)KB * w_sub_bytes);
            for (int kb = 0; kb < KB; ++kb) tma_load_2d_pair(smem_u32(smem_w + (size_t)kb * w_sub_bytes), &mapB, bw, kb * TC_BK, n0 + (int)rank * HB);
            int64_t it = 0;
            for (int64_t i = 0; i < my_tiles && !*abort_flag; ++i) {
                const int m0 = (int)((first_tile + i * stride) * (2 * TC_BM)) + (int)rank * TC_BM;
                for (int kb = 0; kb < KB; ++kb, ++it) {
                    const int s = (int)(it % S);
                    if (it >= S && !mbar_wait(smem_u32(&bar_empty[s]), (uint32_t)(((it / S) & 1) ^ 1), p.wait_ns)) {
                        atomicExch(p.err, 1);
                        *abort_flag = 1;
                        break;
                    }
                    const uint32_t bar = map_to_cta(smem_u32(&bar_full[s]), 0);
                    mbar_expect_tx_remote(bar, a_bytes + (it == 0 && leader ? (uint32_t)p.extra_tx : 0u));
                    tma_load_2d_pair(smem_u32(smem_a + (size_t)s * a_bytes), &mapA, bar, kb * TC_BK, m0);
                }
            }
        } else if (warp == 1 && lane == 0 && leader) {
            // ---- MMA issuer of the pair
            const uint32_t idesc = make_idesc_bf16_pair(BN);
            bool ok = mbar_wait(smem_u32(&bar_w), 0, p.wait_ns);
            if (!ok) { atomicExch(p.err, 4); *abort_flag = 1; }
            int64_t it = 0;
            for (int64_t i = 0; i < my_tiles && ok; ++i) {
                const int b = (int)(i & 1);
                if (i >= 2 && !mbar_wait(smem_u32(&bar_acc_empty[b]), (uint32_t)((((i >> 1) - 1) & 1)), p.wait_ns)) {
                    atomicExch(p.err, 5);
                    *abort_flag = 1;
                    break;
                }
                tc_fence_after();
                const uint32_t tmem_d = tmem_base + (uint32_t)(b * BN);
                for (int kb = 0; kb < KB; ++kb, ++it) {
                    const int s = (int)(it % S);
                    if (!mbar_wait(smem_u32(&bar_full[s]), (uint32_t)((it / S) & 1), p.wait_ns)) {
                        atomicExch(p.err, 2);
                        *abort_flag = 1;
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t sa = smem_u32(smem_a + (size_t)s * a_bytes);
                    const uint32_t sb = smem_u32(smem_w + (size_t)kb * w_sub_bytes);
#pragma unroll
                    for (int k = 0; k < TC_BK / TC_UMMA_K; ++k)
                        umma_bf16_pair(tmem_d, make_smem_desc(sa + k * 32, 16, 1024), make_smem_desc(sb + k * 32, 16, 1024), idesc, (kb | k) != 0 ? 1u : 0u);
                    umma_commit_pair(smem_u32(&bar_empty[s]));  // the stage is free again in both CTAs
                }
                if (ok) umma_commit_pair(smem_u32(&bar_acc_full[b]));  // both CTAs' epilogues may drain their 128 rows
            }
        } else if (warp >= 2) {
            // ---- epilogue (as in kernel 2, on this CTA's 128 rows; the drained accumulator is reported to the leader)
            const int q = warp & 3;
            const int hsel = (warp - 2) >> 2;  // which 32 columns of a 64-column staging box this warp fills
            const uint32_t n_boxes = 2u * (uint32_t)p.out_sets;  // staging boxes, filled in turn by all eight warps
            uint32_t n_stores = 0;
            for (int64_t i = 0; i < my_tiles; ++i) {
                const int b = (int)(i & 1);
                const int m0 = (int)((first_tile + i * stride) * (2 * TC_BM)) + (int)rank * TC_BM;
                const int row_t = q * 32 + lane;
                const bool row_ok = (int64_t)m0 + row_t < p.M;
                // per-row operands of the epilogue are requested before the accumulator is waited for
                const float rs = (p.row_scale && row_ok) ? __ldg(p.row_scale + m0 + row_t) : 1.f;
                uint32_t keep4[4] = {0u, 0u, 0u, 0u};  // sign-bit words of this thread's (up to) four 32-column chunks of the tile
                if (p.mask_in && row_ok) {
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        const int c = 128 * (t >> 1) + 64 * (t & 1) + 32 * hsel;
                        if (c < BN) keep4[t] = __ldg(p.mask_in + (size_t)((n0 + c) >> 5) * (size_t)p.M + (size_t)(m0 + row_t));
                    }
                }
                bool ready = mbar_wait(smem_u32(&bar_acc_full[b]), (uint32_t)((i >> 1) & 1), p.wait_ns);
                if (!ready && lane == 0) { atomicExch(p.err, 3); *abort_flag = 1; }
                if (!__all_sync(0xffffffffu, ready) && lane == 0) *abort_flag = 1;
                epilogue_barrier();
                if (*abort_flag != 0) break;
                tc_fence_after();
                const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(b * BN);
                const bool store_thread = (warp == 2 && lane == 0);
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    const int half = 128 * hh;
                    if (half >= BN) break;
                    uint32_t r[2][32];
                    tmem_ld_32x32_issue(taddr + (uint32_t)(half + 32 * hsel), r[0]);
                    tmem_ld_32x32_issue(taddr + (uint32_t)(half + 64 + 32 * hsel), r[1]);
                    tmem_ld_wait();
#pragma unroll
                    for (int h2 = 0; h2 < 2; ++h2) {
                        // the box about to be filled has been read by the store that used it last: all but the n_boxes - 1 latest are done
                        if (store_thread) { if (n_boxes == 4) tma_store_wait_read_but_three(); else tma_store_wait_read_but_one(); }
                        box_barrier();
                        const uint32_t box_id = n_stores & (n_boxes - 1u);
                        ++n_stores;
                        const int cb = half + 64 * h2;    // first column of the box
                        const int c0 = cb + 32 * hsel;    // first of this thread's 32 columns
                        uint8_t *box = smem_out + (size_t)box_id * 16384 + (size_t)row_t * 128;
                        float v[32];
#pragma unroll
                        for (int j = 0; j < 32; j += 4) {
                            const float4 bb = *reinterpret_cast<const float4 *>(&s_bias[c0 + j]);
                            v[j] = __uint_as_float(r[h2][j]) + bb.x;
                            v[j + 1] = __uint_as_float(r[h2][j + 1]) + bb.y;
                            v[j + 2] = __uint_as_float(r[h2][j + 2]) + bb.z;
                            v[j + 3] = __uint_as_float(r[h2][j + 3]) + bb.w;
                        }
                        if (p.relu) {
#pragma unroll
                            for (int j = 0; j < 32; ++j) v[j] = fmaxf(v[j], 0.f);
                        }
                        if (p.row_scale && n0 + c0 >= p.scale_col0) {
#pragma unroll
                            for (int j = 0; j < 32; ++j) v[j] *= rs;
                        }
                        if (p.mask_in) {
                            const uint32_t keep = keep4[2 * hh + h2];
#pragma unroll
                            for (int j = 0; j < 32; ++j) v[j] = ((keep >> ((j >> 1) + 16 * (j & 1))) & 1u) ? v[j] : 0.f;
                        }
                        const int chunk0 = 4 * hsel;
                        uint32_t positive = 0;
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            Vec16<bf16> o;
                            o.from_float(v + 8 * j);
                            *reinterpret_cast<uint4 *>(box + (((chunk0 + j) ^ (row_t & 7)) << 4)) = o.v;
                            if (p.mask_out) {
                                // a stored value is positive exactly when its magnitude bits are not all zero (the ReLU left no
                                // negative ones): adding 0x7fff carries into bit 15 of each half of a packed pair
                                const uint32_t w4[4] = {o.v.x, o.v.y, o.v.z, o.v.w};
#pragma unroll
                                for (int t = 0; t < 4; ++t) {
                                    const int k = 4 * j + t;  // packed pair k holds columns 2 k and 2 k + 1 of these 32
                                    const uint32_t carry = ((w4[t] & 0x7fff7fffu) + 0x7fff7fffu) >> (15 - k);
                                    positive |= carry & ((1u << k) | (1u << (16 + k)));
                                }
                            }
                        }
                        if (p.mask_out && row_ok) p.mask_out[(size_t)((n0 + c0) >> 5) * (size_t)p.M + (size_t)(m0 + row_t)] = positive;
                        fence_async_proxy();
                        box_barrier();
                        if (store_thread) {
                            tma_store_2d(&mapC, smem_u32(smem_out + (size_t)box_id * 16384), n0 + cb, m0);
                            tma_store_commit();
                        }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_remote(map_to_cta(smem_u32(&bar_acc_empty[b]), 0));
            }
        }
    }
    if (warp == 2 && lane == 0) tma_store_wait_all();
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    cluster_barrier();  // neither CTA frees tensor memory, or leaves with barriers the other may still signal, before both are done
    if (warp == 0) {
        __syncwarp();
        tmem_dealloc_pair(tmem_base, tmem_cols);
    }
}

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
static bool tc_init(TcState &tc, std::string &err)
{
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn) {
        err = "cuTensorMapEncodeTiled is not available from the driver";
        return false;
    }
    tc.encode = (lp_encode_tiled_fn)fn;
    if (cudaMalloc((void **)&tc.err_word, 256) != cudaSuccess || cudaMalloc((void **)&tc.wbuf, sizeof(bf16) * TC_WBUF_ELEMS) != cudaSuccess ||
        cudaMallocHost((void **)&tc.host_err, sizeof(int)) != cudaSuccess) {
        err = "allocation of the tensor-core GEMM state failed";
        return false;
    }
    cudaMemset(tc.err_word, 0, 256);
    if (cudaFuncSetAttribute(tc_linear_persistent_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 225 * 1024 + 512) != cudaSuccess ||
        cudaFuncSetAttribute(tc_linear_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 225 * 1024 + 512) != cudaSuccess ||
        cudaFuncSetAttribute(tc_gemm_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024) != cudaSuccess ||
        cudaFuncSetAttribute(tc_gemm_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024) != cudaSuccess) {
        err = "cannot raise the dynamic shared memory limit of the tensor-core GEMM";
        return false;
    }
    return true;
}

static void tc_destroy(TcState &tc)
{
    cudaFree(tc.err_word);
    cudaFree(tc.wbuf);
    cudaFreeHost(tc.host_err);
    tc = TcState();
}

// Reads the device error word.  `synced` = the stream has already been synchronised by the caller;
// otherwise the word is only inspected when the caller asks for a synchronising check.
// the error word of the bounded waits: requested on the stream (tc_check_enqueue), read after the caller's own synchronise
// (tc_check_result), or both at once with a synchronise in between (tc_check)
static bool tc_check_enqueue(TcState &tc, Exec &ex)
{
    return cudaMemcpyAsync(tc.host_err, tc.err_word, sizeof(int), cudaMemcpyDeviceToHost, ex.st) == cudaSuccess;
}
static lp_status tc_check_result(TcState &tc, Exec &ex, std::string &err);
static lp_status tc_check(TcState &tc, Exec &ex, bool synced, std::string &err)
{
    if (!synced) return LP_OK;
    if (!tc_check_enqueue(tc, ex)) return LP_OK;
    cudaStreamSynchronize(ex.st);
    return tc_check_result(tc, ex, err);
}
static lp_status tc_check_result(TcState &tc, Exec &ex, std::string &err)
{
    if (*tc.host_err != 0) {
        char buf[128];
        snprintf(buf, sizeof buf, "tensor-core GEMM: bounded wait %d expired (1 = stage free, 2 = operands, 3 = accumulator, 4 = operands for the column sums)", *tc.host_err);
        err = buf;
        cudaMemsetAsync(tc.err_word, 0, sizeof(int), ex.st);
        return LP_ETIMEOUT;
    }
    return LP_OK;
}

// 2-D BF16 tensor map over a row-major matrix [rows, cols] with leading dimension ld (elements);
// box = {box_cols (inner, 128 bytes), box_rows}, 128-byte swizzle, zero fill outside.
static bool tc_make_map(const TcState &tc, CUtensorMap *map, const bf16 *base, int64_t rows, int64_t cols, int64_t ld, int box_cols, int box_rows,
                        std::string &err)
{
    if (((uintptr_t)base & 15) != 0 || (ld * 2) % 16 != 0) { err = "operand is not 16-byte aligned"; return false; }
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = tc.encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (void *)base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                           CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { err = "cuTensorMapEncodeTiled failed"; return false; }
    return true;
}

static int tc_pick_bn(int N) { return N <= 256 ? N : 256; }
static bool tc_linear_supported(int K, int N) { return K >= 64 && K % 64 == 0 && N >= 64 && N % 64 == 0 && N <= 512 && (N <= 256 || N % 256 == 0) && (int64_t)K * N <= TC_WBUF_ELEMS; }
static bool tc_weight_grad_supported(int Kin, int N) { return Kin >= 128 && Kin % 128 == 0 && N >= 64 && N % 64 == 0 && N <= 512 && (N <= 256 || N % 256 == 0); }

static int tc_stages(int BN, int num_kb)
{
    // two CTAs per SM when the stage ring allows it (smem per CTA <= ~110 KiB)
    const int stage = TC_BM * TC_BK * 2 + BN * TC_BK * 2;
    int s = (108 * 1024) / stage;
    s = std::max(2, std::min(s, 8));
    return std::max(1, std::min(s, std::max(num_kb, 1)));
}

// C[M, N] (BF16, leading dimension ldc) = act(A[M, K] * Bt[N, K]^T + bias); Bt is BF16, K contiguous.
// Slice width for the persistent kernel: the largest multiple of 64 (at most 256, dividing N) whose
// weight slice BN x K x 2 B fits 128 KiB beside the four 16 KiB A stages and the 32 KiB output staging.  0 = does not fit.
static int tc_persistent_bn(int N, int K)
{
    for (int bn = 256; bn >= 64; bn -= 64)
        if (N % bn == 0 && (int64_t)bn * K * 2 <= 128 * 1024) return bn;
    return 0;
}

// Slice width for the pair kernel: the largest multiple of 128 (at most 256, dividing N) whose half slice BN / 2 x K x 2 B
// fits 128 KiB beside at least two A stages and the output staging.  0 = does not fit.
static int tc_pair_bn(int N, int K)
{
    for (int bn = 256; bn >= 128; bn -= 128)
        if (N % bn == 0 && (int64_t)(bn / 2) * K * 2 <= 128 * 1024) return bn;
    return 0;
}

static int tc_sm_count()
{
    static int sms = 0;
    if (!sms) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (sms <= 0) sms = 148;
    }
    return sms;
}

// whether tc_gemm_kmajor runs this shape on pairs of SMs (the only kernel that reads and writes the sign-bit words)
static bool tc_pair_applies(int64_t M, int N, int K) { return tc_pair_bn(N, K) > 0 && M >= 64 * TC_BM && tc_sm_count() >= 4; }

static bool tc_gemm_kmajor(TcState &tc, Exec &ex, int64_t M, int N, int K, const bf16 *A, int64_t lda, const bf16 *Bt, const float *bias, bool relu,
                           bf16 *C, int64_t ldc, std::string &err, const float *row_scale = nullptr, int scale_col0 = 0, uint32_t *mask_out = nullptr,
                           const uint32_t *mask_in = nullptr)
{
    // pairs of SMs: a slice of up to 256 columns whose half (per CTA) fits 128 KiB; worth it from a few hundred tiles on
    const int pair_bn = tc_pair_bn(N, K);
    if ((mask_out || mask_in) && !(tc_pair_applies(M, N, K) && (!mask_out || relu))) {
        err = "sign-bit words need the pair kernel (and a ReLU when they are written)";
        return false;
    }
    if (tc_pair_applies(M, N, K)) {
        CUtensorMap mapA, mapB, mapC;
        if (!tc_make_map(tc, &mapA, A, M, K, lda, TC_BK, TC_BM, err)) return false;
        if (!tc_make_map(tc, &mapB, Bt, N, K, K, TC_BK, pair_bn / 2, err)) return false;
        if (!tc_make_map(tc, &mapC, C, M, N, ldc, 64, TC_BM, err)) return false;
        TcGemmParams p{};
        const int64_t smem_cap = 225 * 1024 + 512 - 1024;
        const int64_t w_bytes = (int64_t)(K / TC_BK) * (pair_bn / 2) * 128;  // this CTA's half of the slice
        p.M = M; p.N = N; p.K = K; p.BN = pair_bn;
        // a second set of output staging boxes where six A stages still fit beside it
        p.out_sets = (smem_cap - w_bytes - 2 * TCP_STAGE_OUT_BYTES) / (TC_BM * TC_BK * 2) >= 6 ? 2 : 1;
        const int64_t out_bytes = (int64_t)p.out_sets * TCP_STAGE_OUT_BYTES;
        p.stages = (int)std::max<int64_t>(2, std::min<int64_t>(TCP_MAX_STAGES, (smem_cap - w_bytes - out_bytes) / (TC_BM * TC_BK * 2)));
        p.bias = bias; p.relu = relu ? 1 : 0; p.C = C; p.ldc = ldc; p.out_f32 = nullptr; p.err = tc.err_word;
        p.row_scale = row_scale; p.scale_col0 = scale_col0;
        p.mask_out = mask_out; p.mask_in = mask_in;
        p.wait_ns = tc.wait_limit_ns; p.extra_tx = tc.overdeclare_tx; tc.overdeclare_tx = 0;
        const int n_slices = N / pair_bn;
        const int64_t m_tiles = ceil_div64(M, 2 * TC_BM);
        int64_t pairs = std::min<int64_t>((int64_t)tc_sm_count() / 2, m_tiles * n_slices);
        pairs = std::max<int64_t>(n_slices, pairs / n_slices * n_slices);  // a whole number of pairs per slice
        const size_t smem = (size_t)w_bytes + (size_t)p.stages * TC_BM * TC_BK * 2 + (size_t)out_bytes + 1024;
        launch_dep(tc_linear_pair_kernel, dim3((unsigned)(2 * pairs)), dim3(TCP_THREADS), smem, ex.st, mapA, mapB, mapC, p);
        ex.launches += 1;
        return true;
    }
    const int pbn = tc_persistent_bn(N, K);
    if (pbn > 0 && M >= 4 * TC_BM) {
        CUtensorMap mapA, mapB;
        if (!tc_make_map(tc, &mapA, A, M, K, lda, TC_BK, TC_BM, err)) return false;
        if (!tc_make_map(tc, &mapB, Bt, N, K, K, TC_BK, pbn, err)) return false;
        CUtensorMap mapC;
        if (!tc_make_map(tc, &mapC, C, M, N, ldc, 64, TC_BM, err)) return false;
        TcGemmParams p{};
        const int64_t smem_cap = 225 * 1024 + 512 - 1024;
        const int64_t w_bytes = (int64_t)(K / TC_BK) * pbn * 128;
        p.M = M; p.N = N; p.K = K; p.BN = pbn;
        p.stages = (int)std::max<int64_t>(4, std::min<int64_t>(TCP_MAX_STAGES, (smem_cap - w_bytes - TCP_STAGE_OUT_BYTES) / (TC_BM * TC_BK * 2)));
        p.bias = bias; p.relu = relu ? 1 : 0; p.C = C; p.ldc = ldc; p.out_f32 = nullptr; p.err = tc.err_word;
        p.row_scale = row_scale; p.scale_col0 = scale_col0;
        p.wait_ns = tc.wait_limit_ns; p.extra_tx = tc.overdeclare_tx; tc.overdeclare_tx = 0;
        const int n_slices = N / pbn;
        const int64_t m_tiles = ceil_div64(M, TC_BM);
        int64_t ctas = std::min<int64_t>((int64_t)tc_sm_count(), m_tiles * n_slices);
        ctas = std::max<int64_t>(n_slices, ctas / n_slices * n_slices);  // a whole number of CTAs per slice
        const size_t smem = (size_t)w_bytes + (size_t)p.stages * TC_BM * TC_BK * 2 + TCP_STAGE_OUT_BYTES + 1024;
        launch_dep(tc_linear_persistent_kernel, dim3((unsigned)ctas), dim3(TCP_THREADS), smem, ex.st, mapA, mapB, mapC, p);
        ex.launches += 1;
        return true;
    }
    const int BN = tc_pick_bn(N);
    CUtensorMap mapA, mapB;
    if (!tc_make_map(tc, &mapA, A, M, K, lda, TC_BK, TC_BM, err)) return false;
    if (!tc_make_map(tc, &mapB, Bt, N, K, K, TC_BK, BN, err)) return false;
    TcGemmParams p{};
    p.M = M; p.N = N; p.K = K; p.BN = BN;
    p.stages = tc_stages(BN, K / TC_BK);
    p.bias = bias; p.relu = relu ? 1 : 0; p.C = C; p.ldc = ldc; p.out_f32 = nullptr; p.rows = 0; p.rows_per_split = 0; p.err = tc.err_word;
    p.row_scale = row_scale; p.scale_col0 = scale_col0;
    p.wait_ns = tc.wait_limit_ns; p.extra_tx = tc.overdeclare_tx; tc.overdeclare_tx = 0;
    const size_t smem = (size_t)p.stages * (TC_BM * TC_BK * 2 + BN * TC_BK * 2) + 1024;
    dim3 grid((unsigned)ceil_div64(M, TC_BM), (unsigned)(N / BN), 1);
    launch_dep(tc_gemm_kernel<false>, dim3(grid), dim3(TC_THREADS), smem, ex.st, mapA, mapB, p);
    ex.launches += 1;
    return true;
}

// C = act(A B + bias) with a BF16 B operand given as [K, N] (b_is_nk = false: transposed into the scratch first) or [N, K] (b_is_nk = true)
__global__ void transpose_bf16_kernel(const bf16 *__restrict__ B, int K, int N, bf16 *__restrict__ Bt)
{
    LP_DEP_ENTER();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= K * N) return;
    const int k = i / N, n = i - k * N;
    Bt[(size_t)n * K + k] = B[i];
}

static bool tc_linear_bf16_b(TcState &tc, Exec &ex, int64_t M, int N, int K, const bf16 *A, int lda, const bf16 *B, bool b_is_nk, const float *bias,
                             bool relu, bf16 *C, int ldc, std::string &err)
{
    const bf16 *Bt = B;
    if (!b_is_nk) {
        launch_dep(transpose_bf16_kernel, dim3((K * N + 255) / 256), dim3(256), 0, ex.st, B, K, N, tc.wbuf);
        ex.launches += 1;
        Bt = tc.wbuf;
    }
    return tc_gemm_kmajor(tc, ex, M, N, K, A, lda, Bt, bias, relu, C, ldc, err);
}

// weight gradient: dW[Kin, N] (+)= A[rows, Kin]^T dZ[rows, N]; partial tiles per row split, then a
// fixed-order reduction
static int tc_weight_grad_splits(int64_t rows, int Kin, int N)
{
    const int tiles = (Kin / TC_BM) * (N / tc_pick_bn(N));
    int splits = std::max(1, (2 * 148) / std::max(tiles, 1));  // two CTAs per SM (measured: one per SM 156 us, two 145 us, three 207 us per step)
    const int64_t max_by_rows = std::max<int64_t>(1, ceil_div64(rows, 4 * TC_BK));
    return (int)std::min<int64_t>(splits, max_by_rows);
}
static int64_t tc_weight_grad_partials(int64_t rows, int Kin, int N)
{
    if (!tc_weight_grad_supported(Kin, N)) return 0;
    return (int64_t)tc_weight_grad_splits(rows, Kin, N) * (Kin + 1) * N;
}

// With fuse_bias the N floats that follow dW receive the column sums of dZ (the bias gradient): the
// partial tiles get one more row, filled by the first M tile's CTAs, and one reduction serves both.
static bool tc_weight_grad(TcState &tc, Exec &ex, int64_t rows, int Kin, int N, const bf16 *A, int lda, const bf16 *dZ, int ldz, float *dW, int accumulate,
                           float *partials, std::string &err, bool fuse_bias = false)
{
    const int BN = tc_pick_bn(N);
    const int splits = tc_weight_grad_splits(rows, Kin, N);
    CUtensorMap mapA, mapB;
    if (!tc_make_map(tc, &mapA, A, rows, Kin, lda, 64, TC_BK, err)) return false;
    if (!tc_make_map(tc, &mapB, dZ, rows, N, ldz, 64, TC_BK, err)) return false;
    TcGemmParams p{};
    p.M = Kin; p.N = N; p.K = 0; p.BN = BN;
    p.rows = rows;
    p.rows_per_split = ceil_div64(ceil_div64(rows, splits), TC_BK) * TC_BK;
    p.stages = tc_stages(BN, (int)(p.rows_per_split / TC_BK));
    p.bias = nullptr; p.relu = 0; p.C = nullptr; p.ldc = 0; p.out_f32 = partials; p.err = tc.err_word;
    p.colsum = fuse_bias ? 1 : 0;
    p.wait_ns = tc.wait_limit_ns; p.extra_tx = tc.overdeclare_tx; tc.overdeclare_tx = 0;
    const size_t smem = (size_t)p.stages * (TC_BM * TC_BK * 2 + BN * TC_BK * 2) + 1024;
    dim3 grid((unsigned)(Kin / TC_BM), (unsigned)(N / BN), (unsigned)splits);
    launch_dep(tc_gemm_kernel<true>, dim3(grid), dim3(TC_THREADS), smem, ex.st, mapA, mapB, p);
    const int64_t count = (int64_t)(Kin + (fuse_bias ? 1 : 0)) * N;
    launch_dep(reduce_partials_kernel, dim3((unsigned)ceil_div64(count, 256)), dim3(256), 0, ex.st, partials, count, splits, dW, accumulate);
    ex.launches += 2;
    return true;
}
