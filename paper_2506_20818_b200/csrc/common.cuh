// Shared declarations of the link-prediction step library (device helpers, error macros).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <cstdio>
#include <cstring>
#include <string>
#include <vector>

#include "../../include/lp.h"

typedef __nv_bfloat16 bf16;

#define LP_DEVINL __device__ __forceinline__

static inline int64_t ceil_div64(int64_t a, int64_t b) { return (a + b - 1) / b; }

// ---------------------------------------------------------------------------------------------
// Programmatic dependent launch.  A kernel launched through launch_dep may be made resident as the blocks of the kernel
// before it in the stream retire; its own blocks sit at LP_DEP_ENTER until that kernel has completed and its writes
// are visible.  This hides the launch latency between the many short kernels of a step (about 45 us of an 870 us step).
// Every kernel launched this way executes LP_DEP_ENTER as its first statement -- before any early return, so that a grid
// never completes ahead of the one before it.  Launched the ordinary way the statement does nothing.  The kernels do
// not release their dependents early (griddepcontrol.launch_dependents): measured, blocks of the next kernel that take
// up room while this one still runs made the step 9 % slower.
// ---------------------------------------------------------------------------------------------
#define LP_DEP_ENTER() asm volatile("griddepcontrol.wait;" ::: "memory")

template <typename... KArgs, typename... Args>
static inline cudaError_t launch_dep(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args &&...args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// ---------------------------------------------------------------------------------------------
// element conversion helpers: activations are stored as float (FP32 path) or bf16 (BF16 path),
// all arithmetic is done in float.
// ---------------------------------------------------------------------------------------------
template <typename T> struct Vec16;  // 16-byte vector of T
template <> struct Vec16<float> {
    static constexpr int N = 4;
    float4 v;
    LP_DEVINL void load(const float *p) { v = __ldg(reinterpret_cast<const float4 *>(p)); }
    LP_DEVINL void store(float *p) const { *reinterpret_cast<float4 *>(p) = v; }
    LP_DEVINL void zero() { v = make_float4(0.f, 0.f, 0.f, 0.f); }
    LP_DEVINL void load_once(const float *p) { v = __ldcs(reinterpret_cast<const float4 *>(p)); }
    LP_DEVINL void store_once(float *p) const { __stcs(reinterpret_cast<float4 *>(p), v); }
    LP_DEVINL void to_float(float *f) const { f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w; }
    LP_DEVINL void from_float(const float *f) { v = make_float4(f[0], f[1], f[2], f[3]); }
};
template <> struct Vec16<bf16> {
    static constexpr int N = 8;
    uint4 v;
    LP_DEVINL void load(const bf16 *p) { v = __ldg(reinterpret_cast<const uint4 *>(p)); }
    LP_DEVINL void store(bf16 *p) const { *reinterpret_cast<uint4 *>(p) = v; }
    LP_DEVINL void zero() { v = make_uint4(0u, 0u, 0u, 0u); }
    // streaming forms for data touched once per launch (evicted first, so gathered rows keep their place in L2)
    LP_DEVINL void load_once(const bf16 *p) { v = __ldcs(reinterpret_cast<const uint4 *>(p)); }
    LP_DEVINL void store_once(bf16 *p) const { __stcs(reinterpret_cast<uint4 *>(p), v); }
    LP_DEVINL void to_float(float *f) const {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {  // bf16 -> float is a 16-bit shift
            f[2 * i] = __uint_as_float(w[i] << 16);
            f[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
    }
    LP_DEVINL void from_float(const float *f) {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            __nv_bfloat162 h = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
            w[i] = *reinterpret_cast<uint32_t *>(&h);
        }
        v = make_uint4(w[0], w[1], w[2], w[3]);
    }
};

template <typename T> LP_DEVINL float to_f(T x);
template <> LP_DEVINL float to_f<float>(float x) { return x; }
template <> LP_DEVINL float to_f<bf16>(bf16 x) { return __bfloat162float(x); }
template <typename T> LP_DEVINL T from_f(float x);
template <> LP_DEVINL float from_f<float>(float x) { return x; }
template <> LP_DEVINL bf16 from_f<bf16>(float x) { return __float2bfloat16_rn(x); }

// acc += <a, b> over one 16-byte vector, elements in storage order (one FMA each).  BF16 operands go through the
// mixed-precision FMA of sm_100 (fma.rn.f32.bf16: both factors widened exactly, one rounding), which gives the
// same bits as convert-then-fmaf without the conversion instructions.
template <typename T> LP_DEVINL float dot_vec(const Vec16<T> &a, const Vec16<T> &b, float acc)
{
    constexpr int VN = Vec16<T>::N;
    float fa[VN], fb[VN];
    a.to_float(fa);
    b.to_float(fb);
#pragma unroll
    for (int t = 0; t < VN; ++t) acc = fmaf(fa[t], fb[t], acc);
    return acc;
}
template <> LP_DEVINL float dot_vec<bf16>(const Vec16<bf16> &a, const Vec16<bf16> &b, float acc)
{
    const uint32_t x[4] = {a.v.x, a.v.y, a.v.z, a.v.w}, y[4] = {b.v.x, b.v.y, b.v.z, b.v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i)
        asm("{\n\t.reg .b16 alo, ahi, blo, bhi;\n\tmov.b32 {alo, ahi}, %1;\n\tmov.b32 {blo, bhi}, %2;\n\t"
            "fma.rn.f32.bf16 %0, alo, blo, %0;\n\tfma.rn.f32.bf16 %0, ahi, bhi, %0;\n\t}"
            : "+f"(acc)
            : "r"(x[i]), "r"(y[i]));
    return acc;
}
