// Shared host/device helpers of the specverify CUDA library (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <math_constants.h>
#include <stdint.h>

#include "../../include/specverify.h"

namespace sv {

// number of kernels launched by the library since load (reported by sv_launch_count)
extern unsigned long long g_launches;

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// The small kernels of a step (decisions, combine, controller update, cache append) are enqueued as programmatic
// dependent launches: they may be set up on the SMs while their predecessor in the stream drains, which hides the
// launch latency between the several kernels of a step (a third of the step time of the small workloads).  The
// first statement of every kernel, pdl_enter(), waits until the predecessor has completed and its memory is
// visible -- so the order of effects is that of a plain stream -- and then lets its own successor be set up in turn.
// The persistent kernels with a static split of their work (the logit streams, the attention main kernels) are
// launched plainly (early = false): set up early, their blocks start at different times on SMs that the
// predecessor's last blocks still share, and the blocks that start late finish late (+4 % on the largest workload).
template <typename... KArgs, typename... Args>
inline sv_status launch_kernel(bool early, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                               cudaStream_t stream, Args &&...args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = early ? 1 : 0;
    ++g_launches;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
    if (e != cudaSuccess) (void)cudaGetLastError();
    return e == cudaSuccess ? SV_OK : SV_ECUDA;
}

// multiprocessors of the current device (cached per device)
int sm_count();

// first statement of every kernel (see launch_kernel)
__device__ __forceinline__ void pdl_enter()
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}


__device__ __forceinline__ void set_status(uint32_t *status, uint32_t bits)
{
    if (status != nullptr) atomicOr(status, bits);
}

// 128-bit read-only load that does not pollute L1 (streamed once)
__device__ __forceinline__ float4 ld_stream_f4(const float *p)
{
    float4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                 : "l"(p));
    return v;
}

__device__ __forceinline__ float ex2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ double shfl_xor_f64(double v, int mask)
{
    int lo = __double2loint(v), hi = __double2hiint(v);
    lo = __shfl_xor_sync(0xffffffffu, lo, mask);
    hi = __shfl_xor_sync(0xffffffffu, hi, mask);
    return __hiloint2double(hi, lo);
}

__device__ __forceinline__ double shfl_up_f64(double v, int delta)
{
    int lo = __double2loint(v), hi = __double2hiint(v);
    lo = __shfl_up_sync(0xffffffffu, lo, delta);
    hi = __shfl_up_sync(0xffffffffu, hi, delta);
    return __hiloint2double(hi, lo);
}

__device__ __forceinline__ double shfl_idx_f64(double v, int src)
{
    int lo = __double2loint(v), hi = __double2hiint(v);
    lo = __shfl_sync(0xffffffffu, lo, src);
    hi = __shfl_sync(0xffffffffu, hi, src);
    return __hiloint2double(hi, lo);
}

__device__ __forceinline__ double warp_sum_f64(double v)
{
#pragma unroll
    for (int m = 16; m > 0; m >>= 1) v += shfl_xor_f64(v, m);
    return v;
}

// ---- online softmax statistics shared by the kernels that stream logit rows
constexpr float REF_INIT = -1.0e30f;    // running reference before the first element

// x * 2^k for k <= 0, exact while the result is a normal number (x >= 0); a result below the
// normal range, or a shift far below the reference, gives 0
__device__ __forceinline__ double scale_down_pow2(double x, float k)
{
    if (!(k > -800.f) || !(x > 0.0)) return (x != x) ? x : 0.0;     // NaN stays NaN
    if (k == 0.f || x == CUDART_INF) return x;
    const int hi = __double2hiint(x);
    if (((hi >> 20) & 0x7ff) + (int)k < 1) return 0.0;              // the exponent field would wrap
    return __hiloint2double(hi + ((int)k << 20), __double2loint(x));
}

// (ref, sum) pairs combine by rescaling to the larger reference; the factor is a power of two.
__device__ __forceinline__ void merge_stats(float &ref, double &sum, float ref2, double sum2)
{
    const float r = fmaxf(ref, ref2);
    sum = scale_down_pow2(sum, ref - r) + scale_down_pow2(sum2, ref2 - r);
    ref = r;
}

}  // namespace sv
