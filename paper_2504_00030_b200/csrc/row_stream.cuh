// Streaming access to logit rows (float32, or bf16 bit patterns widened exactly to float32), shared by
// the kernels that make one pass over the vocabulary: the accept / resample row statistics and the
// early-stop confidences.
#pragma once

#include "common.cuh"

namespace sv {

// 128-bit read-only load that does not pollute L1 (streamed once)
__device__ __forceinline__ uint4 ld_stream_u4(const void *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// element `idx` of an array of logits
template <bool BF16>
__device__ __forceinline__ float logit_at(const void *base, long long idx)
{
    if (BF16) return __uint_as_float((uint32_t)__ldg(static_cast<const unsigned short *>(base) + idx) << 16);
    return __ldg(static_cast<const float *>(base) + idx);
}

// start of row `row` of a [rows, stride] array of logits
template <bool BF16>
__device__ __forceinline__ const void *logit_row(const void *base, long long row, long long stride)
{
    if (BF16) return static_cast<const unsigned short *>(base) + row * stride;
    return static_cast<const float *>(base) + row * stride;
}

// four consecutive logits starting at k0 (k0 % 4 == 0), -inf past the vocabulary; `vec`: the row is
// 16-byte aligned (float32) / 8-byte aligned (bf16), so one vector load serves
template <bool BF16>
__device__ __forceinline__ void logit_load4(const void *row, int k0, int V, bool vec, float x[4])
{
    if (vec && k0 + 3 < V) {
        if (BF16) {
            const uint2 v = *reinterpret_cast<const uint2 *>(static_cast<const unsigned short *>(row) + k0);
            x[0] = __uint_as_float(v.x << 16); x[1] = __uint_as_float(v.x & 0xffff0000u);
            x[2] = __uint_as_float(v.y << 16); x[3] = __uint_as_float(v.y & 0xffff0000u);
        } else {
            const float4 v = *reinterpret_cast<const float4 *>(static_cast<const float *>(row) + k0);
            x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
        }
    } else {
#pragma unroll
        for (int u = 0; u < 4; ++u) x[u] = (k0 + u < V) ? logit_at<BF16>(row, k0 + u) : -CUDART_INF_F;
    }
}

// One warp streams elements [lo, hi) of a row (lo a multiple of 8) and hands them, four at a time and
// with the index of the first, to consume4(x0, x1, x2, x3, k0); positions past hi arrive as -inf.
// `vec_ok`: 128-bit streaming loads are legal for this row, UNROLL of them per lane are in flight.
template <bool BF16, int UNROLL, typename F>
__device__ __forceinline__ void stream_slice(const void *row, int lo, int hi, bool vec_ok, int lane, F &&consume4)
{
    constexpr int EPV = BF16 ? 8 : 4;          // elements per 128-bit load
    if (vec_ok) {
        const int nv = (hi - lo) / EPV;
        const uint4 *base = reinterpret_cast<const uint4 *>(logit_row<BF16>(row, 0, 0)) + (lo / EPV);
        for (int v0 = lane; v0 < nv; v0 += 32 * UNROLL) {
            uint4 x[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const int v = v0 + u * 32;
                x[u] = (v < nv) ? ld_stream_u4(base + v) : make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const int v = v0 + u * 32;
                if (v >= nv) continue;
                const int k0 = lo + EPV * v;
                if (BF16) {
                    consume4(__uint_as_float(x[u].x << 16), __uint_as_float(x[u].x & 0xffff0000u),
                             __uint_as_float(x[u].y << 16), __uint_as_float(x[u].y & 0xffff0000u), k0);
                    consume4(__uint_as_float(x[u].z << 16), __uint_as_float(x[u].z & 0xffff0000u),
                             __uint_as_float(x[u].w << 16), __uint_as_float(x[u].w & 0xffff0000u), k0 + 4);
                } else {
                    consume4(__uint_as_float(x[u].x), __uint_as_float(x[u].y), __uint_as_float(x[u].z),
                             __uint_as_float(x[u].w), k0);
                }
            }
        }
        // ragged end (fewer than EPV elements): last slice only
        if (lane == 0) {
            for (int k0 = lo + EPV * nv; k0 < hi; k0 += 4) {
                float t[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) t[u] = (k0 + u < hi) ? logit_at<BF16>(row, k0 + u) : -CUDART_INF_F;
                consume4(t[0], t[1], t[2], t[3], k0);
            }
        }
    } else {
        for (int k0 = lo + 4 * lane; k0 < hi; k0 += 4 * 32) {
            float t[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) t[u] = (k0 + u < hi) ? logit_at<BF16>(row, k0 + u) : -CUDART_INF_F;
            consume4(t[0], t[1], t[2], t[3], k0);
        }
    }
}

// 128-bit loads are legal for every row of an array of logits
inline bool logits_vec_ok(const void *base, long long row_stride, bool bf16)
{
    return base == nullptr || (aligned16(base) && row_stride % (bf16 ? 8 : 4) == 0);
}

}  // namespace sv
