// Draft-block attention on CUDA cores: one thread block per (query row, query head).
//
// This is the general-shape path (any head_dim <= 128, any pool strides).  It
// re-reads the keys of a sequence once per query row and head, so it is only
// used where the problem is tiny (latency-bound) or the tensor-core kernel does
// not support the shape.  Scores for 128 keys at a time are computed one key
// per thread with 128-bit loads, combined by an online softmax, and the value
// accumulation runs one output dimension per thread (coalesced over head_dim).
#include "attn_common.cuh"

#include <math_constants.h>

namespace sv {

constexpr int AS_THREADS = 128;

__device__ __forceinline__ float block_max(float v, float *red)
{
#pragma unroll
    for (int m = 16; m > 0; m >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, m));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    v = fmaxf(fmaxf(red[0], red[1]), fmaxf(red[2], red[3]));
    __syncthreads();
    return v;
}

__device__ __forceinline__ float block_sum(float v, float *red)
{
#pragma unroll
    for (int m = 16; m > 0; m >>= 1) v += __shfl_xor_sync(0xffffffffu, v, m);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    v = (red[0] + red[1]) + (red[2] + red[3]);
    __syncthreads();
    return v;
}

__global__ void __launch_bounds__(AS_THREADS)
attn_simple_kernel(sv_attn_params p, sv_kv_pool pool)
{
    pdl_enter();
    __shared__ float s_q[128];
    __shared__ float s_p[AS_THREADS];
    __shared__ int s_page[AS_THREADS];
    __shared__ float s_red[4];
    __shared__ int s_bad;

    const int b = blockIdx.x / (p.gamma_max + 1);
    const int i = blockIdx.x % (p.gamma_max + 1);
    const int h = blockIdx.y;
    int g = p.gamma[b];
    if (g < 0 || g > p.gamma_max) {
        set_status(p.device_status, SV_DEV_BAD_GAMMA);
        g = min(max(g, 0), p.gamma_max);
    }
    if (i > g) return;
    const int L = p.seq_len[b];
    const int R = g + 1;
    if (L < R || (long long)(L + 15) / 16 > p.block_table_stride) {
        set_status(p.device_status, SV_DEV_BAD_LEN);
        return;
    }
    const int pos = L - R + i;                    // row i sees keys 0 .. pos
    const long long row = (long long)p.cu_q[b] + i;
    const int D = p.head_dim;
    const int kvh = h / (p.hq / p.hkv);
    const int tid = threadIdx.x;
    const __nv_bfloat16 *q = static_cast<const __nv_bfloat16 *>(p.q) + (row * p.hq + h) * D;
    const __nv_bfloat16 *kp = static_cast<const __nv_bfloat16 *>(pool.k);
    const __nv_bfloat16 *vp = static_cast<const __nv_bfloat16 *>(pool.v);
    const int32_t *bt = p.block_table + (long long)b * p.block_table_stride;

    if (tid < D) s_q[tid] = __bfloat162float(q[tid]);
    if (tid == 0) s_bad = 0;
    __syncthreads();

    float m_run = -CUDART_INF_F, l_run = 0.f, acc = 0.f;
    for (int t0 = 0; t0 <= pos; t0 += AS_THREADS) {
        const int j = t0 + tid;
        float s = -CUDART_INF_F;
        int page = -1;
        if (j <= pos) {
            page = bt[j >> 4];
            if (page < 0 || page >= pool.n_pages) {
                s_bad = 1;
                page = -1;
            } else {
                const __nv_bfloat16 *k = kp + page * pool.strides[0] + kvh * pool.strides[1] +
                                         (long long)(j & 15) * pool.strides[2];
                float dot = 0.f;
                for (int d = 0; d < D; d += 8) {
                    const uint4 raw = *reinterpret_cast<const uint4 *>(k + d);
                    const __nv_bfloat162 *k2 = reinterpret_cast<const __nv_bfloat162 *>(&raw);
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const float2 kk = __bfloat1622float2(k2[u]);
                        dot = fmaf(s_q[d + 2 * u], kk.x, dot);
                        dot = fmaf(s_q[d + 2 * u + 1], kk.y, dot);
                    }
                }
                s = dot * p.sm_scale;
            }
        }
        s_page[tid] = page;
        const float m_new = fmaxf(m_run, block_max(s, s_red));   // syncs: s_page, s_bad visible
        if (s_bad) break;
        const float pj = (page >= 0) ? __expf(s - m_new) : 0.f;
        s_p[tid] = pj;
        const float psum = block_sum(pj, s_red);                  // syncs: s_p visible
        const float corr = __expf(m_run - m_new);                 // 0 on the first tile
        l_run = l_run * corr + psum;
        acc *= corr;
        m_run = m_new;
        if (tid < D) {
            const int n = min(AS_THREADS, pos + 1 - t0);
            for (int jj = 0; jj < n; ++jj) {
                const __nv_bfloat16 *v = vp + s_page[jj] * pool.strides[0] + kvh * pool.strides[1] +
                                         (long long)((t0 + jj) & 15) * pool.strides[2];
                acc = fmaf(s_p[jj], __bfloat162float(v[tid]), acc);
            }
        }
        __syncthreads();
    }
    if (s_bad) {
        if (tid == 0) set_status(p.device_status, SV_DEV_BAD_PAGE);
        return;
    }
    __nv_bfloat16 *o = static_cast<__nv_bfloat16 *>(p.o) + (row * p.hq + h) * D;
    if (tid < D) o[tid] = __float2bfloat16_rn(acc / l_run);
    if (tid == 0 && p.lse != nullptr) p.lse[row * p.hq + h] = m_run + logf(l_run);
}

sv_status launch_attn_simple(const sv_attn_params &p, cudaStream_t stream)
{
    dim3 grid((unsigned)(p.batch * (p.gamma_max + 1)), (unsigned)p.hq);
    return launch_kernel(true, attn_simple_kernel, grid, AS_THREADS, 0, stream, p, *p.pool);
}

}  // namespace sv
