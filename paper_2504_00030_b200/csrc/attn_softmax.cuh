// The per-tile step of the online softmax shared by the tensor-core attention kernels.
//
// One thread owns one query row = one TMEM lane.  The row's TILE scores are read from the S
// accumulator, masked causally, folded into the running reference (log2 domain, lazy: the
// reference only moves when a tile's maximum exceeds it by RESCALE_THRESHOLD, so P <= 2^8 and
// the accumulator is rarely rescaled), and written back over S as bf16 P for the P V product.
#pragma once

#include "tc_ptx.cuh"

#include <math_constants.h>

namespace sv {

constexpr float RESCALE_THRESHOLD = 8.f;           // log2 units: P <= 2^8 before a lazy rescale

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t *>(&h);
}

// s_addr: this lane's S buffer (TILE fp32 columns; P overlays its first TILE / 2 columns);
// o_addr: this lane's O accumulator (32 * O_CHUNKS fp32 columns); tok0: first token of the tile;
// pos: last key this row may see; first_tile: nothing has been accumulated into O yet.
// wait_prev_pv() must return once the P V product of the previous tile of this row group has
// completed (the accumulator may then be rescaled), or false if the wait was given up.
// Returns false if a wait was given up.  The caller waits for the stores (tcgen05.wait::st),
// fences and hands P over.
template <int TILE, int O_CHUNKS, typename WaitPV>
__device__ __forceinline__ bool softmax_tile(uint32_t s_addr, uint32_t o_addr, int tok0, int pos, bool need_mask,
                                             float c_scale, bool first_tile, float &m_ref, float &l_sum,
                                             WaitPV &&wait_prev_pv)
{
    // the row's scores: all loads in flight, one wait
    uint32_t s[TILE];
#pragma unroll
    for (int ch = 0; ch < TILE / 32; ++ch) tc_ld32_nowait(s_addr + ch * 32, s + ch * 32);
    tc_wait_ld();
    if (need_mask) {
#pragma unroll
        for (int c = 0; c < TILE; ++c)
            if (tok0 + c > pos) s[c] = 0xff800000u;     // -inf
    }
    float m0 = -CUDART_INF_F, m1 = -CUDART_INF_F, m2 = -CUDART_INF_F, m3 = -CUDART_INF_F;
#pragma unroll
    for (int c = 0; c < TILE; c += 4) {
        m0 = fmaxf(m0, __uint_as_float(s[c]));
        m1 = fmaxf(m1, __uint_as_float(s[c + 1]));
        m2 = fmaxf(m2, __uint_as_float(s[c + 2]));
        m3 = fmaxf(m3, __uint_as_float(s[c + 3]));
    }
    const float m_tile = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3)) * c_scale;
    float factor = 1.f;
    bool rescale = false;
    if (m_tile > m_ref + RESCALE_THRESHOLD || m_ref == -CUDART_INF_F) {
        if (m_tile > -CUDART_INF_F) {
            rescale = (m_ref > -CUDART_INF_F);
            factor = rescale ? ex2_approx(m_ref - m_tile) : 1.f;
            m_ref = m_tile;
        }
    }
    const float m_use = (m_ref == -CUDART_INF_F) ? 0.f : m_ref;
    if (rescale) l_sum *= factor;
    // tensor-memory accesses are warp-wide: if any row of the warp has to rescale its
    // accumulator, the whole warp goes through (factor 1 elsewhere)
    if (__any_sync(0xffffffffu, rescale && !first_tile)) {
        if (!wait_prev_pv()) return false;
        tc_fence_after();
        const float f = (rescale && !first_tile) ? factor : 1.f;
#pragma unroll
        for (int ch = 0; ch < O_CHUNKS; ++ch) {
            uint32_t o[32];
            tc_ld32(o_addr + ch * 32, o);
#pragma unroll
            for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * f);
            tc_st32(o_addr + ch * 32, o);
        }
    }
    // P = 2^(s*c - m_ref) as bf16 pairs, written over S (masked scores are -inf -> 0)
    float tile_sum = 0.f;
#pragma unroll
    for (int ch = 0; ch < TILE / 32; ++ch) {
        float sum0 = 0.f, sum1 = 0.f;
        uint32_t pk[16];
#pragma unroll
        for (int c = 0; c < 32; c += 2) {
            const float e0 = ex2_approx(fmaf(__uint_as_float(s[ch * 32 + c]), c_scale, -m_use));
            const float e1 = ex2_approx(fmaf(__uint_as_float(s[ch * 32 + c + 1]), c_scale, -m_use));
            sum0 += e0;
            sum1 += e1;
            pk[c >> 1] = pack_bf16(e0, e1);
        }
        tile_sum += sum0 + sum1;
        // chunk ch of P: 16 packed columns at [16 ch, 16 ch + 16) of the S buffer
        asm volatile(
            "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
            "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};" ::"r"(s_addr + ch * 16),
            "r"(pk[0]), "r"(pk[1]), "r"(pk[2]), "r"(pk[3]), "r"(pk[4]), "r"(pk[5]), "r"(pk[6]), "r"(pk[7]), "r"(pk[8]),
            "r"(pk[9]), "r"(pk[10]), "r"(pk[11]), "r"(pk[12]), "r"(pk[13]), "r"(pk[14]), "r"(pk[15])
            : "memory");
    }
    l_sum += tile_sum;
    return true;
}

}  // namespace sv
