// Appending the draft block to the paged cache (KV caching, paper Section 5).
//
// One thread block per (sequence, new position): its threads copy the position's keys and
// values, 16 bytes at a time, from the packed new rows [n_rows, hkv, head_dim] to slot
// pos % 16 of page block_table[b][pos / 16] in every kv head.  Reads and writes are whole
// 16-byte chunks of contiguous head rows (256 bytes per head at head_dim 128).
#include "attn_common.cuh"
#include "common.cuh"

namespace sv {

constexpr int KA_THREADS = 128;
constexpr int KA_PAGE = 16;

struct KvAppendLaunch {
    sv_kv_append_params p;
    uint4 *k_pool;
    uint4 *v_pool;
    long long n_pages;
    long long stride_page, stride_head, stride_slot;   // in 16-byte chunks
    int hkv;
    int chunks;                                        // 16-byte chunks per head row
};

__global__ void __launch_bounds__(KA_THREADS)
kv_append_kernel(const __grid_constant__ KvAppendLaunch a)
{
    const sv_kv_append_params &p = a.p;
    const int rows_max = p.gamma_max + 1;
    const int b = blockIdx.x / rows_max, i = blockIdx.x % rows_max;
    int g = p.gamma[b];
    if (g < 0 || g > p.gamma_max) {
        if (threadIdx.x == 0 && i == 0) set_status(p.device_status, SV_DEV_BAD_GAMMA);
        g = min(max(g, 0), p.gamma_max);
    }
    const int R = g + 1;
    if (i >= R) return;
    const int L = p.seq_len[b];
    const int pos = L - R + i;
    if (L < R || (long long)(L - 1) / KA_PAGE >= p.block_table_stride) {
        if (threadIdx.x == 0 && i == 0) set_status(p.device_status, SV_DEV_BAD_LEN);
        return;
    }
    const int page = p.block_table[(long long)b * p.block_table_stride + pos / KA_PAGE];
    if (page < 0 || page >= a.n_pages) {
        if (threadIdx.x == 0) set_status(p.device_status, SV_DEV_BAD_PAGE);
        return;
    }
    const long long row = (long long)p.cu_q[b] + i;
    const uint4 *ks = static_cast<const uint4 *>(p.k_new) + row * a.hkv * a.chunks;
    const uint4 *vs = static_cast<const uint4 *>(p.v_new) + row * a.hkv * a.chunks;
    const long long base = (long long)page * a.stride_page + (long long)(pos % KA_PAGE) * a.stride_slot;
    const int n = a.hkv * a.chunks;
    for (int c = threadIdx.x; c < n; c += KA_THREADS) {
        const int head = c / a.chunks, ch = c - head * a.chunks;
        const long long dst = base + (long long)head * a.stride_head + ch;
        a.k_pool[dst] = __ldg(ks + c);
        a.v_pool[dst] = __ldg(vs + c);
    }
}

}  // namespace sv

extern "C" sv_status spec_kv_append(const sv_kv_append_params *p, void *stream)
{
    if (p == nullptr || p->pool == nullptr || p->batch <= 0 || p->gamma_max < 0) return SV_EINVAL;
    if (p->k_new == nullptr || p->v_new == nullptr || p->block_table == nullptr || p->seq_len == nullptr ||
        p->gamma == nullptr || p->cu_q == nullptr || p->block_table_stride <= 0)
        return SV_EINVAL;
    const sv_kv_pool &pool = *p->pool;
    if (pool.page_size != sv::KA_PAGE || pool.head_dim % 8 != 0) return SV_EUNSUPPORTED;
    if (!sv::aligned16(p->k_new) || !sv::aligned16(p->v_new)) return SV_EALIGN;
    if ((long long)p->batch * (p->gamma_max + 1) > 0x7fffffffLL) return SV_EUNSUPPORTED;
    sv::KvAppendLaunch a;
    a.p = *p;
    // the pool was registered through const pointers for the readers; this call is its writer
    a.k_pool = static_cast<uint4 *>(const_cast<void *>(pool.k));
    a.v_pool = static_cast<uint4 *>(const_cast<void *>(pool.v));
    a.n_pages = pool.n_pages;
    a.stride_page = pool.strides[0] / 8;       // registration checked: multiples of 8 elements, dim stride 1
    a.stride_head = pool.strides[1] / 8;
    a.stride_slot = pool.strides[2] / 8;
    a.hkv = pool.hkv;
    a.chunks = pool.head_dim / 8;
    sv::kv_append_kernel<<<(unsigned)(p->batch * (p->gamma_max + 1)), sv::KA_THREADS, 0, (cudaStream_t)stream>>>(a);
    return sv::launch_check();
}
