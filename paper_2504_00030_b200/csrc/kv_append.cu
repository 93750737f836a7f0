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

constexpr int KA_MAX_LAYERS = 24;      // caches per launch (the per-cache pointers travel as kernel arguments)

struct KvAppendTarget {                // one cache and the new rows that go into it
    const uint4 *k_new;
    const uint4 *v_new;
    uint4 *k_pool;
    uint4 *v_pool;
    long long n_pages;
    long long stride_page, stride_head, stride_slot;   // in 16-byte chunks
};

struct KvAppendLaunch {
    sv_kv_append_params p;             // k_new / v_new / pool of p are not used by the kernel: see t[]
    KvAppendTarget t[KA_MAX_LAYERS];   // blockIdx.y selects the cache
    int hkv;
    int chunks;                        // 16-byte chunks per head row
};

__global__ void __launch_bounds__(KA_THREADS)
kv_append_kernel(const __grid_constant__ KvAppendLaunch a)
{
    pdl_enter();
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
    const KvAppendTarget &t = a.t[blockIdx.y];
    const int page = p.block_table[(long long)b * p.block_table_stride + pos / KA_PAGE];
    if (page < 0 || page >= t.n_pages) {
        if (threadIdx.x == 0) set_status(p.device_status, SV_DEV_BAD_PAGE);
        return;
    }
    const long long row = (long long)p.cu_q[b] + i;
    const uint4 *ks = t.k_new + row * a.hkv * a.chunks;
    const uint4 *vs = t.v_new + row * a.hkv * a.chunks;
    const long long base = (long long)page * t.stride_page + (long long)(pos % KA_PAGE) * t.stride_slot;
    const int n = a.hkv * a.chunks;
    for (int c = threadIdx.x; c < n; c += KA_THREADS) {
        const int head = c / a.chunks, ch = c - head * a.chunks;
        const long long dst = base + (long long)head * t.stride_head + ch;
        t.k_pool[dst] = __ldg(ks + c);
        t.v_pool[dst] = __ldg(vs + c);
    }
}

// host side: one cache and its new rows -> a launch target (checks included)
static sv_status make_target(const sv_kv_pool *pool, const void *k_new, const void *v_new, int hkv, int head_dim,
                             KvAppendTarget &t)
{
    if (pool == nullptr || k_new == nullptr || v_new == nullptr) return SV_EINVAL;
    if (pool->page_size != KA_PAGE || pool->head_dim % 8 != 0) return SV_EUNSUPPORTED;
    if (pool->hkv != hkv || pool->head_dim != head_dim) return SV_EINVAL;
    if (!aligned16(k_new) || !aligned16(v_new)) return SV_EALIGN;
    t.k_new = static_cast<const uint4 *>(k_new);
    t.v_new = static_cast<const uint4 *>(v_new);
    // the pool was registered through const pointers for the readers; this call is its writer
    t.k_pool = static_cast<uint4 *>(const_cast<void *>(pool->k));
    t.v_pool = static_cast<uint4 *>(const_cast<void *>(pool->v));
    t.n_pages = pool->n_pages;
    t.stride_page = pool->strides[0] / 8;      // registration checked: multiples of 8 elements, dim stride 1
    t.stride_head = pool->strides[1] / 8;
    t.stride_slot = pool->strides[2] / 8;
    return SV_OK;
}

// Appends the same block structure to n caches (n <= KA_MAX_LAYERS per launch, more in several launches).
sv_status launch_kv_append_layers(const sv_kv_append_params &shared, const sv_kv_pool_t *pools, const void *const *k_new,
                                  const void *const *v_new, int n_layers, cudaStream_t stream)
{
    if (shared.batch <= 0 || shared.gamma_max < 0 || n_layers <= 0 || pools == nullptr || pools[0] == nullptr)
        return SV_EINVAL;
    if (shared.block_table == nullptr || shared.seq_len == nullptr || shared.gamma == nullptr ||
        shared.cu_q == nullptr || shared.block_table_stride <= 0)
        return SV_EINVAL;
    if ((long long)shared.batch * (shared.gamma_max + 1) > 0x7fffffffLL) return SV_EUNSUPPORTED;
    const int hkv = pools[0]->hkv, head_dim = pools[0]->head_dim;
    for (int l0 = 0; l0 < n_layers; l0 += KA_MAX_LAYERS) {
        const int n = n_layers - l0 < KA_MAX_LAYERS ? n_layers - l0 : KA_MAX_LAYERS;
        KvAppendLaunch a;
        a.p = shared;
        a.hkv = hkv;
        a.chunks = head_dim / 8;
        for (int l = 0; l < n; ++l) {
            const sv_status st = make_target(pools[l0 + l], k_new[l0 + l], v_new[l0 + l], hkv, head_dim, a.t[l]);
            if (st != SV_OK) return st;
        }
        const dim3 grid((unsigned)(shared.batch * (shared.gamma_max + 1)), (unsigned)n);
        const sv_status st = launch_kernel(true, kv_append_kernel, grid, KA_THREADS, 0, stream, a);
        if (st != SV_OK) return st;
    }
    return SV_OK;
}

}  // namespace sv

extern "C" sv_status spec_kv_append(const sv_kv_append_params *p, void *stream)
{
    if (p == nullptr || p->pool == nullptr) return SV_EINVAL;
    const sv_kv_pool_t pool = p->pool;
    return sv::launch_kv_append_layers(*p, &pool, &p->k_new, &p->v_new, 1, (cudaStream_t)stream);
}
