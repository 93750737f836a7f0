// C entry points that are not tied to one kernel: status strings, KV-pool
// registration (TMA tensor maps), attention dispatch, the host-buffer step.
#include "attn_common.cuh"

#include <cstdlib>
#include <cstring>
#include <new>

namespace sv {

unsigned long long g_launches = 0;

int sm_count()
{
    static int cached[64];      // per device: one process may drive different GPUs
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (cached[dev] == 0) {
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0)
            cached[dev] = n;
        else
            return 148;   // B200; not cached, so a later call can still ask the device
    }
    return cached[dev];
}

typedef CUresult (*tensor_map_encode_fn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                         const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                         const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                         CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver symbol is looked up at run time so that the library carries no link-time
// dependency on libcuda (it must load on machines without a driver).
static tensor_map_encode_fn encode_fn()
{
    static tensor_map_encode_fn fn = nullptr;
    if (fn == nullptr) {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) ==
                cudaSuccess && q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<tensor_map_encode_fn>(ptr);
    }
    return fn;
}

static bool make_pool_map(CUtensorMap *map, const void *base, const sv_kv_pool &pool)
{
    tensor_map_encode_fn fn = encode_fn();
    if (fn == nullptr) return false;
    // innermost first: dim, slot, head, page
    const cuuint64_t dims[4] = {(cuuint64_t)pool.head_dim, (cuuint64_t)pool.page_size,
                                (cuuint64_t)pool.hkv, (cuuint64_t)pool.n_pages};
    const cuuint64_t strides[3] = {(cuuint64_t)pool.strides[2] * 2, (cuuint64_t)pool.strides[1] * 2,
                                   (cuuint64_t)pool.strides[0] * 2};
    const cuuint32_t box[4] = {64, 16, 1, 1};      // 64 dims (128 B) x 16 slots of one head, one page (head_dim 128: two boxes per page)
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(base), dims, strides, box,
              estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace sv

extern "C" const char *sv_status_str(sv_status s)
{
    switch (s) {
        case SV_OK: return "ok";
        case SV_EINVAL: return "invalid argument";
        case SV_EUNSUPPORTED: return "unsupported shape or option";
        case SV_EALIGN: return "pointer or stride not 16-byte aligned";
        case SV_ECUDA: return "CUDA call failed";
        case SV_EWORKSPACE: return "workspace missing or too small";
        default: return "unknown status";
    }
}

extern "C" uint64_t sv_launch_count(void) { return sv::g_launches; }

extern "C" sv_status spec_kv_pool_register(const void *k_pool, const void *v_pool, int64_t n_pages,
                                           int32_t page_size, int32_t hkv, int32_t head_dim,
                                           const int64_t strides[4], sv_kv_pool_t *out)
{
    if (out == nullptr) return SV_EINVAL;
    *out = nullptr;
    if (k_pool == nullptr || v_pool == nullptr || strides == nullptr || n_pages <= 0 || hkv <= 0)
        return SV_EINVAL;
    if (page_size != 16) return SV_EUNSUPPORTED;
    if (head_dim <= 0 || head_dim > 128 || head_dim % 8 != 0) return SV_EUNSUPPORTED;
    if (strides[3] != 1) return SV_EUNSUPPORTED;
    if (!sv::aligned16(k_pool) || !sv::aligned16(v_pool)) return SV_EALIGN;
    for (int i = 0; i < 3; ++i)
        if (strides[i] <= 0 || strides[i] % 8 != 0) return SV_EALIGN;
    sv_kv_pool *pool = new (std::nothrow) sv_kv_pool;
    if (pool == nullptr) return SV_EINVAL;
    memset(pool, 0, sizeof *pool);
    pool->k = k_pool;
    pool->v = v_pool;
    pool->n_pages = n_pages;
    pool->page_size = page_size;
    pool->hkv = hkv;
    pool->head_dim = head_dim;
    for (int i = 0; i < 4; ++i) pool->strides[i] = strides[i];
    pool->has_maps = false;
    if (head_dim == 128 || head_dim == 64) {
        if (!sv::make_pool_map(&pool->k_map, k_pool, *pool) ||
            !sv::make_pool_map(&pool->v_map, v_pool, *pool)) {
            delete pool;
            return SV_ECUDA;
        }
        pool->has_maps = true;
    }
    *out = pool;
    return SV_OK;
}

extern "C" sv_status spec_kv_pool_release(sv_kv_pool_t pool)
{
    if (pool == nullptr) return SV_EINVAL;
    delete pool;
    return SV_OK;
}

static sv_status check_attn(const sv_attn_params *p)
{
    if (p == nullptr || p->pool == nullptr) return SV_EINVAL;
    if (p->q == nullptr || p->o == nullptr || p->block_table == nullptr || p->seq_len == nullptr ||
        p->gamma == nullptr || p->cu_q == nullptr)
        return SV_EINVAL;
    if (p->batch <= 0 || p->gamma_max < 0 || p->hq <= 0 || p->hkv <= 0 || p->max_seq_len <= 0)
        return SV_EINVAL;
    if (p->hq % p->hkv != 0) return SV_EUNSUPPORTED;
    if (p->hkv != p->pool->hkv || p->head_dim != p->pool->head_dim) return SV_EINVAL;
    if (p->head_dim != 64 && p->head_dim != 128) return SV_EUNSUPPORTED;
    if (p->block_table_stride < (p->max_seq_len + 15) / 16) return SV_EINVAL;
    if (!sv::aligned16(p->q) || !sv::aligned16(p->o)) return SV_EALIGN;
    if (!(p->sm_scale > 0.f)) return SV_EINVAL;
    return SV_OK;
}

extern "C" size_t spec_verify_attn_workspace_bytes(int32_t batch, int32_t gamma_max, int32_t hq,
                                                   int32_t hkv, int32_t head_dim, int32_t max_seq_len)
{
    if (batch <= 0 || gamma_max < 0 || hq <= 0 || hkv <= 0 || head_dim <= 0 || max_seq_len <= 0)
        return 0;
    const size_t n = sv::attn_tc_workspace_bytes(batch, gamma_max, hq, hkv, head_dim, max_seq_len);
    return n > 256 ? n : 256;
}

extern "C" sv_status spec_verify_attn(const sv_attn_params *p, void *workspace,
                                      size_t workspace_bytes, void *stream)
{
    sv_status st = check_attn(p);
    if (st != SV_OK) return st;
    if (sv::attn_tc_supported(*p)) {
        if (workspace == nullptr ||
            workspace_bytes < spec_verify_attn_workspace_bytes(p->batch, p->gamma_max, p->hq, p->hkv,
                                                               p->head_dim, p->max_seq_len))
            return SV_EWORKSPACE;
        if (!sv::aligned16(workspace)) return SV_EALIGN;
        return sv::launch_attn_tc(*p, workspace, workspace_bytes, (cudaStream_t)stream);
    }
    return sv::launch_attn_simple(*p, (cudaStream_t)stream);
}

extern "C" sv_status spec_verify_attn_layers(const sv_attn_layers_params *p, void *workspace,
                                             size_t workspace_bytes, void *stream)
{
    if (p == nullptr || p->n_layers <= 0 || p->pools == nullptr || p->q == nullptr || p->o == nullptr)
        return SV_EINVAL;
    if ((p->k_new == nullptr) != (p->v_new == nullptr)) return SV_EINVAL;
    // every layer's arguments are checked before anything is launched
    for (int l = 0; l < p->n_layers; ++l) {
        sv_attn_params a = p->shared;
        a.pool = p->pools[l];
        a.q = p->q[l];
        a.o = p->o[l];
        a.lse = p->lse != nullptr ? p->lse[l] : nullptr;
        const sv_status st = check_attn(&a);
        if (st != SV_OK) return st;
        if (a.pool->hkv != p->pools[0]->hkv || a.pool->head_dim != p->pools[0]->head_dim) return SV_EINVAL;
    }
    if (p->k_new != nullptr) {
        sv_kv_append_params ka;
        memset(&ka, 0, sizeof ka);
        ka.block_table = p->shared.block_table;
        ka.block_table_stride = p->shared.block_table_stride;
        ka.seq_len = p->shared.seq_len;
        ka.gamma = p->shared.gamma;
        ka.cu_q = p->shared.cu_q;
        ka.batch = p->shared.batch;
        ka.gamma_max = p->shared.gamma_max;
        ka.device_status = p->shared.device_status;
        const sv_status st = sv::launch_kv_append_layers(ka, p->pools, p->k_new, p->v_new, p->n_layers,
                                                         (cudaStream_t)stream);
        if (st != SV_OK) return st;
    }
    for (int l = 0; l < p->n_layers; ++l) {
        sv_attn_params a = p->shared;
        a.pool = p->pools[l];
        a.q = p->q[l];
        a.o = p->o[l];
        a.lse = p->lse != nullptr ? p->lse[l] : nullptr;
        const sv_status st = spec_verify_attn(&a, workspace, workspace_bytes, stream);
        if (st != SV_OK) return st;
    }
    return SV_OK;
}

extern "C" sv_status spec_verify_step_host(const sv_step_host_io *io, const sv_attn_params *attn,
                                           void *attn_ws, size_t attn_ws_bytes,
                                           const sv_accept_params *acc, void *acc_ws,
                                           size_t acc_ws_bytes, const sv_gamma_params *gam,
                                           void *stream)
{
    if (io == nullptr || attn == nullptr || acc == nullptr || gam == nullptr) return SV_EINVAL;
    if (io->q_host == nullptr || io->target_logits_host == nullptr || io->n_accepted_host == nullptr ||
        io->out_tokens_host == nullptr || io->gamma_next_host == nullptr)
        return SV_EINVAL;
    if (io->n_q_rows <= 0 || io->n_d_rows < 0) return SV_EINVAL;
    sv_status st = check_attn(attn);
    if (st != SV_OK) return st;
    cudaStream_t s = (cudaStream_t)stream;
    const size_t q_bytes = (size_t)io->n_q_rows * attn->hq * attn->head_dim * 2;
    const size_t row_bytes = (size_t)acc->row_stride * (acc->logits_bf16 != 0 ? 2 : sizeof(float));
    bool ok = true;
    auto h2d = [&](const void *dst, const void *src, size_t n) {
        if (n != 0 && src != nullptr && dst != nullptr)
            ok = ok && cudaMemcpyAsync(const_cast<void *>(dst), src, n, cudaMemcpyHostToDevice, s) ==
                           cudaSuccess;
    };
    h2d(attn->q, io->q_host, q_bytes);
    h2d(acc->target_logits, io->target_logits_host, (size_t)io->n_q_rows * row_bytes);
    h2d(acc->draft_logits, io->draft_logits_host, (size_t)io->n_d_rows * row_bytes);
    h2d(acc->draft_tokens, io->draft_tokens_host, (size_t)io->n_d_rows * sizeof(int32_t));
    h2d(acc->u_accept, io->u_accept_host, (size_t)io->n_d_rows * sizeof(float));
    h2d(acc->u_sample, io->u_sample_host, (size_t)acc->batch * sizeof(float));
    if (!ok) return SV_ECUDA;
    st = spec_verify_attn(attn, attn_ws, attn_ws_bytes, stream);
    if (st != SV_OK) return st;
    st = spec_accept_sample(acc, acc_ws, acc_ws_bytes, stream);
    if (st != SV_OK) return st;
    st = gamma_tune_update(gam, stream);
    if (st != SV_OK) return st;
    auto d2h = [&](void *dst, const void *src, size_t n) {
        if (n != 0 && src != nullptr && dst != nullptr)
            ok = ok && cudaMemcpyAsync(dst, src, n, cudaMemcpyDeviceToHost, s) == cudaSuccess;
    };
    d2h(io->n_accepted_host, acc->n_accepted, (size_t)acc->batch * sizeof(int32_t));
    d2h(io->out_tokens_host, acc->out_tokens,
        (size_t)acc->batch * (acc->gamma_max + 1) * sizeof(int32_t));
    d2h(io->gamma_next_host, gam->gamma, (size_t)gam->batch * sizeof(int32_t));
    d2h(io->o_host, attn->o, q_bytes);
    return ok ? SV_OK : SV_ECUDA;
}
