// Declarations shared by the attention kernels and the C entry points.
#pragma once

#include <cuda.h>

#include "common.cuh"

struct sv_kv_pool {
    const void *k;
    const void *v;
    int64_t n_pages;
    int32_t page_size, hkv, head_dim;
    int64_t strides[4];     // elements: page, head, slot, dim
    bool has_maps;          // TMA tensor maps built (head_dim 128 and 64)
    CUtensorMap k_map;      // 4-D tiled maps over the pool, box = 64 dims x 16 slots of one
    CUtensorMap v_map;      // head of one page, 128-byte swizzle
};

namespace sv {

// Attention on CUDA cores, one thread block per (query row, head).  Any head_dim <= 128;
// used for shapes the tensor-core kernel does not cover and as a tiny-problem path.
sv_status launch_attn_simple(const sv_attn_params &p, cudaStream_t stream);

// Attention on tcgen05 tensor cores with TMA-staged K/V pages (head_dim 128 and 64).
bool attn_tc_supported(const sv_attn_params &p);
size_t attn_tc_workspace_bytes(int32_t batch, int32_t gamma_max, int32_t hq, int32_t hkv,
                               int32_t head_dim, int32_t max_seq_len);
sv_status launch_attn_tc(const sv_attn_params &p, void *workspace, size_t workspace_bytes,
                         cudaStream_t stream);

// The draft block's keys and values written into n caches that share one block table (kv_append.cu).
sv_status launch_kv_append_layers(const sv_kv_append_params &shared, const sv_kv_pool_t *pools, const void *const *k_new,
                                  const void *const *v_new, int n_layers, cudaStream_t stream);

}  // namespace sv
