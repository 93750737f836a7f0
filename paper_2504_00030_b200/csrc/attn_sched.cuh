// Work schedule shared by the tensor-core attention kernels: the key tiles of the whole batch
// form one list (sequence-major, then kv head, then tile); every persistent block takes an equal
// contiguous share of it.
#pragma once

#include "attn_common.cuh"

namespace sv {

constexpr int HD = 128;                 // head_dim of the tensor-core kernels
constexpr int MAX_BATCH_TC = 1 << 20;

struct AttnTcLaunch {
    sv_attn_params p;
    int64_t n_pool_pages;
    int group;           // query heads per kv head
    int nq;              // row groups of 128 rows (1 or 2)
    int slot_rows;       // query rows per partial-result slot
    int n_slots;         // K/V ring slots
    int32_t *ws_prefix;  // [batch+1] tile prefix, then [2]: total tiles, grid size
    float *ws_part;      // partial results: slot-major
};

// one partial slot: fp32 O rows, then the rows' running maxima, then their running sums
__host__ __device__ inline size_t part_slot_floats(int rows) { return (size_t)rows * (HD + 2); }

// first global tile of block c when `total` tiles are split over `grid` blocks
__device__ __forceinline__ long long share_begin(long long c, long long total, long long grid)
{
    return (c * total) / grid;
}

// Tiles and validated gamma of one sequence; sequences with inconsistent lengths own no tiles.
__device__ __forceinline__ int seq_tiles(const sv_attn_params &p, int b, int *gam_out, bool report, int tile)
{
    int g = p.gamma[b];
    if (g < 0 || g > p.gamma_max) {
        if (report) set_status(p.device_status, SV_DEV_BAD_GAMMA);
        g = min(max(g, 0), p.gamma_max);
    }
    const int L = p.seq_len[b];
    int nt = (L + tile - 1) / tile;
    if (L < g + 1 || (long long)(L + 15) / 16 > p.block_table_stride || L > p.max_seq_len) {
        if (report) set_status(p.device_status, SV_DEV_BAD_LEN);
        nt = 0;
    }
    if (gam_out != nullptr) *gam_out = g;
    return nt;
}

// Walks the (sequence, kv head, tile) triples of a block's share.
struct TileCursor {
    int b, g, t, n_tiles, gam;    // current pair, tile inside it, its tile count and gamma
    int tile_tokens;
    __device__ void seek(const sv_attn_params &p, int start_b, int start_prefix, long long tile, int tokens)
    {
        tile_tokens = tokens;
        b = start_b;
        n_tiles = seq_tiles(p, b, &gam, false, tile_tokens);
        const long long rel = tile - (long long)start_prefix * p.hkv;
        g = (int)(rel / n_tiles);
        t = (int)(rel % n_tiles);
    }
    __device__ void next_pair(const sv_attn_params &p)
    {
        t = 0;
        if (++g == p.hkv) {
            g = 0;
            n_tiles = 0;
            while (n_tiles == 0 && ++b < p.batch) n_tiles = seq_tiles(p, b, &gam, false, tile_tokens);
            if (b >= p.batch) n_tiles = 1;      // past the end: never used
        }
    }
};

// Tensor-memory-Q kernel (attn_tq.cu): up to 128 + 16 query rows per (sequence, kv head).
bool attn_tq_supported(const sv_attn_params &p);
int attn_tq_slot_rows(int rows);
sv_status launch_attn_tq_main(AttnTcLaunch &a, const sv_attn_params &p, int grid, cudaStream_t stream);

}  // namespace sv
