// Work schedule shared by the tensor-core attention kernels: the key tiles of the whole batch
// form one list (sequence-major, then kv head, then tile); every persistent block takes a
// contiguous share of it.  Shares are equal in COST, not in tiles: starting a (sequence, kv
// head) pair -- new query rows, a drained pipeline, an epilogue -- was measured to cost as much
// as a few tiles, so a pair counts as its tiles plus `seg_cost`; otherwise a block whose share
// holds many short sequences finishes long after the others.  Block c writes the first tile of
// its share to bounds[c] in the workspace, where the combine kernel finds it.
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
    int32_t *ws_prefix;  // [batch+1] tile prefix (last = total), grid size, then bounds[grid+1]
    float *ws_part;      // partial results: slot-major
};

// one partial slot: fp32 O rows, then the rows' running maxima, then their running sums
__host__ __device__ inline size_t part_slot_floats(int rows) { return (size_t)rows * (HD + 2); }

// first global tile of block c when `total` tiles are split over `grid` blocks
__device__ __forceinline__ long long share_begin(long long c, long long total, long long grid)
{
    return (c * total) / grid;
}

constexpr int MAX_ATTN_GRID = 1024;     // blocks of a main kernel (bounds table in the workspace)

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

// What a block learns in its prologue.
struct BlockShare {
    int total_tiles;             // tiles of all sequences, per kv head
    long long t_begin, t_end;    // the block's tiles of the global list
    int start_b, start_prefix;   // sequence that holds t_begin and the tiles (per kv head) before it
};

// Computes the calling block's share (whole warp); block 0 also publishes the tile prefix and
// the grid size for the combine kernel, and every block its lower bound.
__device__ __forceinline__ void plan_block_share(const AttnTcLaunch &a, int lane, int tile, int seg_cost,
                                                 BlockShare &o)
{
    const sv_attn_params &p = a.p;
    const int batch = p.batch, hkv = p.hkv;
    int32_t *bounds = a.ws_prefix + batch + 2;
    // pass 1: totals, real and with the per-pair cost added
    int carry = 0, carry_v = 0;
    if (blockIdx.x == 0 && lane == 0) a.ws_prefix[0] = 0;
    for (int base = 0; base < batch; base += 32) {
        const int b = base + lane;
        const int nt = (b < batch) ? seq_tiles(p, b, nullptr, blockIdx.x == 0, tile) : 0;
        int v = nt, vv = nt > 0 ? nt + seg_cost : 0;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, v, d), tv = __shfl_up_sync(0xffffffffu, vv, d);
            if (lane >= d) { v += t; vv += tv; }
        }
        if (blockIdx.x == 0 && b < batch) a.ws_prefix[b + 1] = carry + v;
        carry += __shfl_sync(0xffffffffu, v, 31);
        carry_v += __shfl_sync(0xffffffffu, vv, 31);
    }
    const long long total = (long long)carry * hkv, total_v = (long long)carry_v * hkv;
    const long long xb = share_begin(blockIdx.x, total_v, gridDim.x);
    const long long xe = share_begin(blockIdx.x + 1, total_v, gridDim.x);
    // pass 2: cost positions -> tiles.  A position inside pair j of its sequence maps to that
    // pair's tile at the same offset, or to the next pair's first tile if it falls in the cost part.
    long long tb = total, te = total;
    carry = carry_v = 0;
    for (int base = 0; base < batch; base += 32) {
        const int b = base + lane;
        const int nt = (b < batch) ? seq_tiles(p, b, nullptr, false, tile) : 0;
        const int w = nt > 0 ? nt + seg_cost : 0;
        int v = nt, vv = w;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, v, d), tv = __shfl_up_sync(0xffffffffu, vv, d);
            if (lane >= d) { v += t; vv += tv; }
        }
        const int pr = carry + v - nt, pv = carry_v + vv - w;
        const long long lo = (long long)pv * hkv, hi = (long long)(pv + w) * hkv;
#pragma unroll
        for (int which = 0; which < 2; ++which) {
            const long long x = which == 0 ? xb : xe;
            const unsigned hit = __ballot_sync(0xffffffffu, w > 0 && lo <= x && x < hi);
            if (hit != 0) {
                const int src = __ffs(hit) - 1;
                const int s_nt = __shfl_sync(0xffffffffu, nt, src);
                const int s_pr = __shfl_sync(0xffffffffu, pr, src), s_pv = __shfl_sync(0xffffffffu, pv, src);
                const long long rem = x - (long long)s_pv * hkv;
                const long long j = rem / (s_nt + seg_cost), off = rem - j * (s_nt + seg_cost);
                const long long t = (long long)s_pr * hkv + j * s_nt + (off < s_nt ? off : s_nt);
                if (which == 0) tb = t; else te = t;
            }
        }
        carry += __shfl_sync(0xffffffffu, v, 31);
        carry_v += __shfl_sync(0xffffffffu, vv, 31);
    }
    // pass 3: the sequence whose tiles contain the block's first tile
    int sb = 0, sp = 0;
    carry = 0;
    for (int base = 0; base < batch; base += 32) {
        const int b = base + lane;
        const int nt = (b < batch) ? seq_tiles(p, b, nullptr, false, tile) : 0;
        int v = nt;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, v, d);
            if (lane >= d) v += t;
        }
        const long long lo = (long long)(carry + v - nt) * hkv, hi = (long long)(carry + v) * hkv;
        const unsigned hit = __ballot_sync(0xffffffffu, nt > 0 && lo <= tb && tb < hi);
        if (hit != 0) {
            const int src = __ffs(hit) - 1;
            sb = __shfl_sync(0xffffffffu, b, src);
            sp = __shfl_sync(0xffffffffu, carry + v - nt, src);
        }
        carry += __shfl_sync(0xffffffffu, v, 31);
    }
    if (lane == 0) {
        bounds[blockIdx.x] = (int)tb;
        if (blockIdx.x + 1 == gridDim.x) bounds[gridDim.x] = (int)total;
        if (blockIdx.x == 0) a.ws_prefix[batch + 1] = (int)gridDim.x;
    }
    o.total_tiles = carry;
    o.t_begin = tb;
    o.t_end = te;
    o.start_b = sb;
    o.start_prefix = sp;
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
