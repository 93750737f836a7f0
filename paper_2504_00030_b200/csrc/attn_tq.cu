// Draft-block attention, "queries in tensor memory" variant (tcgen05, sm_100a).
//
// Same schedule and data path as attn_tc.cu (stream-K over 128-token key tiles, TMA-staged
// pages, S = Q K^T and O += P V on the tensor cores with accumulators in tensor memory), with
// two changes that matter when a (sequence, kv head) pair has up to 144 query rows:
//
//  * The 128 query rows of the first row group live in TENSOR memory (64 columns of bf16
//    pairs) and enter S = Q K^T as the A operand from there.  Shared memory then holds nothing
//    but the K/V ring -- six or seven 32 KB slots, i.e. three or more tiles in flight per SM,
//    which is what the HBM latency asks for -- and the Q K^T instructions cost about a third
//    less than with A in shared memory.
//  * Rows 128..143 (8 query heads x 17 positions = 136 rows is the case that matters) do not
//    get a second 128-row tensor-memory group, whose instructions would cost as much as the
//    first group's for 1/16 of the useful work.  Four extra warps take them with warp-level
//    mma.sync (m16n8k16): each warp owns 32 of a tile's 128 tokens, reads the same K/V
//    shared-memory tiles with ldmatrix, keeps its own running max / sum / fp32 O (16 x 128) in
//    registers, and the four partial states are merged through shared memory when the
//    segment ends.
//
// Warps: 0 = TMA producer, 1 = MMA issuer and TMEM owner, 4..7 = softmax / epilogue of rows
// 0..127 (thread = row = TMEM lane), 8..11 = tail rows (template parameter TAIL).  All
// hand-offs are mbarriers; every wait is bounded, an expired wait sets SV_DEV_TIMEOUT and
// drains the block.
#include "attn_sched.cuh"
#include "attn_softmax.cuh"
#include "tc_ptx.cuh"

#include <math_constants.h>

namespace sv {

namespace tq {

constexpr int TILE = 128;                          // tokens per key tile
constexpr int S_COL0 = 0;                          // TMEM columns: two S buffers,
constexpr int O_COL0 = 256;                        // the O accumulator,
constexpr int Q_COL0 = 384;                        // the query rows (bf16 pairs)
constexpr uint32_t TMEM_COLS = 512;
constexpr int TAIL_ROWS = 16;
constexpr int SEG_COST = 6;                        // starting a pair costs about as much as six tiles (fitted: 5.8 us per pair against 1.5 us per tile; 3, 4 and 8 measured slower)

struct Shared {
    uint64_t full[8];        // ring slot filled by TMA
    uint64_t empty[8];       // ring slot released by all its readers
    uint64_t s_full[2];      // S accumulator ready
    uint64_t p_full[2];      // P written by the softmax threads
    uint64_t o_done[2];      // PV of tile u finished (indexed by u & 1)
    uint64_t q_full;         // query rows of a segment are in tensor memory
    uint64_t tail_sync;      // the four tail warps meet here around their merge
    uint32_t tmem_base;
    int abort_flag;
    int total_tiles;
    long long t_begin, t_end;    // this block's tiles of the global list
    int start_b;
    int start_prefix;
};

// merge buffers of the tail warps: [warp][row][dim], then running max and sum [warp][row]
struct TailMerge {
    float o[4][TAIL_ROWS][HD];
    float m[4][TAIL_ROWS];
    float l[4][TAIL_ROWS];
};

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2,
                                                  uint32_t &r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
// D (16x8 fp32) += A (16x16 bf16, row) * B (16x8 bf16, col)
__device__ __forceinline__ void mma_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// transpose of an 8x8 matrix of 16-bit elements held one row (4 x 2 elements) per 4 lanes
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t x)
{
    uint32_t y;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(y) : "r"(x));
    return y;
}

}  // namespace tq

using namespace tq;

// NB: blocks of 8 tail rows beyond row 127 (0: no tail warps).  D: head_dim, 128 or 64.  With 64 dims a K or V
// tile is one 16 KB half (the 128-byte rows of one swizzle atom), Q K^T has four k-steps, O has 64 columns; the
// partial-result slots keep their 128-float row pitch.
template <int NB, int D>
__global__ void __launch_bounds__(NB > 0 ? 384 : 256, 1)
attn_tq_kernel(const AttnTcLaunch a, const __grid_constant__ CUtensorMap k_map,
               const __grid_constant__ CUtensorMap v_map)
{
    static_assert(D == 128 || (D == 64 && NB == 0), "tail rows are built for 128-dim heads only");
    constexpr bool TAIL = NB > 0;
    constexpr int SLOT_BYTES = TILE * D * 2;           // one K or one V tile
    constexpr int NBA = NB > 0 ? NB : 1;               // array extent (no zero-length arrays)
    pdl_enter();
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    // carve: [ring slots][tail merge buffers][Shared]; the swizzled tiles need a 1024-byte aligned base
    uint8_t *ring = smem_raw;
    if ((smem_u32(ring) & 1023u) != 0) {               // never seen; refuse rather than compute garbage
        if (threadIdx.x == 0) set_status(a.p.device_status, SV_DEV_TIMEOUT);
        return;
    }
    const int n_slots = a.n_slots;
    TailMerge *tm = reinterpret_cast<TailMerge *>(ring + (size_t)n_slots * SLOT_BYTES);
    Shared *sh = reinterpret_cast<Shared *>(ring + (size_t)n_slots * SLOT_BYTES + (TAIL ? sizeof(TailMerge) : 0));

    const sv_attn_params &p = a.p;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int batch = p.batch, hkv = p.hkv, G = a.group;

    if (tid == 0) {
        for (int i = 0; i < n_slots; ++i) {
            mbar_init(smem_u32(&sh->full[i]), 1);
            mbar_init(smem_u32(&sh->empty[i]), TAIL ? 5 : 1);    // tensor core + one lane per tail warp
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&sh->s_full[i]), 1);
            mbar_init(smem_u32(&sh->p_full[i]), 128);
            mbar_init(smem_u32(&sh->o_done[i]), 1);
        }
        mbar_init(smem_u32(&sh->q_full), 128);
        mbar_init(smem_u32(&sh->tail_sync), 4);
        sh->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (warp == 0) {
        BlockShare bs;
        plan_block_share(a, lane, TILE, SEG_COST, bs);
        if (lane == 0) {
            sh->total_tiles = bs.total_tiles;
            sh->t_begin = bs.t_begin;
            sh->t_end = bs.t_end;
            sh->start_b = bs.start_b;
            sh->start_prefix = bs.start_prefix;
        }
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                         smem_u32(&sh->tmem_base)),
                     "r"(TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    const long long total = (long long)sh->total_tiles * hkv;
    const long long grid = gridDim.x;
    const long long t_begin = sh->t_begin, t_end = sh->t_end;
    const uint32_t tmem = sh->tmem_base;
    const float c_scale = p.sm_scale * 1.4426950408889634f;   // scores in log2 units
    const int start_b = sh->start_b, start_prefix = sh->start_prefix;
    int *abort_flag = &sh->abort_flag;

    // With the tail warps there are 384 threads and 168 registers each at launch; the producer /
    // MMA warpgroup hands most of its share to the others (128 * (64 + 240 + 200) = 384 * 168).
    if (warp < 4) {
        if (TAIL) asm volatile("setmaxnreg.dec.sync.aligned.u32 64;");
        if (t_end > t_begin && warp != 1) {
            // ================================================================ TMA producers
            // One thread gets a tensor copy under way every ~90 cycles, and a tile needs 32 of
            // them (K and V, 8 pages, two 64-dim halves): one warp cannot keep up with HBM.  Warps
            // 0, 2 and 3 therefore take the ring items (2*tile = K, 2*tile+1 = V) round robin.
            const int pi = warp == 0 ? 0 : warp - 1;       // producer index 0..2
            TileCursor cur;
            cur.seek(p, start_b, start_prefix, t_begin, TILE);
            // lane l < 16: page l/2, dims half l%2 (128 dims); lane l < 8: page l (64 dims, one half)
            const int page_in_tile = D == 128 ? (lane >> 1) & 7 : lane & 7, half = D == 128 ? lane & 1 : 0;
            bool ok = true;
            long long tg = t_begin;
            for (uint32_t item = pi; ok && t_begin + (item >> 1) < t_end; item += 3) {
                while (tg < t_begin + (item >> 1)) {           // advance the cursor to this item's tile
                    ++tg;
                    if (++cur.t == cur.n_tiles) cur.next_pair(p);
                }
                const int b = cur.b;
                const int L = p.seq_len[b];
                const int n_pages = (L + 15) >> 4;
                const int32_t *bt = p.block_table + (long long)b * p.block_table_stride;
                const int lp = cur.t * (TILE / 16) + page_in_tile;
                int phys = (int)a.n_pool_pages;       // out of range: TMA fills zeros, no traffic
                if (lp < n_pages) {
                    const int e = bt[lp];
                    if (e < 0 || e >= a.n_pool_pages) set_status(p.device_status, SV_DEV_BAD_PAGE);
                    else phys = e;
                }
                const uint32_t slot = item % (uint32_t)n_slots;
                const uint32_t use = item / (uint32_t)n_slots;
                const uint32_t full = smem_u32(&sh->full[slot]);
                if (use > 0) ok = bounded_wait(smem_u32(&sh->empty[slot]), (use - 1) & 1, abort_flag, p.device_status);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                if (lane == 0) mbar_expect_tx(full, SLOT_BYTES);
                __syncwarp();
                if (lane < D / 8) {
                    const uint32_t dst = smem_u32(ring + slot * SLOT_BYTES + half * 16384 + page_in_tile * 2048);
                    tma_load_4d(dst, (item & 1) == 0 ? &k_map : &v_map, half * 64, 0, cur.g, phys, full);
                }
            }
        } else if (t_end > t_begin && warp == 1) {
            // ================================================================ MMA issuer
            // the whole warp walks the schedule and waits; one elected lane issues
            const uint32_t idesc_qk = instr_desc(false, TILE), idesc_pv = instr_desc(true, D);
            TileCursor cur;
            cur.seek(p, start_b, start_prefix, t_begin, TILE);
            uint32_t tile_no = 0;      // tiles of this block so far (ring position and S / P buffer parity)
            uint32_t seg_no = 0;
            bool ok = true;
            for (long long tg = t_begin; tg < t_end && ok;) {
                const int seg_tiles = (int)min((long long)(cur.n_tiles - cur.t), t_end - tg);
                ok = bounded_wait(smem_u32(&sh->q_full), seg_no & 1, abort_flag, p.device_status);
                tc_fence_after();
                auto issue_qk = [&](int ti) {
                    const uint32_t gu = tile_no + ti;
                    const uint32_t item = 2 * gu;
                    const uint32_t slot = item % (uint32_t)n_slots;
                    ok = ok && bounded_wait(smem_u32(&sh->full[slot]), (item / n_slots) & 1, abort_flag,
                                            p.device_status);
                    if (!ok) return;
                    tc_fence_after();
                    const uint64_t kd = smem_desc(smem_u32(ring + slot * SLOT_BYTES), 16, 1024);
                    const uint32_t d = tmem + S_COL0 + (gu & 1) * TILE;
                    if (elect_one()) {
#pragma unroll
                        for (int ks = 0; ks < D / 16; ++ks) {
                            const uint32_t koff = ((ks >> 2) * 16384 + (ks & 3) * 32) >> 4;
                            tc_mma_ts(d, tmem + Q_COL0 + ks * 8, kd + koff, idesc_qk, ks > 0);
                        }
                        tc_commit(smem_u32(&sh->s_full[gu & 1]));
                        tc_commit(smem_u32(&sh->empty[slot]));          // K tile consumed
                    }
                    __syncwarp();
                };
                issue_qk(0);
                if (seg_tiles > 1) issue_qk(1);
                for (int ti = 0; ti < seg_tiles && ok; ++ti) {
                    const uint32_t gu = tile_no + ti;
                    ok = bounded_wait(smem_u32(&sh->p_full[gu & 1]), (gu >> 1) & 1, abort_flag, p.device_status);
                    const uint32_t item = 2 * gu + 1;
                    const uint32_t slot = item % (uint32_t)n_slots;
                    if (ok) ok = bounded_wait(smem_u32(&sh->full[slot]), (item / n_slots) & 1, abort_flag, p.device_status);
                    if (!ok) break;
                    tc_fence_after();
                    const uint64_t vd = smem_desc(smem_u32(ring + slot * SLOT_BYTES), 16384, 1024);
                    const uint32_t pa = tmem + S_COL0 + (gu & 1) * TILE;      // P overlays S, TILE/2 columns
                    const uint32_t d = tmem + O_COL0;
                    if (elect_one()) {
#pragma unroll
                        for (int ks = 0; ks < TILE / 16; ++ks)
                            tc_mma_ts(d, pa + ks * 8, vd + (uint64_t)(ks * (2048 >> 4)), idesc_pv,
                                      (ti > 0 || ks > 0) ? 1u : 0u);
                        tc_commit(smem_u32(&sh->o_done[gu & 1]));
                        tc_commit(smem_u32(&sh->empty[slot]));          // V tile consumed
                    }
                    __syncwarp();
                    if (ti + 2 < seg_tiles) issue_qk(ti + 2);
                }
                tile_no += seg_tiles;
                ++seg_no;
                tg += seg_tiles;
                cur.t += seg_tiles;
                if (cur.t == cur.n_tiles) cur.next_pair(p);
            }
        }
    } else if (warp < 8) {
        if (TAIL) asm volatile("setmaxnreg.inc.sync.aligned.u32 240;");
        if (t_end > t_begin) {
            // ================================================================ softmax / epilogue, rows 0..127
            const int quarter = warp & 3;
            const int r = quarter * 32 + lane;                 // row of the pair = TMEM lane
            const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
            const uint32_t o_addr = tmem + lane_addr + O_COL0;
            TileCursor cur;
            cur.seek(p, start_b, start_prefix, t_begin, TILE);
            uint32_t ug = 0;               // tiles of this block so far
            uint32_t seg_no = 0;
            bool ok = true;
            for (long long tg = t_begin; tg < t_end && ok; ++seg_no) {
                const int b = cur.b, g = cur.g;
                const int seg_tiles = (int)min((long long)(cur.n_tiles - cur.t), t_end - tg);
                const int R = cur.gam + 1, L = p.seq_len[b];
                const int n_rows = G * R;
                const bool warp_active = quarter * 32 < n_rows;
                const bool row_ok = r < n_rows;
                const int i = r / G, hh = r - i * G;
                const int pos = L - R + i;                     // last visible key of this row
                const long long q_row = ((long long)p.cu_q[b] + i) * p.hq + (long long)g * G + hh;
                // ---- this thread's query row -> its tensor-memory lane (64 columns of bf16 pairs).
                // Every tensor-core instruction that read the previous segment's rows has completed:
                // this thread has seen the last S of that segment, and S follows all Q K^T in order.
                if (warp_active) {
                    const uint4 *src = reinterpret_cast<const uint4 *>(
                        static_cast<const __nv_bfloat16 *>(p.q) + q_row * D);
#pragma unroll
                    for (int hf = 0; hf < D / 64; ++hf) {
                        uint32_t qv[32];
#pragma unroll
                        for (int c = 0; c < 8; ++c) {
                            const uint4 v = row_ok ? __ldg(src + hf * 8 + c) : make_uint4(0, 0, 0, 0);
                            qv[4 * c] = v.x; qv[4 * c + 1] = v.y; qv[4 * c + 2] = v.z; qv[4 * c + 3] = v.w;
                        }
                        tc_st32(tmem + lane_addr + Q_COL0 + hf * 32, qv);
                    }
                    tc_wait_st();
                    tc_fence_before();
                }
                mbar_arrive(smem_u32(&sh->q_full));
                float m_ref = -CUDART_INF_F, l_sum = 0.f;
                for (int ti = 0; ti < seg_tiles && ok; ++ti) {
                    const uint32_t gu = ug + ti;
                    const uint32_t s_addr = tmem + lane_addr + S_COL0 + (gu & 1) * TILE;
                    ok = bounded_wait(smem_u32(&sh->s_full[gu & 1]), (gu >> 1) & 1, abort_flag, p.device_status);
                    if (!ok) break;
                    if (!warp_active) {                         // all 32 rows are padding
                        mbar_arrive(smem_u32(&sh->p_full[gu & 1]));
                        continue;
                    }
                    tc_fence_after();
                    const int tok0 = (cur.t + ti) * TILE;
                    const bool need_mask = tok0 + TILE - 1 > L - R;    // some row cannot see the whole tile
                    // the accumulator may only be rescaled once the previous PV is complete
                    ok = softmax_tile<TILE, D / 32>(s_addr, o_addr, tok0, pos, need_mask, c_scale, ti == 0, m_ref, l_sum, [&]() {
                        return bounded_wait(smem_u32(&sh->o_done[(gu - 1) & 1]), ((gu - 1) >> 1) & 1, abort_flag,
                                            p.device_status);
                    });
                    if (!ok) break;
                    tc_wait_st();
                    tc_fence_before();
                    mbar_arrive(smem_u32(&sh->p_full[gu & 1]));
                }
                if (!ok) break;
                // ---- epilogue of the segment: wait for the last PV, then read O
                {
                    const uint32_t gl = ug + seg_tiles - 1;
                    if (warp_active)
                        ok = bounded_wait(smem_u32(&sh->o_done[gl & 1]), (gl >> 1) & 1, abort_flag, p.device_status);
                }
                if (!ok) break;
                tc_fence_after();
                const bool whole = (cur.t == 0 && seg_tiles == cur.n_tiles);
                if (!warp_active) {
                    // padding rows: nothing to write
                } else if (whole) {
                    const float inv = 1.f / l_sum;
                    __nv_bfloat16 *dst = static_cast<__nv_bfloat16 *>(p.o) + q_row * D;
#pragma unroll
                    for (int ch = 0; ch < D / 32; ++ch) {
                        uint32_t o[32];
                        tc_ld32(o_addr + ch * 32, o);
                        if (row_ok) {
#pragma unroll
                            for (int c = 0; c < 32; c += 8) {
                                uint4 w;
                                w.x = pack_bf16(__uint_as_float(o[c]) * inv, __uint_as_float(o[c + 1]) * inv);
                                w.y = pack_bf16(__uint_as_float(o[c + 2]) * inv, __uint_as_float(o[c + 3]) * inv);
                                w.z = pack_bf16(__uint_as_float(o[c + 4]) * inv, __uint_as_float(o[c + 5]) * inv);
                                w.w = pack_bf16(__uint_as_float(o[c + 6]) * inv, __uint_as_float(o[c + 7]) * inv);
                                *reinterpret_cast<uint4 *>(dst + ch * 32 + c) = w;
                            }
                        }
                    }
                    if (row_ok && p.lse != nullptr)
                        p.lse[q_row] = (m_ref + log2f(l_sum)) * 0.6931471805599453f;
                } else {
                    // partial: fp32 O row, then max and sum; slot 0 = the block's first segment
                    float *slot = a.ws_part + ((size_t)blockIdx.x * 2 + (seg_no == 0 ? 0 : 1)) * part_slot_floats(a.slot_rows);
                    float *orow = slot + (size_t)r * HD;          // 128-float pitch for both head sizes
#pragma unroll
                    for (int ch = 0; ch < D / 32; ++ch) {
                        uint32_t o[32];
                        tc_ld32(o_addr + ch * 32, o);
                        if (row_ok) {
#pragma unroll
                            for (int c = 0; c < 32; c += 4)
                                *reinterpret_cast<uint4 *>(orow + ch * 32 + c) = make_uint4(o[c], o[c + 1], o[c + 2], o[c + 3]);
                        }
                    }
                    if (row_ok) {
                        slot[(size_t)a.slot_rows * HD + r] = m_ref;
                        slot[(size_t)a.slot_rows * HD + a.slot_rows + r] = l_sum;
                    }
                }
                tc_fence_before();
                ug += seg_tiles;
                tg += seg_tiles;
                cur.t += seg_tiles;
                if (cur.t == cur.n_tiles) cur.next_pair(p);
            }
        }
    } else {
        if (TAIL) asm volatile("setmaxnreg.inc.sync.aligned.u32 200;");
        if (TAIL && t_end > t_begin) {
            // ================================================================ tail rows 128..143
            // Warp tw owns tokens [32 tw, 32 tw + 32) of every tile.  Fragment coordinates of
            // mma.sync m16n8k16: g8 = lane / 4, t4 = lane % 4.
            const int tw = warp - 8;
            const int g8 = lane >> 2, t4 = lane & 3;
            const int mi = lane >> 3, r8 = lane & 7;           // ldmatrix: matrix and row this lane addresses
            TileCursor cur;
            cur.seek(p, start_b, start_prefix, t_begin, TILE);
            uint32_t ug = 0, seg_no = 0, sync_no = 0;
            bool ok = true;
            for (long long tg = t_begin; tg < t_end && ok; ++seg_no) {
                const int b = cur.b, g = cur.g;
                const int seg_tiles = (int)min((long long)(cur.n_tiles - cur.t), t_end - tg);
                const int R = cur.gam + 1, L = p.seq_len[b];
                const int n_rows = G * R;
                const bool active = n_rows > 128;               // the pair has tail rows
                // Transposed products, so that the 8-wide N side of m16n8k16 carries the rows:
                //   S^T (tokens x rows) = K (tokens x dims) Q^T,   O^T (dims x rows) = V^T (dims x tokens) P^T.
                // This thread's rows in block nbk: 8 nbk + 2 t4 + e (accumulator columns) and
                // 8 nbk + g8 (B operand column).
                int pos[NBA][2];
                uint32_t qb[NBA][8][2];                           // B fragments of Q^T: [block][k-step][low / high 8 dims]
#pragma unroll
                for (int nbk = 0; nbk < NBA; ++nbk) {
#pragma unroll
                    for (int e = 0; e < 2; ++e) pos[nbk][e] = L - R + (128 + 8 * nbk + 2 * t4 + e) / G;
                    const int r = 128 + 8 * nbk + g8;
                    const int i = r / G, hh = r - i * G;
                    const bool row_ok = active && r < n_rows;
                    const uint32_t *src = reinterpret_cast<const uint32_t *>(
                        static_cast<const __nv_bfloat16 *>(p.q) +
                        (((long long)p.cu_q[b] + i) * p.hq + (long long)g * G + hh) * HD);
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        qb[nbk][ks][0] = row_ok ? __ldg(src + ks * 8 + t4) : 0u;
                        qb[nbk][ks][1] = row_ok ? __ldg(src + ks * 8 + 4 + t4) : 0u;
                    }
                }
                float m_ref[NBA][2], l_sum[NBA][2];
                float o[8][NBA][4];                               // O^T: [16-dim block][row block][fragment]
#pragma unroll
                for (int nbk = 0; nbk < NBA; ++nbk) {
                    m_ref[nbk][0] = m_ref[nbk][1] = -CUDART_INF_F;
                    l_sum[nbk][0] = l_sum[nbk][1] = 0.f;
#pragma unroll
                    for (int md = 0; md < 8; ++md) o[md][nbk][0] = o[md][nbk][1] = o[md][nbk][2] = o[md][nbk][3] = 0.f;
                }

                for (int ti = 0; ti < seg_tiles && ok; ++ti) {
                    const uint32_t gu = ug + ti;
                    const uint32_t item_k = 2 * gu, item_v = 2 * gu + 1;
                    const uint32_t slot_k = item_k % (uint32_t)n_slots, slot_v = item_v % (uint32_t)n_slots;
                    const int tok0 = (cur.t + ti) * TILE + tw * 32;       // first token of this warp's share
                    const bool work = active && tok0 < L;                  // otherwise nothing visible
                    ok = bounded_wait(smem_u32(&sh->full[slot_k]), (item_k / n_slots) & 1, abort_flag, p.device_status);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    uint32_t pb[2][NBA][2];                                  // B fragments of P^T: [k-step][block][token half]
                    if (work) {
                        // ---- S^T (32 tokens x rows) over 128 dims
                        // two accumulators per (token block, row block), even / odd k-steps: short chains
                        float sacc[2][NBA][4], sodd[2][NBA][4];
                        const uint32_t kbase = smem_u32(ring + slot_k * SLOT_BYTES);
#pragma unroll
                        for (int mb = 0; mb < 2; ++mb)
#pragma unroll
                            for (int nbk = 0; nbk < NBA; ++nbk)
#pragma unroll
                                for (int x = 0; x < 4; ++x) sacc[mb][nbk][x] = sodd[mb][nbk][x] = 0.f;
                        // The loads of four k-steps are issued together, then their MMAs: the asm
                        // statements keep program order, and a load followed at once by its MMA
                        // would cost a full shared-memory latency each time.
#pragma unroll
                        for (int kq = 0; kq < 2; ++kq) {
                            uint32_t ka[4][2][4];
#pragma unroll
                            for (int k4 = 0; k4 < 4; ++k4) {
                                const int c = 2 * (4 * kq + k4) + (mi >> 1);      // 16-byte chunk (8 dims) of the row
#pragma unroll
                                for (int mb = 0; mb < 2; ++mb) {
                                    const int token = tw * 32 + mb * 16 + (mi & 1) * 8 + r8;
                                    const uint32_t addr = kbase + (c >> 3) * (SLOT_BYTES / 2) + token * 128 +
                                                          (((c & 7) ^ (token & 7)) << 4);
                                    ldmatrix_x4(addr, ka[k4][mb][0], ka[k4][mb][1], ka[k4][mb][2], ka[k4][mb][3]);
                                }
                            }
#pragma unroll
                            for (int k4 = 0; k4 < 4; ++k4) {
                                const int ks = 4 * kq + k4;
#pragma unroll
                                for (int mb = 0; mb < 2; ++mb) {
                                    if (ks & 1) {
                                        mma_16816(sodd[mb][0], ka[k4][mb], qb[0][ks][0], qb[0][ks][1]);
                                        if (NB > 1) mma_16816(sodd[mb][NBA - 1], ka[k4][mb], qb[NBA - 1][ks][0], qb[NBA - 1][ks][1]);
                                    } else {
                                        mma_16816(sacc[mb][0], ka[k4][mb], qb[0][ks][0], qb[0][ks][1]);
                                        if (NB > 1) mma_16816(sacc[mb][NBA - 1], ka[k4][mb], qb[NBA - 1][ks][0], qb[NBA - 1][ks][1]);
                                    }
                                }
                            }
                        }
#pragma unroll
                        for (int mb = 0; mb < 2; ++mb)
#pragma unroll
                            for (int nbk = 0; nbk < NBA; ++nbk)
#pragma unroll
                                for (int x = 0; x < 4; ++x) sacc[mb][nbk][x] += sodd[mb][nbk][x];
                        __syncwarp();
                        if (lane == 0) mbar_arrive(smem_u32(&sh->empty[slot_k]));
                        // ---- online softmax; a row's 32 scores sit in the 8 lanes with the same t4
                        float f[NBA][2];
                        bool resc = false;
#pragma unroll
                        for (int nbk = 0; nbk < NBA; ++nbk)
#pragma unroll
                            for (int e = 0; e < 2; ++e) {
                                f[nbk][e] = 1.f;
                                float mt = -CUDART_INF_F;
#pragma unroll
                                for (int mb = 0; mb < 2; ++mb)
#pragma unroll
                                    for (int th = 0; th < 2; ++th) {
                                        float x = sacc[mb][nbk][2 * th + e] * c_scale;
                                        if (tok0 + mb * 16 + th * 8 + g8 > pos[nbk][e]) x = -CUDART_INF_F;
                                        sacc[mb][nbk][2 * th + e] = x;
                                        mt = fmaxf(mt, x);
                                    }
                                mt = fmaxf(mt, __shfl_xor_sync(0xffffffffu, mt, 4));
                                mt = fmaxf(mt, __shfl_xor_sync(0xffffffffu, mt, 8));
                                mt = fmaxf(mt, __shfl_xor_sync(0xffffffffu, mt, 16));
                                float &m = m_ref[nbk][e];
                                if ((mt > m + RESCALE_THRESHOLD || m == -CUDART_INF_F) && mt > -CUDART_INF_F) {
                                    if (m > -CUDART_INF_F) {
                                        f[nbk][e] = ex2_approx(m - mt);
                                        resc = true;
                                    }
                                    m = mt;
                                }
                            }
                        if (__any_sync(0xffffffffu, resc)) {
#pragma unroll
                            for (int nbk = 0; nbk < NBA; ++nbk) {
                                l_sum[nbk][0] *= f[nbk][0];
                                l_sum[nbk][1] *= f[nbk][1];
#pragma unroll
                                for (int md = 0; md < 8; ++md) {
                                    o[md][nbk][0] *= f[nbk][0]; o[md][nbk][1] *= f[nbk][1];
                                    o[md][nbk][2] *= f[nbk][0]; o[md][nbk][3] *= f[nbk][1];
                                }
                            }
                        }
#pragma unroll
                        for (int nbk = 0; nbk < NBA; ++nbk) {
                            const float mu0 = (m_ref[nbk][0] == -CUDART_INF_F) ? 0.f : m_ref[nbk][0];
                            const float mu1 = (m_ref[nbk][1] == -CUDART_INF_F) ? 0.f : m_ref[nbk][1];
#pragma unroll
                            for (int mb = 0; mb < 2; ++mb)
#pragma unroll
                                for (int th = 0; th < 2; ++th) {
                                    const float e0 = ex2_approx(sacc[mb][nbk][2 * th] - mu0);
                                    const float e1 = ex2_approx(sacc[mb][nbk][2 * th + 1] - mu1);
                                    l_sum[nbk][0] += e0;
                                    l_sum[nbk][1] += e1;
                                    // (token g8, rows 2 t4, 2 t4 + 1) -> (row g8, tokens 2 t4, 2 t4 + 1)
                                    pb[mb][nbk][th] = movmatrix_trans(pack_bf16(e0, e1));
                                }
                        }
                    } else {
                        __syncwarp();
                        if (lane == 0) mbar_arrive(smem_u32(&sh->empty[slot_k]));
                    }
                    ok = bounded_wait(smem_u32(&sh->full[slot_v]), (item_v / n_slots) & 1, abort_flag, p.device_status);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    if (work) {
                        // ---- O^T (128 dims x rows) += V^T (dims x 32 tokens) P^T
                        const uint32_t vbase = smem_u32(ring + slot_v * SLOT_BYTES);
#pragma unroll
                        for (int j = 0; j < 2; ++j) {
                            const int token = tw * 32 + 16 * j + (mi >> 1) * 8 + r8;
                            uint32_t va[8][4];                             // all eight loads first, then the MMAs
#pragma unroll
                            for (int md = 0; md < 8; ++md) {
                                const int c = 2 * md + (mi & 1);
                                const uint32_t addr = vbase + (c >> 3) * (SLOT_BYTES / 2) + token * 128 +
                                                      (((c & 7) ^ (token & 7)) << 4);
                                ldmatrix_x4_trans(addr, va[md][0], va[md][1], va[md][2], va[md][3]);
                            }
#pragma unroll
                            for (int md = 0; md < 8; ++md) {
                                mma_16816(o[md][0], va[md], pb[j][0][0], pb[j][0][1]);
                                if (NB > 1) mma_16816(o[md][NBA - 1], va[md], pb[j][NBA - 1][0], pb[j][NBA - 1][1]);
                            }
                        }
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&sh->empty[slot_v]));
                }
                if (!ok) break;
                // ---- merge the four warps' partial states through shared memory
                if (active) {
#pragma unroll
                    for (int nbk = 0; nbk < NBA; ++nbk)
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            float l = l_sum[nbk][e];
                            l += __shfl_xor_sync(0xffffffffu, l, 4);
                            l += __shfl_xor_sync(0xffffffffu, l, 8);
                            l += __shfl_xor_sync(0xffffffffu, l, 16);
                            const int row = 8 * nbk + 2 * t4 + e;
#pragma unroll
                            for (int md = 0; md < 8; ++md) {
                                tm->o[tw][row][16 * md + g8] = o[md][nbk][e];
                                tm->o[tw][row][16 * md + g8 + 8] = o[md][nbk][2 + e];
                            }
                            if (g8 == 0) {
                                tm->m[tw][row] = m_ref[nbk][e];
                                tm->l[tw][row] = l;
                            }
                        }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&sh->tail_sync));
                    ok = bounded_wait(smem_u32(&sh->tail_sync), sync_no & 1, abort_flag, p.device_status);
                    ++sync_no;
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    // thread j of the 128: row j / 8, dims 16 (j % 8) .. + 16
                    const int j = tid - 256;
                    const int row = j >> 3, d0 = (j & 7) * 16;
                    const int r = 128 + row;
                    if (r < n_rows) {
                        float M = -CUDART_INF_F;
#pragma unroll
                        for (int w = 0; w < 4; ++w) M = fmaxf(M, tm->m[w][row]);
                        float acc[16];
#pragma unroll
                        for (int c = 0; c < 16; ++c) acc[c] = 0.f;
                        float lsum = 0.f;
#pragma unroll
                        for (int w = 0; w < 4; ++w) {
                            const float mw = tm->m[w][row];
                            if (mw == -CUDART_INF_F) continue;
                            const float sc = exp2f(mw - M);
                            lsum += sc * tm->l[w][row];
#pragma unroll
                            for (int c = 0; c < 16; c += 4) {
                                const float4 v = *reinterpret_cast<const float4 *>(&tm->o[w][row][d0 + c]);
                                acc[c] += sc * v.x; acc[c + 1] += sc * v.y; acc[c + 2] += sc * v.z; acc[c + 3] += sc * v.w;
                            }
                        }
                        const int i = r / G, hh = r - i * G;
                        const long long qr = ((long long)p.cu_q[b] + i) * p.hq + (long long)g * G + hh;
                        const bool whole = (cur.t == 0 && seg_tiles == cur.n_tiles);
                        if (whole) {
                            const float inv = 1.f / lsum;
                            __nv_bfloat16 *dst = static_cast<__nv_bfloat16 *>(p.o) + qr * HD + d0;
#pragma unroll
                            for (int c = 0; c < 16; c += 8) {
                                uint4 w4;
                                w4.x = pack_bf16(acc[c] * inv, acc[c + 1] * inv);
                                w4.y = pack_bf16(acc[c + 2] * inv, acc[c + 3] * inv);
                                w4.z = pack_bf16(acc[c + 4] * inv, acc[c + 5] * inv);
                                w4.w = pack_bf16(acc[c + 6] * inv, acc[c + 7] * inv);
                                *reinterpret_cast<uint4 *>(dst + c) = w4;
                            }
                            if ((j & 7) == 0 && p.lse != nullptr) p.lse[qr] = (M + log2f(lsum)) * 0.6931471805599453f;
                        } else {
                            float *slot = a.ws_part + ((size_t)blockIdx.x * 2 + (seg_no == 0 ? 0 : 1)) * part_slot_floats(a.slot_rows);
                            float *orow = slot + (size_t)r * HD + d0;
#pragma unroll
                            for (int c = 0; c < 16; c += 4)
                                *reinterpret_cast<float4 *>(orow + c) = make_float4(acc[c], acc[c + 1], acc[c + 2], acc[c + 3]);
                            if ((j & 7) == 0) {
                                slot[(size_t)a.slot_rows * HD + r] = M;
                                slot[(size_t)a.slot_rows * HD + a.slot_rows + r] = lsum;
                            }
                        }
                    }
                    // the buffers are rewritten at the next segment's end: everyone must be done reading
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&sh->tail_sync));
                    ok = bounded_wait(smem_u32(&sh->tail_sync), sync_no & 1, abort_flag, p.device_status);
                    ++sync_no;
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                }
                ug += seg_tiles;
                tg += seg_tiles;
                cur.t += seg_tiles;
                if (cur.t == cur.n_tiles) cur.next_pair(p);
            }
        }
    }
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
    }
}

// ---------------------------------------------------------------------------- host side
bool attn_tq_supported(const sv_attn_params &p)
{
    if ((p.head_dim != 128 && p.head_dim != 64) || p.pool == nullptr || !p.pool->has_maps) return false;
    if (p.batch > MAX_BATCH_TC) return false;
    const int rows = (p.hq / p.hkv) * (p.gamma_max + 1);
    return rows >= 1 && rows <= (p.head_dim == 128 ? 128 + TAIL_ROWS : 128);
}

int attn_tq_slot_rows(int rows) { return rows > 128 ? 128 + TAIL_ROWS : 128; }
static int g_tail_blocks(int rows) { return rows <= 128 ? 0 : (rows - 128 + 7) / 8; }

template <int NB, int D>
static sv_status launch_tq(AttnTcLaunch &a, const sv_attn_params &p, int grid, cudaStream_t stream)
{
    constexpr bool TAIL = NB > 0;
    constexpr int slot_bytes = TILE * D * 2;
    const size_t budget = 227 * 1024;
    const size_t fixed = (TAIL ? sizeof(TailMerge) : 0) + ((sizeof(Shared) + 127) & ~(size_t)127);
    a.n_slots = (int)((budget - fixed) / slot_bytes);
    if (a.n_slots > 8) a.n_slots = 8;
    if (a.n_slots < 4) return SV_EUNSUPPORTED;
    const size_t smem = fixed + (size_t)a.n_slots * slot_bytes;
    if (cudaFuncSetAttribute(attn_tq_kernel<NB, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
        cudaSuccess)
        return SV_ECUDA;
    return launch_kernel(false, attn_tq_kernel<NB, D>, grid, TAIL ? 384 : 256, smem, stream, a, p.pool->k_map, p.pool->v_map);
}

sv_status launch_attn_tq_main(AttnTcLaunch &a, const sv_attn_params &p, int grid, cudaStream_t stream)
{
    if (p.head_dim == 64) return launch_tq<0, 64>(a, p, grid, stream);
    switch (g_tail_blocks(a.group * (p.gamma_max + 1))) {
        case 0: return launch_tq<0, 128>(a, p, grid, stream);
        case 1: return launch_tq<1, 128>(a, p, grid, stream);
        default: return launch_tq<2, 128>(a, p, grid, stream);
    }
}

}  // namespace sv
