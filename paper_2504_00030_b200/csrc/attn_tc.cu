// Draft-block attention on the 5th-generation tensor cores (tcgen05, sm_100a).
//
// Work unit.  A (sequence b, kv head g) pair owns G*(gamma_b+1) query rows (G = hq/hkv query
// heads per kv head, stacked so that the group shares one pass over the keys) and a stream of
// ceil(L_b/128) key tiles of 128 tokens = 8 pages.  The key tiles of the whole batch form one
// global list; each of the grid's persistent thread blocks takes a contiguous share of it
// (lengths live on the device, so the split is computed in the kernel, see attn_sched.cuh),
// which balances ragged contexts.  A block's share is cut into segments, one per (b, g) it touches; a segment
// that covers its pair completely writes the final output, otherwise it leaves an unnormalised
// partial (fp32 O, running max, running sum) in the workspace for attn_combine_kernel.
//
// Data path per tile: the 8 K pages and 8 V pages are fetched by TMA (one 4-D tensor map over
// the pool, box = 64 dims x 16 slots of one head of one page, 128-byte swizzle) into a ring of
// 32 KB shared-memory slots, straight into the layout tcgen05 wants.  S = Q K^T is issued as
// 8 MMAs (M=128 rows, N=128 tokens, K=16) with both operands in shared memory and the
// accumulator in tensor memory; 128 softmax threads (one per query row, the row's scores in
// their own TMEM lane, so max and sum need no shuffles) turn S into bf16 P in place; O += P V
// is 8 MMAs with P read from tensor memory and V (token-major in memory) as the N-major B
// operand.  Rows beyond 128 (e.g. 8 heads x 17 positions = 136) go to a second row group with
// its own S / O accumulators and softmax warps; the two groups alternate on the tensor core.
//
// Warps: 0 = TMA producer, 1 = MMA issuer and TMEM owner, 4..7 = softmax / epilogue of row
// group 0, 8..11 = row group 1 (when needed).  All hand-offs are mbarriers; every wait is
// bounded and an expired wait sets SV_DEV_TIMEOUT and drains the block.
#include "attn_sched.cuh"
#include "attn_softmax.cuh"
#include "tc_ptx.cuh"

#include <math_constants.h>

namespace sv {

// This file's kernel serves pairs with 145..256 query rows (two row groups of 128, key tiles of 128
// tokens, one block per SM); pairs with up to 144 rows go to attn_tq.cu.  Row groups and tile size
// are template parameters.
constexpr int QGROUP_BYTES = 128 * HD * 2;         // 32 KB: 128 query rows



struct Shared {
    uint64_t full[8];        // ring slot filled by TMA
    uint64_t empty[8];       // ring slot released by the tensor core
    uint64_t s_full[2];      // S accumulator ready
    uint64_t p_full[2];      // P written by the softmax threads
    uint64_t o_done[2];      // PV of unit u finished (indexed by u & 1, like s_full / p_full)
    uint64_t q_full;         // query rows of a segment are in shared memory
    uint32_t tmem_base;
    int abort_flag;
    int total_tiles;         // sum over sequences of ceil(L/128)
    int start_b;             // sequence that holds this block's first tile
    int start_prefix;        // tiles (per kv head) of the sequences before it
    long long t_begin, t_end; // this block's tiles of the global list
};



// ---------------------------------------------------------------------------- main kernel
template <int NQ, int TILE>
__global__ void __launch_bounds__(128 + 128 * NQ, 1)
attn_tc_kernel(const AttnTcLaunch a, const __grid_constant__ CUtensorMap k_map,
               const __grid_constant__ CUtensorMap v_map)
{
    constexpr int PAGES_PER_TILE = TILE / 16;
    constexpr int SLOT_BYTES = TILE * HD * 2;          // one K or one V tile
    constexpr int O_COL0 = 2 * TILE;                   // TMEM: two S buffers of TILE columns, then O
    constexpr uint32_t TMEM_COLS = (2 * TILE + 128 * NQ <= 256) ? 256u : 512u;
    pdl_enter();
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    // carve: [Q groups][ring slots][Shared]; the swizzled tiles need a 1024-byte aligned base
    uint8_t *smem = smem_raw;
    if ((smem_u32(smem) & 1023u) != 0) {               // never seen; refuse rather than compute garbage
        if (threadIdx.x == 0) set_status(a.p.device_status, SV_DEV_TIMEOUT);
        return;
    }
    uint8_t *q_smem = smem;
    uint8_t *ring = smem + NQ * QGROUP_BYTES;
    Shared *sh = reinterpret_cast<Shared *>(ring + a.n_slots * SLOT_BYTES);

    const sv_attn_params &p = a.p;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int batch = p.batch, hkv = p.hkv, G = a.group;
    const int n_slots = a.n_slots;

    // ---- tile prefix over the batch (every block computes the same thing)
    if (tid == 0) {
        for (int i = 0; i < n_slots; ++i) {
            mbar_init(smem_u32(&sh->full[i]), 1);
            mbar_init(smem_u32(&sh->empty[i]), 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&sh->s_full[i]), 1);
            mbar_init(smem_u32(&sh->p_full[i]), 128);
            mbar_init(smem_u32(&sh->o_done[i]), 1);
        }
        mbar_init(smem_u32(&sh->q_full), 128 * NQ);
        sh->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (warp == 0) {
        BlockShare bs;
        plan_block_share(a, lane, TILE, 0, bs);
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

    // With two row groups there are 384 threads and 168 registers each; the producer / MMA
    // warpgroup hands part of its share to the softmax warpgroups (128*80 + 256*208 <= 384*168).
    if (warp < 4) {
        if (NQ == 2) asm volatile("setmaxnreg.dec.sync.aligned.u32 80;");
        if (t_end > t_begin && warp == 0) {
            // ================================================================ TMA producer
            TileCursor cur;
            cur.seek(p, sh->start_b, sh->start_prefix, t_begin, TILE);
            uint32_t item = 0;     // ring items: 2*tile = K, 2*tile+1 = V
            for (long long tg = t_begin; tg < t_end; ++tg) {
                const int b = cur.b;
                const int L = p.seq_len[b];
                const int n_pages = (L + 15) >> 4;
                const int32_t *bt = p.block_table + (long long)b * p.block_table_stride;
                // lane l fetches (page l/2, dims half l%2) of K, then of V
                const int page_in_tile = (lane >> 1) % PAGES_PER_TILE, half = lane & 1;
                const int lp = cur.t * PAGES_PER_TILE + page_in_tile;
                int phys = (int)a.n_pool_pages;       // out of range: TMA fills zeros, no traffic
                if (lp < n_pages) {
                    const int e = bt[lp];
                    if (e < 0 || e >= a.n_pool_pages) set_status(p.device_status, SV_DEV_BAD_PAGE);
                    else phys = e;
                }
                bool ok = true;
#pragma unroll
                for (int kv = 0; kv < 2; ++kv) {
                    const uint32_t slot = item % (uint32_t)n_slots;
                    const uint32_t use = item / (uint32_t)n_slots;
                    const uint32_t full = smem_u32(&sh->full[slot]);
                    if (use > 0) ok = ok && bounded_wait(smem_u32(&sh->empty[slot]), (use - 1) & 1, &sh->abort_flag, p.device_status);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    if (lane == 0) mbar_expect_tx(full, SLOT_BYTES);
                    __syncwarp();
                    if (lane < 2 * PAGES_PER_TILE) {
                        const uint32_t dst = smem_u32(ring + slot * SLOT_BYTES + half * (SLOT_BYTES / 2) +
                                                      page_in_tile * 2048);
                        tma_load_4d(dst, kv == 0 ? &k_map : &v_map, half * 64, 0, cur.g, phys, full);
                    }
                    ++item;
                }
                if (!ok) break;
                if (++cur.t == cur.n_tiles) cur.next_pair(p);
            }
        } else if (t_end > t_begin && warp == 1) {
            // ================================================================ MMA issuer
            // the whole warp walks the schedule and waits; one elected lane issues
            {
                const uint32_t idesc_qk = instr_desc(false, TILE), idesc_pv = instr_desc(true, HD);
                const uint64_t q_desc0 = smem_desc(smem_u32(q_smem), 16, 1024);
                const uint64_t q_desc1 = smem_desc(smem_u32(q_smem + (NQ - 1) * QGROUP_BYTES), 16, 1024);
                TileCursor cur;
                cur.seek(p, sh->start_b, sh->start_prefix, t_begin, TILE);
                uint32_t tile_no = 0;      // tiles of this block so far (ring position)
                uint32_t ug = 0;           // global unit counter: unit = (tile, row group)
                uint32_t seg_no = 0;
                bool ok = true;
                for (long long tg = t_begin; tg < t_end && ok;) {
                    const int seg_tiles = (int)min((long long)(cur.n_tiles - cur.t), t_end - tg);
                    // row groups this pair really has (a second group only if it has > 128 rows)
                    const int nq_seg = (NQ == 2 && G * (cur.gam + 1) > 128) ? 2 : 1;
                    const int n_units = seg_tiles * nq_seg;
                    ok = bounded_wait(smem_u32(&sh->q_full), seg_no & 1, &sh->abort_flag, p.device_status);
                    tc_fence_after();
                    auto issue_qk = [&](int u) {       // unit u of this segment
                        const int q = u % nq_seg, ti = u / nq_seg;
                        const uint32_t item = 2 * (tile_no + ti);
                        const uint32_t slot = item % (uint32_t)n_slots;
                        if (q == 0) {
                            ok = ok && bounded_wait(smem_u32(&sh->full[slot]), (item / n_slots) & 1, &sh->abort_flag,
                                                    p.device_status);
                            tc_fence_after();
                        }
                        if (!ok) return;
                        // descriptors are built once; stepping along K only adds to the address field
                        const uint64_t kd = smem_desc(smem_u32(ring + slot * SLOT_BYTES), 16, 1024);
                        const uint64_t qd = q == 0 ? q_desc0 : q_desc1;
                        const uint32_t d = tmem + ((ug + u) & 1) * TILE;
                        if (elect_one()) {
#pragma unroll
                        for (int ks = 0; ks < 8; ++ks) {
                            const uint32_t koff = ((ks >> 2) * (SLOT_BYTES / 2) + (ks & 3) * 32) >> 4;
                            const uint32_t qoff = ((ks >> 2) * (QGROUP_BYTES / 2) + (ks & 3) * 32) >> 4;
                            tc_mma_ss(d, qd + qoff, kd + koff, idesc_qk, ks > 0);
                        }
                        tc_commit(smem_u32(&sh->s_full[(ug + u) & 1]));
                        if (q == nq_seg - 1) tc_commit(smem_u32(&sh->empty[slot]));   // K tile consumed
                        }
                        __syncwarp();
                    };
                    issue_qk(0);
                    if (n_units > 1) issue_qk(1);
                    for (int u = 0; u < n_units && ok; ++u) {
                        const int q = u % nq_seg, ti = u / nq_seg;
                        const uint32_t gu = ug + u;
                        ok = bounded_wait(smem_u32(&sh->p_full[gu & 1]), (gu >> 1) & 1, &sh->abort_flag, p.device_status);
                        const uint32_t item = 2 * (tile_no + ti) + 1;
                        const uint32_t slot = item % (uint32_t)n_slots;
                        if (ok && q == 0)
                            ok = bounded_wait(smem_u32(&sh->full[slot]), (item / n_slots) & 1, &sh->abort_flag,
                                              p.device_status);
                        if (!ok) break;
                        tc_fence_after();
                        const uint64_t vd = smem_desc(smem_u32(ring + slot * SLOT_BYTES), SLOT_BYTES / 2, 1024);
                        const uint32_t pa = tmem + (gu & 1) * TILE;      // P overlays S, TILE/2 columns
                        const uint32_t d = tmem + O_COL0 + q * 128;
                        if (elect_one()) {
#pragma unroll
                        for (int ks = 0; ks < TILE / 16; ++ks)
                            tc_mma_ts(d, pa + ks * 8, vd + (uint64_t)(ks * (2048 >> 4)), idesc_pv,
                                      (ti > 0 || ks > 0) ? 1u : 0u);
                        tc_commit(smem_u32(&sh->o_done[gu & 1]));
                        if (q == nq_seg - 1) tc_commit(smem_u32(&sh->empty[slot]));   // V tile consumed
                        }
                        __syncwarp();
                        if (u + 2 < n_units) issue_qk(u + 2);
                    }
                    ug += n_units;
                    tile_no += seg_tiles;
                    ++seg_no;
                    tg += seg_tiles;
                    cur.t += seg_tiles;
                    if (cur.t == cur.n_tiles) cur.next_pair(p);
                }
            }
        }
    } else {
        if (NQ == 2) asm volatile("setmaxnreg.inc.sync.aligned.u32 208;");
        if (t_end > t_begin) {
            // ================================================================ softmax / epilogue
            const int q = (warp - 4) >> 2;                     // row group of this warp
            const int quarter = warp & 3;
            const int r_in = quarter * 32 + lane;              // TMEM lane = row inside the group
            const int r = q * 128 + r_in;                      // row of the (b, g) pair
            const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
            TileCursor cur;
            cur.seek(p, sh->start_b, sh->start_prefix, t_begin, TILE);
            uint32_t ug = 0;               // global unit counter
            uint32_t seg_no = 0;
            bool ok = true;
            for (long long tg = t_begin; tg < t_end && ok; ++seg_no) {
                const int b = cur.b, g = cur.g;
                const int seg_tiles = (int)min((long long)(cur.n_tiles - cur.t), t_end - tg);
                const int gam = cur.gam;
                const int R = gam + 1, L = p.seq_len[b];
                const int n_rows = G * R;
                const int nq_seg = (NQ == 2 && n_rows > 128) ? 2 : 1;
                const bool grp_active = q < nq_seg;                       // this row group exists for the pair
                const bool warp_active = grp_active && (q * 128 + quarter * 32 < n_rows);
                const bool row_ok = r < n_rows;
                const int i = r / G, hh = r - i * G;
                const int pos = L - R + i;                     // last visible key of this row
                const long long q_row = ((long long)p.cu_q[b] + i) * p.hq + (long long)g * G + hh;
                // ---- this thread's query row -> shared memory (K-major, 128-byte swizzle)
                if (grp_active) {
                    const uint4 *src = reinterpret_cast<const uint4 *>(
                        static_cast<const __nv_bfloat16 *>(p.q) + q_row * HD);
                    uint8_t *dst = q_smem + q * QGROUP_BYTES + r_in * 128;
#pragma unroll
                    for (int c = 0; c < 16; ++c) {
                        const uint4 v = row_ok ? __ldg(src + c) : make_uint4(0, 0, 0, 0);
                        const int half = c >> 3, chunk = (c & 7) ^ (r_in & 7);
                        *reinterpret_cast<uint4 *>(dst + half * (QGROUP_BYTES / 2) + chunk * 16) = v;
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                }
                mbar_arrive(smem_u32(&sh->q_full));
                if (!grp_active) {                              // nothing to do for this pair
                    // Stay in step with the barriers this group will use again later: a parity
                    // wait is only meaningful for a waiter that is at most one phase ahead, so the
                    // idle group follows every phase of q_full and of both s_full barriers.
                    ok = bounded_wait(smem_u32(&sh->q_full), seg_no & 1, &sh->abort_flag, p.device_status);
                    for (int ti = 0; ti < seg_tiles && ok; ++ti) {
                        const uint32_t gu = ug + ti;            // nq_seg == 1 here
                        ok = bounded_wait(smem_u32(&sh->s_full[gu & 1]), (gu >> 1) & 1, &sh->abort_flag, p.device_status);
                    }
                    ug += seg_tiles * nq_seg;
                    tg += seg_tiles;
                    cur.t += seg_tiles;
                    if (cur.t == cur.n_tiles) cur.next_pair(p);
                    continue;
                }
                float m_ref = -CUDART_INF_F, l_sum = 0.f;
                const uint32_t o_addr = tmem + lane_addr + O_COL0 + q * 128;
                for (int ti = 0; ti < seg_tiles && ok; ++ti) {
                    const uint32_t gu = ug + ti * nq_seg + q;
                    const uint32_t s_addr = tmem + lane_addr + (gu & 1) * TILE;
                    ok = bounded_wait(smem_u32(&sh->s_full[gu & 1]), (gu >> 1) & 1, &sh->abort_flag, p.device_status);
                    if (!ok) break;
                    if (!warp_active) {                         // all 32 rows are padding
                        mbar_arrive(smem_u32(&sh->p_full[gu & 1]));
                        continue;
                    }
                    tc_fence_after();
                    const int tok0 = (cur.t + ti) * TILE;
                    const bool need_mask = tok0 + TILE - 1 > L - R;    // some row cannot see the whole tile
                    // The accumulator may only be rescaled once the previous PV of this row group is complete.
                    // The tensor core runs in issue order (PV(u), then QK(u+2)), so having seen S(gu) means
                    // PV(gu-2) is done: with two row groups that IS the previous PV of this group; with one
                    // group it is PV(gu-1), whose barrier is then at most one phase behind.
                    ok = softmax_tile<TILE, 4>(s_addr, o_addr, tok0, pos, need_mask, c_scale, ti == 0, m_ref, l_sum, [&]() {
                        return nq_seg != 1 || bounded_wait(smem_u32(&sh->o_done[(gu - 1) & 1]), ((gu - 1) >> 1) & 1,
                                                           &sh->abort_flag, p.device_status);
                    });
                    if (!ok) break;
                    tc_wait_st();
                    tc_fence_before();
                    mbar_arrive(smem_u32(&sh->p_full[gu & 1]));
                }
                if (!ok) break;
                // ---- epilogue of the segment: wait for the last PV, then read O
                {
                    const uint32_t gl = ug + (seg_tiles - 1) * nq_seg + q;     // this group's last unit
                    if (warp_active)
                        ok = bounded_wait(smem_u32(&sh->o_done[gl & 1]), (gl >> 1) & 1, &sh->abort_flag, p.device_status);
                }
                if (!ok) break;
                tc_fence_after();
                const bool whole = (cur.t == 0 && seg_tiles == cur.n_tiles);
                if (!warp_active) {
                    // padding rows: nothing to write
                } else if (whole) {
                    const float inv = 1.f / l_sum;
                    __nv_bfloat16 *dst = static_cast<__nv_bfloat16 *>(p.o) + q_row * HD;
#pragma unroll
                    for (int ch = 0; ch < 4; ++ch) {
                        uint32_t o[32];
                        tc_ld32(o_addr + ch * 32, o);
                        if (row_ok) {
#pragma unroll
                            for (int c = 0; c < 32; c += 8) {
                                uint4 w;
                                uint32_t *wp = reinterpret_cast<uint32_t *>(&w);
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const __nv_bfloat162 h = __floats2bfloat162_rn(
                                        __uint_as_float(o[c + 2 * e]) * inv, __uint_as_float(o[c + 2 * e + 1]) * inv);
                                    wp[e] = *reinterpret_cast<const uint32_t *>(&h);
                                }
                                *reinterpret_cast<uint4 *>(dst + ch * 32 + c) = w;
                            }
                        }
                    }
                    if (row_ok && p.lse != nullptr)
                        p.lse[q_row] = (m_ref + log2f(l_sum)) * 0.6931471805599453f;
                } else {
                    // partial: fp32 O row, then max and sum; slot 0 = the block's first segment
                    float *slot = a.ws_part + ((size_t)blockIdx.x * 2 + (seg_no == 0 ? 0 : 1)) * part_slot_floats(NQ * 128);
                    float *orow = slot + (size_t)r * HD;
#pragma unroll
                    for (int ch = 0; ch < 4; ++ch) {
                        uint32_t o[32];
                        tc_ld32(o_addr + ch * 32, o);
                        if (row_ok) {
#pragma unroll
                            for (int c = 0; c < 32; c += 4)
                                *reinterpret_cast<uint4 *>(orow + ch * 32 + c) = make_uint4(o[c], o[c + 1], o[c + 2], o[c + 3]);
                        }
                    }
                    if (row_ok) {
                        slot[(size_t)NQ * 128 * HD + r] = m_ref;
                        slot[(size_t)NQ * 128 * HD + NQ * 128 + r] = l_sum;
                    }
                }
                tc_fence_before();
                ug += seg_tiles * nq_seg;
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

// ---------------------------------------------------------------------------- combine kernel
// Merges the partials of pairs whose tiles were shared by several blocks of the main kernel.
// Warp = query row; a row's partials (running max, sum, fp32 O) are all requested before the
// first is used, so a row costs one memory round trip.
constexpr int COMBINE_THREADS = 1024;
constexpr int COMBINE_LIST = 64;      // partial slots merged per pass

__global__ void __launch_bounds__(COMBINE_THREADS)
attn_combine_kernel(const AttnTcLaunch a)
{
    pdl_enter();
    const sv_attn_params &p = a.p;
    __shared__ int s_list[COMBINE_LIST];
    __shared__ int s_n;
    __shared__ long long s_next;
    // One block per block of the main kernel: block c looks at the tile where main block c's
    // share began.  If that tile lies strictly inside a (sequence, kv head) pair, the pair was
    // split there; the block whose bound is the FIRST one inside the pair merges it.
    const int c = blockIdx.x;
    const int slot_rows = a.slot_rows;
    const long long grid = a.ws_prefix[p.batch + 1];
    const long long total = (long long)a.ws_prefix[p.batch] * p.hkv;
    if (c == 0 || c >= grid || total == 0) return;
    // the table of lower bounds is copied to shared memory in one round trip and searched there
    __shared__ int s_bounds[MAX_ATTN_GRID + 1];
    __shared__ int s_b, s_last;
    for (int k = threadIdx.x; k <= grid; k += blockDim.x) s_bounds[k] = a.ws_prefix[p.batch + 2 + k];
    if (threadIdx.x == 0) s_b = -1;
    __syncthreads();
    const long long t = s_bounds[c];
    if (t >= total) return;
    for (int k = threadIdx.x; k < p.batch; k += blockDim.x) {      // the sequence that holds tile t
        const long long lo = (long long)a.ws_prefix[k] * p.hkv, hi = (long long)a.ws_prefix[k + 1] * p.hkv;
        if (lo <= t && t < hi) s_b = k;
    }
    __syncthreads();
    const int b = s_b;
    if (b < 0) return;
    const int n_tiles = a.ws_prefix[b + 1] - a.ws_prefix[b];
    const int g = (int)((t - (long long)a.ws_prefix[b] * p.hkv) / n_tiles);
    const long long T0 = (long long)a.ws_prefix[b] * p.hkv + (long long)g * n_tiles, T1 = T0 + n_tiles;
    if (t == T0 || s_bounds[c - 1] > T0) return;          // not split here, or an earlier bound is inside too
    // shares that hold the pair's first and last tile: c - 1 (the last whose bound is not beyond
    // T0; empty shares repeat their successor's bound and are skipped that way) and the owner of T1 - 1
    if (threadIdx.x == 0) {
        int lo = c, hi = (int)grid;
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (s_bounds[mid] <= T1 - 1) lo = mid; else hi = mid;
        }
        s_last = lo;
    }
    __syncthreads();
    const int *bounds = s_bounds;
    const long long c_first = c - 1, c_last = s_last;
    int gam = p.gamma[b];
    gam = min(max(gam, 0), p.gamma_max);
    const int G = a.group, n_rows = G * (gam + 1);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    const int D = p.head_dim;                              // 128, or 64 (rows keep their 128-float pitch in the slots)
    const bool lane_on = 4 * lane < D;
    const size_t m_off = (size_t)slot_rows * HD, l_off = m_off + (size_t)slot_rows;
    const size_t slot_floats = part_slot_floats(slot_rows);

    // A pair split over more blocks than the list holds is merged in passes: each pass leaves
    // its result in the pass's first slot (only this block touches the pair's slots) and the
    // next pass starts from there.
    int carry = -1;
    for (long long c0 = c_first; c0 <= c_last;) {
        __syncthreads();
        if (threadIdx.x == 0) {
            int n = 0;
            if (carry >= 0) s_list[n++] = carry;
            long long c = c0;
            for (; c <= c_last && n < COMBINE_LIST; ++c) {
                const long long lo = bounds[c];
                if (bounds[c + 1] == lo) continue;
                s_list[n++] = (int)(c * 2 + (lo >= T0 ? 0 : 1));
            }
            s_n = n;
            s_next = c;
        }
        __syncthreads();
        const int n = s_n;
        c0 = s_next;
        const bool last = c0 > c_last;
        carry = s_list[0];
        for (int r = warp; r < n_rows; r += n_warps) {
            float m_run = -CUDART_INF_F, l_run = 0.f;
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int j0 = 0; j0 < n; j0 += 4) {
                float mc[4], lc[4];
                float4 v[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const bool have = j0 + u < n;
                    const float *slot = a.ws_part + (size_t)s_list[have ? j0 + u : 0] * slot_floats;
                    mc[u] = have ? slot[m_off + r] : -CUDART_INF_F;
                    lc[u] = have ? slot[l_off + r] : 0.f;
                    v[u] = (have && lane_on) ? reinterpret_cast<const float4 *>(slot + (size_t)r * HD)[lane]
                                             : make_float4(0.f, 0.f, 0.f, 0.f);
                }
                float m_new = m_run;
#pragma unroll
                for (int u = 0; u < 4; ++u) m_new = fmaxf(m_new, mc[u]);
                if (m_new == -CUDART_INF_F) continue;
                const float w_old = exp2f(m_run - m_new);          // 0 while nothing has been merged
                acc.x *= w_old; acc.y *= w_old; acc.z *= w_old; acc.w *= w_old;
                l_run *= w_old;
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    if (mc[u] == -CUDART_INF_F) continue;
                    const float w = exp2f(mc[u] - m_new);
                    l_run += w * lc[u];
                    acc.x += w * v[u].x; acc.y += w * v[u].y; acc.z += w * v[u].z; acc.w += w * v[u].w;
                }
                m_run = m_new;
            }
            if (!last) {
                float *slot = a.ws_part + (size_t)carry * slot_floats;
                if (lane_on) reinterpret_cast<float4 *>(slot + (size_t)r * HD)[lane] = acc;
                if (lane == 0) { slot[m_off + r] = m_run; slot[l_off + r] = l_run; }
                continue;
            }
            const int i = r / G, hh = r - i * G;
            const long long q_row = ((long long)p.cu_q[b] + i) * p.hq + (long long)g * G + hh;
            const float inv = 1.f / l_run;
            const __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x * inv, acc.y * inv);
            const __nv_bfloat162 hi = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
            uint2 packed;
            packed.x = *reinterpret_cast<const uint32_t *>(&lo);
            packed.y = *reinterpret_cast<const uint32_t *>(&hi);
            if (lane_on) reinterpret_cast<uint2 *>(static_cast<__nv_bfloat16 *>(p.o) + q_row * D)[lane] = packed;
            if (lane == 0 && p.lse != nullptr) p.lse[q_row] = (m_run + log2f(l_run)) * 0.6931471805599453f;
        }
    }
}

// ---------------------------------------------------------------------------- host side
static int rows_groups(const sv_attn_params &p)
{
    const int rows = (p.hq / p.hkv) * (p.gamma_max + 1);
    return (rows + 127) / 128;
}

bool attn_tc_supported(const sv_attn_params &p)
{
    if (p.pool == nullptr || !p.pool->has_maps || p.batch > MAX_BATCH_TC) return false;
    if (attn_tq_supported(p)) return true;               // 128 or 64 dims, one row group (+ tail rows)
    const int nq = rows_groups(p);
    return p.head_dim == HD && nq >= 1 && nq <= 2;       // two row groups: 128 dims only
}

static size_t prefix_bytes(int batch)
{
    return (((size_t)batch + 2 + MAX_ATTN_GRID + 1) * sizeof(int32_t) + 255) & ~(size_t)255;
}

// blocks of the main kernel: one per SM
static int attn_grid(int) { return sm_count(); }

size_t attn_tc_workspace_bytes(int32_t batch, int32_t gamma_max, int32_t hq, int32_t hkv,
                               int32_t head_dim, int32_t max_seq_len)
{
    (void)max_seq_len;
    if ((head_dim != HD && head_dim != 64) || hkv <= 0 || hq % hkv != 0) return 0;
    const int rows = (hq / hkv) * (gamma_max + 1);
    const int nq = (rows + 127) / 128;
    if (nq < 1 || nq > 2 || batch > MAX_BATCH_TC) return 0;
    return prefix_bytes(batch) + (size_t)attn_grid(nq) * 2 * part_slot_floats(nq * 128) * sizeof(float);
}

template <int NQ, int TILE>
static sv_status launch_main(AttnTcLaunch &a, const sv_attn_params &p, int grid, cudaStream_t stream)
{
    constexpr int slot_bytes = TILE * HD * 2;
    // shared memory an SM can give to its one resident block (1 KB per block is reserved)
    const size_t budget = 228 * 1024 - 1024;
    const size_t fixed = (size_t)NQ * QGROUP_BYTES + ((sizeof(Shared) + 127) & ~(size_t)127);
    a.n_slots = (int)((budget - fixed) / slot_bytes);
    if (a.n_slots > 8) a.n_slots = 8;
    if (a.n_slots < 4) return SV_EUNSUPPORTED;
    const size_t smem = fixed + (size_t)a.n_slots * slot_bytes;
    if (cudaFuncSetAttribute(attn_tc_kernel<NQ, TILE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)smem) != cudaSuccess)
        return SV_ECUDA;
    return launch_kernel(false, attn_tc_kernel<NQ, TILE>, grid, 128 + 128 * NQ, smem, stream, a, p.pool->k_map, p.pool->v_map);
}

sv_status launch_attn_tc(const sv_attn_params &p, void *workspace, size_t workspace_bytes,
                         cudaStream_t stream)
{
    AttnTcLaunch a;
    a.p = p;
    a.n_pool_pages = p.pool->n_pages;
    a.group = p.hq / p.hkv;
    a.nq = rows_groups(p);
    const int rows = a.group * (p.gamma_max + 1);
    const bool use_tq = attn_tq_supported(p);
    a.slot_rows = use_tq ? attn_tq_slot_rows(rows) : a.nq * 128;
    const int grid = use_tq ? sm_count() : attn_grid(a.nq);
    if (grid > MAX_ATTN_GRID) return SV_EUNSUPPORTED;
    if (workspace_bytes < prefix_bytes(p.batch) + (size_t)grid * 2 * part_slot_floats(a.slot_rows) * sizeof(float))
        return SV_EWORKSPACE;
    a.ws_prefix = static_cast<int32_t *>(workspace);
    a.ws_part = reinterpret_cast<float *>(static_cast<uint8_t *>(workspace) + prefix_bytes(p.batch));
    sv_status st;
    if (use_tq) st = launch_attn_tq_main(a, p, grid, stream);
    else st = launch_main<2, 128>(a, p, grid, stream);
    if (st != SV_OK) return st;
    return launch_kernel(true, attn_combine_kernel, grid, COMBINE_THREADS, 0, stream, a);
}

}  // namespace sv
