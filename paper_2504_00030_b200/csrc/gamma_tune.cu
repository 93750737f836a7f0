// GammaTune controller (paper Section 4.1, Algorithm 1) with its state on the
// device, plus the sequence-length and row-offset bookkeeping of the next step.
//
// One thread block handles the whole batch: the per-sequence update is O(1) and
// the only cross-sequence work is the prefix sum that rebuilds cu_q / cu_d.
#include "common.cuh"

namespace sv {

constexpr int GT_THREADS = 256;

// Inclusive block scan of one int per thread (two values scanned together).
__device__ __forceinline__ void block_scan2(int &a, int &b, int *smem /* [2 * 8] */)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        int ta = __shfl_up_sync(0xffffffffu, a, d);
        int tb = __shfl_up_sync(0xffffffffu, b, d);
        if (lane >= d) { a += ta; b += tb; }
    }
    if (lane == 31) { smem[warp] = a; smem[8 + warp] = b; }
    __syncthreads();
    int oa = 0, ob = 0;
    for (int w = 0; w < warp; ++w) { oa += smem[w]; ob += smem[8 + w]; }
    a += oa;
    b += ob;
    __syncthreads();
}

template <bool INIT>
__global__ void __launch_bounds__(GT_THREADS)
gamma_tune_kernel(sv_gamma_params p, int gamma0)
{
    pdl_enter();
    __shared__ int scan_smem[16];
    __shared__ int carry[2];
    if (threadIdx.x == 0) {
        carry[0] = 0;
        carry[1] = 0;
        p.cu_q[0] = 0;
        p.cu_d[0] = 0;
    }
    __syncthreads();
    const sv_gamma_config c = p.config;
    for (int base = 0; base < p.batch; base += GT_THREADS) {
        const int b = base + threadIdx.x;
        int g_new = 0;
        if (b < p.batch) {
            if (INIT) {
                g_new = gamma0;
                p.gamma_bar[b] = (double)gamma0;
                p.gamma[b] = gamma0;
            } else {
                int g_old = p.gamma[b];
                if (g_old < 0 || g_old > c.gamma_max) {
                    set_status(p.device_status, SV_DEV_BAD_GAMMA);
                    g_old = min(max(g_old, 0), c.gamma_max);
                }
                int A = p.n_accepted[b];
                A = min(max(A, 0), g_old);
                // GammaTune+ (Section 4.2): the draft may have stopped after n_drafted <= gamma
                // tokens; that many positions (+1) entered the cache, while "A = gamma" below
                // still refers to the gamma this controller issued.
                int rows_old = g_old + 1;
                if (p.n_drafted != nullptr) {
                    int nd = p.n_drafted[b];
                    if (nd < 0 || nd > g_old) {
                        set_status(p.device_status, SV_DEV_BAD_GAMMA);
                        nd = min(max(nd, 0), g_old);
                    }
                    rows_old = nd + 1;
                    A = min(A, nd);
                }
                g_new = g_old;
                if (c.mode == SV_GT_PROPOSED || c.mode == SV_GT_LITERAL) {
                    // Eq. 7: the expansion raises the count fed to the average (proposed
                    // reading); the literal listing feeds A itself.
                    double fed = (double)A;
                    if (A == g_old && c.mode == SV_GT_PROPOSED) fed = __dadd_rn((double)A, c.delta);
                    // Eq. 8, each operation rounded once: no fused multiply-add.
                    const double t1 = __dmul_rn(__dsub_rn(1.0, c.eta), p.gamma_bar[b]);
                    const double t2 = __dmul_rn(c.eta, fed);
                    double s = __dadd_rn(t1, t2);
                    if (s < (double)c.gamma_min) s = (double)c.gamma_min;
                    if (s > (double)c.gamma_max) s = (double)c.gamma_max;
                    p.gamma_bar[b] = s;
                    g_new = (int)ceil(s);
                }
                p.gamma[b] = g_new;
                if (p.seq_len != nullptr)
                    p.seq_len[b] = p.seq_len[b] - rows_old + (A + 1) + (g_new + 1);
                if (p.trajectory != nullptr) p.trajectory[(size_t)p.step * p.batch + b] = g_new;
                if (p.accepted_log != nullptr) p.accepted_log[(size_t)p.step * p.batch + b] = A;
            }
        }
        if (c.padded_rows) {
            if (b < p.batch) {
                p.cu_q[b + 1] = (b + 1) * (c.gamma_max + 1);
                p.cu_d[b + 1] = (b + 1) * c.gamma_max;
            }
        } else {
            int sq = (b < p.batch) ? g_new + 1 : 0;
            int sd = (b < p.batch) ? g_new : 0;
            block_scan2(sq, sd, scan_smem);
            if (b < p.batch) {
                p.cu_q[b + 1] = carry[0] + sq;
                p.cu_d[b + 1] = carry[1] + sd;
            }
            __syncthreads();
            if (threadIdx.x == GT_THREADS - 1) {
                carry[0] += sq;
                carry[1] += sd;
            }
            __syncthreads();
        }
    }
}

static sv_status check_params(const sv_gamma_params *p, bool init)
{
    if (p == nullptr || p->batch <= 0) return SV_EINVAL;
    if (p->gamma_bar == nullptr || p->gamma == nullptr || p->cu_q == nullptr || p->cu_d == nullptr)
        return SV_EINVAL;
    if (!init && p->n_accepted == nullptr) return SV_EINVAL;
    const sv_gamma_config &c = p->config;
    if (c.gamma_min < 0 || c.gamma_max < c.gamma_min) return SV_EINVAL;
    if (!(c.eta >= 0.0 && c.eta <= 1.0) || !(c.delta == c.delta)) return SV_EINVAL;
    if (c.mode != SV_GT_FIXED && c.mode != SV_GT_PROPOSED && c.mode != SV_GT_LITERAL)
        return SV_EUNSUPPORTED;
    if ((p->trajectory != nullptr || p->accepted_log != nullptr) && p->step < 0) return SV_EINVAL;
    return SV_OK;
}

}  // namespace sv

extern "C" sv_status gamma_tune_update(const sv_gamma_params *p, void *stream)
{
    sv_status st = sv::check_params(p, false);
    if (st != SV_OK) return st;
    return sv::launch_kernel(true, sv::gamma_tune_kernel<false>, 1, sv::GT_THREADS, 0, (cudaStream_t)stream, *p, 0);
}

extern "C" sv_status gamma_tune_init(const sv_gamma_params *p, int32_t gamma0, void *stream)
{
    sv_status st = sv::check_params(p, true);
    if (st != SV_OK) return st;
    if (gamma0 < 0 || gamma0 > p->config.gamma_max) return SV_EINVAL;
    return sv::launch_kernel(true, sv::gamma_tune_kernel<true>, 1, sv::GT_THREADS, 0, (cudaStream_t)stream, *p, gamma0);
}
