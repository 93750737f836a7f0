// GammaTune+ confidence-guided early stop of drafting (paper Section 4.2).
//
// Two kernels on the caller's stream:
//
//  1. draft_conf_rowstats_kernel -- streams every draft row once.  One warp per (row, slice of
//     the vocabulary): 128-bit streaming loads, six per lane in flight, running maximum of the
//     logits and a single-pass online softmax sum with a power-of-two reference (float32
//     ex2.approx exponentials accumulated in float64), warp-shuffle reduction, one record per
//     item in the caller's workspace.
//  2. draft_stop_decide_kernel -- one block per sequence, a group of lanes per draft position
//     with its lanes over the slice records: merges them, evaluates the confidence c_i = 2^(max * log2(e)/T - ref) / sum in float64 and
//     takes the first position below tau.
#include "common.cuh"
#include "row_stream.cuh"

namespace sv {

constexpr int DS_THREADS = 256;   // 8 independent warps
constexpr int DS_UNROLL = 6;      // float4 loads in flight per lane
constexpr int DS_MIN_SLICE = 2048;
constexpr int DS_MAX_SLICE = 16384;
constexpr int DS_MAX_GAMMA = 64;

struct __align__(16) ConfPartial {
    double sum;     // sum of 2^(x*c - ref) over the slice
    float ref;      // integer-valued reference exponent
    float amax;     // largest logit of the slice
};

struct DraftStopLaunch {
    sv_draft_stop_params p;
    ConfPartial *partials;   // [batch * gamma_max * n_slices]
    int slice;               // elements per slice (multiple of 1024)
    int n_slices;
    int vec_ok;              // 128-bit loads legal for every row
};

__device__ __forceinline__ float ds_temperature(const sv_draft_stop_params &p, int b)
{
    return p.temperature_per_seq != nullptr ? p.temperature_per_seq[b] : p.temperature;
}

__device__ __forceinline__ int ds_gamma(const sv_draft_stop_params &p, int b)
{
    int g = p.gamma[b];
    if (g < 0 || g > p.gamma_max) {
        set_status(p.device_status, SV_DEV_BAD_GAMMA);
        g = min(max(g, 0), p.gamma_max);
    }
    return g;
}

template <bool BF16>       // logits stored as bf16 bit patterns (widened exactly) instead of float32
__global__ void __launch_bounds__(DS_THREADS)
draft_conf_rowstats_kernel(const __grid_constant__ DraftStopLaunch a)
{
    pdl_enter();
    const sv_draft_stop_params &p = a.p;
    const long long n_items = (long long)p.batch * p.gamma_max * a.n_slices;
    const int lane = threadIdx.x & 31;
    const long long warp0 = (long long)blockIdx.x * (DS_THREADS / 32) + (threadIdx.x >> 5);
    const long long n_warps = (long long)gridDim.x * (DS_THREADS / 32);

    for (long long item = warp0; item < n_items; item += n_warps) {
        const int slice_id = (int)(item % a.n_slices);
        const int dense_row = (int)(item / a.n_slices);
        const int b = dense_row / p.gamma_max, i = dense_row % p.gamma_max;
        const float T = ds_temperature(p, b);
        if (i >= ds_gamma(p, b) || !(T > 0.f)) continue;       // no such position, or a greedy draft
        const void *row = logit_row<BF16>(p.draft_logits, p.cu_d[b] + i, p.row_stride);
        const int lo = slice_id * a.slice;
        const int hi = min(p.vocab, lo + a.slice);

        // c = log2(e)/T split into a float pair with a strictly positive low part, so that
        // x = -inf gives -inf (never inf - inf) and NaN / +inf inputs surface in the sum.
        const double c = 1.4426950408889634 / (double)T;
        float c_hi = __double2float_rd(c);
        float c_lo = (float)(c - (double)c_hi);
        if (!(c_lo > 0.f)) {
            c_hi = __int_as_float(__float_as_int(c_hi) - 1);
            c_lo = (float)(c - (double)c_hi);
        }
        float ref = REF_INIT, amax = -CUDART_INF_F;
        double sum = 0.0;
        auto consume4 = [&](float x0, float x1, float x2, float x3, int) {
            const float m4 = fmaxf(fmaxf(x0, x1), fmaxf(x2, x3));
            amax = fmaxf(amax, m4);
            const float ymax = m4 * c_hi + 1.f;
            if (ymax > ref) {   // rare: the running reference has to grow
                const float nr = ceilf(ymax);
                sum = scale_down_pow2(sum, ref - nr);
                ref = nr;
            }
            const float e0 = ex2_approx(fmaf(x0, c_lo, fmaf(x0, c_hi, -ref)));
            const float e1 = ex2_approx(fmaf(x1, c_lo, fmaf(x1, c_hi, -ref)));
            const float e2 = ex2_approx(fmaf(x2, c_lo, fmaf(x2, c_hi, -ref)));
            const float e3 = ex2_approx(fmaf(x3, c_lo, fmaf(x3, c_hi, -ref)));
            sum += (double)((e0 + e1) + (e2 + e3));
        };
        stream_slice<BF16, DS_UNROLL>(row, lo, hi, a.vec_ok != 0, lane, consume4);
        float r = ref;
#pragma unroll
        for (int m = 16; m > 0; m >>= 1) {
            r = fmaxf(r, __shfl_xor_sync(0xffffffffu, r, m));
            amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, m));
        }
        sum = warp_sum_f64(scale_down_pow2(sum, ref - r));
        if (lane == 0) {
            ConfPartial out;
            out.sum = sum;
            out.ref = r;
            out.amax = amax;
            a.partials[(long long)dense_row * a.n_slices + slice_id] = out;
        }
    }
}

constexpr int DSD_THREADS = 512;     // 16 warps: all positions of a sequence in one or two passes

__global__ void __launch_bounds__(DSD_THREADS)
draft_stop_decide_kernel(const __grid_constant__ DraftStopLaunch a)
{
    pdl_enter();
    const sv_draft_stop_params &p = a.p;
    __shared__ unsigned char s_below[DS_MAX_GAMMA];
    const int b = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = ds_gamma(p, b);
    const float Tf = ds_temperature(p, b);
    const double tau = (double)p.tau;
    // groups of `lpr` lanes (a power of two covering the slices, at most a warp) take one draft
    // position each, their lanes over the slice records of its row (a shuffle butterfly)
    int lpr = 1;
    while (lpr < 32 && lpr < a.n_slices) lpr <<= 1;
    const int per_pass = (DSD_THREADS / 32) * (32 / lpr);
    const int sub = lane / lpr, sl = lane % lpr;
    for (int i0 = 0; i0 < g; i0 += per_pass) {
        const int i = i0 + warp * (32 / lpr) + sub;
        const bool have = i < g;
        double conf = 1.0;                             // greedy draft: the drafted token has probability one
        if (Tf > 0.f) {                                // the same for the whole block
            const ConfPartial *pp = a.partials + ((long long)b * p.gamma_max + i) * a.n_slices;
            float ref = REF_INIT, amax = -CUDART_INF_F;
            double sum = 0.0;
            if (have) {
                for (int s = sl; s < a.n_slices; s += lpr) {
                    const ConfPartial q = pp[s];
                    merge_stats(ref, sum, q.ref, q.sum);
                    amax = fmaxf(amax, q.amax);
                }
            }
            for (int m = lpr >> 1; m > 0; m >>= 1) {
                merge_stats(ref, sum, __shfl_xor_sync(0xffffffffu, ref, m), shfl_xor_f64(sum, m));
                amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, m));
            }
            // top probability = exp(max/T) / sum_k exp(x_k/T) = 2^(max c - ref) / sum
            if (have) conf = exp2((double)amax * (1.4426950408889634 / (double)Tf) - (double)ref) / sum;
        }
        if (have && sl == 0) {
            if (!(conf == conf)) set_status(p.device_status, SV_DEV_NONFINITE);
            if (p.top_prob != nullptr) p.top_prob[p.cu_d[b] + i] = conf;
            s_below[i] = conf < tau;
        }
    }
    __syncthreads();
    if (warp != 0) return;
    int first = g;                                     // first position whose confidence is below tau
    for (int i0 = 0; i0 < g; i0 += 32) {
        const int i = i0 + lane;
        const unsigned m = __ballot_sync(0xffffffffu, i < g && s_below[i] != 0);
        if (m != 0 && first == g) first = i0 + __ffs(m) - 1;
    }
    if (lane == 0) p.n_drafted[b] = first < g ? first + 1 : g;
}

static size_t ds_align256(size_t n) { return (n + 255) & ~(size_t)255; }

static int ds_pick_slice(const sv_draft_stop_params *p)
{
    const long long rows = (long long)p->batch * p->gamma_max;
    const long long want = 4LL * sm_count() * 32;
    int slice = DS_MAX_SLICE;
    while (slice > DS_MIN_SLICE && rows * ((p->vocab + slice - 1) / slice) < want) slice >>= 1;
    return slice;
}

}  // namespace sv

extern "C" size_t spec_draft_stop_workspace_bytes(int32_t batch, int32_t gamma_max, int32_t vocab)
{
    if (batch <= 0 || gamma_max < 0 || vocab <= 0) return 0;
    const size_t n_slices = ((size_t)vocab + sv::DS_MIN_SLICE - 1) / sv::DS_MIN_SLICE;
    const size_t n = sv::ds_align256((size_t)batch * (size_t)gamma_max * n_slices * sizeof(sv::ConfPartial));
    return n > 256 ? n : 256;
}

extern "C" sv_status spec_draft_stop(const sv_draft_stop_params *p, void *workspace, size_t workspace_bytes,
                                     void *stream)
{
    if (p == nullptr || p->batch <= 0 || p->vocab <= 0 || p->gamma_max < 0) return SV_EINVAL;
    if (p->gamma_max > sv::DS_MAX_GAMMA) return SV_EUNSUPPORTED;
    if (p->gamma == nullptr || p->cu_d == nullptr || p->n_drafted == nullptr) return SV_EINVAL;
    if (p->gamma_max > 0 && p->draft_logits == nullptr) return SV_EINVAL;
    if (p->row_stride < p->vocab) return SV_EINVAL;
    if (!(p->temperature >= 0.f) || !(p->tau >= 0.f) || !(p->tau <= 1.f)) return SV_EINVAL;
    if (workspace == nullptr ||
        workspace_bytes < spec_draft_stop_workspace_bytes(p->batch, p->gamma_max, p->vocab))
        return SV_EWORKSPACE;
    if (!sv::aligned16(workspace)) return SV_EALIGN;
    cudaStream_t s = (cudaStream_t)stream;
    sv::DraftStopLaunch a;
    a.p = *p;
    a.partials = static_cast<sv::ConfPartial *>(workspace);
    a.slice = sv::ds_pick_slice(p);
    a.n_slices = (p->vocab + a.slice - 1) / a.slice;
    const bool bf16 = p->logits_bf16 != 0;
    a.vec_ok = sv::logits_vec_ok(p->draft_logits, p->row_stride, bf16);
    const long long n_items = (long long)p->batch * p->gamma_max * a.n_slices;
    if (n_items > 0) {
        static int blocks_per_sm_of[64][2]; // resident blocks per SM, asked once per device and logit type
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SV_ECUDA;
        if (blocks_per_sm_of[dev][bf16] == 0) {
            int n = 0;
            const cudaError_t e =
                bf16 ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, sv::draft_conf_rowstats_kernel<true>, sv::DS_THREADS, 0)
                     : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, sv::draft_conf_rowstats_kernel<false>, sv::DS_THREADS, 0);
            if (e != cudaSuccess || n < 1) n = 2;
            blocks_per_sm_of[dev][bf16] = n;
        }
        const int blocks_per_sm = blocks_per_sm_of[dev][bf16];
        const long long blocks_needed = (n_items + sv::DS_THREADS / 32 - 1) / (sv::DS_THREADS / 32);
        const long long cap = (long long)blocks_per_sm * sv::sm_count();
        const int grid = (int)(blocks_needed < cap ? blocks_needed : cap);
        const sv_status st = bf16 ? sv::launch_kernel(false, sv::draft_conf_rowstats_kernel<true>, grid, sv::DS_THREADS, 0, s, a)
                                  : sv::launch_kernel(false, sv::draft_conf_rowstats_kernel<false>, grid, sv::DS_THREADS, 0, s, a);
        if (st != SV_OK) return st;
    }
    return sv::launch_kernel(true, sv::draft_stop_decide_kernel, p->batch, sv::DSD_THREADS, 0, s, a);
}
