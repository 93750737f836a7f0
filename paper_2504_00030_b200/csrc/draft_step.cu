// One drafting step with the confidence stop of GammaTune+ (paper Section 4.2): for every sequence
// that is still drafting, the next draft token is drawn from its row of draft logits, the row's top
// probability is compared with tau, and the drafting state is advanced.
//
// Four kernels on the caller's stream:
//
//  1. draft_step_rowstats_kernel -- streams the rows of the active sequences once.  One warp per
//     (sequence, slice of the vocabulary): running maximum and single-pass online softmax sum with
//     a power-of-two reference (float32 ex2.approx exponentials accumulated in float64); greedy
//     rows (T == 0) keep the largest logit and its lowest index instead.
//  2. draft_step_decide_kernel -- one warp per sequence: merges the slice records, forms the
//     confidence c = 2^(max * log2(e)/T - ref) / sum in float64, leaves the record the sampling
//     pass needs, and takes the greedy token directly.
//  3. the float64 inverse-CDF pass of accept_sample.cu over each active row (row_sample.cuh).
//  4. draft_step_commit_kernel -- stores token and confidence at the sequence's next draft
//     position and advances n_drafted / active.
#include "common.cuh"
#include "row_sample.cuh"
#include "row_stream.cuh"

#include <math_constants.h>

namespace sv {

constexpr int DP_THREADS = 256;   // 8 independent warps
constexpr int DP_UNROLL = 6;      // 128-bit loads in flight per lane
constexpr int DP_MIN_SLICE = 1024;
constexpr int DP_MAX_SLICE = 16384;

struct __align__(16) StepPartial {
    double sum;     // sum of 2^(x*c - ref) over the slice
    float ref;      // integer-valued reference exponent
    float amax;     // largest logit of the slice
    int32_t aidx;   // greedy rows: its lowest index
    int32_t bad;    // greedy rows: nonzero if the slice held a NaN
};

// per sequence, between the decision and the commit
struct StepDecision {
    double conf;
    int32_t token;      // greedy token, or -1
    int32_t state;      // 0: not drafting this step, 1: token comes from the sampling pass, 2: token is set here
};

struct DraftStepLaunch {
    sv_draft_step_params p;
    StepPartial *partials;   // [batch * n_slices]
    StepDecision *decisions; // [batch]
    SeqRecord *records;      // [batch]
    unsigned int *done;      // [batch]
    int32_t *sampled;        // [batch] tokens of the sampling pass
    int slice, n_slices;
    int vec_ok;
};

__device__ __forceinline__ float dp_temperature(const sv_draft_step_params &p, int b)
{
    return p.temperature_per_seq != nullptr ? p.temperature_per_seq[b] : p.temperature;
}

// does sequence b draft a token in this step?
__device__ __forceinline__ bool dp_drafting(const sv_draft_step_params &p, int b)
{
    if (p.active[b] == 0) return false;
    int g = p.gamma[b];
    if (g < 0 || g > p.gamma_max) {
        set_status(p.device_status, SV_DEV_BAD_GAMMA);
        g = min(max(g, 0), p.gamma_max);
    }
    const int n = p.n_drafted[b];
    return n >= 0 && n < g;
}

template <bool BF16>
__global__ void __launch_bounds__(DP_THREADS)
draft_step_rowstats_kernel(const __grid_constant__ DraftStepLaunch a)
{
    pdl_enter();
    const sv_draft_step_params &p = a.p;
    const long long n_items = (long long)p.batch * a.n_slices;
    const int lane = threadIdx.x & 31;
    const long long warp0 = (long long)blockIdx.x * (DP_THREADS / 32) + (threadIdx.x >> 5);
    const long long n_warps = (long long)gridDim.x * (DP_THREADS / 32);

    for (long long item = warp0; item < n_items; item += n_warps) {
        const int slice_id = (int)(item % a.n_slices);
        const int b = (int)(item / a.n_slices);
        if (!dp_drafting(p, b)) continue;
        const float T = dp_temperature(p, b);
        const bool greedy = !(T > 0.f);
        const void *row = logit_row<BF16>(p.draft_logits, b, p.row_stride);
        const int lo = slice_id * a.slice;
        const int hi = min(p.vocab, lo + a.slice);

        // c = log2(e)/T split into a float pair with a strictly positive low part, so that
        // x = -inf gives -inf (never inf - inf) and NaN / +inf inputs surface in the sum.
        float c_hi = 0.f, c_lo = 0.f;
        if (!greedy) {
            const double c = 1.4426950408889634 / (double)T;
            c_hi = __double2float_rd(c);
            c_lo = (float)(c - (double)c_hi);
            if (!(c_lo > 0.f)) {
                c_hi = __int_as_float(__float_as_int(c_hi) - 1);
                c_lo = (float)(c - (double)c_hi);
            }
        }
        float ref = REF_INIT, amax = -CUDART_INF_F;
        double sum = 0.0;
        int aidx = 0x7fffffff, bad = 0;
        auto consume4 = [&](float x0, float x1, float x2, float x3, int k0) {
            if (greedy) {
                const float s4 = (x0 + x1) + (x2 + x3);       // NaN if any of the four is (padding is -inf)
                if (!(s4 == s4)) bad = 1;
                if (x0 > amax) { amax = x0; aidx = k0; }
                if (x1 > amax) { amax = x1; aidx = k0 + 1; }
                if (x2 > amax) { amax = x2; aidx = k0 + 2; }
                if (x3 > amax) { amax = x3; aidx = k0 + 3; }
            } else {
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
            }
        };
        stream_slice<BF16, DP_UNROLL>(row, lo, hi, a.vec_ok != 0, lane, consume4);

        if (greedy) {
#pragma unroll
            for (int m = 16; m > 0; m >>= 1) {
                const float v2 = __shfl_xor_sync(0xffffffffu, amax, m);
                const int i2 = __shfl_xor_sync(0xffffffffu, aidx, m);
                if (v2 > amax || (v2 == amax && i2 < aidx)) { amax = v2; aidx = i2; }
            }
            bad = __any_sync(0xffffffffu, bad != 0) ? 1 : 0;
        } else {
            float r = ref;
#pragma unroll
            for (int m = 16; m > 0; m >>= 1) {
                r = fmaxf(r, __shfl_xor_sync(0xffffffffu, r, m));
                amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, m));
            }
            sum = warp_sum_f64(scale_down_pow2(sum, ref - r));
            ref = r;
        }
        if (lane == 0) {
            StepPartial out;
            out.sum = sum;
            out.ref = ref;
            out.amax = amax;
            out.aidx = aidx;
            out.bad = bad;
            a.partials[(long long)b * a.n_slices + slice_id] = out;
        }
    }
}

// One warp per sequence: the slice records of its row -> confidence, sampling record or greedy token.
__global__ void __launch_bounds__(32)
draft_step_decide_kernel(const __grid_constant__ DraftStepLaunch a)
{
    pdl_enter();
    const sv_draft_step_params &p = a.p;
    const int b = blockIdx.x, lane = threadIdx.x;
    SeqRecord rec;
    rec.sum_p_hat = rec.sum_q_hat = 0.0;
    rec.ref_p = rec.ref_q = 0.f;
    rec.n = 0;
    rec.mode = 0;
    StepDecision dec;
    dec.conf = 1.0;
    dec.token = -1;
    dec.state = 0;
    if (dp_drafting(p, b)) {                             // the same for the whole warp
        const float T = dp_temperature(p, b);
        const StepPartial *pp = a.partials + (long long)b * a.n_slices;
        if (T > 0.f) {
            float ref = REF_INIT, amax = -CUDART_INF_F;
            double sum = 0.0;
            for (int s = lane; s < a.n_slices; s += 32) {
                const StepPartial q = pp[s];
                merge_stats(ref, sum, q.ref, q.sum);
                amax = fmaxf(amax, q.amax);
            }
#pragma unroll
            for (int m = 16; m > 0; m >>= 1) {
                merge_stats(ref, sum, __shfl_xor_sync(0xffffffffu, ref, m), shfl_xor_f64(sum, m));
                amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, m));
            }
            // top probability = exp(max/T) / sum_k exp(x_k/T) = 2^(max c - ref) / sum
            const double conf = exp2((double)amax * (1.4426950408889634 / (double)T) - (double)ref) / sum;
            if (!(sum > 0.0) || !(sum < CUDART_INF) || !(conf == conf)) {
                set_status(p.device_status, SV_DEV_NONFINITE);
                dec.conf = CUDART_NAN;
                dec.state = 2;                           // token -1
            } else {
                dec.conf = conf;
                dec.state = 1;
                rec.mode = 2;
                rec.ref_p = ref;
                rec.sum_p_hat = sum;
            }
        } else {
            float amax = -CUDART_INF_F;
            int aidx = 0x7fffffff, bad = 0;
            for (int s = lane; s < a.n_slices; s += 32) {
                const StepPartial q = pp[s];
                if (q.amax > amax || (q.amax == amax && q.aidx < aidx)) { amax = q.amax; aidx = q.aidx; }
                bad |= q.bad;
            }
#pragma unroll
            for (int m = 16; m > 0; m >>= 1) {
                const float v2 = __shfl_xor_sync(0xffffffffu, amax, m);
                const int i2 = __shfl_xor_sync(0xffffffffu, aidx, m);
                if (v2 > amax || (v2 == amax && i2 < aidx)) { amax = v2; aidx = i2; }
            }
            bad = __any_sync(0xffffffffu, bad != 0) ? 1 : 0;
            dec.state = 2;
            if (bad || aidx == 0x7fffffff) {             // a NaN in the row, or nothing above -inf
                set_status(p.device_status, SV_DEV_NONFINITE);
                dec.conf = CUDART_NAN;
            } else {
                dec.token = aidx;
            }
        }
    }
    if (lane == 0) {
        a.records[b] = rec;
        a.decisions[b] = dec;
        a.done[b] = 0u;
    }
}

constexpr int DC_THREADS = 128;

__global__ void __launch_bounds__(DC_THREADS)
draft_step_commit_kernel(const __grid_constant__ DraftStepLaunch a)
{
    pdl_enter();
    const sv_draft_step_params &p = a.p;
    const int b = blockIdx.x * DC_THREADS + threadIdx.x;
    if (b >= p.batch) return;
    const StepDecision dec = a.decisions[b];
    const int g = min(max(p.gamma[b], 0), p.gamma_max);
    if (dec.state == 0) {
        if (p.active[b] != 0 && p.n_drafted[b] >= g) p.active[b] = 0;    // the cap was reached earlier
        return;
    }
    const int tok = dec.state == 1 ? a.sampled[b] : dec.token;
    const int n = p.n_drafted[b];
    const long long pos = (long long)p.cu_d[b] + n;
    p.draft_tokens[pos] = tok;
    if (p.top_prob != nullptr) p.top_prob[pos] = dec.conf;
    p.n_drafted[b] = n + 1;
    p.active[b] = (tok >= 0 && dec.conf >= (double)p.tau && n + 1 < g) ? 1 : 0;
}

static size_t dp_align256(size_t n) { return (n + 255) & ~(size_t)255; }

struct DraftStepLayout {
    size_t partials, decisions, records, done, sampled, sampler, total;
};

static DraftStepLayout draft_step_layout(int batch, int vocab)
{
    DraftStepLayout l;
    const size_t n_slices = ((size_t)vocab + DP_MIN_SLICE - 1) / DP_MIN_SLICE;
    l.partials = 0;
    l.decisions = dp_align256((size_t)batch * n_slices * sizeof(StepPartial));
    l.records = l.decisions + dp_align256((size_t)batch * sizeof(StepDecision));
    l.done = l.records + dp_align256((size_t)batch * sizeof(SeqRecord));
    l.sampled = l.done + dp_align256((size_t)batch * sizeof(unsigned int));
    l.sampler = l.sampled + dp_align256((size_t)batch * sizeof(int32_t));
    l.total = l.sampler + row_sample_scratch_bytes(batch, vocab);
    return l;
}

static int dp_pick_slice(const sv_draft_step_params *p)
{
    // one warp per (row, slice): enough items to fill the resident warps, slices of 1K..16K elements
    const long long want = 4LL * sm_count() * 32;
    int slice = DP_MAX_SLICE;
    while (slice > DP_MIN_SLICE && (long long)p->batch * ((p->vocab + slice - 1) / slice) < want) slice >>= 1;
    return slice;
}

}  // namespace sv

extern "C" size_t spec_draft_step_workspace_bytes(int32_t batch, int32_t vocab)
{
    if (batch <= 0 || vocab <= 0) return 0;
    return sv::draft_step_layout(batch, vocab).total;
}

extern "C" sv_status spec_draft_step(const sv_draft_step_params *p, void *workspace, size_t workspace_bytes,
                                     void *stream)
{
    if (p == nullptr || p->batch <= 0 || p->vocab <= 0 || p->gamma_max < 0) return SV_EINVAL;
    if (p->draft_logits == nullptr || p->gamma == nullptr || p->cu_d == nullptr || p->n_drafted == nullptr ||
        p->active == nullptr || p->draft_tokens == nullptr)
        return SV_EINVAL;
    if (p->row_stride < p->vocab) return SV_EINVAL;
    if (!(p->temperature >= 0.f) || !(p->tau >= 0.f) || !(p->tau <= 1.f)) return SV_EINVAL;
    const bool any_sampling = p->temperature_per_seq != nullptr || p->temperature > 0.f;
    if (any_sampling && p->u_sample == nullptr) return SV_EINVAL;
    if (workspace == nullptr || workspace_bytes < spec_draft_step_workspace_bytes(p->batch, p->vocab))
        return SV_EWORKSPACE;
    if (!sv::aligned16(workspace)) return SV_EALIGN;
    cudaStream_t s = (cudaStream_t)stream;
    const sv::DraftStepLayout l = sv::draft_step_layout(p->batch, p->vocab);
    uint8_t *base = static_cast<uint8_t *>(workspace);
    sv::DraftStepLaunch a;
    a.p = *p;
    a.partials = reinterpret_cast<sv::StepPartial *>(base + l.partials);
    a.decisions = reinterpret_cast<sv::StepDecision *>(base + l.decisions);
    a.records = reinterpret_cast<sv::SeqRecord *>(base + l.records);
    a.done = reinterpret_cast<unsigned int *>(base + l.done);
    a.sampled = reinterpret_cast<int32_t *>(base + l.sampled);
    a.slice = sv::dp_pick_slice(p);
    a.n_slices = (p->vocab + a.slice - 1) / a.slice;
    const bool bf16 = p->logits_bf16 != 0;
    a.vec_ok = sv::logits_vec_ok(p->draft_logits, p->row_stride, bf16);

    const long long n_items = (long long)p->batch * a.n_slices;
    const long long blocks_needed = (n_items + sv::DP_THREADS / 32 - 1) / (sv::DP_THREADS / 32);
    const long long cap = 4LL * sv::sm_count();
    const int grid = (int)(blocks_needed < cap ? blocks_needed : cap);
    sv_status st = bf16 ? sv::launch_kernel(false, sv::draft_step_rowstats_kernel<true>, grid, sv::DP_THREADS, 0, s, a)
                        : sv::launch_kernel(false, sv::draft_step_rowstats_kernel<false>, grid, sv::DP_THREADS, 0, s, a);
    if (st != SV_OK) return st;
    st = sv::launch_kernel(true, sv::draft_step_decide_kernel, p->batch, 32, 0, s, a);
    if (st != SV_OK) return st;
    if (any_sampling) {
        sv::RowSampleArgs r;
        r.logits = p->draft_logits;
        r.logits_bf16 = p->logits_bf16;
        r.row_stride = p->row_stride;
        r.vocab = p->vocab;
        r.batch = p->batch;
        r.temperature = p->temperature;
        r.temperature_per_seq = p->temperature_per_seq;
        r.u_sample = p->u_sample;
        r.out_tokens = a.sampled;
        r.records = a.records;
        r.done = a.done;
        r.scratch = base + l.sampler;
        r.device_status = p->device_status;
        st = sv::launch_row_sample(r, s);
        if (st != SV_OK) return st;
    }
    return sv::launch_kernel(true, sv::draft_step_commit_kernel, (p->batch + sv::DC_THREADS - 1) / sv::DC_THREADS,
                             sv::DC_THREADS, 0, s, a);
}
