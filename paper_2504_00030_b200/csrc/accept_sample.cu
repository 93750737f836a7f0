// Fused speculative-sampling acceptance over the vocabulary (paper Section 3).
//
// Two kernels per step:
//
//  1. accept_rowstats_kernel -- the streaming pass.  Every target and draft
//     logit is read exactly once with 128-bit loads; for each (row, slice of the
//     vocabulary) one thread block produces the single-pass online softmax
//     statistics (a power-of-two reference exponent and the sum of
//     2^(x*log2e/T - ref)) or, for greedy sequences, the (max, lowest index).
//     Exponentials are float32 (ex2.approx); sums are carried in float64 and
//     every rescale is by an exact power of two, so the only error in a row's
//     partition function is the per-element float32 rounding.
//
//  2. accept_finish_kernel -- one thread block per sequence: merges the slice
//     statistics into ln Z per row, evaluates ratio_i = min(1, p_i[x_i]/q_i[x_i])
//     and the comparison with u_i in float64, finds the first rejection, and
//     draws the next token from the residual max(0, p_n - q_n) (or the bonus
//     row) by inverse CDF.  That last part re-reads only the one or two rows it
//     samples from and works entirely in float64.
#include "common.cuh"

#include <math_constants.h>

namespace sv {

constexpr int RS_THREADS = 256;   // rowstats block
constexpr int RS_UNROLL = 4;      // float4 loads in flight per thread
constexpr int FIN_THREADS = 512;  // finish block
constexpr int SEG = 128;          // vocabulary elements per sampling segment (one warp, float4 per lane)
constexpr int MIN_SLICE = 2048;
constexpr float REF_INIT = -1.0e30f;

struct __align__(16) RowPartial {
    double sum;     // sum of 2^(x*c - ref) over the slice
    float ref;      // integer-valued reference exponent
    float amax;     // greedy rows: largest logit of the slice
    int32_t aidx;   // ... and its lowest index
    int32_t pad;
};

struct AcceptLaunch {
    sv_accept_params p;
    RowPartial *partials;
    int slice;       // elements per slice (multiple of 1024)
    int n_slices;
    int vec_ok;      // 128-bit loads legal for every row
};

__device__ __forceinline__ float seq_temperature(const sv_accept_params &p, int b)
{
    return p.temperature_per_seq != nullptr ? p.temperature_per_seq[b] : p.temperature;
}

__device__ __forceinline__ int seq_gamma(const sv_accept_params &p, int b)
{
    int g = p.gamma[b];
    if (g < 0 || g > p.gamma_max) {
        set_status(p.device_status, SV_DEV_BAD_GAMMA);
        g = min(max(g, 0), p.gamma_max);
    }
    return g;
}

// (ref, sum) pairs combine by rescaling to the larger reference; the factor is a power of two.
__device__ __forceinline__ void merge_stats(float &ref, double &sum, float ref2, double sum2)
{
    const float r = fmaxf(ref, ref2);
    const float d1 = fmaxf(ref - r, -2000.f), d2 = fmaxf(ref2 - r, -2000.f);
    sum = scalbn(sum, (int)d1) + scalbn(sum2, (int)d2);
    ref = r;
}

__device__ __forceinline__ void merge_argmax(float &v, int &i, float v2, int i2)
{
    if (v2 > v || (v2 == v && i2 < i)) { v = v2; i = i2; }
}

// ---------------------------------------------------------------------------------------------
// Kernel 1: streaming row statistics.
// Dense row numbering: sequence b owns rows b*(2*gmax+1) + j; j <= gmax is target row j,
// j > gmax is draft row j-gmax-1.  Rows a sequence does not have this step are skipped.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(RS_THREADS)
accept_rowstats_kernel(AcceptLaunch a)
{
    const sv_accept_params &p = a.p;
    const int rows_per_seq = 2 * p.gamma_max + 1;
    const long long n_items = (long long)p.batch * rows_per_seq * a.n_slices;
    __shared__ double s_sum[RS_THREADS / 32];
    __shared__ float s_ref[RS_THREADS / 32];
    __shared__ float s_amax[RS_THREADS / 32];
    __shared__ int s_aidx[RS_THREADS / 32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

    for (long long item = blockIdx.x; item < n_items; item += gridDim.x) {
        const int slice_id = (int)(item % a.n_slices);
        const int dense_row = (int)(item / a.n_slices);
        const int b = dense_row / rows_per_seq;
        const int j = dense_row % rows_per_seq;
        const int g = seq_gamma(p, b);
        const float T = seq_temperature(p, b);
        const bool greedy = !(T > 0.f);
        const float *row;
        if (j <= p.gamma_max) {
            if (j > g) continue;
            row = p.target_logits + (long long)(p.cu_q[b] + j) * p.row_stride;
        } else {
            const int i = j - p.gamma_max - 1;
            if (i >= g || greedy) continue;
            row = p.draft_logits + (long long)(p.cu_d[b] + i) * p.row_stride;
        }
        const int lo = slice_id * a.slice;
        const int hi = min(p.vocab, lo + a.slice);

        float ref = REF_INIT;
        double sum = 0.0;
        float amax = -CUDART_INF_F;
        int aidx = 0x7fffffff;

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

        auto consume4 = [&](float x0, float x1, float x2, float x3, int k0) {
            if (greedy) {
                if (x0 > amax) { amax = x0; aidx = k0; }
                if (x1 > amax) { amax = x1; aidx = k0 + 1; }
                if (x2 > amax) { amax = x2; aidx = k0 + 2; }
                if (x3 > amax) { amax = x3; aidx = k0 + 3; }
            } else {
                const float m4 = fmaxf(fmaxf(x0, x1), fmaxf(x2, x3));
                const float ymax = m4 * c_hi + 1.f;
                if (ymax > ref) {   // rare: the running reference has to grow
                    const float nr = ceilf(ymax);
                    sum = scalbn(sum, (int)fmaxf(ref - nr, -2000.f));
                    ref = nr;
                }
                const float e0 = ex2_approx(fmaf(x0, c_lo, fmaf(x0, c_hi, -ref)));
                const float e1 = ex2_approx(fmaf(x1, c_lo, fmaf(x1, c_hi, -ref)));
                const float e2 = ex2_approx(fmaf(x2, c_lo, fmaf(x2, c_hi, -ref)));
                const float e3 = ex2_approx(fmaf(x3, c_lo, fmaf(x3, c_hi, -ref)));
                sum += (double)((e0 + e1) + (e2 + e3));
            }
        };

        if (a.vec_ok) {
            // lo is a multiple of 4; the row base is 16-byte aligned
            const int n4 = (hi - lo) >> 2;
            const float *base = row + lo;
            for (int v0 = threadIdx.x; v0 < n4; v0 += RS_THREADS * RS_UNROLL) {
                float4 x[RS_UNROLL];
#pragma unroll
                for (int u = 0; u < RS_UNROLL; ++u) {
                    const int v = v0 + u * RS_THREADS;
                    x[u] = (v < n4) ? ld_stream_f4(base + 4 * (long long)v)
                                    : make_float4(-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F,
                                                  -CUDART_INF_F);
                }
#pragma unroll
                for (int u = 0; u < RS_UNROLL; ++u) {
                    const int v = v0 + u * RS_THREADS;
                    if (v < n4) consume4(x[u].x, x[u].y, x[u].z, x[u].w, lo + 4 * v);
                }
            }
            // ragged tail (vocab not a multiple of 4): at most 3 elements, last slice only
            const int tail0 = lo + 4 * n4;
            if (threadIdx.x == 0 && tail0 < hi) {
                float t[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) t[u] = (tail0 + u < hi) ? row[tail0 + u] : -CUDART_INF_F;
                consume4(t[0], t[1], t[2], t[3], tail0);
            }
        } else {
            for (int k0 = lo + 4 * threadIdx.x; k0 < hi; k0 += 4 * RS_THREADS) {
                float t[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) t[u] = (k0 + u < hi) ? __ldg(row + k0 + u) : -CUDART_INF_F;
                consume4(t[0], t[1], t[2], t[3], k0);
            }
        }

        // block reduction: warp shuffles, then one value per warp through shared memory
#pragma unroll
        for (int m = 16; m > 0; m >>= 1) {
            if (greedy) {
                const float v2 = __shfl_xor_sync(0xffffffffu, amax, m);
                const int i2 = __shfl_xor_sync(0xffffffffu, aidx, m);
                merge_argmax(amax, aidx, v2, i2);
            } else {
                const float r2 = __shfl_xor_sync(0xffffffffu, ref, m);
                const double s2 = shfl_xor_f64(sum, m);
                merge_stats(ref, sum, r2, s2);
            }
        }
        __syncthreads();   // previous item's readers are done with the shared arrays
        if (lane == 0) {
            s_sum[warp] = sum;
            s_ref[warp] = ref;
            s_amax[warp] = amax;
            s_aidx[warp] = aidx;
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            for (int w = 1; w < RS_THREADS / 32; ++w) {
                if (greedy) merge_argmax(amax, aidx, s_amax[w], s_aidx[w]);
                else merge_stats(ref, sum, s_ref[w], s_sum[w]);
            }
            RowPartial out;
            out.sum = sum;
            out.ref = ref;
            out.amax = amax;
            out.aidx = aidx;
            out.pad = 0;
            a.partials[(long long)dense_row * a.n_slices + slice_id] = out;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Kernel 2: decisions and sampling, one block per sequence.
// ---------------------------------------------------------------------------------------------
// four consecutive logits starting at k0 (k0 % 4 == 0), -inf past the vocabulary
__device__ __forceinline__ void load4(const float *row, int k0, int V, bool vec, float x[4])
{
    if (vec && k0 + 3 < V) {
        const float4 v = *reinterpret_cast<const float4 *>(row + k0);
        x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
    } else {
#pragma unroll
        for (int u = 0; u < 4; ++u) x[u] = (k0 + u < V) ? row[k0 + u] : -CUDART_INF_F;
    }
}

__global__ void __launch_bounds__(FIN_THREADS)
accept_finish_kernel(AcceptLaunch a)
{
    const sv_accept_params &p = a.p;
    extern __shared__ double dyn[];          // [3 * n_seg]: positive-part sums of a, of b, all of a
    __shared__ double s_logz[2 * 64 + 1];    // ln Z per dense row (natural log, of exp(x/T))
    __shared__ double s_rsum[2 * 64 + 1];    // merged sum and reference of each dense row
    __shared__ float s_rref[2 * 64 + 1];
    __shared__ int s_amax_idx[64 + 1];
    __shared__ int s_n, s_ok;
    __shared__ double s_red[2 * (FIN_THREADS / 32)];
    __shared__ double s_ratio[64];
    __shared__ unsigned char s_code[64];

    const int b = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int gmax = p.gamma_max;
    const int rows_per_seq = 2 * gmax + 1;
    const int g = seq_gamma(p, b);
    const float Tf = seq_temperature(p, b);
    const bool greedy = !(Tf > 0.f);
    const double T = (double)Tf;
    const int V = p.vocab;
    const float *t_rows = p.target_logits + (long long)p.cu_q[b] * p.row_stride;
    const float *d_rows = greedy ? nullptr : p.draft_logits + (long long)p.cu_d[b] * p.row_stride;
    const int32_t *x = p.draft_tokens + p.cu_d[b];
    int32_t *out = p.out_tokens + (long long)b * (gmax + 1);

    // ---- merge the slice statistics of every row this sequence has
    for (int j = tid; j < rows_per_seq; j += FIN_THREADS) {
        const bool is_target = j <= gmax;
        const int i = is_target ? j : j - gmax - 1;
        const bool have = is_target ? (i <= g) : (i < g && !greedy);
        if (!have) continue;
        const RowPartial *pp = a.partials + ((long long)b * rows_per_seq + j) * a.n_slices;
        if (greedy) {
            float v = pp[0].amax;
            int ix = pp[0].aidx;
            for (int s = 1; s < a.n_slices; ++s) merge_argmax(v, ix, pp[s].amax, pp[s].aidx);
            s_amax_idx[i] = ix;
        } else {
            float ref = pp[0].ref;
            double sum = pp[0].sum;
            for (int s = 1; s < a.n_slices; ++s) merge_stats(ref, sum, pp[s].ref, pp[s].sum);
            s_rref[j] = ref;
            s_rsum[j] = sum;
            // ln sum exp(x/T) = (ref + log2(sum)) * ln 2
            const double lz = ((double)ref + log2(sum)) * 0.6931471805599453;
            s_logz[j] = lz;
            if (is_target) { if (p.logZ_p != nullptr) p.logZ_p[p.cu_q[b] + i] = lz; }
            else           { if (p.logZ_q != nullptr) p.logZ_q[p.cu_d[b] + i] = lz; }
        }
    }
    for (int i = tid; i <= gmax; i += FIN_THREADS) out[i] = -1;
    __syncthreads();

    // ---- ratio and decision of every draft position in parallel (float64) ...
    for (int i = tid; i < g; i += FIN_THREADS) {
        const int xi = x[i];
        double r = 0.0;
        int code;   // 0 reject, 1 accept, 2 non-finite partition function
        int flag = 0;
        if (xi < 0 || xi >= V) {
            set_status(p.device_status, SV_DEV_BAD_TOKEN);
            code = 0;
        } else if (greedy) {
            code = (s_amax_idx[i] == xi) ? 1 : 0;
            r = (double)code;
        } else {
            const double lzp = s_logz[i], lzq = s_logz[gmax + 1 + i];
            if (!(isfinite(lzp) && isfinite(lzq))) {
                code = 2;
            } else {
                const double lp = (double)t_rows[(long long)i * p.row_stride + xi] / T - lzp;
                const double lq = (double)d_rows[(long long)i * p.row_stride + xi] / T - lzq;
                // ratio = min(1, p/q); q == 0 (a token the draft could not have produced) -> 1
                r = (lq == -CUDART_INF) ? 1.0 : exp(fmin(lp - lq, 0.0));
                const double u = (double)p.u_accept[p.cu_d[b] + i];
                code = (u < r) ? 1 : 0;
                flag = fabs(u - r) < 1e-6;
            }
        }
        s_ratio[i] = r;
        s_code[i] = (unsigned char)(code | (flag << 2));
    }
    __syncthreads();
    // ... then the first rejection, which is sequential by definition: one thread
    if (tid == 0) {
        int n = g, ok = 1;
        uint32_t flags = 0;
        for (int i = 0; i < g; ++i) {
            const int code = s_code[i] & 3;
            if (code == 2) { ok = 0; n = i; break; }
            flags += (s_code[i] >> 2) & 1;
            if (p.ratio != nullptr) p.ratio[p.cu_d[b] + i] = s_ratio[i];
            if (code == 0) { n = i; break; }
        }
        if (p.ratio != nullptr)
            for (int i = n + 1; i < g; ++i) p.ratio[p.cu_d[b] + i] = CUDART_NAN;
        if (!greedy && ok && !isfinite(s_logz[n])) ok = 0;
        if (!ok) set_status(p.device_status, SV_DEV_NONFINITE);
        if (flags != 0 && p.flag_count != nullptr) atomicAdd(p.flag_count, flags);
        s_n = n;
        s_ok = ok;
        p.n_accepted[b] = ok ? n : 0;
        if (ok) {
            for (int i = 0; i < n; ++i) out[i] = x[i];
            if (greedy) out[n] = s_amax_idx[n];
        }
    }
    __syncthreads();
    if (greedy || !s_ok) return;

    // ---- sample the next token from row n: residual max(0, p_n - q_n), or p_gamma (bonus)
    const int n = s_n;
    const bool residual = n < g;
    const float *trow = t_rows + (long long)n * p.row_stride;
    const float *drow = residual ? d_rows + (long long)n * p.row_stride : nullptr;
    const bool vec = a.vec_ok != 0;
    const int n_seg = (V + SEG - 1) / SEG;
    double *seg_ap = dyn, *seg_bp = dyn + n_seg, *seg_a = dyn + 2 * n_seg;
    const double c = 1.4426950408889634 / T;
    const double ref_p = (double)s_rref[n];
    const double ref_q = residual ? (double)s_rref[gmax + 1 + n] : 0.0;
    // first-pass partition sums, good to ~1e-7: only used to decide the sign of p_k - q_k
    const double inv_zp_hat = 1.0 / s_rsum[n];
    const double inv_zq_hat = residual ? 1.0 / s_rsum[gmax + 1 + n] : 0.0;

    double tot_a = 0.0, tot_b = 0.0;
    for (int s = warp; s < n_seg; s += FIN_THREADS / 32) {
        const int k0 = s * SEG + 4 * lane;
        float xt[4], xd[4];
        load4(trow, k0, V, vec, xt);
        double sa = 0.0, sap = 0.0, sbp = 0.0, sb = 0.0;
        if (residual) load4(drow, k0, V, vec, xd);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const double ak = exp2((double)xt[u] * c - ref_p);
            sa += ak;
            if (residual) {
                const double bk = exp2((double)xd[u] * c - ref_q);
                sb += bk;
                if (ak * inv_zp_hat > bk * inv_zq_hat) { sap += ak; sbp += bk; }
            }
        }
        tot_a += sa;
        tot_b += sb;
        sa = warp_sum_f64(sa);
        if (residual) { sap = warp_sum_f64(sap); sbp = warp_sum_f64(sbp); }
        if (lane == 0) { seg_a[s] = sa; seg_ap[s] = sap; seg_bp[s] = sbp; }
    }
    tot_a = warp_sum_f64(tot_a);
    tot_b = warp_sum_f64(tot_b);
    if (lane == 0) { s_red[warp] = tot_a; s_red[FIN_THREADS / 32 + warp] = tot_b; }
    __syncthreads();
    if (warp != 0) return;   // the rest is one warp's work

    double Zp = 0.0, Zq = 0.0;
    for (int w = 0; w < FIN_THREADS / 32; ++w) { Zp += s_red[w]; Zq += s_red[FIN_THREADS / 32 + w]; }
    const double inv_zp = 1.0 / Zp, inv_zq = residual ? 1.0 / Zq : 0.0;

    // total mass; lane l owns the contiguous segments [l*per, (l+1)*per)
    const int per = (n_seg + 31) / 32;
    const int s_lo = min(lane * per, n_seg), s_hi = min(s_lo + per, n_seg);
    auto seg_w = [&](int s, bool use_resid) {
        return use_resid ? seg_ap[s] * inv_zp - seg_bp[s] * inv_zq : seg_a[s] * inv_zp;
    };
    double mine = 0.0;
    if (residual) for (int s = s_lo; s < s_hi; ++s) mine += seg_w(s, true);
    double W = warp_sum_f64(mine);
    bool use_resid = residual && (W > 0.0);     // no residual mass: fall back to p_n
    if (!use_resid) {
        mine = 0.0;
        for (int s = s_lo; s < s_hi; ++s) mine += seg_w(s, false);
        W = warp_sum_f64(mine);
    }
    const double target = (double)p.u_sample[b] * W;

    // exclusive prefix of the lanes' masses, then the first segment whose inclusive
    // cumulative mass exceeds the target
    double incl = mine;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const double t = shfl_up_f64(incl, d);
        if (lane >= d) incl += t;
    }
    double cum = incl - mine;
    int seg_found = n_seg;
    double seg_base = 0.0;
    for (int s = s_lo; s < s_hi; ++s) {
        const double w = seg_w(s, use_resid);
        if (seg_found == n_seg && cum + w > target) { seg_found = s; seg_base = cum; }
        cum += w;
    }
    // lowest segment over the warp
    int best = seg_found;
#pragma unroll
    for (int m = 16; m > 0; m >>= 1) best = min(best, __shfl_xor_sync(0xffffffffu, best, m));
    const unsigned who = __ballot_sync(0xffffffffu, seg_found == best && best < n_seg);
    double base = 0.0;
    if (who != 0) base = shfl_idx_f64(seg_base, __ffs(who) - 1);

    // resolve inside the segment with exact float64 weights; if rounding pushed the target
    // past this segment, walk on; if nothing qualifies, take the last positive weight.
    int y = -1, last_pos = -1;
    int s = best;
    if (best >= n_seg) { s = 0; base = 0.0; }    // target at or beyond the total: walk everything
    for (; s < n_seg && y < 0; ++s) {
        const int k0 = s * SEG + 4 * lane;
        float xt[4], xd[4];
        load4(trow, k0, V, vec, xt);
        if (use_resid) load4(drow, k0, V, vec, xd);
        double w[4], loc = 0.0;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const double pk = exp2((double)xt[u] * c - ref_p) * inv_zp;
            double wk = pk;
            if (use_resid) wk = fmax(pk - exp2((double)xd[u] * c - ref_q) * inv_zq, 0.0);
            w[u] = wk;
            loc += wk;
        }
        double inc = loc;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const double t = shfl_up_f64(inc, d);
            if (lane >= d) inc += t;
        }
        double run = base + inc - loc;
        int cand = -1, lp = -1;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            run += w[u];
            if (w[u] > 0.0) {
                lp = k0 + u;
                if (cand < 0 && run > target) cand = k0 + u;
            }
        }
        const unsigned hit = __ballot_sync(0xffffffffu, cand >= 0);
        if (hit != 0) y = __shfl_sync(0xffffffffu, cand, __ffs(hit) - 1);
        const unsigned pos = __ballot_sync(0xffffffffu, lp >= 0);
        if (pos != 0) last_pos = __shfl_sync(0xffffffffu, lp, 31 - __clz(pos));
        base = shfl_idx_f64(inc, 31) + base;
    }
    if (y < 0) {
        // target at or beyond the total mass: last token with positive weight
        if (last_pos < 0) {
            for (int s2 = n_seg - 1; s2 >= 0 && last_pos < 0; --s2) {
                const int k0 = s2 * SEG + 4 * lane;
                float xt[4], xd[4];
                load4(trow, k0, V, vec, xt);
                if (use_resid) load4(drow, k0, V, vec, xd);
                int lp = -1;
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const double pk = exp2((double)xt[u] * c - ref_p) * inv_zp;
                    double wk = pk;
                    if (use_resid) wk = fmax(pk - exp2((double)xd[u] * c - ref_q) * inv_zq, 0.0);
                    if (wk > 0.0) lp = k0 + u;
                }
                const unsigned pos = __ballot_sync(0xffffffffu, lp >= 0);
                if (pos != 0) last_pos = __shfl_sync(0xffffffffu, lp, 31 - __clz(pos));
            }
        }
        y = last_pos;
    }
    if (lane == 0) out[n] = y;
}

static int pick_slice(const sv_accept_params *p)
{
    // aim for at least ~4 blocks per SM worth of (row, slice) items, slices of 2K..16K elements
    const long long rows = (long long)p->batch * (2 * p->gamma_max + 1);
    const long long want = 4LL * sm_count();
    int slice = 16384;
    while (slice > MIN_SLICE && rows * ((p->vocab + slice - 1) / slice) < want) slice >>= 1;
    return slice;
}

}  // namespace sv

extern "C" size_t spec_accept_sample_workspace_bytes(int32_t batch, int32_t gamma_max, int32_t vocab)
{
    if (batch <= 0 || gamma_max < 0 || vocab <= 0) return 0;
    const size_t n_slices = ((size_t)vocab + sv::MIN_SLICE - 1) / sv::MIN_SLICE;
    return (size_t)batch * (2 * (size_t)gamma_max + 1) * n_slices * sizeof(sv::RowPartial);
}

extern "C" sv_status spec_accept_sample(const sv_accept_params *p, void *workspace,
                                        size_t workspace_bytes, void *stream)
{
    if (p == nullptr || p->batch <= 0 || p->vocab <= 0 || p->gamma_max < 0) return SV_EINVAL;
    if (p->gamma_max > 64) return SV_EUNSUPPORTED;
    if (p->target_logits == nullptr || p->gamma == nullptr || p->cu_q == nullptr ||
        p->cu_d == nullptr || p->n_accepted == nullptr || p->out_tokens == nullptr)
        return SV_EINVAL;
    const bool any_sampling = p->temperature_per_seq != nullptr || p->temperature > 0.f;
    if (any_sampling && (p->draft_logits == nullptr || p->u_accept == nullptr || p->u_sample == nullptr))
        return SV_EINVAL;
    if (p->gamma_max > 0 && p->draft_tokens == nullptr) return SV_EINVAL;
    if (p->row_stride < p->vocab) return SV_EINVAL;
    if (!(p->temperature >= 0.f)) return SV_EINVAL;
    if (workspace == nullptr ||
        workspace_bytes < spec_accept_sample_workspace_bytes(p->batch, p->gamma_max, p->vocab))
        return SV_EWORKSPACE;
    if (!sv::aligned16(workspace)) return SV_EALIGN;

    const int n_seg = (p->vocab + sv::SEG - 1) / sv::SEG;
    const size_t dyn = 3 * sizeof(double) * (size_t)n_seg;
    if (dyn > 200 * 1024) return SV_EUNSUPPORTED;

    sv::AcceptLaunch a;
    a.p = *p;
    a.partials = static_cast<sv::RowPartial *>(workspace);
    a.slice = sv::pick_slice(p);
    a.n_slices = (p->vocab + a.slice - 1) / a.slice;
    a.vec_ok = (p->row_stride % 4 == 0) && sv::aligned16(p->target_logits) &&
               (p->draft_logits == nullptr || sv::aligned16(p->draft_logits));

    const long long n_items = (long long)p->batch * (2 * p->gamma_max + 1) * a.n_slices;
    const long long cap = 8LL * sv::sm_count();
    const int grid = (int)(n_items < cap ? n_items : cap);
    sv::accept_rowstats_kernel<<<grid, sv::RS_THREADS, 0, (cudaStream_t)stream>>>(a);
    sv_status st = sv::launch_check();
    if (st != SV_OK) return st;

    if (dyn > 48 * 1024) {
        if (cudaFuncSetAttribute(sv::accept_finish_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)dyn) != cudaSuccess)
            return SV_ECUDA;
    }
    sv::accept_finish_kernel<<<p->batch, sv::FIN_THREADS, dyn, (cudaStream_t)stream>>>(a);
    return sv::launch_check();
}

// ---------------------------------------------------------------------------------------------
// Variant without caller-provided scratch.
// ---------------------------------------------------------------------------------------------
namespace sv {

// Slice statistics of one call live here instead of in a caller's workspace.  The array is part
// of the library image: every GPU that loads the library holds these bytes until the process
// exits.  All calls on a device share it.
static __device__ __align__(256) unsigned char g_accept_static_scratch[SV_ACCEPT_STATIC_SCRATCH_BYTES];

constexpr int MAX_DEVICES = 64;
static void *g_static_scratch_ptr[MAX_DEVICES];   // device address of the array, per device

}  // namespace sv

extern "C" sv_status spec_accept_sample_static(const sv_accept_params *p, void *stream)
{
    if (p == nullptr || p->batch <= 0 || p->vocab <= 0 || p->gamma_max < 0) return SV_EINVAL;
    if (p->gamma_max > 64) return SV_EUNSUPPORTED;
    if (p->target_logits == nullptr || p->gamma == nullptr || p->cu_q == nullptr ||
        p->cu_d == nullptr || p->n_accepted == nullptr || p->out_tokens == nullptr)
        return SV_EINVAL;
    const bool any_sampling = p->temperature_per_seq != nullptr || p->temperature > 0.f;
    if (any_sampling && (p->draft_logits == nullptr || p->u_accept == nullptr || p->u_sample == nullptr))
        return SV_EINVAL;
    if (p->gamma_max > 0 && p->draft_tokens == nullptr) return SV_EINVAL;
    if (p->row_stride < p->vocab) return SV_EINVAL;
    if (!(p->temperature >= 0.f)) return SV_EINVAL;
    const int n_seg = (p->vocab + sv::SEG - 1) / sv::SEG;
    const size_t dyn = 3 * sizeof(double) * (size_t)n_seg;
    if (dyn > 200 * 1024) return SV_EUNSUPPORTED;

    sv::AcceptLaunch a;
    a.p = *p;
    a.slice = sv::pick_slice(p);
    a.n_slices = (p->vocab + a.slice - 1) / a.slice;
    a.vec_ok = (p->row_stride % 4 == 0) && sv::aligned16(p->target_logits) &&
               (p->draft_logits == nullptr || sv::aligned16(p->draft_logits));
    const unsigned long long n_items =
        (unsigned long long)p->batch * (2ull * p->gamma_max + 1) * (unsigned long long)a.n_slices;
    // the problem must fit the built-in array: one 32-byte record per (row, slice)
    if (n_items * sizeof(sv::RowPartial) > (unsigned long long)SV_ACCEPT_STATIC_SCRATCH_BYTES)
        return SV_EWORKSPACE;

    // In host code the array's name is only a handle; its device address has to be asked for,
    // once per device, with that device current.
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= sv::MAX_DEVICES) return SV_ECUDA;
    if (sv::g_static_scratch_ptr[dev] == nullptr) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, sv::g_accept_static_scratch) != cudaSuccess || ptr == nullptr)
            return SV_ECUDA;
        sv::g_static_scratch_ptr[dev] = ptr;
    }
    a.partials = static_cast<sv::RowPartial *>(sv::g_static_scratch_ptr[dev]);

    const long long cap = 8LL * sv::sm_count();
    const int grid = (int)((long long)n_items < cap ? (long long)n_items : cap);
    sv::accept_rowstats_kernel<<<grid, sv::RS_THREADS, 0, (cudaStream_t)stream>>>(a);
    sv_status st = sv::launch_check();
    if (st != SV_OK) return st;
    if (dyn > 48 * 1024) {
        if (cudaFuncSetAttribute(sv::accept_finish_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)dyn) != cudaSuccess)
            return SV_ECUDA;
    }
    sv::accept_finish_kernel<<<p->batch, sv::FIN_THREADS, dyn, (cudaStream_t)stream>>>(a);
    return sv::launch_check();
}
