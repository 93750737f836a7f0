// Fused speculative-sampling acceptance over the vocabulary (paper Section 3).
//
// Three kernels per step, all on the caller's stream:
//
//  1. accept_rowstats_kernel -- the streaming pass and the only one that touches every
//     logit.  Each (row, slice of the vocabulary) item is owned by ONE WARP: 128-bit
//     streaming loads, six per lane in flight, a single-pass online softmax with a
//     power-of-two running reference (so every rescale is exact), float32 ex2.approx
//     exponentials summed four at a time into a float64 accumulator, and a warp-shuffle
//     reduction at the end.  No block-level synchronisation at all.  Greedy sequences
//     (T = 0) only track (max, lowest index) of their target rows.
//  2. accept_decide_kernel -- one block per sequence: its warps merge the slice statistics
//     into ln Z per row (float64, lanes over slices), then one warp evaluates ratio_i = min(1, p_i[x_i]/q_i[x_i]) against u_i in float64
//     for all positions in parallel, then takes the first rejection.
//  3. accept_sample_kernel -- several blocks per sequence: float64 pass over the one or two
//     rows the next token is drawn from (residual max(0, p_n - q_n) or the bonus row), sums
//     per 128-token segment, the sign of p_k - q_k decided with the first-pass partition
//     sums.  The block that finishes a sequence last runs the inverse CDF over the segment
//     sums and resolves the token exactly inside the chosen segment.
//
// (Letting the streaming kernel's warps take the decisions or the float64 pass as they
// become possible was measured and is slower: code that a warp runs once in a while is
// fetched through an instruction cache that the streaming loop owns, under a saturated
// memory system -- the decision alone then costs more than the whole kernel 2 and 3.)
#include "common.cuh"
#include "row_stream.cuh"

#include "row_sample.cuh"

#include <math_constants.h>

namespace sv {

constexpr int RS_THREADS = 256;   // rowstats block (8 independent warps)
constexpr int RS_UNROLL = 6;      // float4 loads in flight per lane: 61 registers, 32 warps per SM (4, 8, 12, 16 measured slower)
constexpr int CHUNK = 128;        // vocabulary elements a warp takes at a time (float4 per lane)
constexpr int SEG_SUB = 4;         // chunks per sampling segment: one reduction and one record per segment
constexpr int SEG = CHUNK * SEG_SUB;
constexpr int SEG_THREADS = 256;
constexpr int MAX_SPLITS = 64;    // blocks per sequence in the sampling kernel (small batches: enough blocks to fill the GPU)
constexpr int MIN_SLICE = 2048;
constexpr int MAX_SLICE = 16384;
constexpr int MAX_GAMMA = 64;
constexpr int MAX_DEVICES = 64;

struct __align__(16) RowPartial {
    double sum;     // sum of 2^(x*c - ref) over the slice
    float ref;      // integer-valued reference exponent
    float amax;     // greedy rows: largest logit of the slice
    int32_t aidx;   // ... and its lowest index
    int32_t bad;    // greedy rows: nonzero if the slice held a NaN (or +inf beside -inf)
};


struct AcceptLaunch {
    sv_accept_params p;
    RowPartial *partials;   // [batch * (2 gmax + 1) * n_slices]
    SeqRecord *records;     // [batch] written by the decision, read by the sampling kernel
    unsigned int *done;     // [batch] blocks of the sampling kernel that finished (cleared by the decision kernel)
    double *seg;            // [batch][3][n_seg]: positive-part sums of a, of b, all of a
    double *totals;         // [batch][MAX_SPLITS][2]
    int slice;              // elements per slice (multiple of 1024)
    int n_slices;
    int n_seg;
    int splits;
    int vec_ok;             // 128-bit loads legal for every row
    int row_per_seq;        // the sampling pass alone, on row b of target_logits for sequence b, token to out_tokens[b]
};

// shared scratch of the decision
struct DecideScratch {
    double logz[2 * MAX_GAMMA + 1];    // ln Z per dense row (natural log, of exp(x/T))
    double rsum[2 * MAX_GAMMA + 1];    // merged sum and reference of each dense row
    double ratio[MAX_GAMMA];
    float rref[2 * MAX_GAMMA + 1];
    int amax_idx[MAX_GAMMA + 1];
    unsigned char code[MAX_GAMMA];
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

__device__ __forceinline__ void merge_argmax(float &v, int &i, float v2, int i2)
{
    if (v2 > v || (v2 == v && i2 < i)) { v = v2; i = i2; }
}

// 2^(j/128), j = 0..127, correctly rounded
__device__ const double g_exp2_table[128] = {
    1.0, 1.0054299011128027, 1.0108892860517005, 1.016378314910953,
    1.0218971486541166, 1.0274459491187637, 1.0330248790212284, 1.0386341019613787,
    1.0442737824274138, 1.0499440858006872, 1.0556451783605572, 1.061377227289262,
    1.0671404006768237, 1.0729348675259756, 1.0787607977571199, 1.0846183622133092,
    1.0905077326652577, 1.0964290818163769, 1.102382583307841, 1.1083684117236787,
    1.1143867425958924, 1.1204377524096067, 1.1265216186082418, 1.1326385195987192,
    1.1387886347566916, 1.1449721444318042, 1.1511892299529827, 1.1574400736337511,
    1.1637248587775775, 1.1700437696832502, 1.1763969916502812, 1.182784710984341,
    1.189207115002721, 1.1956643920398273, 1.202156731452703, 1.2086843236265816,
    1.215247359980469, 1.2218460329727576, 1.22848053610687, 1.2351510639369334,
    1.241857812073484, 1.2486009771892048, 1.255380757024691, 1.2621973503942507,
    1.2690509571917332, 1.275941778396392, 1.2828700160787783, 1.2898358734066657,
    1.2968395546510096, 1.3038812651919358, 1.3109612115247644, 1.318079601266064,
    1.3252366431597413, 1.3324325470831615, 1.339667524053303, 1.3469417862329458,
    1.3542555469368927, 1.3616090206382248, 1.3690024229745905, 1.3764359707545302,
    1.383909881963832, 1.3914243757719262, 1.3989796725383112, 1.4065759938190154,
    1.4142135623730951, 1.4218926021691656, 1.42961333839197, 1.4373759974489824,
    1.4451808069770467, 1.4530279958490526, 1.460917794180647, 1.4688504333369818,
    1.4768261459394993, 1.4848451658727524, 1.4929077282912648, 1.5010140696264256,
    1.5091644275934228, 1.5173590411982147, 1.5255981507445384, 1.533881997840956,
    1.5422108254079407, 1.550584877685, 1.559004400237837, 1.567469639965553,
    1.5759808451078865, 1.5845382652524937, 1.593142151342267, 1.6017927556826934,
    1.6104903319492543, 1.6192351351948637, 1.6280274218573478, 1.6368674497669644,
    1.645755478153965, 1.6546917676561943, 1.6636765803267364, 1.6727101796415966,
    1.681792830507429, 1.6909247992693053, 1.7001063537185235, 1.709337763100463,
    1.718619298122478, 1.7279512309618377, 1.7373338352737062, 1.746767386199169,
    1.7562521603732995, 1.7657884359332727, 1.7753764925265212, 1.785016611318935,
    1.7947090750031072, 1.804454167806624, 1.8142521755003989, 1.8241033854070534,
    1.8340080864093424, 1.843966568958626, 1.8539791250833855, 1.864046048397789,
    1.8741676341103, 1.8843441790323345, 1.8945759815869656, 1.9048633418176741,
    1.9152065613971474, 1.925605943636125, 1.9360617934922943, 1.9465744175792332,
    1.9571441241754002, 1.9677712232331759, 1.978456026387951, 1.9891988469672663,
};

// 2^y in float64 for y <= ~4 (anything below -1000, -inf or NaN gives 0).  y is split into
// k/128 + r with k = rint(128 y): 2^y = 2^(k >> 7) * table[k & 127] * 2^r, |r| <= 1/256, 2^r by
// its degree-3 Taylor polynomial: the first dropped term is (r ln 2)^4 / 24 <= 2.2e-12, a relative
// error far below the 1e-9 window inside which a sampled token counts as a near tie, and common
// to numerator and denominator of every cumulative fraction.  The power of two goes straight
// into the exponent field.  N values at once, each step taken for all of them before the
// next, so that the N dependent chains overlap in the pipeline; no branches.  `tab` is a
// shared-memory copy of g_exp2_table.
template <int N>
__device__ __forceinline__ void exp2_f64_n(const double (&y)[N], double (&out)[N], const double *tab)
{
    constexpr double MAGIC = 6755399441055744.0;      // 1.5 * 2^52: adding it rounds to an integer
    double r[N], t[N], q[N];
    int k[N];
#pragma unroll
    for (int i = 0; i < N; ++i) {
        const double yc = (y[i] > -1000.0) ? y[i] : -1000.0;     // NaN and -inf take this branch too
        const double m = fma(yc, 128.0, MAGIC);
        k[i] = __double2loint(m);
        r[i] = fma(m - MAGIC, -0.0078125, yc);
        t[i] = tab[k[i] & 127];
        q[i] = 0.055504108664821576;                  // (ln 2)^3 / 6
    }
    constexpr double C[3] = {0.2402265069591007, 0.6931471805599453, 1.0};
#pragma unroll
    for (int c = 0; c < 3; ++c)
#pragma unroll
        for (int i = 0; i < N; ++i) q[i] = fma(q[i], r[i], C[c]);
#pragma unroll
    for (int i = 0; i < N; ++i) {
        const double v = q[i] * t[i];
        const double s = __hiloint2double(__double2hiint(v) + ((k[i] >> 7) << 20), __double2loint(v));
        out[i] = (y[i] > -1000.0) ? s : 0.0;
    }
}

// ---------------------------------------------------------------------------------------------
// Kernel 1: streaming row statistics, one warp per (row, slice).
// Dense row numbering: sequence b owns rows b*(2*gmax+1) + j; j <= gmax is target row j,
// j > gmax is draft row j-gmax-1.  Rows a sequence does not have this step are skipped.
// ---------------------------------------------------------------------------------------------
template <bool BF16>       // logits stored as bf16 bit patterns (widened exactly) instead of float32
__global__ void __launch_bounds__(RS_THREADS)
accept_rowstats_kernel(const __grid_constant__ AcceptLaunch a)
{
    pdl_enter();
    const sv_accept_params &p = a.p;
    const int rows_per_seq = 2 * p.gamma_max + 1;
    const long long n_items = (long long)p.batch * rows_per_seq * a.n_slices;
    const int lane = threadIdx.x & 31;
    const long long warp0 = (long long)blockIdx.x * (RS_THREADS / 32) + (threadIdx.x >> 5);
    const long long n_warps = (long long)gridDim.x * (RS_THREADS / 32);

    for (long long item = warp0; item < n_items; item += n_warps) {
        const int slice_id = (int)(item % a.n_slices);
        const int dense_row = (int)(item / a.n_slices);
        const int b = dense_row / rows_per_seq;
        const int j = dense_row % rows_per_seq;
        const int g = seq_gamma(p, b);
        const float T = seq_temperature(p, b);
        const bool greedy = !(T > 0.f);
        const void *row;
        if (j <= p.gamma_max) {
            if (j > g) continue;
            row = logit_row<BF16>(p.target_logits, p.cu_q[b] + j, p.row_stride);
        } else {
            const int i = j - p.gamma_max - 1;
            if (i >= g || greedy) continue;
            row = logit_row<BF16>(p.draft_logits, p.cu_d[b] + i, p.row_stride);
        }
        const int lo = slice_id * a.slice;
        const int hi = min(p.vocab, lo + a.slice);

        float ref = REF_INIT;
        double sum = 0.0;
        float amax = -CUDART_INF_F;
        int aidx = 0x7fffffff, bad = 0;

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
                const float s4 = (x0 + x1) + (x2 + x3);       // NaN if any of the four is (padding is -inf)
                if (!(s4 == s4)) bad = 1;
                if (x0 > amax) { amax = x0; aidx = k0; }
                if (x1 > amax) { amax = x1; aidx = k0 + 1; }
                if (x2 > amax) { amax = x2; aidx = k0 + 2; }
                if (x3 > amax) { amax = x3; aidx = k0 + 3; }
            } else {
                const float m4 = fmaxf(fmaxf(x0, x1), fmaxf(x2, x3));
                const float ymax = m4 * c_hi + 1.f;
                if (ymax > ref) {   // rare: the running reference has to grow
                    const float nr = ceilf(ymax);
                    sum = scale_down_pow2(sum, ref - nr);
                    ref = nr;
                }
                if (BF16) {
                    // With bf16 logits the pass is bound by instruction issue, not by memory: two logits
                    // per instruction (packed float32 pairs; each half rounds as the scalar form does).
                    // With float32 logits the scalar form measured slightly faster.
                    const float2 ch2 = make_float2(c_hi, c_hi), cl2 = make_float2(c_lo, c_lo), nr2 = make_float2(-ref, -ref);
                    const float2 xa = make_float2(x0, x2), xb = make_float2(x1, x3);
                    const float2 ya = __ffma2_rn(xa, cl2, __ffma2_rn(xa, ch2, nr2));
                    const float2 yb = __ffma2_rn(xb, cl2, __ffma2_rn(xb, ch2, nr2));
                    const float2 e = __fadd2_rn(make_float2(ex2_approx(ya.x), ex2_approx(ya.y)),
                                                make_float2(ex2_approx(yb.x), ex2_approx(yb.y)));    // (e0 + e1, e2 + e3)
                    sum += (double)(e.x + e.y);
                } else {
                    const float e0 = ex2_approx(fmaf(x0, c_lo, fmaf(x0, c_hi, -ref)));
                    const float e1 = ex2_approx(fmaf(x1, c_lo, fmaf(x1, c_hi, -ref)));
                    const float e2 = ex2_approx(fmaf(x2, c_lo, fmaf(x2, c_hi, -ref)));
                    const float e3 = ex2_approx(fmaf(x3, c_lo, fmaf(x3, c_hi, -ref)));
                    sum += (double)((e0 + e1) + (e2 + e3));
                }
            }
        };

        stream_slice<BF16, RS_UNROLL>(row, lo, hi, a.vec_ok != 0, lane, consume4);

        // warp reduction
        if (greedy) {
#pragma unroll
            for (int m = 16; m > 0; m >>= 1) {
                const float v2 = __shfl_xor_sync(0xffffffffu, amax, m);
                const int i2 = __shfl_xor_sync(0xffffffffu, aidx, m);
                merge_argmax(amax, aidx, v2, i2);
            }
            bad = __any_sync(0xffffffffu, bad != 0) ? 1 : 0;
        } else {
            float r = ref;
#pragma unroll
            for (int m = 16; m > 0; m >>= 1) r = fmaxf(r, __shfl_xor_sync(0xffffffffu, r, m));
            sum = warp_sum_f64(scale_down_pow2(sum, ref - r));
            ref = r;
        }
        if (lane == 0) {
            RowPartial out;
            out.sum = sum;
            out.ref = ref;
            out.amax = amax;
            out.aidx = aidx;
            out.bad = bad;
            a.partials[(long long)dense_row * a.n_slices + slice_id] = out;
        }
    }
}

// a slice record written by the streaming kernel
__device__ __forceinline__ RowPartial load_partial(const RowPartial *q)
{
    const int4 v = __ldcg(reinterpret_cast<const int4 *>(q));
    const int4 w = __ldcg(reinterpret_cast<const int4 *>(q) + 1);
    RowPartial r;
    r.sum = __hiloint2double(v.y, v.x);
    r.ref = __int_as_float(v.z);
    r.amax = __int_as_float(v.w);
    r.aidx = w.x;
    r.bad = w.y;
    return r;
}

// ---------------------------------------------------------------------------------------------
// Decision of one sequence (one block of DEC_THREADS): ln Z per row, ratios, first rejection; the
// record for the sampling kernel goes to *rec_out.  The slice statistics of the rows are merged
// by groups of lanes, one group per row, its lanes over the slices (a shuffle butterfly);
// warp 0 then evaluates the positions in parallel and lane 0 walks to the first rejection.
// ---------------------------------------------------------------------------------------------
constexpr int DEC_THREADS = 512;   // 16 warps: the rows of a sequence merged in one or two passes (128 threads: six at c3, +14 us)

template <bool BF16>
__device__ __forceinline__ void decide_seq(const AcceptLaunch &a, int b, DecideScratch *sc, int tid, SeqRecord *rec_out)
{
    constexpr bool write = true;
    const int lane = tid & 31, warp = tid >> 5;
    const sv_accept_params &p = a.p;
    const int gmax = p.gamma_max;
    const int rows_per_seq = 2 * gmax + 1;
    const int g = seq_gamma(p, b);
    const float Tf = seq_temperature(p, b);
    const bool greedy = !(Tf > 0.f);
    const double T = (double)Tf;
    const int V = p.vocab;
    const void *t_rows = logit_row<BF16>(p.target_logits, p.cu_q[b], p.row_stride);
    const void *d_rows = greedy ? nullptr : logit_row<BF16>(p.draft_logits, p.cu_d[b], p.row_stride);
    const int32_t *x = p.draft_tokens + p.cu_d[b];
    int32_t *out = p.out_tokens + (long long)b * (gmax + 1);

    // ---- merge the slice statistics of every row this sequence has: groups of `lpr` lanes (a
    // power of two covering the slices, at most a warp) take one row each
    int lpr = 1;
    while (lpr < 32 && lpr < a.n_slices) lpr <<= 1;
    const int rows_per_pass = (DEC_THREADS / 32) * (32 / lpr);
    const int sub = lane / lpr, sl = lane % lpr;
    for (int j0 = 0; j0 < rows_per_seq; j0 += rows_per_pass) {
        const int j = j0 + warp * (32 / lpr) + sub;
        const bool is_target = j <= gmax;
        const int i = is_target ? j : j - gmax - 1;
        const bool have = j < rows_per_seq && (is_target ? (i <= g) : (i < g && !greedy));
        const RowPartial *pp = a.partials + ((long long)b * rows_per_seq + j) * a.n_slices;
        float ref = REF_INIT, v = -CUDART_INF_F;
        double sum = 0.0;
        int ix = 0x7fffffff, bad = 0;
        if (have) {
            for (int s0 = sl; s0 < a.n_slices; s0 += lpr) {
                const RowPartial q = load_partial(pp + s0);
                if (greedy) { merge_argmax(v, ix, q.amax, q.aidx); bad |= q.bad; }
                else merge_stats(ref, sum, q.ref, q.sum);
            }
        }
        // rows that are absent ride along with neutral values: the shuffles need every lane
        if (greedy) {
            for (int m = lpr >> 1; m > 0; m >>= 1) {
                merge_argmax(v, ix, __shfl_xor_sync(0xffffffffu, v, m), __shfl_xor_sync(0xffffffffu, ix, m));
                bad |= __shfl_xor_sync(0xffffffffu, bad, m);
            }
            // a row with a NaN or +inf logit, or with nothing above -inf, has no argmax
            if (have && sl == 0) sc->amax_idx[i] = (bad != 0 || v == CUDART_INF_F) ? 0x7fffffff : ix;
        } else {
            for (int m = lpr >> 1; m > 0; m >>= 1)
                merge_stats(ref, sum, __shfl_xor_sync(0xffffffffu, ref, m), shfl_xor_f64(sum, m));
            if (have && sl == 0) {
                sc->rref[j] = ref;
                sc->rsum[j] = sum;
                // ln sum exp(x/T) = (ref + log2(sum)) * ln 2
                const double lz = ((double)ref + log2(sum)) * 0.6931471805599453;
                sc->logz[j] = lz;
                if (is_target) { if (write && p.logZ_p != nullptr) p.logZ_p[p.cu_q[b] + i] = lz; }
                else           { if (write && p.logZ_q != nullptr) p.logZ_q[p.cu_d[b] + i] = lz; }
            }
        }
    }
    __syncthreads();
    if (warp != 0) return;
    if (write)
        for (int i = lane; i <= gmax; i += 32) out[i] = -1;
    __syncwarp();

    // ---- ratio and decision of every draft position in parallel (float64) ...
    for (int i = lane; i < g; i += 32) {
        const int xi = x[i];
        double r = 0.0;
        int code;   // 0 reject, 1 accept, 2 non-finite partition function
        int flag = 0;
        if (xi < 0 || xi >= V) {
            if (write) set_status(p.device_status, SV_DEV_BAD_TOKEN);
            code = 0;
        } else if (greedy) {
            code = (sc->amax_idx[i] == 0x7fffffff) ? 2 : (sc->amax_idx[i] == xi) ? 1 : 0;
            r = (code == 1) ? 1.0 : 0.0;
        } else {
            const double lzp = sc->logz[i], lzq = sc->logz[gmax + 1 + i];
            if (!(isfinite(lzp) && isfinite(lzq))) {
                code = 2;
            } else {
                const double lp = (double)logit_at<BF16>(t_rows, (long long)i * p.row_stride + xi) / T - lzp;
                const double lq = (double)logit_at<BF16>(d_rows, (long long)i * p.row_stride + xi) / T - lzq;
                // ratio = min(1, p/q); q == 0 (a token the draft could not have produced) -> 1
                r = (lq == -CUDART_INF) ? 1.0 : exp(fmin(lp - lq, 0.0));
                const double u = (double)p.u_accept[p.cu_d[b] + i];
                code = (u < r) ? 1 : 0;
                flag = fabs(u - r) < 1e-6;
            }
        }
        sc->ratio[i] = r;
        sc->code[i] = (unsigned char)(code | (flag << 2));
    }
    __syncwarp();
    // ... then the first rejection, which is sequential by definition: one lane
    if (lane == 0) {
        int n = g, ok = 1;
        uint32_t flags = 0;
        for (int i = 0; i < g; ++i) {
            const int code = sc->code[i] & 3;
            if (code == 2) { ok = 0; n = i; break; }
            flags += (sc->code[i] >> 2) & 1;
            if (write && p.ratio != nullptr) p.ratio[p.cu_d[b] + i] = sc->ratio[i];
            if (code == 0) { n = i; break; }
        }
        if (write && p.ratio != nullptr)
            for (int i = n + 1; i < g; ++i) p.ratio[p.cu_d[b] + i] = CUDART_NAN;
        if (!greedy && ok && !isfinite(sc->logz[n])) ok = 0;
        if (greedy && ok && sc->amax_idx[n] == 0x7fffffff) ok = 0;
        if (write && !ok) set_status(p.device_status, SV_DEV_NONFINITE);
        if (write && flags != 0 && p.flag_count != nullptr) atomicAdd(p.flag_count, flags);
        if (write) p.n_accepted[b] = ok ? n : 0;
        if (write && ok) {
            for (int i = 0; i < n; ++i) out[i] = x[i];
            if (greedy) out[n] = sc->amax_idx[n];
        }
        SeqRecord rec;
        rec.n = n;
        rec.mode = (greedy || !ok) ? 0 : (n < g ? 1 : 2);
        rec.ref_p = rec.ref_q = 0.f;
        rec.sum_p_hat = rec.sum_q_hat = 1.0;
        if (rec.mode != 0) {
            rec.ref_p = sc->rref[n];
            rec.sum_p_hat = sc->rsum[n];
            if (rec.mode == 1) {
                rec.ref_q = sc->rref[gmax + 1 + n];
                rec.sum_q_hat = sc->rsum[gmax + 1 + n];
            }
        }
        *rec_out = rec;
    }
    __syncwarp();
}

// Kernel 2: one block per sequence takes the decision; it also clears the sequence's completion
// counter for kernel 3.
template <bool BF16>
__global__ void __launch_bounds__(DEC_THREADS)
accept_decide_kernel(const __grid_constant__ AcceptLaunch a)
{
    pdl_enter();
    __shared__ DecideScratch s_dec;
    const int b = blockIdx.x;
    if (threadIdx.x == 0) a.done[b] = 0u;
    decide_seq<BF16>(a, b, &s_dec, threadIdx.x, a.records + b);
}

// ---------------------------------------------------------------------------------------------
// Inverse CDF of one sequence (after all blocks of the sequence have stored their sums).  Called
// by the whole block: all threads bring the segments' normalised masses into shared memory at
// once (one round of loads instead of a warp's serial walk through global memory; this phase is
// exposed when the batch is small), then warp 0 finds the segment and the token.  Rows with
// more than PICK_SEGS segments are read in place.
// ---------------------------------------------------------------------------------------------
constexpr int PICK_SEGS = 2048;     // 2 x 16 KB of shared memory: vocabularies up to 262144

template <bool BF16>
__device__ __forceinline__ void pick_seq(const AcceptLaunch &a, int b, const SeqRecord &rec, int tid, const double *tab,
                                         double (*s_w)[PICK_SEGS])
{
    const int lane = tid & 31;
    const sv_accept_params &p = a.p;
    const bool residual = rec.mode == 1;
    const int V = p.vocab, n_seg = a.n_seg, n = rec.n;
    const double c = 1.4426950408889634 / (double)seq_temperature(p, b);
    const void *trow = logit_row<BF16>(p.target_logits, a.row_per_seq ? b : p.cu_q[b] + n, p.row_stride);
    const void *drow = residual ? logit_row<BF16>(p.draft_logits, p.cu_d[b] + n, p.row_stride) : nullptr;
    const bool vec = a.vec_ok != 0;
    const double ref_p = (double)rec.ref_p, ref_q = (double)rec.ref_q;
    const double *seg_ap = a.seg + (size_t)b * 3 * n_seg, *seg_bp = seg_ap + n_seg, *seg_a = seg_bp + n_seg;

    double Zp = 0.0, Zq = 0.0;
    for (int sp = 0; sp < a.splits; ++sp) {
        Zp += __ldcg(&a.totals[((size_t)b * MAX_SPLITS + sp) * 2]);
        Zq += __ldcg(&a.totals[((size_t)b * MAX_SPLITS + sp) * 2 + 1]);
    }
    const double inv_zp = 1.0 / Zp, inv_zq = residual ? 1.0 / Zq : 0.0;

    auto seg_w_global = [&](int s, bool use_r) {
        return use_r ? __ldcg(&seg_ap[s]) * inv_zp - __ldcg(&seg_bp[s]) * inv_zq : __ldcg(&seg_a[s]) * inv_zp;
    };
    const bool staged = n_seg <= PICK_SEGS;
    if (staged) {
        for (int s = tid; s < n_seg; s += SEG_THREADS) {
            s_w[0][s] = seg_w_global(s, false);
            if (residual) s_w[1][s] = seg_w_global(s, true);
        }
    }
    __syncthreads();
    if (tid >= 32) return;
    auto seg_w = [&](int s, bool use_r) { return staged ? s_w[use_r ? 1 : 0][s] : seg_w_global(s, use_r); };

    // total mass; lane l owns the contiguous segments [l*per, (l+1)*per)
    const int per = (n_seg + 31) / 32;
    const int s_lo = min(lane * per, n_seg), s_hi = min(s_lo + per, n_seg);
    double mine = 0.0;
    if (residual) for (int s = s_lo; s < s_hi; ++s) mine += seg_w(s, true);
    double W = warp_sum_f64(mine);
    const bool use_resid = residual && (W > 0.0);     // no residual mass: fall back to p_n
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
    int best = seg_found;
#pragma unroll
    for (int m = 16; m > 0; m >>= 1) best = min(best, __shfl_xor_sync(0xffffffffu, best, m));
    const unsigned who = __ballot_sync(0xffffffffu, seg_found == best && best < n_seg);
    double base = 0.0;
    if (who != 0) base = shfl_idx_f64(seg_base, __ffs(who) - 1);

    // exact float64 weights of four consecutive tokens
    auto weights4 = [&](int k0, double w[4]) {
        float xt[4], xd[4];
        logit_load4<BF16>(trow, k0, V, vec, xt);
        if (use_resid) logit_load4<BF16>(drow, k0, V, vec, xd);
        double y[8], e[8];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            y[u] = (double)xt[u] * c - ref_p;
            y[4 + u] = use_resid ? (double)xd[u] * c - ref_q : -2000.0;
        }
        exp2_f64_n<8>(y, e, tab);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const double pk = e[u] * inv_zp;
            w[u] = use_resid ? fmax(pk - e[4 + u] * inv_zq, 0.0) : pk;
        }
    };

    // resolve inside the segment; if rounding pushed the target past it, walk on; if nothing
    // qualifies, take the last positive weight.
    int y = -1, last_pos = -1;
    const int n_chunk = (V + CHUNK - 1) / CHUNK;
    int s = best * SEG_SUB;                      // from here on in chunks of 128 tokens
    if (best >= n_seg) { s = 0; base = 0.0; }    // target at or beyond the total: walk everything
    for (; s < n_chunk && y < 0; ++s) {
        const int k0 = s * CHUNK + 4 * lane;
        double w[4], loc = 0.0;
        weights4(k0, w);
#pragma unroll
        for (int u = 0; u < 4; ++u) loc += w[u];
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
        for (int s2 = n_chunk - 1; s2 >= 0 && last_pos < 0; --s2) {
            const int k0 = s2 * CHUNK + 4 * lane;
            double w[4];
            weights4(k0, w);
            int lp = -1;
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (w[u] > 0.0) lp = k0 + u;
            const unsigned pos = __ballot_sync(0xffffffffu, lp >= 0);
            if (pos != 0) last_pos = __shfl_sync(0xffffffffu, lp, 31 - __clz(pos));
        }
        y = last_pos;
    }
    if (lane == 0) p.out_tokens[a.row_per_seq ? (long long)b : (long long)b * (p.gamma_max + 1) + n] = y;
}

// ---------------------------------------------------------------------------------------------
// Kernel 3: float64 segment sums of the sampled row(s), inverse CDF.
// grid = batch * splits.
//   a_k = 2^(t_k c - ref_p), b_k = 2^(d_k c - ref_q), c = log2(e)/T
//   per segment: sum of a over {p_k > q_k}, sum of b over the same set, sum of all a
//   per block: sum of all a and all b (the exact partition sums, up to 2^ref)
// ---------------------------------------------------------------------------------------------
// Four blocks (32 warps) per SM: the pass is a mix of float64 arithmetic and shuffles that no
// pipe saturates, so throughput follows the number of resident warps; 64 registers suffice.
template <bool BF16>
__global__ void __launch_bounds__(SEG_THREADS, 4)
accept_sample_kernel(const __grid_constant__ AcceptLaunch a)
{
    pdl_enter();
    const sv_accept_params &p = a.p;
    __shared__ double s_tab[128];
    __shared__ double s_red[2 * (SEG_THREADS / 32)];
    __shared__ int s_last;
    __shared__ double s_w[2][PICK_SEGS];
    const int b = blockIdx.x / a.splits, sp = blockIdx.x % a.splits;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid >= 128) s_tab[tid - 128] = g_exp2_table[tid - 128];
    __syncthreads();
    const SeqRecord rec = a.records[b];
    if (rec.mode == 0) return;                        // greedy, or the sequence failed: nothing to sample
    const bool residual = rec.mode == 1;
    const int V = p.vocab, n_seg = a.n_seg;
    const double c = 1.4426950408889634 / (double)seq_temperature(p, b);
    const void *trow = logit_row<BF16>(p.target_logits, a.row_per_seq ? b : p.cu_q[b] + rec.n, p.row_stride);
    const void *drow = residual ? logit_row<BF16>(p.draft_logits, p.cu_d[b] + rec.n, p.row_stride) : nullptr;
    const bool vec = a.vec_ok != 0;
    const double ref_p = (double)rec.ref_p, ref_q = (double)rec.ref_q;
    // first-pass partition sums, good to ~1e-7: only used to decide the sign of p_k - q_k
    const double z_ratio = rec.sum_q_hat / rec.sum_p_hat;     // p_k > q_k  <=>  a_k * Zq > b_k * Zp
    double *seg_ap = a.seg + (size_t)b * 3 * n_seg, *seg_bp = seg_ap + n_seg, *seg_a = seg_bp + n_seg;

    const int per = (n_seg + a.splits - 1) / a.splits;
    const int s_begin = sp * per, s_end = min(n_seg, s_begin + per);
    double tot_a = 0.0, tot_b = 0.0;
    constexpr int NW = SEG_THREADS / 32;
    for (int s = s_begin + warp; s < s_end; s += NW) {
        {
            double sa = 0.0, sap = 0.0, sbp = 0.0, sb = 0.0;
#pragma unroll 1
            for (int sub = 0; sub < SEG_SUB; ++sub) {
                const int k0 = s * SEG + sub * CHUNK + 4 * lane;
                if (k0 - 4 * lane >= V) break;                   // past the vocabulary (last segment)
                float xt[4], xd[4];
                logit_load4<BF16>(trow, k0, V, vec, xt);
                if (residual) {
                    logit_load4<BF16>(drow, k0, V, vec, xd);
                    // the eight exponentials of this lane (four tokens, two rows) as overlapping chains
                    double y[8], w[8];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        y[u] = (double)xt[u] * c - ref_p;
                        y[4 + u] = (double)xd[u] * c - ref_q;
                    }
                    exp2_f64_n<8>(y, w, s_tab);
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const double ak = w[u], bk = w[4 + u];
                        sa += ak;
                        sb += bk;
                        if (ak * z_ratio > bk) { sap += ak; sbp += bk; }
                    }
                } else {
                    double y[4], w[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) y[u] = (double)xt[u] * c - ref_p;
                    exp2_f64_n<4>(y, w, s_tab);
#pragma unroll
                    for (int u = 0; u < 4; ++u) sa += w[u];
                }
            }
            tot_a += sa;
            tot_b += sb;
            if (residual) {
                // the three sums in one butterfly: after the first exchange the lower half-warp
                // carries (sa, sap) and the upper half sbp; after the second each quarter carries
                // one of them; the totals end in lanes 0, 8 and 16
                const bool up16 = (lane & 16) != 0, up8 = (lane & 8) != 0;
                double x0 = (up16 ? sbp : sa) + shfl_xor_f64(up16 ? sa : sbp, 16);
                double x1 = (up16 ? 0.0 : sap) + shfl_xor_f64(up16 ? sap : 0.0, 16);
                double y1 = (up8 ? x1 : x0) + shfl_xor_f64(up8 ? x0 : x1, 8);
                y1 += shfl_xor_f64(y1, 4);
                y1 += shfl_xor_f64(y1, 2);
                y1 += shfl_xor_f64(y1, 1);
                if (lane == 0) seg_a[s] = y1;
                if (lane == 8) seg_ap[s] = y1;
                if (lane == 16) seg_bp[s] = y1;
            } else {
                sa = warp_sum_f64(sa);
                if (lane == 0) { seg_a[s] = sa; seg_ap[s] = 0.0; seg_bp[s] = 0.0; }
            }
        }
    }
    tot_a = warp_sum_f64(tot_a);
    tot_b = warp_sum_f64(tot_b);
    if (lane == 0) { s_red[warp] = tot_a; s_red[NW + warp] = tot_b; }
    __syncthreads();          // also orders every warp's segment stores before the counter below
    if (tid == 0) {
        double za = 0.0, zb = 0.0;
        for (int w = 0; w < NW; ++w) { za += s_red[w]; zb += s_red[NW + w]; }
        a.totals[((size_t)b * MAX_SPLITS + sp) * 2] = za;
        a.totals[((size_t)b * MAX_SPLITS + sp) * 2 + 1] = zb;
        __threadfence();
        s_last = atomicAdd(&a.done[b], 1u) + 1 == (unsigned)a.splits;
    }
    __syncthreads();
    if (s_last) {             // the same for the whole block
        __threadfence();
        pick_seq<BF16>(a, b, rec, tid, s_tab, s_w);
    }
}

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
static int pick_slice(const sv_accept_params *p)
{
    // one warp per (row, slice): aim for a few items per resident warp, slices of 2K..16K elements
    const long long rows = (long long)p->batch * (2 * p->gamma_max + 1);
    const long long want = 4LL * sm_count() * 40;
    int slice = MAX_SLICE;
    while (slice > MIN_SLICE && rows * ((p->vocab + slice - 1) / slice) < want) slice >>= 1;
    return slice;
}

static size_t align256(size_t n) { return (n + 255) & ~(size_t)255; }

struct AcceptLayout {
    size_t partials, records, ctl, seg, totals, total;
};

static AcceptLayout accept_layout(int batch, int gamma_max, int vocab, int slice)
{
    AcceptLayout l;
    const size_t n_slices = ((size_t)vocab + slice - 1) / slice;
    const size_t n_seg = ((size_t)vocab + SEG - 1) / SEG;
    l.partials = 0;
    l.records = align256((size_t)batch * (2 * (size_t)gamma_max + 1) * n_slices * sizeof(RowPartial));
    l.ctl = l.records + align256((size_t)batch * sizeof(SeqRecord));
    l.seg = l.ctl + align256((size_t)batch * sizeof(unsigned int));
    l.totals = l.seg + align256((size_t)batch * 3 * n_seg * sizeof(double));
    l.total = l.totals + align256((size_t)batch * MAX_SPLITS * 2 * sizeof(double));
    return l;
}

static sv_status check_accept(const sv_accept_params *p)
{
    if (p == nullptr || p->batch <= 0 || p->vocab <= 0 || p->gamma_max < 0) return SV_EINVAL;
    if (p->gamma_max > MAX_GAMMA) return SV_EUNSUPPORTED;
    if (p->target_logits == nullptr || p->gamma == nullptr || p->cu_q == nullptr ||
        p->cu_d == nullptr || p->n_accepted == nullptr || p->out_tokens == nullptr)
        return SV_EINVAL;
    const bool any_sampling = p->temperature_per_seq != nullptr || p->temperature > 0.f;
    if (any_sampling && (p->draft_logits == nullptr || p->u_accept == nullptr || p->u_sample == nullptr))
        return SV_EINVAL;
    if (p->gamma_max > 0 && p->draft_tokens == nullptr) return SV_EINVAL;
    if (p->row_stride < p->vocab) return SV_EINVAL;
    if (!(p->temperature >= 0.f)) return SV_EINVAL;
    return SV_OK;
}

template <bool BF16>
static sv_status launch_kernels(const AcceptLaunch &a, int rs_grid, cudaStream_t stream)
{
    sv_status st = launch_kernel(false, accept_rowstats_kernel<BF16>, rs_grid, RS_THREADS, 0, stream, a);
    if (st != SV_OK) return st;
    st = launch_kernel(true, accept_decide_kernel<BF16>, a.p.batch, DEC_THREADS, 0, stream, a);
    if (st != SV_OK) return st;
    return launch_kernel(true, accept_sample_kernel<BF16>, (unsigned)(a.splits * a.p.batch), SEG_THREADS, 0, stream, a);
}

// the three launches; `scratch` holds accept_layout(..., slice).total bytes
static sv_status launch_accept(const sv_accept_params *p, void *scratch, int slice, cudaStream_t stream)
{
    const AcceptLayout l = accept_layout(p->batch, p->gamma_max, p->vocab, slice);
    uint8_t *base = static_cast<uint8_t *>(scratch);
    AcceptLaunch a;
    a.p = *p;
    a.partials = reinterpret_cast<RowPartial *>(base + l.partials);
    a.records = reinterpret_cast<SeqRecord *>(base + l.records);
    a.done = reinterpret_cast<unsigned int *>(base + l.ctl);
    a.seg = reinterpret_cast<double *>(base + l.seg);
    a.totals = reinterpret_cast<double *>(base + l.totals);
    a.slice = slice;
    a.n_slices = (p->vocab + slice - 1) / slice;
    a.n_seg = (p->vocab + SEG - 1) / SEG;
    const bool bf16 = p->logits_bf16 != 0;
    a.vec_ok = logits_vec_ok(p->target_logits, p->row_stride, bf16) && logits_vec_ok(p->draft_logits, p->row_stride, bf16);
    // blocks per sequence in the sampling kernel: the float64 pass is bound by arithmetic, so
    // several small blocks per SM balance better than one wave of large ones -- two full waves
    // of the four blocks an SM holds (4, 10, 13, 16 blocks per sequence measured slower than 9
    // at batch 128); at least 8 segments per block; one block when nothing samples
    const bool any_sampling = p->temperature_per_seq != nullptr || p->temperature > 0.f;
    int splits = (2 * 4 * sm_count()) / p->batch;
    if (splits > MAX_SPLITS) splits = MAX_SPLITS;
    if (splits > (a.n_seg + 7) / 8) splits = (a.n_seg + 7) / 8;
    if (splits < 1 || !any_sampling) splits = 1;
    a.splits = splits;
    a.row_per_seq = 0;

    const long long n_items = (long long)p->batch * (2 * p->gamma_max + 1) * a.n_slices;
    const long long blocks_needed = (n_items + RS_THREADS / 32 - 1) / (RS_THREADS / 32);
    static int blocks_per_sm_of[MAX_DEVICES][2];   // resident blocks per SM, asked once per device and logit type
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return SV_ECUDA;
    if (blocks_per_sm_of[dev][bf16] == 0) {
        int n = 0;
        const cudaError_t e = bf16 ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, accept_rowstats_kernel<true>, RS_THREADS, 0)
                                   : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, accept_rowstats_kernel<false>, RS_THREADS, 0);
        if (e != cudaSuccess || n < 1) n = 2;
        blocks_per_sm_of[dev][bf16] = n;
    }
    const long long cap = (long long)blocks_per_sm_of[dev][bf16] * sm_count();
    const int rs_grid = (int)(blocks_needed < cap ? blocks_needed : cap);
    return bf16 ? launch_kernels<true>(a, rs_grid, stream) : launch_kernels<false>(a, rs_grid, stream);
}

// ---------------------------------------------------------------------------------------------
// The sampling pass alone (row_sample.cuh): one row per sequence, records prepared by the caller's kernel.
// ---------------------------------------------------------------------------------------------
static int row_sample_splits(int batch, int n_seg)
{
    int splits = (2 * 4 * sm_count()) / batch;
    if (splits > MAX_SPLITS) splits = MAX_SPLITS;
    if (splits > (n_seg + 7) / 8) splits = (n_seg + 7) / 8;
    return splits < 1 ? 1 : splits;
}

size_t row_sample_scratch_bytes(int batch, int vocab)
{
    const size_t n_seg = ((size_t)vocab + SEG - 1) / SEG;
    return align256((size_t)batch * 3 * n_seg * sizeof(double)) + align256((size_t)batch * MAX_SPLITS * 2 * sizeof(double));
}

sv_status launch_row_sample(const RowSampleArgs &r, cudaStream_t stream)
{
    AcceptLaunch a;
    memset(&a, 0, sizeof(a));
    a.p.target_logits = static_cast<const float *>(r.logits);
    a.p.logits_bf16 = r.logits_bf16;
    a.p.row_stride = r.row_stride;
    a.p.vocab = r.vocab;
    a.p.batch = r.batch;
    a.p.temperature = r.temperature;
    a.p.temperature_per_seq = r.temperature_per_seq;
    a.p.u_sample = r.u_sample;
    a.p.out_tokens = r.out_tokens;
    a.p.device_status = r.device_status;
    a.records = const_cast<SeqRecord *>(r.records);
    a.done = r.done;
    a.n_seg = (r.vocab + SEG - 1) / SEG;
    a.seg = static_cast<double *>(r.scratch);
    a.totals = reinterpret_cast<double *>(static_cast<uint8_t *>(r.scratch) +
                                          align256((size_t)r.batch * 3 * a.n_seg * sizeof(double)));
    a.splits = row_sample_splits(r.batch, a.n_seg);
    a.vec_ok = logits_vec_ok(r.logits, r.row_stride, r.logits_bf16 != 0);
    a.row_per_seq = 1;
    const unsigned grid = (unsigned)(a.splits * r.batch);
    return r.logits_bf16 ? launch_kernel(true, accept_sample_kernel<true>, grid, SEG_THREADS, 0, stream, a)
                         : launch_kernel(true, accept_sample_kernel<false>, grid, SEG_THREADS, 0, stream, a);
}

}  // namespace sv

extern "C" size_t spec_accept_sample_workspace_bytes(int32_t batch, int32_t gamma_max, int32_t vocab)
{
    if (batch <= 0 || gamma_max < 0 || vocab <= 0) return 0;
    return sv::accept_layout(batch, gamma_max, vocab, sv::MIN_SLICE).total;
}

extern "C" sv_status spec_accept_sample(const sv_accept_params *p, void *workspace,
                                        size_t workspace_bytes, void *stream)
{
    sv_status st = sv::check_accept(p);
    if (st != SV_OK) return st;
    if (workspace == nullptr ||
        workspace_bytes < spec_accept_sample_workspace_bytes(p->batch, p->gamma_max, p->vocab))
        return SV_EWORKSPACE;
    if (!sv::aligned16(workspace)) return SV_EALIGN;
    return sv::launch_accept(p, workspace, sv::pick_slice(p), (cudaStream_t)stream);
}

// ---------------------------------------------------------------------------------------------
// Variant without caller-provided scratch.
// ---------------------------------------------------------------------------------------------
namespace sv {

// The intermediate results of one call live here instead of in a caller's workspace.  The array
// is part of the library image: every GPU that loads the library holds these bytes until the
// process exits.  All calls on a device share it.
static __device__ __align__(256) unsigned char g_accept_static_scratch[SV_ACCEPT_STATIC_SCRATCH_BYTES];

static void *g_static_scratch_ptr[MAX_DEVICES];   // device address of the array, per device

}  // namespace sv

extern "C" sv_status spec_accept_sample_static(const sv_accept_params *p, void *stream)
{
    sv_status st = sv::check_accept(p);
    if (st != SV_OK) return st;
    // the problem must fit the built-in array
    const int slice = sv::pick_slice(p);
    if (sv::accept_layout(p->batch, p->gamma_max, p->vocab, slice).total >
        (size_t)SV_ACCEPT_STATIC_SCRATCH_BYTES)
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
    return sv::launch_accept(p, sv::g_static_scratch_ptr[dev], slice, (cudaStream_t)stream);
}
