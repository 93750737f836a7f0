/*
 * Float64 CPU oracle for the speculative-decoding verify step
 * (appending the draft block to the paged cache, attention of the draft block,
 * accept / resample, GammaTune controller, GammaTune+ early stop of drafting).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
 * CUDA library is checked against.  It shares no code with the CUDA path and
 * must never be called from it; only the tests, the smoke check and the
 * benchmark's CPU-baseline leg may load it.
 *
 * Every routine is written as the definition (attention) or as the steps of
 * the procedure in the order the paper and the speculative-sampling rule state
 * them (accept / resample, Algorithm 1): no blocking, no fusion, no
 * reordering.  The only parallelism is an OpenMP loop over independent
 * sequences / query rows, which does not change any arithmetic.
 *
 * Compile with -ffp-contract=off so that (1-eta)*gbar + eta*A is two
 * multiplications and one addition, each rounded once (IEEE binary64).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------- */
/* bf16 storage format: the upper 16 bits of an IEEE binary32 value.          */
static double bf16_bits_to_f64(uint16_t h)
{
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* =========================================================================
 * 1. Attention of the draft block against the paged KV cache.
 *
 * Paper, Section 3 ("Background"): the target model verifies the gamma drafted
 * tokens in one parallel forward; with KV caching (Section 5) the part of that
 * forward that grows with context is causal softmax attention of the
 * gamma+1 new positions against the cache.  This is the textbook definition:
 *
 *   s_j = scale * sum_d q[d] k_j[d]          j = 0 .. n_keys-1
 *   m   = max_j s_j ;  Z = sum_j exp(s_j - m)
 *   o[d] = sum_j exp(s_j - m) v_j[d] / Z ;   lse = m + ln Z
 *
 * KV token j of a sequence lives in physical page block_table[j / page_size],
 * slot j % page_size.  kv_strides = element strides of the pool for
 * (page, kv head, slot, dim).
 * ========================================================================= */
void oracle_attn_row(const uint16_t *q_row, const uint16_t *k_pool, const uint16_t *v_pool,
                     const int64_t *kv_strides, const int32_t *block_table_row, int page_size,
                     int kv_head, int head_dim, int n_keys, double scale, double *o, double *lse)
{
    double *s = (double *)malloc(sizeof(double) * (size_t)(n_keys > 0 ? n_keys : 1));
    double m = -INFINITY;
    for (int j = 0; j < n_keys; ++j) {
        int64_t page = block_table_row[j / page_size];
        int64_t slot = j % page_size;
        const uint16_t *k = k_pool + page * kv_strides[0] + (int64_t)kv_head * kv_strides[1] +
                            slot * kv_strides[2];
        double dot = 0.0;
        for (int d = 0; d < head_dim; ++d)
            dot += bf16_bits_to_f64(q_row[d]) * bf16_bits_to_f64(k[(int64_t)d * kv_strides[3]]);
        s[j] = dot * scale;
        if (s[j] > m) m = s[j];
    }
    double Z = 0.0;
    for (int d = 0; d < head_dim; ++d) o[d] = 0.0;
    for (int j = 0; j < n_keys; ++j) {
        int64_t page = block_table_row[j / page_size];
        int64_t slot = j % page_size;
        const uint16_t *v = v_pool + page * kv_strides[0] + (int64_t)kv_head * kv_strides[1] +
                            slot * kv_strides[2];
        double e = exp(s[j] - m);
        Z += e;
        for (int d = 0; d < head_dim; ++d)
            o[d] += e * bf16_bits_to_f64(v[(int64_t)d * kv_strides[3]]);
    }
    for (int d = 0; d < head_dim; ++d) o[d] /= Z;
    if (lse) *lse = m + log(Z);
    free(s);
}

/*
 * All rows of a ragged batch.  Sequence b has gamma[b]+1 query rows, stored at
 * rows cu_q[b] .. cu_q[b+1]-1 of q [sum R, hq, head_dim]; they are the LAST
 * gamma[b]+1 positions of the sequence (seq_len[b] counts them), so row i sees
 * keys 0 .. seq_len[b]-(gamma[b]+1)+i inclusive.  Query head h reads kv head
 * h / (hq / hkv).
 */
void oracle_verify_attn(const uint16_t *q, const uint16_t *k_pool, const uint16_t *v_pool,
                        const int64_t *kv_strides, const int32_t *block_table,
                        int64_t block_table_stride, const int32_t *seq_len, const int32_t *gamma,
                        const int32_t *cu_q, int batch, int hq, int hkv, int head_dim,
                        int page_size, double scale, double *o, double *lse)
{
    int group = hq / hkv;
    for (int b = 0; b < batch; ++b) {
        int R = gamma[b] + 1;
        int L = seq_len[b];
        int64_t n_items = (int64_t)R * hq;
#pragma omp parallel for schedule(dynamic, 1)
        for (int64_t it = 0; it < n_items; ++it) {
            int i = (int)(it / hq);
            int h = (int)(it % hq);
            int pos = L - R + i;
            int64_t row = (int64_t)cu_q[b] + i;
            oracle_attn_row(q + (row * hq + h) * head_dim, k_pool, v_pool, kv_strides,
                            block_table + (int64_t)b * block_table_stride, page_size, h / group,
                            head_dim, pos + 1, scale, o + (row * hq + h) * head_dim,
                            lse ? lse + row * hq + h : NULL);
        }
    }
}

/* -------------------------------------------------------------------------
 * 1b. Appending the draft block to the cache (KV caching, paper Section 5,
 *     experimental setup).  Before the verify attention runs, the keys and
 *     values of the gamma[b]+1 new positions are written behind the context:
 *     new row i of sequence b is token  pos = seq_len[b] - (gamma[b]+1) + i
 *     (seq_len already counts the block), which lives in physical page
 *     block_table[b][pos / page_size], slot pos % page_size.  A plain copy of
 *     bf16 bit patterns; every other element of the pools is left alone.
 *     k_new, v_new: [sum R, hkv, head_dim].
 * ------------------------------------------------------------------------- */
void oracle_kv_append(const uint16_t *k_new, const uint16_t *v_new, uint16_t *k_pool, uint16_t *v_pool,
                      const int64_t *kv_strides, const int32_t *block_table, int64_t block_table_stride,
                      const int32_t *seq_len, const int32_t *gamma, const int32_t *cu_q, int batch,
                      int hkv, int head_dim, int page_size)
{
    for (int b = 0; b < batch; ++b) {
        int R = gamma[b] + 1;
        for (int i = 0; i < R; ++i) {
            int pos = seq_len[b] - R + i;
            int64_t page = block_table[(int64_t)b * block_table_stride + pos / page_size];
            int64_t slot = pos % page_size;
            for (int g = 0; g < hkv; ++g) {
                int64_t dst = page * kv_strides[0] + (int64_t)g * kv_strides[1] + slot * kv_strides[2];
                int64_t src = (((int64_t)cu_q[b] + i) * hkv + g) * head_dim;
                for (int d = 0; d < head_dim; ++d) {
                    k_pool[dst + (int64_t)d * kv_strides[3]] = k_new[src + d];
                    v_pool[dst + (int64_t)d * kv_strides[3]] = v_new[src + d];
                }
            }
        }
    }
}

/* =========================================================================
 * 2. Accept / resample (speculative sampling, paper Section 3, first
 *    paragraph, by reference to Leviathan et al. and Chen et al.).
 * ========================================================================= */

/* softmax of x/T in float64: p_k = exp(x_k/T - m) / sum_j exp(x_j/T - m).
 * Returns ln sum_j exp(x_j / T). */
static double softmax_f64(const float *x, int V, double T, double *p)
{
    double m = -INFINITY;
    for (int k = 0; k < V; ++k) {
        double z = (double)x[k] / T;
        if (z > m) m = z;
    }
    double Z = 0.0;
    for (int k = 0; k < V; ++k) {
        p[k] = exp((double)x[k] / T - m);
        Z += p[k];
    }
    for (int k = 0; k < V; ++k) p[k] /= Z;
    return m + log(Z);
}

/* index of the largest element, lowest index on ties */
static int argmax_lowest(const float *x, int V)
{
    int best = 0;
    for (int k = 1; k < V; ++k)
        if (x[k] > x[best]) best = k;
    return best;
}

/*
 * Inverse CDF in vocabulary order: smallest k with sum_{j<=k} w_j > u * W,
 * W = sum_j w_j.  Zero-weight tokens are never chosen; if rounding leaves no
 * such k the last token with positive weight is taken.
 * Near-edge report: if u*W lies within tol*W of the lower (upper) CDF edge of
 * the chosen token, *alt is the previous (next) token with positive weight
 * and *flag is set; both tokens are then legal answers for a float32 device.
 */
static int inv_cdf(const double *w, int V, double u, double tol, int *alt, uint8_t *flag)
{
    double W = 0.0;
    for (int k = 0; k < V; ++k) W += w[k];
    double target = u * W;
    double c = 0.0, lower = 0.0, upper = 0.0;
    int y = -1;
    for (int k = 0; k < V; ++k) {
        double c_next = c + w[k];
        if (w[k] > 0.0 && c_next > target) {
            y = k;
            lower = c;
            upper = c_next;
            break;
        }
        c = c_next;
    }
    if (y < 0) {
        for (int k = V - 1; k >= 0; --k)
            if (w[k] > 0.0) { y = k; break; }
        lower = W - (y >= 0 ? w[y] : 0.0);
        upper = W;
    }
    *alt = -1;
    *flag = 0;
    if (y >= 0) {
        if (target - lower < tol * W) {
            for (int k = y - 1; k >= 0; --k)
                if (w[k] > 0.0) { *alt = k; *flag = 1; break; }
        } else if (upper - target < tol * W) {
            for (int k = y + 1; k < V; ++k)
                if (w[k] > 0.0) { *alt = k; *flag = 1; break; }
        }
    }
    return y;
}

/*
 * One verify step for a ragged batch.
 *
 * Row layout: sequence b owns target rows cu_q[b] .. cu_q[b]+gamma[b]
 * (row i is the target distribution for draft position i; row gamma[b] is the
 * bonus position) and draft rows / tokens / uniforms cu_d[b] .. cu_d[b]+gamma[b]-1.
 *
 * T > 0, for i = 0 .. gamma-1 in order:
 *     p_i = softmax(t_i / T), q_i = softmax(d_i / T)
 *     ratio_i = min(1, p_i[x_i] / q_i[x_i])            (1 if q_i[x_i] == 0)
 *     accept iff u_i < ratio_i ; the first rejection ends the scan: n = i
 *   n < gamma : next token ~ normalise(max(0, p_n - q_n))   (p_n if that mass is 0)
 *   n = gamma : next token ~ p_gamma                         (bonus token)
 *   both by inverse CDF with u_sample[b].
 * T == 0: n = first i with argmax(t_i) != x_i, next token = argmax(t_n).
 *
 * force (nullable, one per draft position): -1 = decide by the rule,
 * 0 / 1 = take this decision instead.  A comparison harness uses it to follow
 * the device through a position the oracle itself reports as a near tie.
 *
 * Outputs: n_accepted[b] (accepted draft tokens, 0..gamma, the extra token not
 * counted); out_tokens[b, 0..n-1] = accepted drafts, [n] = next token, rest -1;
 * ratio / accept_flag per draft position (NaN / 0 where the scan never got);
 * logZ_p per target row, logZ_q per draft row (ln sum exp(x/T); NaN if T == 0);
 * alt_token / sample_flag / resid_mass per sequence.
 */
void oracle_accept_sample(const float *target_logits, const float *draft_logits, int64_t row_stride,
                          int V, const int32_t *draft_tokens, const float *u_accept,
                          const float *u_sample, const float *temperature, const int32_t *gamma,
                          const int32_t *cu_q, const int32_t *cu_d, int batch, int gamma_max,
                          const int8_t *force, double accept_tol, double sample_tol,
                          int32_t *n_accepted, int32_t *out_tokens, double *ratio, double *logZ_p,
                          double *logZ_q, uint8_t *accept_flag, int32_t *alt_token,
                          uint8_t *sample_flag, double *resid_mass)
{
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < batch; ++b) {
        int g = gamma[b];
        double T = (double)temperature[b];
        const float *t_rows = target_logits + (int64_t)cu_q[b] * row_stride;
        const float *d_rows = draft_logits + (int64_t)cu_d[b] * row_stride;
        const int32_t *x = draft_tokens + cu_d[b];
        int32_t *out = out_tokens + (int64_t)b * (gamma_max + 1);
        for (int i = 0; i <= gamma_max; ++i) out[i] = -1;
        for (int i = 0; i < g; ++i) {
            ratio[cu_d[b] + i] = NAN;
            accept_flag[cu_d[b] + i] = 0;
            logZ_q[cu_d[b] + i] = NAN;
        }
        for (int i = 0; i <= g; ++i) logZ_p[cu_q[b] + i] = NAN;
        alt_token[b] = -1;
        sample_flag[b] = 0;
        resid_mass[b] = NAN;

        int n = g;
        int y;
        if (T == 0.0) {
            for (int i = 0; i < g; ++i) {
                int top = argmax_lowest(t_rows + (int64_t)i * row_stride, V);
                int ok = (top == x[i]);
                if (force && force[cu_d[b] + i] >= 0) ok = force[cu_d[b] + i];
                if (!ok) { n = i; break; }
            }
            y = argmax_lowest(t_rows + (int64_t)n * row_stride, V);
        } else {
            double *p = (double *)malloc(sizeof(double) * (size_t)V);
            double *q = (double *)malloc(sizeof(double) * (size_t)V);
            double *w = (double *)malloc(sizeof(double) * (size_t)V);
            for (int i = 0; i < g; ++i) {
                logZ_p[cu_q[b] + i] = softmax_f64(t_rows + (int64_t)i * row_stride, V, T, p);
                logZ_q[cu_d[b] + i] = softmax_f64(d_rows + (int64_t)i * row_stride, V, T, q);
                double r = 1.0;
                if (q[x[i]] > 0.0) {
                    r = p[x[i]] / q[x[i]];
                    if (r > 1.0) r = 1.0;
                }
                double u = (double)u_accept[cu_d[b] + i];
                ratio[cu_d[b] + i] = r;
                accept_flag[cu_d[b] + i] = (fabs(u - r) < accept_tol) ? 1 : 0;
                int ok = (u < r);
                if (force && force[cu_d[b] + i] >= 0) ok = force[cu_d[b] + i];
                if (!ok) { n = i; break; }
            }
            /* p, q still hold rows n when the scan stopped at a rejection */
            if (n < g) {
                double W = 0.0;
                for (int k = 0; k < V; ++k) {
                    w[k] = p[k] - q[k];
                    if (w[k] < 0.0) w[k] = 0.0;
                    W += w[k];
                }
                resid_mass[b] = W;
                if (!(W > 0.0))
                    for (int k = 0; k < V; ++k) w[k] = p[k];
            } else {
                logZ_p[cu_q[b] + g] = softmax_f64(t_rows + (int64_t)g * row_stride, V, T, w);
            }
            int alt;
            uint8_t fl;
            y = inv_cdf(w, V, (double)u_sample[b], sample_tol, &alt, &fl);
            alt_token[b] = alt;
            sample_flag[b] = fl;
            free(p);
            free(q);
            free(w);
        }
        n_accepted[b] = n;
        for (int i = 0; i < n; ++i) out[i] = x[i];
        out[n] = y;
    }
}

/* =========================================================================
 * 3. GammaTune controller, paper Section 4.1, Algorithm 1, per sequence.
 *
 *   mode 1 (reading "proposed"): the expansion rule of Eq. 7 raises the
 *       acceptance count that feeds the moving average, as the prose of the
 *       "Adaptive Expansion" paragraph says:
 *           A' = A + delta  if A == gamma  else A
 *           gbar <- min(gmax, max(gmin, (1-eta)*gbar + eta*A'))      (Eq. 8)
 *           gamma <- ceil(gbar)
 *   mode 2 (reading "literal"): Algorithm 1 exactly as printed, where the
 *       assignment gamma <- A + delta is overwritten by the last line, so
 *       the average is fed A itself.
 *   mode 0: fixed gamma (plain speculative decoding); state is left alone.
 *
 * Bookkeeping around it (implied by KV caching): the block just verified had
 * gamma+1 positions appended; A+1 of them stay; the next block appends
 * gamma_next+1:  seq_len <- seq_len - (gamma+1) + (A+1) + (gamma_next+1).
 * cu_q / cu_d are rebuilt as prefix sums of gamma_next+1 / gamma_next (packed
 * rows), or as b*(gamma_max+1) / b*gamma_max when padded_rows is set (every
 * sequence owns a fixed slab of rows, of which it uses the first gamma+1).
 * ========================================================================= */
void oracle_gamma_tune_update(const int32_t *n_accepted, double *gamma_bar, int32_t *gamma,
                              int32_t *seq_len, int32_t *cu_q, int32_t *cu_d, int batch,
                              double eta, double delta, int gamma_min, int gamma_max, int mode,
                              int padded_rows, const int32_t *n_drafted)
{
    /* n_drafted (GammaTune+, Section 4.2; NULL for plain GammaTune): the draft stopped after
     * n_drafted[b] <= gamma[b] tokens, so that many rows (+1) were appended to the cache; the
     * comparison "A = gamma" still uses the gamma the controller issued. */
    cu_q[0] = 0;
    cu_d[0] = 0;
    for (int b = 0; b < batch; ++b) {
        int A = n_accepted[b];
        int g_old = gamma[b];
        int rows_old = (n_drafted != NULL ? n_drafted[b] : g_old) + 1;
        int g_new = g_old;
        if (mode == 1 || mode == 2) {
            double a_eff = (double)A;
            if (A == g_old) {
                if (mode == 1) a_eff = (double)A + delta;
                /* mode 2: gamma <- A + delta here, but it is overwritten below */
            }
            double t1 = (1.0 - eta) * gamma_bar[b];
            double t2 = eta * a_eff;
            double s = t1 + t2;
            if (s < (double)gamma_min) s = (double)gamma_min;
            if (s > (double)gamma_max) s = (double)gamma_max;
            gamma_bar[b] = s;
            g_new = (int)ceil(s);
        }
        gamma[b] = g_new;
        seq_len[b] = seq_len[b] - rows_old + (A + 1) + (g_new + 1);
        cu_q[b + 1] = padded_rows ? (b + 1) * (gamma_max + 1) : cu_q[b] + g_new + 1;
        cu_d[b + 1] = padded_rows ? (b + 1) * gamma_max : cu_d[b] + g_new;
    }
}

/*
 * GammaTune+ (Section 4.2): confidence-guided early stop of drafting.  The draft's confidence
 * at position i is its top probability c_i = max_k softmax(d_i / T)_k.  The paper only says
 * that drafting stops when it falls below tau; the reading taken here: the token drafted at
 * the first such position is still part of the block, nothing is drafted after it, so
 *     n_drafted = min(gamma, 1 + first i with c_i < tau)      (gamma if there is none).
 * T = 0 (greedy draft): c_i = 1, never below tau <= 1.
 * flag[row] = 1 when |c_i - tau| < tol (either decision is legal there).
 */
void oracle_draft_stop(const float *draft_logits, int64_t row_stride, int vocab, const float *temperature,
                       double tau, const int32_t *gamma, const int32_t *cu_d, int batch, double tol,
                       int32_t *n_drafted, double *top_prob, uint8_t *flag)
{
    for (int b = 0; b < batch; ++b) {
        const int g = gamma[b];
        const double T = (double)temperature[b];
        int n = g;
        for (int i = 0; i < g; ++i) {
            const float *d = draft_logits + (int64_t)(cu_d[b] + i) * row_stride;
            double c = 1.0;
            if (T > 0.0) {
                double m = -INFINITY;
                for (int k = 0; k < vocab; ++k)
                    if ((double)d[k] > m) m = (double)d[k];
                double z = 0.0;
                for (int k = 0; k < vocab; ++k) z += exp(((double)d[k] - m) / T);
                c = 1.0 / z;
            }
            top_prob[cu_d[b] + i] = c;
            flag[cu_d[b] + i] = fabs(c - tau) < tol ? 1 : 0;
            if (n == g && c < tau) n = i + 1 < g ? i + 1 : g;
        }
        n_drafted[b] = n;
    }
}

/*
 * One drafting step with the confidence stop (paper Section 4.2: the draft model's top
 * probability is looked at while it drafts, and drafting ends once it falls below tau).
 *
 * Row b of draft_logits holds sequence b's draft logits for its next position.  For every
 * sequence with active[b] != 0 (and n_drafted[b] < gamma[b]):
 *     q = softmax(d / T);  token ~ q by inverse CDF with u[b]  (T == 0: token = argmax d, lowest index)
 *     c = max_k q_k                                                (T == 0: c = 1)
 *     draft_tokens[cu_d[b] + n_drafted[b]] = token, top_prob[same] = c, n_drafted[b] += 1
 *     active[b] = (c >= tau) && (n_drafted[b] < gamma[b])
 * The token drawn at a position whose confidence is below tau is kept (it is the last one
 * drafted), as in oracle_draft_stop.  Sequences that are not active are left untouched.
 * alt_token / sample_flag report a draw within tol of a CDF edge (see inv_cdf); conf_flag[b] = 1
 * when |c - tau| < conf_tol (either decision is legal there).
 */
void oracle_draft_step(const float *draft_logits, int64_t row_stride, int vocab, const float *temperature,
                       double tau, const float *u, const int32_t *gamma, const int32_t *cu_d, int batch,
                       double tol, double conf_tol, int32_t *n_drafted, int32_t *active,
                       int32_t *draft_tokens, double *top_prob, int32_t *alt_token, uint8_t *sample_flag,
                       uint8_t *conf_flag)
{
    double *q = (double *)malloc((size_t)(vocab > 0 ? vocab : 1) * sizeof(double));
    for (int b = 0; b < batch; ++b) {
        alt_token[b] = -1;
        sample_flag[b] = 0;
        conf_flag[b] = 0;
        if (!active[b]) continue;
        if (n_drafted[b] >= gamma[b]) { active[b] = 0; continue; }
        const float *d = draft_logits + (int64_t)b * row_stride;
        const double T = (double)temperature[b];
        int token;
        double c = 1.0;
        if (T > 0.0) {
            softmax_f64(d, vocab, T, q);
            int alt; uint8_t fl;
            token = inv_cdf(q, vocab, (double)u[b], tol, &alt, &fl);
            alt_token[b] = alt;
            sample_flag[b] = fl;
            c = 0.0;
            for (int k = 0; k < vocab; ++k)
                if (q[k] > c) c = q[k];
        } else {
            token = argmax_lowest(d, vocab);
        }
        const int pos = cu_d[b] + n_drafted[b];
        draft_tokens[pos] = token;
        top_prob[pos] = c;
        conf_flag[b] = fabs(c - tau) < conf_tol ? 1 : 0;
        n_drafted[b] += 1;
        active[b] = (c >= tau) && (n_drafted[b] < gamma[b]);
    }
    free(q);
}

/* gamma = gamma0, gbar = gamma0 for every sequence, plus the prefix sums. */
void oracle_gamma_tune_init(double *gamma_bar, int32_t *gamma, int32_t *cu_q, int32_t *cu_d,
                            int batch, int gamma0, int gamma_max, int padded_rows)
{
    cu_q[0] = 0;
    cu_d[0] = 0;
    for (int b = 0; b < batch; ++b) {
        gamma_bar[b] = (double)gamma0;
        gamma[b] = gamma0;
        cu_q[b + 1] = padded_rows ? (b + 1) * (gamma_max + 1) : cu_q[b] + gamma0 + 1;
        cu_d[b + 1] = padded_rows ? (b + 1) * gamma_max : cu_d[b] + gamma0;
    }
}

/* =========================================================================
 * 4. Cost model of paper Section 3 (Eq. 2-6), in units of T_draft:
 *    cost = N / (alpha*gamma + 1) * (c + gamma).  Analysis only.
 * ========================================================================= */
double oracle_cost_model(double n_tokens, double alpha, double gamma, double c)
{
    double n_steps = n_tokens / (alpha * gamma + 1.0);      /* Eq. 3 */
    double calls_target = n_steps;                          /* Eq. 4 */
    double calls_draft = gamma * n_steps;                   /* Eq. 5 */
    return c * calls_target + 1.0 * calls_draft;            /* Eq. 2 with T_draft = 1, T_target = c */
}
