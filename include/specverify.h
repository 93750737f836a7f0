/*
 * specverify -- the target model's verify step of speculative decoding with a
 * draft length gamma that changes every step (GammaTune, "Token-Driven
 * GammaTune: Adaptive Calibration for Enhanced Speculative Decoding").
 *
 * C ABI of a CUDA library for NVIDIA B200 (sm_100a).  Three operations make up
 * one verify step; they run back to back on one stream and never synchronise
 * with or read back to the host:
 *
 *   spec_verify_attn    attention of the gamma+1 draft positions against the
 *                       paged bf16 KV cache                     (Section 3 / 5)
 *   spec_accept_sample  accept / reject the drafts, resample or draw the bonus
 *                       token                                   (Section 3)
 *   gamma_tune_update   choose the next gamma from the number accepted
 *                                                               (Section 4.1, Algorithm 1)
 * and, for GammaTune+, spec_draft_stop in front of them         (Section 4.2).
 *
 * General conventions
 *   - Pointers named "device" point to device memory owned by the caller; the
 *     library allocates no device memory and keeps no state between calls
 *     except registered KV-pool handles (host memory), a few per-device facts
 *     it caches on the host (multiprocessor count, occupancy), and the one
 *     built-in scratch array of spec_accept_sample_static with its cached
 *     device address (see there).
 *   - "host" pointers are plain host memory (spec_verify_step_host prefers
 *     pinned memory so that its copies are asynchronous).
 *   - Every call is asynchronous on the given stream (a cudaStream_t passed as
 *     void*; NULL = the default stream) and returns after enqueueing.
 *   - A negative sv_status is an error found on the host before anything was
 *     launched.  Conditions found on the device (a page id outside the pool, a
 *     token id outside the vocabulary, a non-finite softmax sum, gamma outside
 *     [0, gamma_max], a bounded wait that expired) set bits in the caller's
 *     device_status word; the affected sequence is skipped or clamped and the
 *     kernel returns normally.  Nothing traps or asserts on the device.
 *   - Batch notation: B sequences; sequence b has draft length gamma[b] and
 *     R_b = gamma[b]+1 query / target rows starting at row cu_q[b], and
 *     gamma[b] draft rows / tokens / uniforms starting at cu_d[b].  seq_len[b]
 *     is the KV length INCLUDING those R_b positions (their K/V are already in
 *     the cache).  gamma, seq_len, cu_q, cu_d live on the device.
 */
#ifndef SPECVERIFY_H
#define SPECVERIFY_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t sv_status;
enum {
    SV_OK = 0,
    SV_EINVAL = -1,        /* null pointer, non-positive size, inconsistent arguments */
    SV_EUNSUPPORTED = -2,  /* head_dim not 64/128, page_size not 16, hq % hkv != 0, ... */
    SV_EALIGN = -3,        /* a pointer or stride misses the alignment stated below */
    SV_ECUDA = -4,         /* a CUDA runtime / driver call failed (launch, tensor map) */
    SV_EWORKSPACE = -5     /* workspace missing or smaller than the size query says */
};

/* bits of the device status word */
enum {
    SV_DEV_BAD_GAMMA = 1,   /* gamma[b] outside [0, gamma_max]: clamped */
    SV_DEV_BAD_PAGE = 2,    /* block-table entry outside [0, n_pages): attention reads that page as zeros
                               and the outputs of that sequence are unspecified (other sequences are
                               unaffected); the cache append skips that position */
    SV_DEV_BAD_TOKEN = 4,   /* draft token outside [0, vocab): position rejected */
    SV_DEV_NONFINITE = 8,   /* softmax sum not finite (NaN / +Inf logit): sequence emits -1 */
    SV_DEV_TIMEOUT = 16,    /* a bounded device-side wait expired (also: a kernel found its shared
                               memory misaligned and did nothing) */
    SV_DEV_BAD_LEN = 32     /* seq_len[b] < gamma[b]+1 or beyond the block table: sequence skipped */
};

const char *sv_status_str(sv_status s);

/* ---------------------------------------------------------------- KV pool */
/*
 * A paged KV pool: K and V arrays of n_pages pages, each page holding
 * page_size (= 16) token slots for hkv heads of head_dim bf16 values.
 * strides[4] = element strides for (page, kv head, slot, dim); dim stride must
 * be 1, the others multiples of 8 elements (16 bytes); both base pointers
 * 16-byte aligned.  [page, head, slot, dim] and [page, slot, head, dim] are
 * both expressible.  Registration builds the TMA tensor maps on the host; the
 * handle is host memory released by spec_kv_pool_release.  Slots past a
 * sequence's seq_len inside its last page are read (and multiplied by zero
 * weights), so pool memory must hold finite values.
 */
typedef struct sv_kv_pool *sv_kv_pool_t;

sv_status spec_kv_pool_register(const void *k_pool_device, const void *v_pool_device,
                                int64_t n_pages, int32_t page_size, int32_t hkv, int32_t head_dim,
                                const int64_t strides[4], sv_kv_pool_t *out);
sv_status spec_kv_pool_release(sv_kv_pool_t pool);

/* ---------------------------------------------------------------- attention */
/*
 * Paper Section 3: the target verifies the gamma drafted tokens in one parallel
 * forward; with KV caching (Section 5) the context-dependent part of it is
 * this causal attention.  For sequence b, row i in [0, gamma[b]], query head h:
 *     pos = seq_len[b] - (gamma[b]+1) + i ;  kv head = h / (hq / hkv)
 *     s_j = sm_scale * <q, k_j>   for j = 0 .. pos
 *     o   = sum_j softmax(s)_j v_j ;   lse = ln sum_j exp(s_j)
 * bf16 inputs, fp32 accumulation and softmax, bf16 output.
 */
typedef struct sv_attn_params {
    const void *q;              /* device bf16 [n_rows, hq, head_dim], 16-byte aligned */
    void *o;                    /* device bf16 [n_rows, hq, head_dim], 16-byte aligned */
    float *lse;                 /* device fp32 [n_rows, hq], or NULL */
    sv_kv_pool_t pool;
    const int32_t *block_table; /* device [batch, block_table_stride]: physical page of logical page */
    int64_t block_table_stride; /* elements between rows; >= ceil(max_seq_len / 16) */
    const int32_t *seq_len;     /* device [batch] */
    const int32_t *gamma;       /* device [batch] */
    const int32_t *cu_q;        /* device [batch+1] */
    int32_t batch;
    int32_t gamma_max;          /* upper bound of gamma[b]; sizes the row tile */
    int32_t hq, hkv, head_dim;
    int32_t max_seq_len;        /* upper bound of seq_len[b]; sizes the grid and the workspace */
    float sm_scale;             /* usually 1/sqrt(head_dim) */
    uint32_t *device_status;    /* device, one word, OR-ed into; may be NULL */
} sv_attn_params;

/* Bytes of device scratch spec_verify_attn needs for these bounds (partial
 * results of sequences whose keys are split over several thread blocks). */
size_t spec_verify_attn_workspace_bytes(int32_t batch, int32_t gamma_max, int32_t hq, int32_t hkv,
                                        int32_t head_dim, int32_t max_seq_len);

sv_status spec_verify_attn(const sv_attn_params *p, void *workspace_device, size_t workspace_bytes,
                           void *stream);

/* ---------------------------------------------------------------- cache append */
/*
 * KV caching (paper Section 5, experimental setup): before the verify
 * attention runs, the keys and values of the gamma[b]+1 new positions are
 * written behind each sequence's context.  New row i of sequence b (row
 * cu_q[b]+i of k_new / v_new) is token
 *     pos = seq_len[b] - (gamma[b]+1) + i
 * (seq_len already counts the block) and goes to physical page
 * block_table[b][pos / 16], slot pos % 16 of every kv head.  A copy of bf16
 * bit patterns; nothing else in the pools is touched.  Rolling rejected
 * positions back needs no copy: gamma_tune_update shortens seq_len, and the
 * next append overwrites them.
 * The pool memory (registered through const pointers for the attention) is
 * written by this call; the caller owns it and orders the call before the
 * attention on the same stream.
 * Device-detected: gamma[b] out of range -> SV_DEV_BAD_GAMMA, clamped;
 * seq_len[b] < gamma[b]+1 or a position beyond the block table row ->
 * SV_DEV_BAD_LEN, sequence skipped; a page id outside [0, n_pages) ->
 * SV_DEV_BAD_PAGE, that position skipped.
 */
typedef struct sv_kv_append_params {
    const void *k_new;          /* device bf16 [n_rows, hkv, head_dim], 16-byte aligned */
    const void *v_new;          /* device bf16 [n_rows, hkv, head_dim], 16-byte aligned */
    sv_kv_pool_t pool;          /* head_dim a multiple of 8 */
    const int32_t *block_table; /* device [batch, block_table_stride] */
    int64_t block_table_stride;
    const int32_t *seq_len;     /* device [batch] */
    const int32_t *gamma;       /* device [batch] */
    const int32_t *cu_q;        /* device [batch+1] */
    int32_t batch;
    int32_t gamma_max;          /* upper bound of gamma[b]; sizes the grid */
    uint32_t *device_status;    /* device, one word, OR-ed into; may be NULL */
} sv_kv_append_params;

sv_status spec_kv_append(const sv_kv_append_params *p, void *stream);

/* ---------------------------------------------------------------- all layers of a step */
/*
 * A target model keeps one KV cache per layer (KV caching, paper Section 5), all
 * with the same paging: one block table, one set of lengths.  This call runs the
 * cache append and the verify attention of n_layers caches in one enqueue: first
 * ONE launch writes every layer's new keys and values (spec_kv_append for all
 * layers at once; skipped when k_new is NULL), then the attention of layer 0, 1,
 * ... in order, each reading its own pool, queries and writing its own output.
 * In a real model layer l+1's queries depend on layer l's output through the
 * projections in between, which are outside this library; here they are inputs.
 * pools / q / o / k_new / v_new / lse are HOST arrays of n_layers entries
 * (device pointers inside); everything else is shared and means what it means in
 * sv_attn_params.  The workspace is the one spec_verify_attn asks for (it is
 * reused layer after layer).  Errors: as spec_verify_attn / spec_kv_append; the
 * pools must agree in hkv and head_dim.
 */
typedef struct sv_attn_layers_params {
    int32_t n_layers;
    const sv_kv_pool_t *pools;    /* host [n_layers] */
    const void *const *q;         /* host [n_layers] of device bf16 [n_rows, hq, head_dim] */
    void *const *o;               /* host [n_layers] of device bf16 [n_rows, hq, head_dim] */
    float *const *lse;            /* host [n_layers] of device fp32 [n_rows, hq], or NULL */
    const void *const *k_new;     /* host [n_layers] of device bf16 [n_rows, hkv, head_dim], or NULL: no append */
    const void *const *v_new;     /* host [n_layers], NULL exactly when k_new is */
    sv_attn_params shared;        /* q, o, lse and pool of this struct are ignored */
} sv_attn_layers_params;

sv_status spec_verify_attn_layers(const sv_attn_layers_params *p, void *workspace_device,
                                  size_t workspace_bytes, void *stream);

/* ---------------------------------------------------------------- accept / resample */
/*
 * Speculative sampling (paper Section 3, after Leviathan et al. and Chen et
 * al.).  Per sequence, with T = its temperature, target rows t_0..t_gamma and
 * draft rows d_0..d_{gamma-1}, draft tokens x_i, uniforms u_i and u_s:
 *   T > 0:  p_i = softmax(t_i / T), q_i = softmax(d_i / T)
 *           ratio_i = min(1, p_i[x_i] / q_i[x_i]); accept while u_i < ratio_i;
 *           n = index of the first rejection (gamma if none)
 *           n < gamma: next ~ normalise(max(0, p_n - q_n))  (p_n if that is all zero)
 *           n = gamma: next ~ p_gamma                        (the bonus token)
 *           both by inverse CDF in vocabulary order with u_s
 *           (smallest k with sum_{j<=k} w_j > u_s * sum_j w_j).
 *   T == 0: n = first i with argmax(t_i) != x_i (lowest index wins ties),
 *           next = argmax(t_n); draft logits and uniforms are not read.
 * Softmax sums are accumulated in float64 from float32 exponentials; the
 * ratio, the comparison and the sampled row are evaluated in float64.
 * The paper's largest target runs with reduced precision (Section 5); logits
 * stored as bf16 are accepted too (logits_bf16), which halves the bytes of
 * this step.
 */
typedef struct sv_accept_params {
    const float *target_logits;   /* device fp32 [n_q_rows, row_stride] */
    const float *draft_logits;    /* device fp32 [n_d_rows, row_stride]; may be NULL if all T == 0 */
    int64_t row_stride;           /* elements between rows (>= vocab); a multiple of 4 with
                                     16-byte aligned bases enables 128-bit loads */
    int32_t vocab;
    const int32_t *draft_tokens;  /* device [n_d_rows] */
    const float *u_accept;        /* device [n_d_rows], in [0,1) */
    const float *u_sample;        /* device [batch], in [0,1) */
    float temperature;            /* used when temperature_per_seq is NULL */
    const float *temperature_per_seq; /* device [batch] or NULL */
    const int32_t *gamma;         /* device [batch] */
    const int32_t *cu_q;          /* device [batch+1] */
    const int32_t *cu_d;          /* device [batch+1] */
    int32_t batch;
    int32_t gamma_max;
    int32_t *n_accepted;          /* device out [batch]: accepted drafts, 0..gamma (extra token not counted) */
    int32_t *out_tokens;          /* device out [batch, gamma_max+1]: accepted drafts, next token, then -1 */
    double *ratio;                /* device out [n_d_rows] or NULL (NaN past the first rejection) */
    double *logZ_p;               /* device out [n_q_rows] or NULL: ln sum exp(t/T) */
    double *logZ_q;               /* device out [n_d_rows] or NULL: ln sum exp(d/T) */
    uint32_t *flag_count;         /* device, one word or NULL: += positions with |u - ratio| < 1e-6 */
    uint32_t *device_status;      /* device, one word or NULL */
    int32_t logits_bf16;          /* 0: the logits are float32 (as declared).  1: target_logits / draft_logits
                                     point to bf16 values (2 bytes each, row_stride still in elements; a
                                     multiple of 8 with 16-byte aligned bases enables 128-bit loads); every
                                     value is widened exactly to float32 and the arithmetic is unchanged, so
                                     the result is that of the float32 call on the widened values at half
                                     the bytes */
} sv_accept_params;

size_t spec_accept_sample_workspace_bytes(int32_t batch, int32_t gamma_max, int32_t vocab);

sv_status spec_accept_sample(const sv_accept_params *p, void *workspace_device,
                             size_t workspace_bytes, void *stream);

/*
 * spec_accept_sample without a workspace argument and without any allocation.
 * The paper has no counterpart to this entry point; it exists for callers that
 * are not able to obtain device scratch memory themselves: code running where
 * every device buffer was fixed at start-up (a serving engine whose memory pool
 * is fully handed out, a plugin that is only given its input and output
 * tensors), or code that must not call cudaMalloc at this point because an
 * allocation would synchronise the device or is forbidden by the host
 * framework's rules.  The computation and the results are those of
 * spec_accept_sample; only the place of the intermediate slice statistics
 * differs: they go to an array of SV_ACCEPT_STATIC_SCRATCH_BYTES bytes that is
 * built into the library (each GPU that loads the library carries it until the
 * process ends).
 *   - Limit: the intermediate results -- 32 bytes per (row, slice of the
 *     vocabulary) with batch * (2*gamma_max + 1) rows and slices of 2048 to 16384
 *     elements (the library picks larger slices when there are many rows), plus
 *     24 bytes per 128 vocabulary entries per sequence for the sampling pass --
 *     must fit in SV_ACCEPT_STATIC_SCRATCH_BYTES.  The largest configuration of
 *     the tests (batch 128, gamma_max 16, vocab 128256) needs about 4.2 MB.  A
 *     larger problem is refused with SV_EWORKSPACE before anything is launched;
 *     use spec_accept_sample then.
 *   - The first call on each device looks up the array's device address
 *     (cudaGetSymbolAddress) with that device current; make that first call
 *     outside any stream capture.  No call allocates or frees memory.
 *   - All calls on one device share the array and it keeps whatever the previous
 *     call left there.  Nothing needs clearing: every record a call reads was
 *     written earlier in that same call.  Two calls whose kernels can overlap on
 *     the GPU (different streams without an ordering between them) race on the
 *     array and give wrong results; keep such calls on one stream or order them
 *     with events.
 */
#define SV_ACCEPT_STATIC_SCRATCH_BYTES (8u << 20)
sv_status spec_accept_sample_static(const sv_accept_params *p, void *stream);

/* ---------------------------------------------------------------- GammaTune */
/*
 * Paper Section 4.1, Algorithm 1, one update per sequence, state on the device:
 *   SV_GT_PROPOSED  A' = A + delta if A == gamma else A      (Eq. 7 feeding the average,
 *                   gbar <- min(gmax, max(gmin, (1-eta) gbar + eta A'))   (Eq. 8)   as the prose says)
 *                   gamma <- ceil(gbar)
 *   SV_GT_LITERAL   the listing as printed: the average is fed A itself
 *   SV_GT_FIXED     gamma and gbar stay (plain speculative decoding)
 * binary64 throughout, each product and the sum rounded separately (no fused
 * multiply-add), so trajectories are reproducible bit for bit.
 * Bookkeeping done in the same kernel:
 *   seq_len <- seq_len - (gamma+1) + (A+1) + (gamma_next+1)
 *   cu_q, cu_d <- prefix sums of gamma_next+1 / gamma_next, or b*(gamma_max+1) /
 *   b*gamma_max when padded_rows != 0 (fixed row slabs per sequence).
 */
enum { SV_GT_FIXED = 0, SV_GT_PROPOSED = 1, SV_GT_LITERAL = 2 };

typedef struct sv_gamma_config {
    double eta;          /* adaptation rate in [0, 1] */
    double delta;        /* expansion offset */
    int32_t gamma_min;   /* >= 0 */
    int32_t gamma_max;   /* >= gamma_min */
    int32_t mode;        /* SV_GT_* */
    int32_t padded_rows; /* row-offset convention, see above */
} sv_gamma_config;

typedef struct sv_gamma_params {
    const int32_t *n_accepted;  /* device [batch] */
    double *gamma_bar;          /* device in/out [batch] */
    int32_t *gamma;             /* device in/out [batch] */
    int32_t *seq_len;           /* device in/out [batch], or NULL */
    int32_t *cu_q;              /* device out [batch+1] */
    int32_t *cu_d;              /* device out [batch+1] */
    int32_t batch;
    sv_gamma_config config;
    int32_t *trajectory;        /* device out or NULL: gamma_next written to trajectory[step*batch + b] */
    int32_t *accepted_log;      /* device out or NULL: A written to accepted_log[step*batch + b] */
    int32_t step;
    uint32_t *device_status;    /* device, one word or NULL */
    const int32_t *n_drafted;   /* device [batch] or NULL: drafts actually produced this step when
                                   drafting stopped early (spec_draft_stop); gamma[b] stays the
                                   length the controller issued and is what A is compared with,
                                   n_drafted[b]+1 is the number of positions the cache gained */
} sv_gamma_params;

sv_status gamma_tune_update(const sv_gamma_params *p, void *stream);
/* gamma = gamma0 and gamma_bar = gamma0 for every sequence, cu_q / cu_d built; n_accepted,
 * seq_len, trajectory are not touched. */
sv_status gamma_tune_init(const sv_gamma_params *p, int32_t gamma0, void *stream);

/* ---------------------------------------------------------------- GammaTune+ early stop */
/*
 * Paper Section 4.2 (GammaTune+): drafting stops when the draft model's top
 * probability falls below a threshold tau.  For sequence b and draft position
 * i < gamma[b] the confidence is c_i = max_k softmax(d_i / T)_k (one streaming
 * pass over the draft row: running max and sum).  The paper does not say
 * whether the low-confidence token itself is kept; here it is, and nothing is
 * drafted after it:
 *     n_drafted[b] = min(gamma[b], 1 + first i with c_i < tau)   (gamma[b] if none).
 * T == 0 (greedy draft): c_i = 1, drafting never stops early.
 * The verify step then runs with n_drafted as its gamma array (attention,
 * accept) and gamma_tune_update takes both (see sv_gamma_params.n_drafted).
 * Confidences are float32 exponentials summed in float64; c_i and the
 * comparison with tau are evaluated in float64.
 */
typedef struct sv_draft_stop_params {
    const float *draft_logits;    /* device fp32 [n_d_rows, row_stride] */
    int64_t row_stride;           /* elements between rows (>= vocab) */
    int32_t vocab;
    float temperature;            /* used when temperature_per_seq is NULL */
    const float *temperature_per_seq; /* device [batch] or NULL */
    float tau;                    /* threshold in [0, 1] */
    const int32_t *gamma;         /* device [batch]: draft lengths issued by the controller */
    const int32_t *cu_d;          /* device [batch+1] */
    int32_t batch;
    int32_t gamma_max;
    int32_t *n_drafted;           /* device out [batch] */
    double *top_prob;             /* device out [n_d_rows] or NULL: c_i of every draft row */
    uint32_t *device_status;      /* device, one word or NULL */
    int32_t logits_bf16;          /* as in sv_accept_params: 1 = draft_logits holds bf16 values */
} sv_draft_stop_params;

size_t spec_draft_stop_workspace_bytes(int32_t batch, int32_t gamma_max, int32_t vocab);

sv_status spec_draft_stop(const sv_draft_stop_params *p, void *workspace_device, size_t workspace_bytes,
                          void *stream);

/* ---------------------------------------------------------------- GammaTune+ drafting step */
/*
 * Paper Section 4.2, the draft side: one drafting step of every sequence that
 * is still drafting.  Row b of draft_logits holds sequence b's draft logits for
 * its next position.  For every b with active[b] != 0 and n_drafted[b] < gamma[b]:
 *     q = softmax(d_b / T);  token ~ q by inverse CDF in vocabulary order with
 *     u_sample[b] (the smallest k with sum_{j<=k} q_j > u * sum_j q_j;
 *     T == 0: token = argmax, lowest index on ties);  c = max_k q_k (T == 0: 1)
 *     draft_tokens[cu_d[b] + n_drafted[b]] = token, top_prob[same] = c,
 *     n_drafted[b] += 1,  active[b] = (c >= tau) && (n_drafted[b] < gamma[b]).
 * The token drawn at a position whose confidence is below tau is kept, as in
 * spec_draft_stop; a loop of these steps from n_drafted = 0 and active = 1 ends
 * with the n_drafted that spec_draft_stop gives for the same rows, and with the
 * tokens where spec_accept_sample reads them.  Sequences that are not active are
 * not read and not written; one with n_drafted[b] >= gamma[b] only has active[b]
 * cleared.  A row whose softmax sum is not finite (NaN or +inf logits) sets
 * SV_DEV_NONFINITE, stores token -1 and clears active[b].
 * Arithmetic: the top probability from float32 exponentials summed in float64
 * (as spec_draft_stop), evaluated and compared with tau in float64; the token
 * from a float64 pass over the row (as the bonus token of spec_accept_sample).
 */
typedef struct sv_draft_step_params {
    const float *draft_logits;    /* device fp32 [batch, row_stride] (bf16 values if logits_bf16) */
    int64_t row_stride;           /* elements between rows (>= vocab) */
    int32_t vocab;
    float temperature;            /* used when temperature_per_seq is NULL */
    const float *temperature_per_seq; /* device [batch] or NULL */
    float tau;                    /* threshold in [0, 1] */
    const float *u_sample;        /* device [batch], in [0,1); may be NULL if every temperature is 0 */
    const int32_t *gamma;         /* device [batch]: draft lengths issued by the controller */
    const int32_t *cu_d;          /* device [batch+1]: first draft row of each sequence */
    int32_t batch;
    int32_t gamma_max;            /* bound on gamma[b] */
    int32_t *n_drafted;           /* device in/out [batch] */
    int32_t *active;              /* device in/out [batch] */
    int32_t *draft_tokens;        /* device out [n_d_rows] */
    double *top_prob;             /* device out [n_d_rows] or NULL */
    uint32_t *device_status;      /* device, one word or NULL */
    int32_t logits_bf16;          /* as in sv_accept_params */
} sv_draft_step_params;

size_t spec_draft_step_workspace_bytes(int32_t batch, int32_t vocab);

/* Four launches on `stream`; nothing is read back.  Errors before any launch: SV_EINVAL (null pointers,
 * sizes <= 0, row_stride < vocab, tau outside [0, 1], u_sample NULL with a positive temperature),
 * SV_EWORKSPACE, SV_EALIGN (workspace not 16-byte aligned). */
sv_status spec_draft_step(const sv_draft_step_params *p, void *workspace_device, size_t workspace_bytes,
                          void *stream);

/* ---------------------------------------------------------------- whole step from host buffers */
/*
 * One verify step whose per-step inputs start in HOST memory: copies q,
 * logits, draft tokens and uniforms to the caller's device staging buffers,
 * runs spec_verify_attn, spec_accept_sample, gamma_tune_update on `stream`,
 * and copies n_accepted, out_tokens, gamma (next) and the attention output
 * back to host buffers.  All asynchronous; the caller synchronises the stream
 * before reading the host outputs.  The KV pool, block table and controller
 * state stay resident on the device (that is what a KV cache is).
 * n_q_rows / n_d_rows are the numbers of rows to copy (host knows the layout
 * it filled).  Device pointers inside attn / accept / gamma are used as the
 * staging destinations.
 */
typedef struct sv_step_host_io {
    const void *q_host;             /* bf16 [n_q_rows, hq, head_dim] */
    const float *target_logits_host;
    const float *draft_logits_host;
    const int32_t *draft_tokens_host;
    const float *u_accept_host;
    const float *u_sample_host;
    int64_t n_q_rows, n_d_rows;
    int32_t *n_accepted_host;       /* out [batch] */
    int32_t *out_tokens_host;       /* out [batch, gamma_max+1] */
    int32_t *gamma_next_host;       /* out [batch] */
    void *o_host;                   /* out bf16 [n_q_rows, hq, head_dim], or NULL */
} sv_step_host_io;

sv_status spec_verify_step_host(const sv_step_host_io *io, const sv_attn_params *attn,
                                void *attn_workspace, size_t attn_workspace_bytes,
                                const sv_accept_params *accept, void *accept_workspace,
                                size_t accept_workspace_bytes, const sv_gamma_params *gamma,
                                void *stream);

/*
 * Self-test of the bounded waits (no counterpart in the paper).  Every wait of
 * the tensor-core kernels has a cycle budget; when it runs out the kernel sets
 * SV_DEV_TIMEOUT and returns instead of hanging.  This call launches one thread
 * block that waits, with a budget of limit_cycles (1 .. 2e9 SM cycles), on a
 * barrier nothing ever arrives at.  Afterwards *device_status has
 * SV_DEV_TIMEOUT set and *device_result is 0 (1 would mean the wait was
 * satisfied); the context stays usable.
 */
sv_status sv_selftest_wait_expiry(uint32_t *device_status, int32_t *device_result, int64_t limit_cycles,
                                  void *stream);

/* Kernel launches issued by the library since it was loaded (for reporting). */
uint64_t sv_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* SPECVERIFY_H */
