// The float64 inverse-CDF sampling pass of accept_sample.cu as a step other callers can enqueue: one token per
// sequence from one row of logits (softmax of x / T, the smallest index whose cumulative mass exceeds u * total).
#pragma once

#include "common.cuh"

namespace sv {

// what a decision kernel leaves for the sampling pass, one per sequence
struct SeqRecord {
    double sum_p_hat, sum_q_hat;  // first-pass sums of the sampled rows (at ref_p / ref_q)
    float ref_p, ref_q;           // integer-valued reference exponents: the pass forms 2^(x * log2(e)/T - ref)
    int32_t n;                    // accept: first rejection (gamma if none)
    int32_t mode;                 // 0: nothing to sample (greedy or failed), 1: residual, 2: the row itself
};

struct RowSampleArgs {
    const void *logits;               // [batch][row_stride], float32 or bf16 bit patterns; row b belongs to sequence b
    int logits_bf16;
    long long row_stride;
    int vocab, batch;
    float temperature;
    const float *temperature_per_seq; // nullable
    const float *u_sample;            // [batch]
    int32_t *out_tokens;              // [batch]; written for sequences whose record has mode 2
    const SeqRecord *records;         // [batch], mode 0 or 2, ref_p at or above the row's largest x * log2(e)/T
    unsigned int *done;               // [batch], zero when the pass starts
    void *scratch;                    // row_sample_scratch_bytes(), 256-byte aligned
    uint32_t *device_status;
};

size_t row_sample_scratch_bytes(int batch, int vocab);
// enqueues the pass as a dependent launch behind the kernel that wrote `records` and cleared `done`
sv_status launch_row_sample(const RowSampleArgs &r, cudaStream_t stream);

}  // namespace sv
