// Internal interface between the host entry points (api.cu) and the kernel launchers.
#pragma once

#include "ciar_device.cuh"

namespace ciar {

struct QuantifyArgs {
    const void *logits;
    int64_t rows;  // logical rows of this launch
    int64_t row_stride;
    int32_t vb, n;
    RowMap rm;
    int32_t radius_mode, radius_is_raw;
    const void *radius;
    float r_scalar, r_max, lo_cap, hi_cap;
    int32_t policy;
    float tau;
    const float *u_flag;
    ciar_quantify_out out;  // indexed by logical row
    // streaming kernels: bound of every device-side wait, in SM clocks, and (test hook, off when negative)
    // the CTA and the place in its walk of one row whose copy is never issued
    int64_t wait_cycles;
    int32_t drop_cta, drop_k;
};

// Scratch of one verify launch, carved out of the caller's workspace.
struct VerifyScratch {
    int32_t *window_done;  // [windows] arrival counters, zero before the launch
    int32_t *candidate;    // [rows] residual sample of each rejected row
    uint8_t *accept;       // [rows] accept bits when the caller did not ask for them
    // streaming path only
    int32_t *tested;       // [rows + 1] logical rows the cloud tests, in order; tested[rows] = how many
    float *tq_max, *tq_sum;  // [rows] maximum and sum of exp(. - max) of the target rows that were tested
};

struct VerifyArgs {
    const void *draft, *target;
    int64_t rows;  // logical rows, a multiple of the window
    int64_t row_stride;
    int32_t vocab, vb, n;
    RowMap rm;
    const int32_t *tokens;       // by physical row
    const uint8_t *flag;         // by logical row
    const float *draft_row_max;  // by logical row, nullable (then recomputed)
    const float *draft_sum_exp;
    const float *u_accept, *u_resample;  // by physical row
    int32_t window, mode;
    ciar_verify_out out;  // by logical row / logical window
    VerifyScratch ws;
};

struct DecodeUpdateArgs {
    ciar_decode_state st;
    int32_t window, mode;
    const int32_t *tokens;  // draft token pool
    const uint8_t *flag;    // [requests * window] flags of this step
    const int32_t *first_flag, *accepted_len, *resampled_token;  // [requests]
};

struct TopkArgs {
    const void *logits;
    int64_t rows, row_stride;
    int32_t vb, n, k;
    int32_t radius_mode, radius_is_raw;
    const void *radius;
    float r_scalar, r_max, lo_cap, hi_cap, tau;
    ciar_topk_out out;
};

struct EnsembleArgs {
    const void *heads;
    int32_t n_heads;
    int64_t head_stride;
    int64_t rows, row_stride;
    int32_t vb, n;
    int32_t radius_mode, radius_is_raw;
    const float *radius;  // [n_heads, rows] when PER_ROW
    float r_scalar, r_max, lo_cap, hi_cap, tau;
    ciar_quantify_out out;
};

struct InterDroArgs {
    const void *center, *radius, *cloud;
    int64_t rows, row_stride;
    int32_t vb, n;
    ciar_interdro_params prm;
    ciar_interdro_out out;
    double *ws;  // [7, rows]: L1 mid / up / lo, CE mid / up / lo, KL of every row, kept in double for the batch step
};

cudaError_t launch_quantify(const QuantifyArgs &a, int dtype, cudaStream_t stream);
cudaError_t launch_topk(const TopkArgs &a, int dtype, cudaStream_t stream);
cudaError_t launch_rescore(int64_t rows, int32_t n, const float *omega, const float *sigma, const ciar_score_params &p,
                           float *score_out, uint8_t *flag_out, cudaStream_t stream);
cudaError_t launch_ensemble(const EnsembleArgs &a, int dtype, cudaStream_t stream);
cudaError_t launch_vote(int32_t n_heads, int64_t rows, const uint8_t *flags, uint8_t *flag_out, int32_t *votes_out,
                        cudaStream_t stream);
cudaError_t launch_interdro(const InterDroArgs &a, int dtype, cudaStream_t stream);
// The streaming (TMA ring) quantifier and the test that says whether it covers a call.
bool quantify_stream_eligible(const QuantifyArgs &a, int dtype);
cudaError_t launch_quantify_stream(const QuantifyArgs &a, int dtype, cudaStream_t stream);
// The streaming quantifier for rows wider than that one takes (two passes over a row, chunk by chunk).
bool quantify_wide_eligible(const QuantifyArgs &a, int dtype);
cudaError_t launch_quantify_wide(const QuantifyArgs &a, int dtype, cudaStream_t stream);
// The streaming quantifier for one radius per code (logits and radii through the same TMA ring).
bool quantify_percode_eligible(const QuantifyArgs &a, int dtype);
cudaError_t launch_quantify_percode(const QuantifyArgs &a, int dtype, cudaStream_t stream);
cudaError_t launch_verify(const VerifyArgs &a, int dtype, cudaStream_t stream);
// The streaming (plan, TMA-ring accept sweep, per-window finish) verifier and the test that says whether it covers a call.
bool verify_stream_eligible(const VerifyArgs &a, int dtype);
cudaError_t launch_verify_stream(const VerifyArgs &a, int dtype, cudaStream_t stream);
cudaError_t launch_decode_init(const ciar_decode_state &st, int32_t pos0, cudaStream_t stream);
cudaError_t launch_decode_update(const DecodeUpdateArgs &a, cudaStream_t stream);

int sm_count();       // SMs of the current device (cached per device)
void count_launch();  // bumps the process-wide launch counter

}  // namespace ciar
