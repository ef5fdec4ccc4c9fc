// Per-row epilogues on the quantifier's outputs: the score variants of the uncertainty appendix's practical
// remarks, and hard voting over the flags of several Inter-Heads.  One thread per row.
#include "ciar_internal.h"

namespace ciar {

namespace {

__global__ void rescore_kernel(int64_t rows, double n, const float *__restrict__ omega, const float *__restrict__ sigma,
                               ciar_score_params p, float *__restrict__ score_out, uint8_t *__restrict__ flag_out)
{
    const int64_t row = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (row >= rows) return;
    const double om = (double)omega[row], sg = (double)sigma[row];
    double v;
    switch (p.variant) {
    case CIAR_SCORE_PRODUCT: v = om * sg; break;
    case CIAR_SCORE_PER_N: v = om * sg / n; break;
    case CIAR_SCORE_PER_OMEGA2: v = sg / om; break;
    case CIAR_SCORE_SMOOTHED: v = om * sqrt(sg * sg + (double)p.eps); break;
    default: v = (double)p.lambda1 * om + (double)p.lambda2 * om * sg; break;
    }
    if (score_out) score_out[row] = (float)v;
    if (flag_out) flag_out[row] = (v != v) ? (uint8_t)1 : (uint8_t)(v > (double)p.tau);
}

__global__ void vote_kernel(int32_t n_heads, int64_t rows, const uint8_t *__restrict__ flags, uint8_t *__restrict__ flag_out,
                            int32_t *__restrict__ votes_out)
{
    const int64_t row = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (row >= rows) return;
    int cnt = 0;
    for (int h = 0; h < n_heads; ++h) cnt += flags[(int64_t)h * rows + row] != 0;
    if (votes_out) votes_out[row] = cnt;
    if (flag_out) flag_out[row] = (uint8_t)(2 * cnt > n_heads);
}

}  // namespace

cudaError_t launch_rescore(int64_t rows, int32_t n, const float *omega, const float *sigma, const ciar_score_params &p,
                           float *score_out, uint8_t *flag_out, cudaStream_t stream)
{
    if (rows == 0) return cudaSuccess;
    rescore_kernel<<<(unsigned)((rows + 255) / 256), 256, 0, stream>>>(rows, (double)n, omega, sigma, p, score_out, flag_out);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_vote(int32_t n_heads, int64_t rows, const uint8_t *flags, uint8_t *flag_out, int32_t *votes_out,
                        cudaStream_t stream)
{
    if (rows == 0) return cudaSuccess;
    vote_kernel<<<(unsigned)((rows + 255) / 256), 256, 0, stream>>>(n_heads, rows, flags, flag_out, votes_out);
    count_launch();
    return cudaGetLastError();
}

}  // namespace ciar
