// Cloud-side verification of draft windows: target-row softmax statistics, the accept test on
// the drafted token, the residual inverse-CDF sample of rejected rows, and the per-window
// combine (first flag, accepted length, resampled token) done by whichever CTA of the window
// finishes last -- no CTA ever waits for another.
#include "ciar_internal.h"
#include "verify_resample.cuh"

namespace ciar {

namespace {

// First flagged row of a window (wlen if none).
__device__ __forceinline__ int32_t first_flag_of(const uint8_t *flag, int64_t row0, int32_t wlen)
{
    for (int32_t j = 0; j < wlen; ++j)
        if (flag[row0 + j]) return j;
    return wlen;
}

__device__ __forceinline__ bool row_tested(int mode, int32_t j, int32_t f, int32_t wlen, const uint8_t *flag, int64_t lr)
{
    if (j >= wlen) return false;
    if (mode == CIAR_VERIFY_ALL) return true;
    if (mode == CIAR_VERIFY_ANCHORED) return j >= f;
    return flag[lr] != 0;
}

template <typename T>
__global__ void __launch_bounds__(kThreads) verify_kernel(VerifyArgs a)
{
    constexpr int V = Elem<T>::kVec;
    __shared__ float fs[kWarps];
    __shared__ double ds[3 * kWarps];
    __shared__ double scan_warp[kWarps];
    __shared__ double sh_d[4];
    __shared__ int sh_i[4];  // 0: accept bit, 2..3: scratch of the resampler
    const T *dbase = reinterpret_cast<const T *>(a.draft);
    const T *tbase = reinterpret_cast<const T *>(a.target);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint8_t *accept_arr = a.out.accept ? a.out.accept : a.ws.accept;

    for (int64_t lr = blockIdx.x; lr < a.rows; lr += gridDim.x) {
        const int64_t w = lr / a.window;
        const int32_t j = (int32_t)(lr - w * a.window);
        const int32_t wlen = window_len(a.rm, w);
        int64_t pr;
        map_row(a.rm, lr, pr);
        const int32_t f = (a.mode == CIAR_VERIFY_ALL) ? 0 : first_flag_of(a.flag, w * a.window, wlen);
        const bool tested = row_tested(a.mode, j, f, wlen, a.flag, lr);

        int acc = 1, status = 0, cand = -1;
        float px_out = 0.f, qx_out = 0.f;
        if (tested) {
            const RowView<T> rd(dbase + pr * a.row_stride, a.vb, a.n);
            const RowView<T> rt(tbase + pr * a.row_stride, a.vb, a.n);
            float mp;
            double zp;
            bool have_stats = a.draft_row_max != nullptr;
            if (have_stats) {
                mp = a.draft_row_max[lr];
                zp = (double)a.draft_sum_exp[lr];
                // the quantifier marks unusable rows with NaN: recompute to learn which kind it is
                if (!(zp > 0.0) || !(zp < INFINITY) || !(mp == mp)) have_stats = false;
            }
            if (!have_stats) {
                RowStats sd;
                row_stats(rd, fs, ds, sd);
                mp = sd.m;
                zp = sd.z;
                if (sd.m == -INFINITY) status |= CIAR_ROW_NO_FINITE;
                else if (!(sd.z_raw < INFINITY) || !(sd.z_raw > 0.0)) status |= CIAR_ROW_NAN;
            }
            RowStats sq;
            row_stats(rt, fs, ds, sq);
            if (sq.m == -INFINITY) status |= CIAR_ROW_NO_FINITE;
            else if (!(sq.z_raw < INFINITY) || !(sq.z_raw > 0.0)) status |= CIAR_ROW_NAN;
            const float mq = sq.m;
            const double zq = sq.z;
            const int32_t x = a.tokens[pr];
            const bool bad_token = (x < 0 || x >= a.vocab);

            if (status) {
                acc = 0;  // unusable logits: rejected, nothing to resample from
                px_out = qx_out = __int_as_float(0x7fc00000);
                if (bad_token) status |= CIAR_ROW_BAD_TOKEN;
            } else {
                // accept test on the drafted token, in double: u * p_x < q_x
                if (threadIdx.x == 0) {
                    double px = 0.0, qx = 0.0;
                    if (x >= a.vb && x < a.vb + a.n) {  // a code outside the valid slice has probability 0
                        const double cx = (double)Elem<T>::widen(dbase[pr * a.row_stride + x]);
                        const double tx = (double)Elem<T>::widen(tbase[pr * a.row_stride + x]);
                        px = exp(cx - (double)mp) / zp;
                        qx = exp(tx - (double)mq) / zq;
                    }
                    sh_d[0] = px;
                    sh_d[1] = qx;
                    sh_i[0] = (!bad_token && (double)a.u_accept[pr] * px < qx) ? 1 : 0;
                }
                __syncthreads();
                acc = sh_i[0];
                px_out = (float)sh_d[0];
                qx_out = (float)sh_d[1];
                __syncthreads();
                if (bad_token) {  // an id outside [0, vocab): rejected; the replacement comes from the residual
                    status |= CIAR_ROW_BAD_TOKEN;
                    px_out = qx_out = __int_as_float(0x7fc00000);
                }

                if (!acc) {
                    cand = resample_row<T, kThreads>(rd, rt, mp, zp, mq, zq, a.u_resample[pr], a.vb, scan_warp, sh_i + 2);
                }
            }
        }

        // publish this row, then count it in; the CTA that completes the window combines it
        if (threadIdx.x == 0) {
            if (j < wlen || a.rm.pos == nullptr) {
                accept_arr[lr] = (uint8_t)acc;
                a.ws.candidate[lr] = cand;
                if (a.out.p_draft_tok) a.out.p_draft_tok[lr] = px_out;
                if (a.out.p_target_tok) a.out.p_target_tok[lr] = qx_out;
                if (a.out.row_status) a.out.row_status[lr] = (uint8_t)status;
            } else {
                accept_arr[lr] = 1;
                a.ws.candidate[lr] = -1;
                if (a.out.p_draft_tok) a.out.p_draft_tok[lr] = 0.f;
                if (a.out.p_target_tok) a.out.p_target_tok[lr] = 0.f;
                if (a.out.row_status) a.out.row_status[lr] = 0;
            }
            __threadfence();
            const int old = atomicAdd(&a.ws.window_done[w], 1);
            if (old == a.window - 1) {
                __threadfence();
                int32_t acc_len = wlen;
                for (int32_t jj = 0; jj < wlen; ++jj) {
                    const int64_t r2 = w * a.window + jj;
                    if (row_tested(a.mode, jj, f, wlen, a.flag, r2) &&
                        *reinterpret_cast<volatile uint8_t *>(accept_arr + r2) == 0) {
                        acc_len = jj;
                        break;
                    }
                }
                int32_t tok = -1;
                if (acc_len < wlen) tok = *reinterpret_cast<volatile int32_t *>(a.ws.candidate + w * a.window + acc_len);
                if (a.out.first_flag) a.out.first_flag[w] = f;
                if (a.out.accepted_len) a.out.accepted_len[w] = acc_len;
                if (a.out.resampled_token) a.out.resampled_token[w] = tok;
                if (a.out.cloud_call) a.out.cloud_call[w] = (uint8_t)(f < wlen);
                a.ws.window_done[w] = 0;  // ready for the next launch
            }
        }
        __syncthreads();
    }
}

}  // namespace

cudaError_t launch_verify(const VerifyArgs &a, int dtype, cudaStream_t stream)
{
    if (a.rows == 0) return cudaSuccess;
    const int64_t cap = (int64_t)sm_count() * 16;
    const unsigned grid = (unsigned)(a.rows < cap ? a.rows : cap);
    if (dtype == CIAR_F32) verify_kernel<float><<<grid, kThreads, 0, stream>>>(a);
    else verify_kernel<__nv_bfloat16><<<grid, kThreads, 0, stream>>>(a);
    count_launch();
    return cudaGetLastError();
}

}  // namespace ciar
