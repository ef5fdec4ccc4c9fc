// Residual resampling of one rejected row by a whole CTA (NT threads): the token drawn from
// norm(max(0, q - p)) by inverse CDF, p = softmax(draft row), q = softmax(target row).
#pragma once

#include "ciar_device.cuh"

namespace ciar {

__device__ __forceinline__ float residual_term(float t, float c, float mq, float mp, float ratio)
{
    // exp(t - mq) - ratio * exp(c - mp) = zq * (q_i - p_i) with ratio = zq / zp
    const float eq = ex2_approx((t - mq) * kLog2e);
    const float ep = ex2_approx((c - mp) * kLog2e);
    return fmaxf(fmaf(-ratio, ep, eq), 0.0f);
}

// Smallest code k whose cumulative residual exceeds u * total (cumulated in code order); the last
// code with a positive residual if rounding leaves none; the mode of q (lowest index) when the
// residual mass is zero.  Returns the global code id.  (mp, zp) / (mq, zq): maximum and sum of
// exp(. - max) of the draft / target row.  scan_warp: NT / 32 doubles, sh_i: 2 ints of shared
// memory.  Every thread of the CTA must call it; all get the result.
template <typename T, int NT>
__device__ __forceinline__ int32_t resample_row(const RowView<T> &rd, const RowView<T> &rt, float mp, double zp, float mq,
                                                double zq, float u_res, int32_t vb, double *scan_warp, int *sh_i)
{
    constexpr int V = Elem<T>::kVec;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    __shared__ double sh_excl;      // of the thread whose run holds the crossing: its exclusive prefix ...
    __shared__ int32_t sh_run[2];  // ... and its run of vectors
    if (threadIdx.x == 0) {
        sh_i[0] = -1;
        sh_i[1] = 0x7fffffff;
        sh_run[0] = sh_run[1] = 0;
        sh_excl = 0.0;
    }
    // Thread t owns a contiguous run of vectors so that a block scan gives code-order prefixes.
    const float ratio = (float)(zq / zp);
    const int32_t nvec = rt.vec_end - rt.vec_begin;
    const int32_t vpt = (nvec + NT - 1) / NT;
    const int32_t v0 = rt.vec_begin + threadIdx.x * vpt;
    const int32_t v1 = min(v0 + vpt, rt.vec_end);
    double part = 0.0;
    for (int32_t vi = v0; vi < v1; ++vi) {
        float tv[V], cv[V];
        rt.load(vi, tv, -INFINITY);
        rd.load(vi, cv, -INFINITY);
        float s = 0.f;
#pragma unroll
        for (int k = 0; k < V; ++k) s += residual_term(tv[k], cv[k], mq, mp, ratio);
        part += (double)s;
    }
    // inclusive block scan of the per-thread partials (double)
    double incl = part;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += up;
    }
    if (lane == 31) scan_warp[warp] = incl;
    __syncthreads();
    double woff = 0.0, total = 0.0;
#pragma unroll
    for (int ww = 0; ww < NT / 32; ++ww) {
        if (ww < warp) woff += scan_warp[ww];
        total += scan_warp[ww];
    }
    incl += woff;
    // exclusive prefix = the previous thread's inclusive prefix, bit for bit, so that the
    // half-open intervals [excl, incl) tile [0, total) without gaps or overlaps
    double excl = __shfl_up_sync(0xffffffffu, incl, 1);
    if (lane == 0) excl = woff;
    int32_t result;
    if (total > 0.0) {
        const double thr = (double)u_res * total;
        // exactly one thread has excl <= thr < incl (threads with part == 0 never qualify): its run of vectors holds the
        // crossing.  The first warp walks that run, a code per lane, 32 codes at a time in code order.
        if (excl <= thr && thr < incl) {
            sh_run[0] = v0;
            sh_run[1] = v1;
            sh_excl = excl;
        }
        __syncthreads();
        if (warp == 0) {
            const int32_t r0 = sh_run[0], ncodes = (sh_run[1] - sh_run[0]) * V;
            double cum = sh_excl;
            int32_t pick = -1, last_pos = -1;
            for (int32_t c0 = 0; c0 < ncodes && pick < 0; c0 += 32) {
                const int32_t e = r0 * V + c0 + lane;  // element of the row
                float rs = 0.f;
                if (c0 + lane < ncodes && e >= rt.vb && e < rt.vb + rt.n)
                    rs = residual_term(Elem<T>::widen(rt.row[e]), Elem<T>::widen(rd.row[e]), mq, mp, ratio);
                double run = (double)rs;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const double up = __shfl_up_sync(0xffffffffu, run, o);
                    if (lane >= o) run += up;
                }
                const unsigned pos = __ballot_sync(0xffffffffu, rs > 0.f);
                const unsigned hit = __ballot_sync(0xffffffffu, rs > 0.f && cum + run > thr);
                if (hit) pick = r0 * V + c0 + (__ffs((int)hit) - 1) - rt.vb;
                else if (pos) last_pos = r0 * V + c0 + (31 - __clz((int)pos)) - rt.vb;
                cum += __shfl_sync(0xffffffffu, run, 31);
            }
            if (pick < 0) pick = last_pos;  // rounding: the crossing is at the run's end
            if (lane == 0) sh_i[0] = pick;
        }
        __syncthreads();
        result = sh_i[0] >= 0 ? sh_i[0] + vb : -1;
    } else {
        // p == q wherever q > 0: fall back to the mode of q (lowest index at the maximum)
        int32_t amin = 0x7fffffff;
        for (int32_t vi = rt.vec_begin + threadIdx.x; vi < rt.vec_end; vi += NT) {
            float tv[V];
            const int32_t i0 = rt.load(vi, tv, -INFINITY);
#pragma unroll
            for (int k = 0; k < V; ++k)
                if (tv[k] == mq) amin = min(amin, i0 + k);
        }
        atomicMin(&sh_i[1], amin);
        __syncthreads();
        result = sh_i[1] + vb;
    }
    __syncthreads();  // the shared scratch may be reused
    return result;
}

}  // namespace ciar
