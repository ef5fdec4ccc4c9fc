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
    if (threadIdx.x == 0) {
        sh_i[0] = -1;
        sh_i[1] = 0x7fffffff;
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
        // exactly one thread has excl <= thr < incl (threads with part == 0 never qualify)
        if (excl <= thr && thr < incl) {
            double cum = excl;
            int32_t pick = -1, last_pos = -1;
            for (int32_t vi = v0; vi < v1 && pick < 0; ++vi) {
                float tv[V], cv[V], rs[V];
                const int32_t i0 = rt.load(vi, tv, -INFINITY);
                rd.load(vi, cv, -INFINITY);
                float s = 0.f;
#pragma unroll
                for (int k = 0; k < V; ++k) {
                    rs[k] = residual_term(tv[k], cv[k], mq, mp, ratio);
                    s += rs[k];
                }
                if (cum + (double)s > thr) {
                    double c2 = cum;
#pragma unroll
                    for (int k = 0; k < V; ++k) {
                        if (rs[k] > 0.f) last_pos = i0 + k;
                        c2 += (double)rs[k];
                        if (pick < 0 && rs[k] > 0.f && c2 > thr) pick = i0 + k;
                    }
                    if (pick < 0) pick = last_pos;  // rounding: the crossing is at the vector's end
                } else {
                    cum += (double)s;
#pragma unroll
                    for (int k = 0; k < V; ++k)
                        if (rs[k] > 0.f) last_pos = i0 + k;
                }
            }
            if (pick < 0) pick = last_pos;
            sh_i[0] = pick;
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
