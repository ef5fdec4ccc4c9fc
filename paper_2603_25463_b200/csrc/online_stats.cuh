// Softmax statistics of a row that arrives in chunks: every warp keeps a running maximum of the codes it has
// seen and, per lane, the sums of exp and of exp * exponent relative to that maximum (in double across chunks,
// in float within one).  When the maximum moves the sums are rescaled; codes whose exponential equals the
// maximum's are counted instead of summed (a term near 1 would cost the small terms their low bits in float).
// The exponent of code c under maximum m is fma(c, log2e, -fl(m * log2e)), as in the on-chip kernels, so the
// joined sums are in the same units as theirs.  sm_100a only.
#pragma once

#include "stream_common.cuh"

namespace ciar {

struct OnlineStats {
    float m_w;      // the warp's running maximum (the same in all its lanes)
    double zd, td;  // this lane's sums of exp and of exp * exponent, codes equal to the maximum left out of zd
    int cnt;        // this lane's codes whose exponential equals the maximum's
    int chunk;      // the first chunk in which the warp met its running maximum

    __device__ __forceinline__ void reset()
    {
        m_w = -INFINITY;
        zd = td = 0.0;
        cnt = 0;
        chunk = 0;
    }
};

// Takes chunk c, landed in `stage`, into the warp's statistics: thread `tg` of the NT that share the chunk owns
// its vectors tg, tg + NT, ... (JV of them when WHOLE, else nj).  WITH_T: the entropy sum is kept too.
template <typename T, int NT, int JV, bool WHOLE, bool WITH_T>
__device__ __forceinline__ void online_sweep(OnlineStats &st, const unsigned char *stage, int tg, int nj, int c)
{
    typedef Vec<T> V;
    constexpr int VEC = Elem<T>::kVec;
    constexpr int NPV = V::kPairs;
    typename V::Max mx = V::max_init();
#pragma unroll
    for (int j = 0; j < JV; ++j)
        if (WHOLE || j < nj) mx = V::fold_max(mx, stage_vec(stage, tg + j * NT));
    const float tmax = V::max_value(mx);
    const float wmc = warp_redux_max(tmax);
    if (wmc > st.m_w) {  // the maximum moves: what was summed so far is rescaled to it (in double)
        if (st.m_w > -INFINITY) {
            const float m2o = st.m_w * kLog2e;
            const double dl = (double)m2o - (double)(wmc * kLog2e);  // change of every exponent
            const double f = exp2(dl);
            const double tot = st.zd + (double)st.cnt * (double)ex2_approx(fmaf(st.m_w, kLog2e, -m2o));
            st.td = f * (st.td + dl * tot);
            st.zd = tot * f;
            st.cnt = 0;
        }
        st.m_w = wmc;
        st.chunk = c;
    }
    if (st.m_w > -INFINITY) {  // else nothing finite so far
        const float m2w = st.m_w * kLog2e;
        float2 z2 = f2(0.f), t2 = f2(0.f);
        {
            const float2 L2 = f2(kLog2e), nm2 = f2(-m2w);
#pragma unroll
            for (int j = 0; j < JV; ++j) {
                if (WHOLE || j < nj) {
                    float2 cc[NPV];
                    V::pairs(stage_vec(stage, tg + j * NT), cc);
#pragma unroll
                    for (int q = 0; q < NPV; ++q) {
                        const float2 d = __ffma2_rn(cc[q], L2, nm2);
                        const float2 ev = make_float2(ex2_approx(d.x), ex2_approx(d.y));  // a NaN logit poisons the sums on purpose
                        z2 = __fadd2_rn(z2, ev);
                        if (WITH_T) t2 = __ffma2_rn(ev, d, t2);  // 0 * -inf = NaN for a -inf logit: redone below
                    }
                }
            }
        }
        float zs = z2.x + z2.y, ts = t2.x + t2.y;
        if (WITH_T && !(ts == ts)) {  // a -inf logit or a real NaN: the product of such a code is taken as 0 (a NaN still shows in zs)
            ts = 0.f;
            for (int j = 0; j < nj; ++j) {
                const T *v = reinterpret_cast<const T *>(stage + (size_t)(tg + j * NT) * 16);
#pragma unroll
                for (int q = 0; q < VEC; ++q) {
                    const float d = fmaf(Elem<T>::widen(v[q]), kLog2e, -m2w);
                    ts = fmaf(ex2_approx(d), fmaxf(d, kNegHuge), ts);
                }
            }
        }
        if (wmc == st.m_w) {
            // This chunk holds codes equal to the warp's maximum.  The sum of a thread that holds one is formed again
            // without them, by the whole warp, a code per lane; they are counted instead.
            const float e0w = ex2_approx(fmaf(st.m_w, kLog2e, -m2w));
            const int lane = threadIdx.x & 31;
            for (unsigned holders = __ballot_sync(0xffffffffu, tmax == st.m_w); holders != 0; holders &= holders - 1) {
                const int h = __ffs((int)holders) - 1;
                const int htg = (tg & ~31) + h;
                const int hn = (WHOLE ? JV : __shfl_sync(0xffffffffu, nj, h)) * VEC;  // the thread's codes in this chunk
                float zz = 0.f;
                int cnt = 0;
                for (int i = lane; i < hn; i += 32) {
                    const T *v = reinterpret_cast<const T *>(stage + (size_t)(htg + (i / VEC) * NT) * 16);
                    const float ev = ex2_approx(fmaf(Elem<T>::widen(v[i % VEC]), kLog2e, -m2w));
                    if (ev == e0w) ++cnt; else zz += ev;
                }
                zz = warp_sum_f(zz);
                cnt = __reduce_add_sync(0xffffffffu, cnt);
                if (lane == h) {
                    zs = zz;
                    st.cnt += cnt;
                }
            }
        }
        st.zd += (double)zs;
        if (WITH_T) st.td += (double)ts;
    }
}

// The warp's share, summed over its lanes (all lanes get the sums).
__device__ __forceinline__ void online_warp_totals(const OnlineStats &st, double &zw, double &tw, int &cw)
{
    zw = st.zd;
    tw = st.td;
    cw = st.cnt;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        zw += __shfl_xor_sync(0xffffffffu, zw, o);
        tw += __shfl_xor_sync(0xffffffffu, tw, o);
        cw += __shfl_xor_sync(0xffffffffu, cw, o);
    }
}

// Joins the shares of NW warps (NW a power of two up to 32; arrays in shared memory, complete): lane w takes
// warp w's share, rescales it to the row maximum, and the lanes add up.  Every lane of the calling warp gets the
// row maximum m, the sum zc of exponentials without the nc codes equal to the maximum, and the entropy sum tc.
template <int NW>
__device__ __forceinline__ void online_join(const float *wm, const double *wz, const double *wt, const int *wcnt, int lane, float &m,
                                            double &zc, double &tc, int &nc)
{
    const int w = lane & (NW - 1);
    const float mw = wm[w];
    m = warp_redux_max(mw);
    const float m2 = m * kLog2e;
    zc = tc = 0.0;
    nc = 0;
    if (mw > -INFINITY) {
        const double zw = wz[w], tw = wt ? wt[w] : 0.0;
        const int cw = wcnt[w];
        if (mw == m) {
            zc = zw;
            tc = tw;
            nc = cw;
        } else {
            const float mw2 = mw * kLog2e;
            const double dl = (double)mw2 - (double)m2;
            const double f = exp2(dl);
            const double tot = zw + (double)cw * (double)ex2_approx(fmaf(mw, kLog2e, -mw2));
            zc = tot * f;
            tc = f * (tw + dl * tot);
        }
    }
#pragma unroll
    for (int o = NW / 2; o > 0; o >>= 1) {
        zc += __shfl_xor_sync(0xffffffffu, zc, o);
        tc += __shfl_xor_sync(0xffffffffu, tc, o);
        nc += __shfl_xor_sync(0xffffffffu, nc, o);
    }
}

}  // namespace ciar
