// Soft voting over several Inter-Heads: the heads' softmax distributions are averaged code by code and the
// interval quantities are formed around the averaged distribution with the mean of the heads' radii.
//
// One CTA of 256 threads per row.  Per head a statistics pass (maximum, sum of exponentials); then one sweep
// over the codes that forms pbar_i = (1/H) sum_h exp(c^h_i - m_h) / Z_h (one exponential per head and code),
// its entropy term, and the bounds of the code from pbar_i (InterFuse rewritten in the probability).  A code
// that holds more than half of the mass is kept out of the sweep: its 1 - p is the sum of the others, known
// only after the reduction, and its terms are added then.  Each head's row comes from HBM once; the second
// visit (and the third, for rows with nearly equal widths or a dense dump) hits L1 / L2.
#include "ciar_internal.h"
#include "interval_math.cuh"

namespace ciar {

namespace {

struct HeadsShared {
    float fs[kWarps];
    double ds[8 * kWarps];
    float m2[CIAR_MAX_HEADS];
    float inv[CIAR_MAX_HEADS];  // 1 / (H * Z_h), Z_h as summed (same exponent offset as the sweep's terms)
};

template <typename T>
__global__ void __launch_bounds__(kThreads) ensemble_kernel(EnsembleArgs a)
{
    constexpr int V = Elem<T>::kVec;
    __shared__ HeadsShared sh;
    const int tid = threadIdx.x;
    const ciar_quantify_out &o = a.out;
    const int H = a.n_heads;
    const int vec_begin = a.vb / V, vec_end = (a.vb + a.n + V - 1) / V;

    for (int64_t row = blockIdx.x; row < a.rows; row += gridDim.x) {
        const T *hrow = reinterpret_cast<const T *>(a.heads) + row * a.row_stride;
        int status = 0;
        double rsum = 0.0;
        for (int h = 0; h < H; ++h) {
            const RowView<T> rv(hrow + (size_t)h * a.head_stride, a.vb, a.n);
            RowStats st;
            row_stats(rv, sh.fs, sh.ds, st);
            if (st.m == -INFINITY) status |= CIAR_ROW_NO_FINITE;
            else if (!(st.z_raw < INFINITY) || !(st.z_raw > 0.0)) status |= CIAR_ROW_NAN;
            double r = (double)a.r_scalar;
            if (a.radius_mode == CIAR_RADIUS_PER_ROW) r = (double)a.radius[(int64_t)h * a.rows + row];
            if (!(r == r)) status |= CIAR_ROW_NAN;
            rsum += clamp_radius(r, a.radius_is_raw, (double)a.r_max);
            __syncthreads();  // the statistics' scratch is free again
            if (tid == 0) {
                sh.m2[h] = st.m2;
                sh.inv[h] = (float)(1.0 / ((double)H * st.z_raw));
            }
        }
        __syncthreads();
        float *dp = o.dense_p ? o.dense_p + row * (int64_t)a.n : nullptr;
        if (status) {
            const float nanv = __int_as_float(0x7fc00000);
            if (tid == 0) {
                if (o.p_max) o.p_max[row] = nanv;
                if (o.entropy) o.entropy[row] = nanv;
                if (o.S_lo) o.S_lo[row] = nanv;
                if (o.S_up) o.S_up[row] = nanv;
                if (o.omega) o.omega[row] = nanv;
                if (o.sigma) o.sigma[row] = nanv;
                if (o.score) o.score[row] = nanv;
                if (o.flag) o.flag[row] = 1;
                if (o.row_status) o.row_status[row] = (uint8_t)status;
            }
            if (dp)
                for (int i = tid; i < a.n; i += kThreads) dp[i] = nanv;
            continue;
        }
        const RadiusConst krow = radius_const(rsum / (double)H);

        // the averaged probability of the V codes of vector vi
        auto averaged = [&](int vi, float (&p)[V]) -> int {
            int i0 = 0;
#pragma unroll
            for (int k = 0; k < V; ++k) p[k] = 0.f;
            for (int h = 0; h < H; ++h) {
                const RowView<T> rv(hrow + (size_t)h * a.head_stride, a.vb, a.n);
                float v[V];
                i0 = rv.load(vi, v, -INFINITY);
                const float m2 = sh.m2[h], inv = sh.inv[h];
#pragma unroll
                for (int k = 0; k < V; ++k) p[k] = fmaf(ex2_approx(fmaf(v[k], kLog2e, -m2)), inv, p[k]);
            }
            return i0;
        };

        double acc[8] = { 0, 0, 0, 0, 0, 0, 0, 0 };  // A, B, AA, AB, BB, sum p ln p, sum of the non-dominant p, dominant p
        float pm = 0.f;
        for (int vi = vec_begin + tid; vi < vec_end; vi += kThreads) {
            float p[V];
            const int i0 = averaged(vi, p);
            float sA = 0.f, sB = 0.f, sAA = 0.f, sAB = 0.f, sBB = 0.f, sH = 0.f, sP = 0.f;
#pragma unroll
            for (int k = 0; k < V; ++k) {
                const int i = i0 + k;
                if (i < 0 || i >= a.n) continue;
                const float pk = p[k];
                pm = fmaxf(pm, pk);
                if (pk > 0.f) sH = fmaf(pk, __logf(pk), sH);
                if (pk > 0.5f) {
                    acc[7] += (double)pk;  // at most one code of the row
                    continue;
                }
                sP += pk;
                float pl, d;
                bounds_from_p_omp(pk, 1.0f - pk, krow, pl, d);
                sA += d;
                sB += pl;
                sAA = fmaf(d, d, sAA);
                sAB = fmaf(d, pl, sAB);
                sBB = fmaf(pl, pl, sBB);
            }
            acc[0] += (double)sA; acc[1] += (double)sB; acc[2] += (double)sAA; acc[3] += (double)sAB;
            acc[4] += (double)sBB; acc[5] += (double)sH; acc[6] += (double)sP;
        }
        block_sum<8>(acc, sh.ds);
        pm = block_max(pm, sh.fs);
        const float pdom = (float)acc[7], omp_dom = (float)acc[6];
        if (acc[7] > 0.0) {
            float pl, d;
            bounds_from_p_omp(pdom, omp_dom, krow, pl, d);
            acc[0] += (double)d;
            acc[1] += (double)pl;
            acc[2] += (double)d * (double)d;
            acc[3] += (double)d * (double)pl;
            acc[4] += (double)pl * (double)pl;
        }
        const double nn = (double)a.n;
        const ScoreParts sp = score_parts(acc[0], acc[1], acc[2], acc[3], acc[4], nn, (double)a.lo_cap, (double)a.hi_cap);
        double var = sp.var;
        const bool low_cv = !(var >= 0.1 * sp.mu * sp.mu);
        if (low_cv || dp) {
            const float fku = (float)sp.k_up, fg = (float)sp.g, fmu = (float)sp.mu;
            double dev[1] = { 0.0 };
            for (int vi = vec_begin + tid; vi < vec_end; vi += kThreads) {
                float p[V];
                const int i0 = averaged(vi, p);
                float s = 0.f;
#pragma unroll
                for (int k = 0; k < V; ++k) {
                    const int i = i0 + k;
                    if (i < 0 || i >= a.n) continue;
                    const float pk = p[k];
                    float pl, d;
                    bounds_from_p_omp(pk, pk > 0.5f ? omp_dom : 1.0f - pk, krow, pl, d);
                    const float x = fmaf(fku, d, fg * pl) - fmu;
                    s = fmaf(x, x, s);
                    if (dp) dp[i] = pk;
                }
                dev[0] += (double)s;
            }
            block_sum<1>(dev, sh.ds);
            if (low_cv) var = dev[0] / nn;
        }
        const double sigma = sqrt(var > 0.0 ? var : 0.0);
        const double score = sp.omega * sigma;
        if (tid == 0) {
            if (o.p_max) o.p_max[row] = pm;
            if (o.entropy) o.entropy[row] = (float)(-acc[5]);
            if (o.S_lo) o.S_lo[row] = (float)sp.S_lo;
            if (o.S_up) o.S_up[row] = (float)sp.S_up;
            if (o.omega) o.omega[row] = (float)sp.omega;
            if (o.sigma) o.sigma[row] = (float)sigma;
            if (o.score) o.score[row] = (float)score;
            if (o.flag) o.flag[row] = (uint8_t)(score > (double)a.tau);
            if (o.row_status) o.row_status[row] = 0;
        }
    }
}

}  // namespace

cudaError_t launch_ensemble(const EnsembleArgs &a, int dtype, cudaStream_t stream)
{
    if (a.rows == 0) return cudaSuccess;
    const int64_t cap = (int64_t)sm_count() * 8;
    const unsigned grid = (unsigned)(a.rows < cap ? a.rows : cap);
    if (dtype == CIAR_F32) ensemble_kernel<float><<<grid, kThreads, 0, stream>>>(a);
    else ensemble_kernel<__nv_bfloat16><<<grid, kThreads, 0, stream>>>(a);
    count_launch();
    return cudaGetLastError();
}

}  // namespace ciar
