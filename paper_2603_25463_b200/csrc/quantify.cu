// Device-side uncertainty quantification: row softmax statistics, InterFuse interval sums,
// Omega * Sigma score and the cloud flag.  One CTA per token row; the row is read from HBM once
// (the later sweeps hit L1 / L2).
#include "ciar_internal.h"
#include "interval_math.cuh"

namespace ciar {

namespace {

template <typename T>
__device__ __forceinline__ RadiusConst code_radius(const RowView<T> &, float rho, int raw, float r_max)
{
    float r = rho;
    if (raw) r = (rho > 0.f) ? rho + log1pf(expf(-rho)) : log1pf(expf(rho));
    r = !(r > r_max) ? r : r_max;  // (a NaN radius stays NaN and marks the row)
    RadiusConst k;
    k.alpha = -expm1f(-r);
    k.beta = expm1f(r);
    k.a = 1.0f - k.alpha;
    k.bma = k.alpha + k.beta;
    return k;
}

struct Sums {
    double A, B, AA, AB, BB;  // sum d, sum p^l, sum d^2, sum d p^l, sum (p^l)^2 (raw bounds)
};

template <typename T, bool PER_CODE>
__global__ void __launch_bounds__(kThreads) quantify_kernel(QuantifyArgs a)
{
    constexpr int V = Elem<T>::kVec;
    __shared__ float fs[kWarps];
    __shared__ double ds[5 * kWarps];
    __shared__ int is[kWarps];
    const T *base = reinterpret_cast<const T *>(a.logits);
    const T *rbase = reinterpret_cast<const T *>(a.radius);
    const ciar_quantify_out &o = a.out;

    for (int64_t lr = blockIdx.x; lr < a.rows; lr += gridDim.x) {
        int64_t pr;
        const bool active = map_row(a.rm, lr, pr);
        if (!active) {  // a position past the end of the sequence: nothing to quantify
            if (threadIdx.x == 0) {
                if (o.flag) o.flag[lr] = 0;
                if (o.row_status) o.row_status[lr] = 0;
            }
            continue;
        }
        const RowView<T> rv(base + pr * a.row_stride, a.vb, a.n);
        const RowView<T> rr(rbase + (PER_CODE ? pr * a.row_stride : 0), a.vb, a.n);
        RowStats st;
        row_stats(rv, fs, ds, st);

        int status = 0;
        if (st.m == -INFINITY) status |= CIAR_ROW_NO_FINITE;
        else if (!(st.z_raw < INFINITY) || !(st.z_raw > 0.0)) status |= CIAR_ROW_NAN;  // NaN or +inf logit
        double r_row = (double)a.r_scalar;
        if (!PER_CODE && a.radius_mode == CIAR_RADIUS_PER_ROW) r_row = (double)reinterpret_cast<const float *>(a.radius)[pr];
        if (!PER_CODE && !(r_row == r_row)) status |= CIAR_ROW_NAN;

        float *dp = o.dense_p ? o.dense_p + lr * (int64_t)a.n : nullptr;
        float *dl = o.dense_lo ? o.dense_lo + lr * (int64_t)a.n : nullptr;
        float *du = o.dense_up ? o.dense_up + lr * (int64_t)a.n : nullptr;

        if (status) {
            const float nanv = __int_as_float(0x7fc00000);
            if (threadIdx.x == 0) {
                if (o.row_max) o.row_max[lr] = nanv;
                if (o.sum_exp) o.sum_exp[lr] = nanv;
                if (o.lse) o.lse[lr] = nanv;
                if (o.p_max) o.p_max[lr] = nanv;
                if (o.entropy) o.entropy[lr] = nanv;
                if (o.S_lo) o.S_lo[lr] = nanv;
                if (o.S_up) o.S_up[lr] = nanv;
                if (o.omega) o.omega[lr] = nanv;
                if (o.sigma) o.sigma[lr] = nanv;
                if (o.score) o.score[lr] = nanv;
                if (o.argmax) o.argmax[lr] = -1;
                if (o.flag) o.flag[lr] = 1;
                if (o.row_status) o.row_status[lr] = (uint8_t)status;
            }
            for (int32_t i = threadIdx.x; i < a.n; i += kThreads) {
                if (dp) dp[i] = nanv;
                if (dl) dl[i] = nanv;
                if (du) du[i] = nanv;
            }
            continue;
        }

        const RadiusConst krow = radius_const(clamp_radius(r_row, a.radius_is_raw, (double)a.r_max));
        const float invz = (float)(1.0 / st.z_raw);
        const float m = st.m, m2 = st.m2;

        // interval sweep: the sums that Omega and Sigma are built from, and the arg-max
        double acc[5] = { 0, 0, 0, 0, 0 };
        int32_t amin = 0x7fffffff;
        {
            int32_t vi = rv.vec_begin + threadIdx.x;
            while (vi < rv.vec_end) {
                float sA = 0.f, sB = 0.f, sAA = 0.f, sAB = 0.f, sBB = 0.f;
#pragma unroll 2
                for (int it = 0; it < 8 && vi < rv.vec_end; ++it, vi += kThreads) {
                    float v[V], rho[V];
                    const int32_t i0 = rv.load(vi, v, -INFINITY);
                    if (PER_CODE) rr.load(vi, rho, 0.f);
#pragma unroll
                    for (int k = 0; k < V; ++k) {
                        const float e = ex2_approx(fmaf(v[k], kLog2e, -m2));
                        const float p = e * invz;
                        float pl, d;
                        if (PER_CODE) bounds_from_p(p, code_radius(rr, rho[k], a.radius_is_raw, a.r_max), pl, d);
                        else bounds_from_p(p, krow, pl, d);
                        sA += d;
                        sB += pl;
                        sAA = fmaf(d, d, sAA);
                        sAB = fmaf(d, pl, sAB);
                        sBB = fmaf(pl, pl, sBB);
                        if (v[k] == m) amin = min(amin, i0 + k);
                    }
                }
                acc[0] += (double)sA; acc[1] += (double)sB; acc[2] += (double)sAA;
                acc[3] += (double)sAB; acc[4] += (double)sBB;
            }
        }
        block_sum<5>(acc, ds);
#pragma unroll
        for (int o2 = 16; o2 > 0; o2 >>= 1) amin = min(amin, __shfl_xor_sync(0xffffffffu, amin, o2));
        if ((threadIdx.x & 31) == 0) is[threadIdx.x >> 5] = amin;
        __syncthreads();
        amin = is[0];
#pragma unroll
        for (int w = 1; w < kWarps; ++w) amin = min(amin, is[w]);

        // normalisation step and score, in double (every thread computes the same values)
        const double A = acc[0], B = acc[1], AA = acc[2], AB = acc[3], BB = acc[4];
        if (PER_CODE && (!(A == A) || !(B == B))) {  // a NaN radius among the row's codes: the row is unusable
            const float nanv = __int_as_float(0x7fc00000);
            if (threadIdx.x == 0) {
                if (o.row_max) o.row_max[lr] = nanv;
                if (o.sum_exp) o.sum_exp[lr] = nanv;
                if (o.lse) o.lse[lr] = nanv;
                if (o.p_max) o.p_max[lr] = nanv;
                if (o.entropy) o.entropy[lr] = nanv;
                if (o.S_lo) o.S_lo[lr] = nanv;
                if (o.S_up) o.S_up[lr] = nanv;
                if (o.omega) o.omega[lr] = nanv;
                if (o.sigma) o.sigma[lr] = nanv;
                if (o.score) o.score[lr] = nanv;
                if (o.argmax) o.argmax[lr] = -1;
                if (o.flag) o.flag[lr] = 1;
                if (o.row_status) o.row_status[lr] = (uint8_t)CIAR_ROW_NAN;
            }
            for (int32_t i = threadIdx.x; i < a.n; i += kThreads) {
                if (dp) dp[i] = nanv;
                if (dl) dl[i] = nanv;
                if (du) du[i] = nanv;
            }
            continue;
        }
        const double S_lo = B, S_up = A + B;
        double k_lo = 1.0, k_up = 1.0;
        if (S_lo > 0.0 && (double)a.lo_cap / S_lo < 1.0) k_lo = (double)a.lo_cap / S_lo;
        if (S_up > 0.0 && (double)a.hi_cap / S_up > 1.0) k_up = (double)a.hi_cap / S_up;
        const double g = k_up - k_lo;  // delta_i = k_up d_i + g p^l_i, every term >= 0
        const double omega = k_up * A + g * B;
        const double nn = (double)a.n;
        const double mu = omega / nn;
        double var = (k_up * k_up * AA + 2.0 * k_up * g * AB + g * g * BB) / nn - mu * mu;
        const bool need_dense = dp || dl || du;
        const bool low_cv = !(var >= 0.1 * mu * mu);  // nearly uniform widths: the moment form cancels
        if (low_cv || need_dense) {
            // second look at the row with the scales known: sum (delta_i - mu)^2 directly, dense dumps
            const float fku = (float)k_up, fkl = (float)k_lo, fg = (float)g, fmu = (float)mu;
            double dev[1] = { 0.0 };
            int32_t vi = rv.vec_begin + threadIdx.x;
            while (vi < rv.vec_end) {
                float s = 0.f;
                for (int it = 0; it < 8 && vi < rv.vec_end; ++it, vi += kThreads) {
                    float v[V], rho[V];
                    const int32_t i0 = rv.load(vi, v, -INFINITY);
                    if (PER_CODE) rr.load(vi, rho, 0.f);
#pragma unroll
                    for (int k = 0; k < V; ++k) {
                        const int32_t i = i0 + k;
                        if (i < 0 || i >= a.n) continue;
                        const float e = ex2_approx(fmaf(v[k], kLog2e, -m2));
                        const float p = e * invz;
                        float pl, d;
                        if (PER_CODE) bounds_from_p(p, code_radius(rr, rho[k], a.radius_is_raw, a.r_max), pl, d);
                        else bounds_from_p(p, krow, pl, d);
                        const float x = fmaf(fku, d, fg * pl) - fmu;
                        s = fmaf(x, x, s);
                        if (dp) dp[i] = p;
                        if (dl) dl[i] = fkl * pl;
                        if (du) du[i] = fku * (pl + d);
                    }
                }
                dev[0] += (double)s;
            }
            block_sum<1>(dev, ds);
            if (low_cv) var = dev[0] / nn;
        }
        const double sigma = sqrt(var > 0.0 ? var : 0.0);
        const double score = omega * sigma;
        const double lnz = log(st.z);
        const double entropy = lnz - kLn2D * st.t / st.z;
        const double p_max = 1.0 / st.z;

        if (threadIdx.x == 0) {
            int fl;
            switch (a.policy) {
            case CIAR_POLICY_INTERVAL: fl = score > (double)a.tau; break;
            case CIAR_POLICY_ENTROPY: fl = entropy > (double)a.tau; break;
            case CIAR_POLICY_MAXPROB: fl = p_max < (double)a.tau; break;
            case CIAR_POLICY_RANDOM: fl = a.u_flag[pr] < a.tau; break;
            default: fl = 1; break;
            }
            if (o.row_max) o.row_max[lr] = m;
            if (o.sum_exp) o.sum_exp[lr] = (float)st.z;
            if (o.lse) o.lse[lr] = (float)((double)m + lnz);
            if (o.p_max) o.p_max[lr] = (float)p_max;
            if (o.entropy) o.entropy[lr] = (float)entropy;
            if (o.S_lo) o.S_lo[lr] = (float)S_lo;
            if (o.S_up) o.S_up[lr] = (float)S_up;
            if (o.omega) o.omega[lr] = (float)omega;
            if (o.sigma) o.sigma[lr] = (float)sigma;
            if (o.score) o.score[lr] = (float)score;
            if (o.argmax) o.argmax[lr] = amin + a.vb;
            if (o.flag) o.flag[lr] = (uint8_t)fl;
            if (o.row_status) o.row_status[lr] = 0;
        }
    }
}

}  // namespace

cudaError_t launch_quantify(const QuantifyArgs &a, int dtype, cudaStream_t stream)
{
    if (a.rows == 0) return cudaSuccess;
    if (quantify_stream_eligible(a, dtype)) return launch_quantify_stream(a, dtype, stream);
    if (quantify_wide_eligible(a, dtype)) return launch_quantify_wide(a, dtype, stream);
    if (quantify_percode_eligible(a, dtype)) return launch_quantify_percode(a, dtype, stream);
    const int64_t cap = (int64_t)sm_count() * 16;
    const unsigned grid = (unsigned)(a.rows < cap ? a.rows : cap);
    const bool per_code = a.radius_mode == CIAR_RADIUS_PER_CODE;
    if (dtype == CIAR_F32) {
        if (per_code) quantify_kernel<float, true><<<grid, kThreads, 0, stream>>>(a);
        else quantify_kernel<float, false><<<grid, kThreads, 0, stream>>>(a);
    } else {
        if (per_code) quantify_kernel<__nv_bfloat16, true><<<grid, kThreads, 0, stream>>>(a);
        else quantify_kernel<__nv_bfloat16, false><<<grid, kThreads, 0, stream>>>(a);
    }
    count_launch();
    return cudaGetLastError();
}

}  // namespace ciar
