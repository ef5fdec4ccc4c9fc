// Forward value of the Inter-DRO loss: per row the L1 distances and cross-entropies of the three device
// distributions (centre, upper, lower logits) against the cloud distribution and the KL term of the centre,
// then one small kernel for the batch means and the softmax re-weighting of the lower bound's cross-entropies.
//
// Row kernel: one CTA of 256 threads per row; the row's three tensors (centre logits, radii, cloud logits) are
// copied to shared memory once when they fit (3 x 32 KB), so HBM is read once, and three sweeps run from there:
//   1. maxima of c, c + r, c - r and t;
//   2. sums of 2^(o L - m2) for the four, and the cloud-weighted sums  sum e_t c, sum e_t r, sum e_t (t - c):
//      with q_i = e_t,i / Z_t they give CE_x = lse_x - E_q[o_x] and KL = E_q[t - c] - (lse_t - lse_mid) without a
//      pass of their own;
//   3. the L1 distances from normalised probabilities p = 2^(o L - lse2), lse2 = m2 + log2 Z held as a float pair.
// L is the float constant log2(e); m2 = fl(m L).  The exponent of c +- r is formed as (c L - ref) +- r L, never from
// the float sum c + r, whose rounding (1e-6 of a logit near 30) would show in the probabilities of the large codes.
#include "ciar_internal.h"

namespace ciar {

namespace {

constexpr int kDroStageBytes = 96 * 1024;

struct DroShared {
    float fs[4 * kWarps];
    double ds[8 * kWarps];
};

// Block-wide maxima of four values at once.
__device__ __forceinline__ void block_max4(float (&v)[4], float *scratch)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int k = 0; k < 4; ++k) v[k] = warp_max(v[k]);
    __syncthreads();
    if (lane == 0) {
#pragma unroll
        for (int k = 0; k < 4; ++k) scratch[k * kWarps + warp] = v[k];
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        float r = scratch[k * kWarps];
#pragma unroll
        for (int w = 1; w < kWarps; ++w) r = fmaxf(r, scratch[k * kWarps + w]);
        v[k] = r;
    }
}

// r = min(Softplus(rho), r_max) (or min(rho, r_max) for a stored radius)
__device__ __forceinline__ float code_radius_f(float rho, int raw, float r_max)
{
    float r = rho;
    if (raw) r = fmaxf(rho, 0.f) + __logf(1.0f + ex2_approx(-fabsf(rho) * kLog2e));
    return fminf(r, r_max);
}

template <typename T>
__global__ void __launch_bounds__(kThreads) interdro_rows_kernel(InterDroArgs a, int staged)
{
    constexpr int V = Elem<T>::kVec;
    extern __shared__ __align__(16) unsigned char dro_stage[];
    __shared__ DroShared sh;
    const int tid = threadIdx.x;
    const int vec_begin = a.vb / V, vec_end = (a.vb + a.n + V - 1) / V, nvec = vec_end - vec_begin;
    const int raw = a.prm.radius_is_raw;
    const float r_max = a.prm.r_max;

    for (int64_t row = blockIdx.x; row < a.rows; row += gridDim.x) {
        const T *gc = reinterpret_cast<const T *>(a.center) + row * a.row_stride;
        const T *gr = reinterpret_cast<const T *>(a.radius) + row * a.row_stride;
        const T *gt = reinterpret_cast<const T *>(a.cloud) + row * a.row_stride;
        __syncthreads();  // the previous row is no longer read
        if (staged) {
            uint4 *dst = reinterpret_cast<uint4 *>(dro_stage);
            const uint4 *s0 = reinterpret_cast<const uint4 *>(gc) + vec_begin;
            const uint4 *s1 = reinterpret_cast<const uint4 *>(gr) + vec_begin;
            const uint4 *s2 = reinterpret_cast<const uint4 *>(gt) + vec_begin;
            for (int vi = tid; vi < nvec; vi += kThreads) {
                dst[vi] = s0[vi];
                dst[nvec + vi] = s1[vi];
                dst[2 * nvec + vi] = s2[vi];
            }
            __syncthreads();
        }
        const T *sbase = reinterpret_cast<const T *>(dro_stage);
        const RowView<T> vc(staged ? sbase - (size_t)vec_begin * V : gc, a.vb, a.n);
        const RowView<T> vr(staged ? sbase + (size_t)nvec * V - (size_t)vec_begin * V : gr, a.vb, a.n);
        const RowView<T> vt(staged ? sbase + (size_t)2 * nvec * V - (size_t)vec_begin * V : gt, a.vb, a.n);

        // ---- 1. maxima: [0] c, [1] c + r, [2] c - r, [3] t
        float mx[4] = { -INFINITY, -INFINITY, -INFINITY, -INFINITY };
        for (int vi = vec_begin + tid; vi < vec_end; vi += kThreads) {
            float c[V], rho[V], t[V];
            vc.load(vi, c, -INFINITY);
            vr.load(vi, rho, 0.f);
            vt.load(vi, t, -INFINITY);
#pragma unroll
            for (int k = 0; k < V; ++k) {
                const float r = code_radius_f(rho[k], raw, r_max);
                mx[0] = fmaxf(mx[0], c[k]);
                mx[1] = fmaxf(mx[1], c[k] + r);
                mx[2] = fmaxf(mx[2], c[k] - r);
                mx[3] = fmaxf(mx[3], t[k]);
            }
        }
        block_max4(mx, sh.fs);
        float m2[4];
#pragma unroll
        for (int x = 0; x < 4; ++x) m2[x] = mx[x] * kLog2e;

        // ---- 2. sums: [0..3] Z of c, c + r, c - r, t; [4] sum e_t c, [5] sum e_t r, [6] sum e_t (t - c)
        double acc[8] = { 0, 0, 0, 0, 0, 0, 0, 0 };
        for (int vi = vec_begin + tid; vi < vec_end; vi += kThreads) {
            float c[V], rho[V], t[V];
            vc.load(vi, c, -INFINITY);
            vr.load(vi, rho, 0.f);
            vt.load(vi, t, -INFINITY);
            float s[7] = { 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f };
#pragma unroll
            for (int k = 0; k < V; ++k) {
                const float r = code_radius_f(rho[k], raw, r_max);
                s[0] += ex2_approx(fmaf(c[k], kLog2e, -m2[0]));
                s[1] += ex2_approx(fmaf(r, kLog2e, fmaf(c[k], kLog2e, -m2[1])));
                s[2] += ex2_approx(fmaf(-r, kLog2e, fmaf(c[k], kLog2e, -m2[2])));
                const float et = ex2_approx(fmaf(t[k], kLog2e, -m2[3]));
                s[3] += et;
                if (et > 0.f) {  // a code the cloud gives no mass: its terms are 0 whatever the device logits
                    s[4] = fmaf(et, c[k], s[4]);
                    s[5] = fmaf(et, r, s[5]);
                    s[6] = fmaf(et, t[k] - c[k], s[6]);
                }
            }
#pragma unroll
            for (int q = 0; q < 7; ++q) acc[q] += (double)s[q];
        }
        block_sum<8>(acc, sh.ds);
        // base-2 log-sum-exp of o L for the four logit vectors, natural lse = lse2 / L
        double lse2[4], lse[4];
        float hi[4], lo[4];
#pragma unroll
        for (int x = 0; x < 4; ++x) {
            lse2[x] = (double)m2[x] + log2(acc[x]);
            lse[x] = lse2[x] / (double)kLog2e;
            hi[x] = (float)lse2[x];
            lo[x] = (float)(lse2[x] - (double)hi[x]);
        }
        const double eq_c = acc[4] / acc[3], eq_r = acc[5] / acc[3], eq_d = acc[6] / acc[3];
        const double ce_mid = lse[0] - eq_c, ce_up = lse[1] - (eq_c + eq_r), ce_lo = lse[2] - (eq_c - eq_r);
        const double kl = eq_d - (lse[3] - lse[0]);

        // ---- 3. L1 distances.  A code that holds more than half of the mass on both sides is left out of the
        // sum: the difference of two probabilities near 1 has no digits left in float, while their complements
        // (the sums over all the other codes) do, and p - q = (1 - q) - (1 - p).
        double l1[3] = { 0, 0, 0 };
        double oth[8] = { 0, 0, 0, 0, 0, 0, 0, 0 };  // per x: sum of the other codes' p, of their q; [6] codes left out
        for (int vi = vec_begin + tid; vi < vec_end; vi += kThreads) {
            float c[V], rho[V], t[V];
            const int i0 = vc.load(vi, c, -INFINITY);
            vr.load(vi, rho, 0.f);
            vt.load(vi, t, -INFINITY);
            float s[3] = { 0.f, 0.f, 0.f }, sp[3] = { 0.f, 0.f, 0.f }, sq[3] = { 0.f, 0.f, 0.f };
            int left_out = 0;
#pragma unroll
            for (int k = 0; k < V; ++k) {
                if (i0 + k < 0 || i0 + k >= a.n) continue;
                const float r = code_radius_f(rho[k], raw, r_max);
                const float q = ex2_approx(fmaf(t[k], kLog2e, -hi[3]) - lo[3]);
                float px[3];
                px[0] = ex2_approx(fmaf(c[k], kLog2e, -hi[0]) - lo[0]);
                px[1] = ex2_approx(fmaf(r, kLog2e, fmaf(c[k], kLog2e, -hi[1])) - lo[1]);
                px[2] = ex2_approx(fmaf(-r, kLog2e, fmaf(c[k], kLog2e, -hi[2])) - lo[2]);
#pragma unroll
                for (int x = 0; x < 3; ++x) {
                    if (q > 0.5f && px[x] > 0.5f) {
                        left_out |= 1 << x;
                    } else {
                        s[x] += fabsf(px[x] - q);
                        sp[x] += px[x];
                        sq[x] += q;
                    }
                }
            }
#pragma unroll
            for (int x = 0; x < 3; ++x) {
                l1[x] += (double)s[x];
                oth[2 * x] += (double)sp[x];
                oth[2 * x + 1] += (double)sq[x];
            }
            oth[6] += (double)left_out;  // at most one code of a row is left out per x: the bits add up without carries
        }
        block_sum<3>(l1, sh.ds);
        block_sum<8>(oth, sh.ds);
        {
            const int left_out = (int)oth[6];
#pragma unroll
            for (int x = 0; x < 3; ++x)
                if ((left_out >> x) & 1) l1[x] += fabs(oth[2 * x + 1] - oth[2 * x]);
        }
        if (tid == 0) {
            const double vals[7] = { l1[0], l1[1], l1[2], ce_mid, ce_up, ce_lo, kl };
#pragma unroll
            for (int q = 0; q < 7; ++q) a.ws[(int64_t)q * a.rows + row] = vals[q];
            if (a.out.l1) {
                a.out.l1[row] = (float)l1[0];
                a.out.l1[a.rows + row] = (float)l1[1];
                a.out.l1[2 * a.rows + row] = (float)l1[2];
            }
            if (a.out.ce) {
                a.out.ce[row] = (float)ce_mid;
                a.out.ce[a.rows + row] = (float)ce_up;
                a.out.ce[2 * a.rows + row] = (float)ce_lo;
            }
            if (a.out.kl) a.out.kl[row] = (float)kl;
        }
    }
}

constexpr int kRedThreads = 1024;

// Sum (or maximum) of one double per thread over the CTA, in a fixed order; every thread gets the result.
template <bool MAX>
__device__ __forceinline__ double red_block(double v, double *scratch)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const double u = __shfl_xor_sync(0xffffffffu, v, o);
        v = MAX ? fmax(v, u) : v + u;
    }
    __syncthreads();
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    double r = scratch[0];
    for (int w = 1; w < kRedThreads / 32; ++w) r = MAX ? fmax(r, scratch[w]) : r + scratch[w];
    return r;
}

// Batch reduction: means of the per-row terms, softmax weights of alpha * CE_lo over the rows, the loss parts.
__global__ void __launch_bounds__(kRedThreads) interdro_reduce_kernel(InterDroArgs a)
{
    __shared__ double scratch[kRedThreads / 32];
    const int64_t rows = a.rows;
    double mean[7];
    for (int q = 0; q < 7; ++q) {
        double s = 0.0;
        for (int64_t r = threadIdx.x; r < rows; r += kRedThreads) s += a.ws[(int64_t)q * rows + r];
        mean[q] = red_block<false>(s, scratch) / (double)rows;
    }
    const double *cel = a.ws + 5 * rows;
    const double alpha = (double)a.prm.alpha;
    double mx = -INFINITY;
    for (int64_t r = threadIdx.x; r < rows; r += kRedThreads) mx = fmax(mx, alpha * cel[r]);
    mx = red_block<true>(mx, scratch);
    double zs = 0.0;
    for (int64_t r = threadIdx.x; r < rows; r += kRedThreads) zs += exp(alpha * cel[r] - mx);
    zs = red_block<false>(zs, scratch);
    double dro = 0.0;
    for (int64_t r = threadIdx.x; r < rows; r += kRedThreads) {
        const double w = exp(alpha * cel[r] - mx) / zs;
        if (a.out.weights) a.out.weights[r] = (float)w;
        dro += w * cel[r];
    }
    dro = red_block<false>(dro, scratch);
    if (threadIdx.x == 0 && a.out.loss) {
        const double lv = (double)a.prm.lambda_v, lp = (double)a.prm.lambda_p;
        const double anchor_mid = lv * mean[0] + lp * mean[3];
        const double anchor_up = lv * mean[1] + lp * mean[4];
        const double anchor_lo = lv * mean[2] + lp * mean[5];
        const double align = (double)a.prm.lambda_beta * mean[6];
        a.out.loss[1] = (float)(anchor_mid + align);
        a.out.loss[2] = (float)anchor_up;
        a.out.loss[3] = (float)(anchor_lo + dro);
        a.out.loss[4] = (float)dro;
        a.out.loss[5] = (float)align;
        a.out.loss[0] = (float)(anchor_mid + align + anchor_up + anchor_lo + dro);
    }
}

template <typename T>
cudaError_t launch_interdro_typed(const InterDroArgs &a, cudaStream_t stream)
{
    constexpr int V = Elem<T>::kVec;
    const int nvec = (a.vb + a.n + V - 1) / V - a.vb / V;
    const int staged = (size_t)nvec * 48 <= (size_t)kDroStageBytes ? 1 : 0;
    const size_t smem = staged ? (size_t)nvec * 48 : 0;
    static bool attr_set = false;
    if (!attr_set) {
        const cudaError_t err = cudaFuncSetAttribute(interdro_rows_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, kDroStageBytes);
        if (err != cudaSuccess) return err;
        attr_set = true;
    }
    const int64_t cap = (int64_t)sm_count() * 2;
    const unsigned grid = (unsigned)(a.rows < cap ? a.rows : cap);
    interdro_rows_kernel<T><<<grid, kThreads, smem, stream>>>(a, staged);
    count_launch();
    cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) return err;
    interdro_reduce_kernel<<<1, kRedThreads, 0, stream>>>(a);
    count_launch();
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_interdro(const InterDroArgs &a, int dtype, cudaStream_t stream)
{
    if (dtype == CIAR_F32) return launch_interdro_typed<float>(a, stream);
    return launch_interdro_typed<__nv_bfloat16>(a, stream);
}

}  // namespace ciar
