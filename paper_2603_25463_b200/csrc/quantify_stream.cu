// Streaming quantifier for rows that fit on chip (up to 16384 codes, scalar or per-row radius).
//
// One persistent CTA walks rows blockIdx.x, blockIdx.x + gridDim.x, ...  Rows arrive through a
// ring of shared-memory stages filled by bulk (TMA) copies that one thread issues several rows
// ahead, so HBM always has requests in flight.  16 consumer warps take a landed row into
// registers (32 codes per thread), find the maximum, exponentiate once (one MUFU op per code),
// and accumulate the interval sums from the exponentials they still hold; a 17th warp, fed
// through a small hand-off buffer, does the per-row double-precision arithmetic and the stores,
// off the consumers' critical path.  Each logit is read from HBM once and from shared memory once.
#include <climits>

#include "ciar_internal.h"
#include "stream_common.cuh"

namespace ciar {

namespace {

constexpr int kQConsumers = 512;
constexpr int kQWarps = kQConsumers / 32;
constexpr int kQBlock = kQConsumers + 32;  // + the finalizer warp
constexpr int kQStages = 3;
constexpr int kBarConsumers = 1, kBarFull = 2, kBarFree = 3;  // named barriers
constexpr long long kWaitCycles = 2000000000ll;                // bound of a wait for a row (about a second)
constexpr long long kDrainCycles = 20000000ll;                 // bound of each wait while leaving after a failure
// Logits at or below -2^120 are treated as -inf (their exponential is 0 either way); the floor
// keeps 0 * (-inf) out of the entropy sum.
constexpr float kLogitFloor = -1.329227995784916e36f;
constexpr uint32_t kLogitFloorBf16x2 = 0xFB80FB80u;

// Interval constants of one row.  With x = softmax probability and s = 1 - x the raw bounds are
//   p^l = a1 x / den_l,  p^u - p^l = kd x s / (den_l den_u),  den_l = a1 + b1 s,  den_u = a1 + b1 x,
// where (a1, b1, kd) = (1, beta, beta (2 + beta)) for beta = e^r - 1 <= 1 and (1 / beta, 1, 1 + 2 / beta)
// otherwise (the second form keeps every term in range for radii up to 80).
struct RowConst {
    float a1, b1;
    float pl0, dd0;  // the two raw terms at x = 1 / n: the sums are accumulated about these values
    float r;         // clamped radius; NaN marks an unusable radius
    int big;
};

struct RowInfo {
    long long lr, pr;
    float m, e0;  // row maximum; the exponential of a code equal to it, as the consumers computed it
    int argmin, nmax;
    int status;  // CIAR_ROW_* bits found by the consumers (0 = a regular row)
    int cmd;     // 0 = finalize this row, 1 = no more rows
    RowConst rc;
    float2 zt[kQWarps];  // per-warp sums of exp and of exp * exponent
};

struct QShared {
    unsigned long long full[kQStages];
    float wmax[kQWarps];
    float wz[kQWarps];
    RowConst rc[2];
    int argmin, nmax;  // lowest index holding the row maximum, number of codes equal to it
    int bad_nan, bad_finite;
    int abort;
    RowInfo info;
    float part[5][kQConsumers];
};

__device__ __forceinline__ RowConst make_row_const(float rho, int raw, float r_max, int n)
{
    RowConst k;
    float r = rho;
    if (raw) r = (rho > 0.f) ? rho + log1pf(expf(-rho)) : log1pf(expf(rho));  // Softplus, beta = 1
    r = fminf(r, r_max);                                                     // NaN stays NaN
    if (!(rho == rho)) r = rho;
    k.r = r;
    const float beta = expm1f(r);
    k.big = beta > 1.0f;
    if (k.big) {
        k.a1 = 1.0f / beta;
        k.b1 = 1.0f;
    } else {
        k.a1 = 1.0f;
        k.b1 = beta;
    }
    const float x0 = 1.0f / (float)n, s0 = 1.0f - x0;
    const float den_l = fmaf(k.b1, s0, k.a1), den_u = fmaf(k.b1, x0, k.a1);
    const float xr = x0 / (den_l * den_u);
    k.pl0 = k.a1 * (xr * den_u);
    k.dd0 = xr * s0;
    return k;
}

// The codes one consumer thread owns: JV 16-byte vectors, vector j being number tid + 512 j of
// the row.  load() takes them from the landed stage and returns the thread's maximum.
template <typename T, int JV>
struct ThreadRow;

template <int JV>
struct ThreadRow<__nv_bfloat16, JV> {
    uint4 w[JV];

    __device__ __forceinline__ float load(const unsigned char *stage, int tid, int nj)
    {
        uint32_t mx = kLogitFloorBf16x2;
#pragma unroll
        for (int j = 0; j < JV; ++j) {
            if (j < nj) {
                uint4 v = *reinterpret_cast<const uint4 *>(stage + (size_t)(tid + j * kQConsumers) * 16);
                // floor the logits (NaN is kept so that it still poisons the sums), then the running maximum
                asm("max.NaN.bf16x2 %0, %0, %1;" : "+r"(v.x) : "r"(kLogitFloorBf16x2));
                asm("max.NaN.bf16x2 %0, %0, %1;" : "+r"(v.y) : "r"(kLogitFloorBf16x2));
                asm("max.NaN.bf16x2 %0, %0, %1;" : "+r"(v.z) : "r"(kLogitFloorBf16x2));
                asm("max.NaN.bf16x2 %0, %0, %1;" : "+r"(v.w) : "r"(kLogitFloorBf16x2));
                mx = bf16x2_max(mx, bf16x2_max(bf16x2_max(v.x, v.y), bf16x2_max(v.z, v.w)));
                w[j] = v;
            }
        }
        const float2 p = unpack_bf16x2(mx);
        return fmaxf(p.x, p.y);
    }
    // slice-relative index of the first owned code equal to m (INT_MAX if none)
    __device__ __forceinline__ int find(float m, int tid, int nj) const
    {
        int best = INT_MAX;
#pragma unroll
        for (int j = JV - 1; j >= 0; --j) {
            if (j < nj) {
                const uint32_t ws[4] = { w[j].x, w[j].y, w[j].z, w[j].w };
#pragma unroll
                for (int q = 3; q >= 0; --q) {
                    const float2 c = unpack_bf16x2(ws[q]);
                    const int i0 = (tid + j * kQConsumers) * 8 + q * 2;
                    if (c.y == m) best = i0 + 1;
                    if (c.x == m) best = i0;
                }
            }
        }
        return best;
    }
    __device__ __forceinline__ float2 pair(int j, int q) const
    {
        const uint32_t ws[4] = { w[j].x, w[j].y, w[j].z, w[j].w };
        return unpack_bf16x2(ws[q]);
    }
    static __device__ __forceinline__ float2 exponent_for_entropy(float2 d) { return d; }  // floored already
};

template <int JV>
struct ThreadRow<float, JV> {
    float4 w[JV];

    __device__ __forceinline__ float load(const unsigned char *stage, int tid, int nj)
    {
        float mx = -INFINITY;
#pragma unroll
        for (int j = 0; j < JV; ++j) {
            if (j < nj) {
                const float4 v = *reinterpret_cast<const float4 *>(stage + (size_t)(tid + j * kQConsumers) * 16);
                mx = fmaxf(mx, fmaxf(fmaxf(v.x, v.y), fmaxf(v.z, v.w)));
                w[j] = v;
            }
        }
        return mx;
    }
    __device__ __forceinline__ int find(float m, int tid, int nj) const
    {
        int best = INT_MAX;
#pragma unroll
        for (int j = JV - 1; j >= 0; --j) {
            if (j < nj) {
                const int i0 = (tid + j * kQConsumers) * 4;
                if (w[j].w == m) best = i0 + 3;
                if (w[j].z == m) best = i0 + 2;
                if (w[j].y == m) best = i0 + 1;
                if (w[j].x == m) best = i0;
            }
        }
        return best;
    }
    __device__ __forceinline__ float2 pair(int j, int q) const
    {
        return q == 0 ? make_float2(w[j].x, w[j].y) : make_float2(w[j].z, w[j].w);
    }
    // -inf logit: exp = 0 and the exponent is floored so that the product is 0, not NaN
    static __device__ __forceinline__ float2 exponent_for_entropy(float2 d)
    {
        return make_float2(fmaxf(d.x, kNegHuge), fmaxf(d.y, kNegHuge));
    }
};

__device__ __forceinline__ double warp_sum_d(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Marks a row as unusable: NaN scores, no arg-max, flagged for the cloud.
__device__ __forceinline__ void write_unusable(const ciar_quantify_out &o, long long lr, int status)
{
    const float nanv = __int_as_float(0x7fc00000);
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

// One row's outputs from its reduced sums (normalisation step, Omega, Sigma, U, entropy, flag).
__device__ __forceinline__ void finalize_one(const QuantifyArgs &a, const double (&s)[5], double zr, double tr,
                                             long long lr, long long pr, float m, int argmin, int status,
                                             const RowConst &rc)
{
    const ciar_quantify_out &o = a.out;
    if (status) {
        write_unusable(o, lr, status);
        return;
    }
    const double nn = (double)a.n;
    const double P1 = s[0], D1 = s[1], PP = s[2], PD = s[3], DD = s[4];
    const double a1 = (double)rc.a1, b1 = (double)rc.b1;
    const double kd = rc.big ? 1.0 + 2.0 * a1 : b1 * (2.0 + b1);
    const double B = nn * (double)rc.pl0 + P1;       // sum of the raw lower bounds
    const double Dsum = nn * (double)rc.dd0 + D1;
    const double A = kd * Dsum;                      // sum of the raw widths
    const double S_lo = B, S_up = A + B;
    double k_lo = 1.0, k_up = 1.0;
    if (S_lo > 0.0 && (double)a.lo_cap / S_lo < 1.0) k_lo = (double)a.lo_cap / S_lo;
    if (S_up > 0.0 && (double)a.hi_cap / S_up > 1.0) k_up = (double)a.hi_cap / S_up;
    // delta_i = k_up d_i + (k_up - k_lo) p^l_i = c1 dd_i + c2 pl_i
    const double c1 = k_up * kd, c2 = k_up - k_lo;
    const double omega = c1 * Dsum + c2 * B;
    const double lin = c1 * D1 + c2 * P1;
    double ss = c1 * c1 * DD + 2.0 * c1 * c2 * PD + c2 * c2 * PP - lin * lin / nn;
    if (!(ss > 0.0)) ss = 0.0;
    const double sigma = sqrt(ss / nn);
    const double score = omega * sigma;
    // exponent actually used: c * log2e_f - m2 = (c - m) * log2e_f + off with off = m * log2e_f - m2
    const double off = (double)m * (double)kLog2e - (double)(m * kLog2e);
    const double unscale = exp2(-off);
    const double z = zr * unscale;
    const double t = tr * unscale - off * z;
    const double lnz = log(z);
    const double entropy = lnz - kLn2D * t / z;
    const double p_max = 1.0 / z;
    int fl;
    switch (a.policy) {
    case CIAR_POLICY_INTERVAL: fl = score > (double)a.tau; break;
    case CIAR_POLICY_ENTROPY: fl = entropy > (double)a.tau; break;
    case CIAR_POLICY_MAXPROB: fl = p_max < (double)a.tau; break;
    case CIAR_POLICY_RANDOM: fl = a.u_flag[pr] < a.tau; break;
    default: fl = 1; break;
    }
    if (o.row_max) o.row_max[lr] = m;
    if (o.sum_exp) o.sum_exp[lr] = (float)z;
    if (o.lse) o.lse[lr] = (float)((double)m + lnz);
    if (o.p_max) o.p_max[lr] = (float)p_max;
    if (o.entropy) o.entropy[lr] = (float)entropy;
    if (o.S_lo) o.S_lo[lr] = (float)S_lo;
    if (o.S_up) o.S_up[lr] = (float)S_up;
    if (o.omega) o.omega[lr] = (float)omega;
    if (o.sigma) o.sigma[lr] = (float)sigma;
    if (o.score) o.score[lr] = (float)score;
    if (o.argmax) o.argmax[lr] = argmin + a.vb;
    if (o.flag) o.flag[lr] = (uint8_t)fl;
    if (o.row_status) o.row_status[lr] = 0;
}

// The finalizer warp: takes the per-thread partial sums of one row from the hand-off buffer,
// adds them up in double and turns them into the row's outputs (normalisation step, Omega,
// Sigma, U, entropy, the flag).
__device__ __noinline__ void finalize_rows(const QuantifyArgs &a, QShared &sh, int lane)
{
    named_bar_arrive(kBarFree, kQBlock);
    for (;;) {
        named_bar_sync(kBarFull, kQBlock);
        if (sh.info.cmd) break;
        double s[5];
#pragma unroll
        for (int k = 0; k < 5; ++k) {
            double acc = 0.0;
#pragma unroll
            for (int i = 0; i < kQConsumers / 32; ++i) acc += (double)sh.part[k][lane + 32 * i];
            s[k] = acc;
        }
        double zr = 0.0, tr = 0.0;
        if (lane < kQWarps) {
            zr = (double)sh.info.zt[lane].x;
            tr = (double)sh.info.zt[lane].y;
        }
        const long long lr = sh.info.lr, pr = sh.info.pr;
        const float m = sh.info.m;
        const int argmin = sh.info.argmin;
        const double zmax = (double)sh.info.nmax * (double)sh.info.e0;  // the maxima, left out of the partial sums
        const int status = sh.info.status;
        const RowConst rc = sh.info.rc;
        named_bar_arrive(kBarFree, kQBlock);  // the consumers may refill the buffer from here on
#pragma unroll
        for (int k = 0; k < 5; ++k) s[k] = warp_sum_d(s[k]);
        zr = warp_sum_d(zr) + zmax;
        tr = warp_sum_d(tr);
        if (lane == 0) finalize_one(a, s, zr, tr, lr, pr, m, argmin, status, rc);
        __syncwarp();
    }
}

template <typename T, int JV, int MINB>
__global__ void __launch_bounds__(kQBlock, MINB) quantify_stream_kernel(QuantifyArgs a)
{
    constexpr int VEC = Elem<T>::kVec;
    constexpr int NPV = VEC / 2;  // float2 pairs per 16-byte vector
    constexpr int NP = JV * NPV;  // pairs per thread
    constexpr int kStageBytes = kQConsumers * JV * 16;
    extern __shared__ __align__(128) unsigned char smem[];
    QShared &sh = *reinterpret_cast<QShared *>(smem + (size_t)kQStages * kStageBytes);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    if (tid == 0) {
#pragma unroll
        for (int s = 0; s < kQStages; ++s) mbar_init(&sh.full[s], 1);
        sh.abort = 0;
        sh.info.cmd = 0;
        mbar_init_fence();
    }
    __syncthreads();
    if (warp == kQWarps) {
        finalize_rows(a, sh, lane);
        return;
    }

    const int nvec = a.n / VEC;
    const uint32_t row_bytes = (uint32_t)nvec * 16u;
    int nj = (nvec - tid + kQConsumers - 1) / kQConsumers;
    nj = nj < 0 ? 0 : (nj > JV ? JV : nj);
    const T *base = reinterpret_cast<const T *>(a.logits) + a.vb;
    const ciar_quantify_out &o = a.out;
    const int64_t stride_rows = gridDim.x;

    // issues the copy of this CTA's k-th row into its stage (thread 0 only)
    auto issue = [&](int k) {
        const int64_t lr = blockIdx.x + (int64_t)k * stride_rows;
        int64_t pr;
        if (lr < a.rows && map_row(a.rm, lr, pr)) {
            const int s = k % kQStages;
            mbar_arrive_expect_tx(&sh.full[s], row_bytes);
            bulk_copy_g2s(smem + (size_t)s * kStageBytes, base + pr * a.row_stride, row_bytes, &sh.full[s]);
        }
    };
    if (tid == 0) {
#pragma unroll
        for (int s = 0; s < kQStages; ++s) issue(s);
    }
    // thread 32 owns the interval constants; a radius shared by all rows is worked out once
    const bool per_row = a.radius_mode == CIAR_RADIUS_PER_ROW;
    if (tid == 32 && !per_row) {
        const RowConst k0 = make_row_const(a.r_scalar, a.radius_is_raw, a.r_max, a.n);
        sh.rc[0] = k0;
        sh.rc[1] = k0;
    }
    float rho_next = 0.f;  // thread 32: the next row's radius, fetched one row ahead
    if (tid == 32 && per_row) {
        int64_t pr;
        if ((int64_t)blockIdx.x < a.rows && map_row(a.rm, blockIdx.x, pr)) rho_next = reinterpret_cast<const float *>(a.radius)[pr];
    }

    uint32_t phases = 0;
    int k = 0;
    bool aborted = false;
    for (;; ++k) {
        const int64_t lr = blockIdx.x + (int64_t)k * stride_rows;
        if (lr >= a.rows) break;
        const int s = k % kQStages;
        int64_t pr;
        const bool active = map_row(a.rm, lr, pr);
        float rho = rho_next;
        if (tid == 32 && per_row) {  // fetch the following row's radius now, use it one trip later
            const int64_t lr2 = lr + stride_rows;
            int64_t pr2;
            if (lr2 < a.rows && map_row(a.rm, lr2, pr2)) rho_next = reinterpret_cast<const float *>(a.radius)[pr2];
        }
        if (!active) {  // a position past the end of the sequence: nothing to quantify
            if (tid == 0) {
                if (o.flag) o.flag[lr] = 0;
                if (o.row_status) o.row_status[lr] = 0;
                issue(k + kQStages);
            }
            continue;
        }
        const unsigned char *stage = smem + (size_t)s * kStageBytes;
        if (mbar_wait_bounded(&sh.full[s], (phases >> s) & 1u, kWaitCycles)) phases ^= 1u << s;
        else sh.abort = 1;

        // ---- sweep 1: the row into registers, its maximum
        ThreadRow<T, JV> row;
        const float tm = row.load(stage, tid, nj);
        const float wm = warp_redux_max(tm);
        if (lane == 0) sh.wmax[warp] = wm;
        if (tid == 0) {
            sh.argmin = INT_MAX;
            sh.nmax = 0;
        }
        if (tid == 32 && per_row) sh.rc[k & 1] = make_row_const(rho, a.radius_is_raw, a.r_max, a.n);
        named_bar_sync(kBarConsumers, kQConsumers);
        if (sh.abort) {
            aborted = true;
            break;
        }
        const float m = warp_redux_max(sh.wmax[lane & (kQWarps - 1)]);
        if (tm == m) {
            const int idx = row.find(m, tid, nj);
            if (idx != INT_MAX) atomicMin(&sh.argmin, idx);
        }

        // ---- sweep 2: exponentials (kept in registers), their sum and the entropy sum
        const float m2 = m * kLog2e;
        float2 e[NP];
        float2 z2 = f2(0.f), t2 = f2(0.f);
        const float2 L2 = f2(kLog2e), nm2 = f2(-m2);
#pragma unroll
        for (int j = 0; j < JV; ++j) {
#pragma unroll
            for (int q = 0; q < NPV; ++q) {
                float2 ev = f2(0.f);
                if (j < nj) {
                    const float2 d = __ffma2_rn(row.pair(j, q), L2, nm2);
                    ev = make_float2(ex2_approx(d.x), ex2_approx(d.y));  // a NaN logit poisons the sums on purpose
                    z2 = __fadd2_rn(z2, ev);
                    t2 = __ffma2_rn(ev, ThreadRow<T, JV>::exponent_for_entropy(d), t2);
                }
                e[j * NPV + q] = ev;
            }
        }
        float zs = z2.x + z2.y;
        if (tm == m) {
            // This thread owns a maximum.  A term near 1 would cost the small terms their low bits, so its
            // partial sum is formed again without the maxima; they come back exactly, as a count times e0.
            float zz = 0.f;
            int cnt = 0;
#pragma unroll
            for (int j = 0; j < JV; ++j) {
#pragma unroll
                for (int q = 0; q < NPV; ++q) {
                    if (j < nj) {
                        const float2 c = row.pair(j, q), ev = e[j * NPV + q];
                        if (c.x == m) ++cnt; else zz += ev.x;
                        if (c.y == m) ++cnt; else zz += ev.y;
                    }
                }
            }
            zs = zz;
            atomicAdd(&sh.nmax, cnt);
        }
        const float zt = warp_sum_pair(zs, t2.x + t2.y, lane);  // lanes 0..15: z, lanes 16..31: t
        if (lane == 0) sh.wz[warp] = zt;
        named_bar_sync(kBarConsumers, kQConsumers);
        float z = sh.wz[lane & (kQWarps - 1)];
#pragma unroll
        for (int ofs = 8; ofs > 0; ofs >>= 1) z += __shfl_xor_sync(0xffffffffu, z, ofs);
        const float e0 = ex2_approx(fmaf(m, kLog2e, -m2));  // the exponential every maximum got
        const int nmax = sh.nmax;
        z = fmaf((float)nmax, e0, z);
        const RowConst rc = sh.rc[k & 1];

        int status = 0;
        if (!(m > kLogitFloor) || !(z > 0.f) || !(z < INFINITY) || !(rc.r == rc.r)) {
            // an unusable row (NaN / +inf logit, no finite logit, NaN radius): classify it from the
            // landed bytes exactly as the row-status bits are defined
            if (tid == 0) sh.bad_nan = sh.bad_finite = 0;
            named_bar_sync(kBarConsumers, kQConsumers);
            int has_nan = 0, has_finite = 0;
#pragma unroll
            for (int j = 0; j < JV; ++j) {
                if (j < nj) {
                    const T *v = reinterpret_cast<const T *>(stage + (size_t)(tid + j * kQConsumers) * 16);
#pragma unroll
                    for (int q = 0; q < VEC; ++q) {
                        const float c = Elem<T>::widen(v[q]);
                        if (!(c == c) || c == INFINITY) has_nan = 1;
                        if (c == c && fabsf(c) != INFINITY) has_finite = 1;
                    }
                }
            }
            if (has_nan) sh.bad_nan = 1;
            if (has_finite) sh.bad_finite = 1;
            named_bar_sync(kBarConsumers, kQConsumers);
            if (sh.bad_nan || !(rc.r == rc.r)) status |= CIAR_ROW_NAN;
            if (!sh.bad_finite) status |= CIAR_ROW_NO_FINITE;
            if (!status) status = CIAR_ROW_NAN;  // sums overflowed without any single bad logit
        }
        if (tid == 0) {  // every consumer has read the stage: refill it
            fence_proxy_async_smem();
            issue(k + kQStages);
        }

        // ---- sweep 3: interval sums from the exponentials in registers
        float2 P1 = f2(0.f), D1 = f2(0.f), PP = f2(0.f), PD = f2(0.f), DD = f2(0.f);
        if (!status) {
            const float invz = 1.0f / z;
            const float2 iz = f2(invz), niz = f2(-invz), one = f2(1.0f);
            const float2 a1 = f2(rc.a1), b1 = f2(rc.b1), npl0 = f2(-rc.pl0), ndd0 = f2(-rc.dd0);
#pragma unroll
            for (int i = 0; i < NP; ++i) {
                if (i / NPV < nj) {
                    const float2 x = __fmul2_rn(e[i], iz);
                    const float2 sx = __ffma2_rn(e[i], niz, one);
                    const float2 den_l = __ffma2_rn(b1, sx, a1);
                    const float2 den_u = __ffma2_rn(b1, x, a1);
                    const float2 q = __fmul2_rn(den_l, den_u);
                    const float2 xr = __fmul2_rn(x, make_float2(rcp_approx(q.x), rcp_approx(q.y)));
                    const float2 pl = __ffma2_rn(__fmul2_rn(xr, den_u), a1, npl0);  // p^l term minus its centre
                    const float2 dd = __ffma2_rn(xr, sx, ndd0);                     // width term minus its centre
                    P1 = __fadd2_rn(P1, pl);
                    D1 = __fadd2_rn(D1, dd);
                    PP = __ffma2_rn(pl, pl, PP);
                    PD = __ffma2_rn(pl, dd, PD);
                    DD = __ffma2_rn(dd, dd, DD);
                }
            }
        }

        // ---- hand the row to the finalizer warp
        named_bar_sync(kBarFree, kQBlock);
        sh.part[0][tid] = P1.x + P1.y;
        sh.part[1][tid] = D1.x + D1.y;
        sh.part[2][tid] = PP.x + PP.y;
        sh.part[3][tid] = PD.x + PD.y;
        sh.part[4][tid] = DD.x + DD.y;
        if (lane == 0) sh.info.zt[warp].x = zt;
        if (lane == 16) sh.info.zt[warp].y = zt;
        if (tid == 0) {
            sh.info.lr = lr;
            sh.info.pr = pr;
            sh.info.m = m;
            sh.info.argmin = sh.argmin;
            sh.info.nmax = nmax;
            sh.info.e0 = e0;
            sh.info.status = status;
        }
        if (tid == 32) sh.info.rc = rc;
        named_bar_arrive(kBarFull, kQBlock);
    }

    if (aborted) {
        // A copy never arrived.  Mark this row and the rest of this CTA's rows, then give the
        // copies still in flight a last bounded chance to land before the CTA leaves.
        if (tid == 0) {
            for (int k2 = k;; ++k2) {
                const int64_t lr = blockIdx.x + (int64_t)k2 * stride_rows;
                if (lr >= a.rows) break;
                write_unusable(o, lr, CIAR_ROW_TIMEOUT);
            }
            for (int s = 0; s < kQStages; ++s) mbar_wait_bounded(&sh.full[s], (phases >> s) & 1u, kDrainCycles);
        }
    }
    named_bar_sync(kBarFree, kQBlock);
    if (tid == 0) sh.info.cmd = 1;
    named_bar_arrive(kBarFull, kQBlock);
}

template <typename T, int JV, int MINB>
cudaError_t launch_one(const QuantifyArgs &a, cudaStream_t stream)
{
    constexpr size_t smem = (size_t)kQStages * kQConsumers * JV * 16 + sizeof(QShared);
    static bool configured[64] = {};
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!configured[dev]) {
        err = cudaFuncSetAttribute(quantify_stream_kernel<T, JV, MINB>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (err != cudaSuccess) return err;
        configured[dev] = true;
    }
    const int64_t cap = (int64_t)sm_count() * MINB;
    const unsigned grid = (unsigned)(a.rows < cap ? a.rows : cap);
    quantify_stream_kernel<T, JV, MINB><<<grid, kQBlock, smem, stream>>>(a);
    count_launch();
    return cudaGetLastError();
}

}  // namespace

bool quantify_stream_eligible(const QuantifyArgs &a, int dtype)
{
    const int vec = dtype == CIAR_F32 ? 4 : 8;
    if (a.radius_mode == CIAR_RADIUS_PER_CODE) return false;
    if (a.out.dense_p || a.out.dense_lo || a.out.dense_up) return false;
    if (a.vb % vec != 0 || a.n % vec != 0) return false;
    return a.n >= 2048 && a.n <= 16384;
}

cudaError_t launch_quantify_stream(const QuantifyArgs &a, int dtype, cudaStream_t stream)
{
    if (a.rows == 0) return cudaSuccess;
    if (dtype == CIAR_F32) {
        if (a.n <= 4096) return launch_one<float, 2, 2>(a, stream);
        if (a.n <= 8192) return launch_one<float, 4, 2>(a, stream);
        return launch_one<float, 8, 1>(a, stream);
    }
    if (a.n <= 4096) return launch_one<__nv_bfloat16, 1, 2>(a, stream);
    if (a.n <= 8192) return launch_one<__nv_bfloat16, 2, 2>(a, stream);
    return launch_one<__nv_bfloat16, 4, 2>(a, stream);
}

}  // namespace ciar
