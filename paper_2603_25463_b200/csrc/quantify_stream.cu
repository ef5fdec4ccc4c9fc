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

// Interval constants of one row, worked out by one consumer thread per row.
//
// With x = softmax probability, s = 1 - x and beta = e^r - 1 the raw InterFuse bounds are
//   p^l = x / (1 + beta s),   p^u = (1 + beta) x / (1 + beta x),
//   p^u - p^l = beta (2 + beta) x s / ((1 + beta s)(1 + beta x)).
// Rows with r <= 1 take the "series" route: every code with x below theta = 2^-8 / (1 + beta) enters
// only through the power sums of (e - c0) up to the fourth (c0 = Z / n), from which the finalizer
// rebuilds the sums of p^l, of the widths and of their squares by a fourth-order Taylor expansion
// about x0 = 1 / n (terms beyond it are below 1e-7 of the result); the few codes above theta are
// clamped to it in the power sums, listed, and put back exactly.  Rows with r > 1 take the
// "direct" route: both bounds of every code from the formulas above, in the scaled form
//   den_l = a1 + b1 s, den_u = a1 + b1 x, (a1, b1) = (1, beta) or (1 / beta, 1) for beta > 1,
// which keeps every term in range for radii up to 80.
struct RowConst {
    float rho;       // radius as stored (before Softplus when raw); NaN marks an unusable radius
    float r;         // clamped radius
    float theta_p;   // series route: probability above which a code is treated exactly
    float a1, b1;    // direct route
    float pl0, dd0;  // direct route: the two raw terms at x = 1 / n, about which its sums are taken
    int series;
    int big;
};

constexpr int kListCap = 704;  // > 256 (1 + beta) for r <= 1: more codes than that cannot exceed theta

struct RowInfo {
    long long lr, pr;
    float m, e0;   // row maximum; the exponential of a code equal to it, as the consumers computed it
    float c0, th;  // series route: centre of the power sums and clamp level, in units of exp(c - m)
    int argmin, nmax;
    int status;  // CIAR_ROW_* bits found by the consumers (0 = a regular row)
    int cmd;     // 0 = finalize this row, 1 = no more rows
    RowConst rc;
    float2 zt[kQWarps];  // per-warp sums of exp (maxima left out) and of exp * exponent
};

struct QShared {
    unsigned long long full[kQStages];
    float wmax[kQWarps];
    float wz[kQWarps];
    RowConst rc[2];
    int argmin, nmax;  // lowest index holding the row maximum, number of codes whose exponential equals e0
    int bad_nan, bad_finite;
    int abort;
    int nlist;  // codes above theta in the row being swept (reset by the finalizer when it has read them)
    RowInfo info;
    float part[5][kQConsumers];
    float list[kListCap];
};

__device__ __forceinline__ RowConst make_row_const(float rho, int raw, float r_max, int n)
{
    RowConst k;
    k.rho = rho;
    float r = rho;
    if (raw) r = (rho > 0.f) ? rho + log1pf(expf(-rho)) : log1pf(expf(rho));  // Softplus, beta = 1
    r = fminf(r, r_max);
    k.r = r;
    const float beta = expm1f(r);
    k.series = r <= 1.0f;
    k.theta_p = 0.00390625f / (1.0f + beta);
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

// What the consumers hand over for one row, reduced over the CTA (lane 0 of the finalizer).
struct RowSums {
    double s[5];    // series route: s[0..2] = sums of (e - c0)^2, ^3, ^4; direct route: the five centred sums
    double zpart;   // sum of exp(c - m) without the maxima
    double tr;      // sum of exp * exponent
    double excess;  // series route: sum over listed codes of (e - clamp level)
};

// Omega, Sigma and the raw bound sums of a series-route row.  Listed codes are handled by all lanes.
__device__ __forceinline__ void series_sums(const QuantifyArgs &a, const QShared &sh, const RowSums &rs, double beta,
                                            float e0f, int nmax, float c0f, float thf, int nlist, float e_first, int lane,
                                            double &S_lo, double &S_up, double &omega, double &sigma)
{
    const double nn = (double)a.n;
    const double e0 = (double)e0f, zd = rs.zpart + (double)nmax * e0;  // the row's sum of exponentials
    const double invz = 1.0 / zd;
    const double b = 1.0 + beta, kap = beta * (2.0 + beta);
    const double x0 = (double)c0f * invz, hth = ((double)thf - (double)c0f) * invz;
    const double iz2 = invz * invz;
    const double H1 = (zd - rs.excess - nn * (double)c0f) * invz;  // sum of (clamped x - x0)
    const double H2 = rs.s[0] * iz2, H3 = rs.s[1] * iz2 * invz, H4 = rs.s[2] * iz2 * iz2;
    // Taylor coefficients about x0 of p^l(x) = x / (b - beta x) and p^u(x) = b x / (1 + beta x)
    const double u = b - beta * x0, v = 1.0 + beta * x0;
    const double iuv = 1.0 / (u * v), iu = v * iuv, iv = u * iuv;
    const double rl = beta * iu, ru = -beta * iv;
    const double PL0 = x0 * iu, PL1 = b * iu * iu, PL2 = PL1 * rl, PL3 = PL2 * rl, PL4 = PL3 * rl;
    const double PU1 = b * iv * iv, PU2 = PU1 * ru, PU3 = PU2 * ru, PU4 = PU3 * ru;
    const double DD0 = kap * x0 * (1.0 - x0) * iuv;                        // p^u - p^l at x0, no cancellation
    const double DD1 = b * beta * (1.0 - 2.0 * x0) * (u + v) * iuv * iuv;  // PU1 - PL1, no cancellation
    const double DD2 = PU2 - PL2, DD3 = PU3 - PL3, DD4 = PU4 - PL4;
    const double h2 = hth * hth, h3 = h2 * hth, h4 = h2 * h2;
    const double pl_th = PL0 + PL1 * hth + PL2 * h2 + PL3 * h3 + PL4 * h4;  // what a clamped code contributed
    const double dd_th = DD0 + DD1 * hth + DD2 * h2 + DD3 * h3 + DD4 * h4;
    // listed codes, exactly: first their share of the bound sums
    double bl = 0.0, dl = 0.0;
    for (int i = lane; i < nlist; i += 32) {
        const double e = i < 32 ? (double)e_first : (double)sh.list[i];
        const double x = e * invz;
        const double sx = (e == e0 ? rs.zpart + (double)(nmax - 1) * e0 : zd - e) * invz;  // 1 - x from the other codes
        const double den = 1.0 / ((1.0 + beta * sx) * (1.0 + beta * x));
        bl += x * (1.0 + beta * x) * den - pl_th;
        dl += kap * x * sx * den - dd_th;
    }
    bl = warp_sum_d(bl);
    dl = warp_sum_d(dl);
    const double B = nn * PL0 + PL1 * H1 + PL2 * H2 + PL3 * H3 + PL4 * H4 + bl;  // sum of raw lower bounds
    const double A = nn * DD0 + DD1 * H1 + DD2 * H2 + DD3 * H3 + DD4 * H4 + dl;  // sum of raw widths
    S_lo = B;
    S_up = A + B;
    double k_lo = 1.0, k_up = 1.0;
    if (S_lo > 0.0 && (double)a.lo_cap / S_lo < 1.0) k_lo = (double)a.lo_cap / S_lo;
    if (S_up > 0.0 && (double)a.hi_cap / S_up > 1.0) k_up = (double)a.hi_cap / S_up;
    const double g = k_up - k_lo;  // delta = k_up (p^u - p^l) + g p^l
    omega = k_up * A + g * B;
    const double mu = omega / nn;
    const double E0 = k_up * DD0 + g * PL0 - mu, E1 = k_up * DD1 + g * PL1, E2 = k_up * DD2 + g * PL2,
                 E3 = k_up * DD3 + g * PL3, E4 = k_up * DD4 + g * PL4;
    const double q11 = E1 * E1, q12 = 2.0 * E1 * E2, q22 = 2.0 * E1 * E3 + E2 * E2;
    double ss = nn * E0 * E0 + 2.0 * E0 * (E1 * H1 + E2 * H2 + E3 * H3 + E4 * H4) + q11 * H2 + q12 * H3 + q22 * H4;
    const double sq_th = E0 * E0 + 2.0 * E0 * (E1 * hth + E2 * h2 + E3 * h3 + E4 * h4) + q11 * h2 + q12 * h3 + q22 * h4;
    double sl = 0.0;
    for (int i = lane; i < nlist; i += 32) {
        const double e = i < 32 ? (double)e_first : (double)sh.list[i];
        const double x = e * invz;
        const double sx = (e == e0 ? rs.zpart + (double)(nmax - 1) * e0 : zd - e) * invz;
        const double den = 1.0 / ((1.0 + beta * sx) * (1.0 + beta * x));
        const double dev = k_up * (kap * x * sx * den) + g * (x * (1.0 + beta * x) * den) - mu;
        sl += dev * dev - sq_th;
    }
    ss += warp_sum_d(sl);
    sigma = sqrt((ss > 0.0 ? ss : 0.0) / nn);
}

// Omega, Sigma and the raw bound sums of a direct-route row (lane 0 only needs them).
__device__ __forceinline__ void direct_sums(const QuantifyArgs &a, const RowSums &rs, const RowConst &rc, double &S_lo,
                                            double &S_up, double &omega, double &sigma)
{
    const double nn = (double)a.n;
    const double P1 = rs.s[0], D1 = rs.s[1], PP = rs.s[2], PD = rs.s[3], DD = rs.s[4];
    const double a1 = (double)rc.a1, b1 = (double)rc.b1;
    const double kd = rc.big ? 1.0 + 2.0 * a1 : b1 * (2.0 + b1);
    const double B = nn * (double)rc.pl0 + P1;  // sum of the raw lower bounds
    const double Dsum = nn * (double)rc.dd0 + D1;
    const double A = kd * Dsum;  // sum of the raw widths
    S_lo = B;
    S_up = A + B;
    double k_lo = 1.0, k_up = 1.0;
    if (S_lo > 0.0 && (double)a.lo_cap / S_lo < 1.0) k_lo = (double)a.lo_cap / S_lo;
    if (S_up > 0.0 && (double)a.hi_cap / S_up > 1.0) k_up = (double)a.hi_cap / S_up;
    // delta_i = k_up d_i + (k_up - k_lo) p^l_i = c1 dd_i + c2 pl_i
    const double c1 = k_up * kd, c2 = k_up - k_lo;
    omega = c1 * Dsum + c2 * B;
    const double lin = c1 * D1 + c2 * P1;
    const double ss = c1 * c1 * DD + 2.0 * c1 * c2 * PD + c2 * c2 * PP - lin * lin / nn;
    sigma = sqrt((ss > 0.0 ? ss : 0.0) / nn);
}

// The finalizer warp: takes the per-thread partial sums of one row from the hand-off buffer,
// adds them up in double and turns them into the row's outputs (normalisation step, Omega,
// Sigma, U, entropy, the flag).
__device__ __noinline__ void finalize_rows(const QuantifyArgs &a, QShared &sh, int lane)
{
    const ciar_quantify_out &o = a.out;
    float beta_key = __int_as_float(0x7fc00000);  // stored radius whose e^r - 1 is cached in beta_val
    double beta_val = 0.0;
    named_bar_arrive(kBarFree, kQBlock);
    for (;;) {
        named_bar_sync(kBarFull, kQBlock);
        if (sh.info.cmd) break;
        const RowConst rc = sh.info.rc;
        const int status = sh.info.status;
        const int nk = rc.series ? 3 : 5;
        RowSums rs;
#pragma unroll
        for (int k = 0; k < 5; ++k) {
            double acc = 0.0;
            if (k < nk) {
#pragma unroll
                for (int i = 0; i < kQConsumers / 32; ++i) acc += (double)sh.part[k][lane + 32 * i];
            }
            rs.s[k] = acc;
        }
        rs.zpart = rs.tr = 0.0;
        if (lane < kQWarps) {
            rs.zpart = (double)sh.info.zt[lane].x;
            rs.tr = (double)sh.info.zt[lane].y;
        }
        const long long lr = sh.info.lr, pr = sh.info.pr;
        const float m = sh.info.m, e0 = sh.info.e0, c0 = sh.info.c0, th = sh.info.th;
        const int argmin = sh.info.argmin, nmax = sh.info.nmax;
        int nlist = sh.nlist;
        nlist = nlist > kListCap ? kListCap : nlist;
        const bool series = !status && rc.series;
        double ex = 0.0;
        float e_first = 0.f;  // this lane's listed code among the first 32
        if (series) {
            if (lane < nlist) e_first = sh.list[lane];
            for (int i = lane; i < nlist; i += 32) ex += (double)sh.list[i] - (double)th;
        }
        rs.excess = ex;
        // Up to 32 listed codes travel in registers and the buffer goes back to the consumers at
        // once; a longer list is read in place, so the buffer is held until the row is done.
        const bool hold = series && nlist > 32;
        if (!hold) {
            __syncwarp();
            if (lane == 0) sh.nlist = 0;
            named_bar_arrive(kBarFree, kQBlock);
        }
#pragma unroll
        for (int k = 0; k < 5; ++k) rs.s[k] = warp_sum_d(rs.s[k]);
        rs.zpart = warp_sum_d(rs.zpart);
        rs.tr = warp_sum_d(rs.tr);
        rs.excess = warp_sum_d(rs.excess);

        double S_lo = 0.0, S_up = 0.0, omega = 0.0, sigma = 0.0;
        if (series) {
            if (!(rc.rho == beta_key)) {
                double r = (double)rc.rho;
                if (a.radius_is_raw) r = (r > 0.0) ? r + log1p(exp(-r)) : log1p(exp(r));  // Softplus, beta = 1
                if (r > (double)a.r_max) r = (double)a.r_max;
                beta_val = expm1(r);
                beta_key = rc.rho;
            }
            series_sums(a, sh, rs, beta_val, e0, nmax, c0, th, nlist, e_first, lane, S_lo, S_up, omega, sigma);
        } else if (!status) {
            direct_sums(a, rs, rc, S_lo, S_up, omega, sigma);
        }
        if (hold) {
            __syncwarp();
            if (lane == 0) sh.nlist = 0;
            named_bar_arrive(kBarFree, kQBlock);
        }
        if (lane == 0) {
            if (status) {
                write_unusable(o, lr, status);
            } else {
                const double score = omega * sigma;
                // exponent actually used: c * log2e_f - m2 = (c - m) * log2e_f + off with off = m * log2e_f - m2
                const double off = (double)m * (double)kLog2e - (double)(m * kLog2e);
                const double unscale = exp2(-off);
                const double z = (rs.zpart + (double)nmax * (double)e0) * unscale;
                const double t = rs.tr * unscale - off * z;
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
        }
        __syncwarp();
    }
}

template <typename T, int JV, int MINB>
__global__ void __launch_bounds__(kQBlock, MINB) quantify_stream_kernel(const __grid_constant__ QuantifyArgs a)
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
        sh.nlist = 0;
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
    const float inv_n = 1.0f / (float)a.n;

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
        const float e0 = ex2_approx(fmaf(m, kLog2e, -m2));  // the exponential every maximum got
        if (tm == m) {
            // This thread owns a maximum.  A term near 1 would cost the small terms their low bits, so its
            // partial sum is formed again without the terms equal to e0; they come back exactly, as a count.
            float zz = 0.f;
            int cnt = 0;
#pragma unroll
            for (int i = 0; i < NP; ++i) {
                if (i / NPV < nj) {
                    if (e[i].x == e0) ++cnt; else zz += e[i].x;
                    if (e[i].y == e0) ++cnt; else zz += e[i].y;
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
        const int nmax = sh.nmax;
        z = fmaf((float)nmax, e0, z);
        const RowConst rc = sh.rc[k & 1];

        int status = 0;
        if (!(m > kLogitFloor) || !(z > 0.f) || !(z < INFINITY) || !(rc.rho == rc.rho)) {
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
            if (sh.bad_nan || !(rc.rho == rc.rho)) status |= CIAR_ROW_NAN;
            if (!sh.bad_finite) status |= CIAR_ROW_NO_FINITE;
            if (!status) status = CIAR_ROW_NAN;  // sums overflowed without any single bad logit
        }
        const bool direct = !status && !rc.series;
        if (tid == 0 && !direct) {  // every consumer has read the stage: refill it
            fence_proxy_async_smem();
            issue(k + kQStages);
        }
        // the hand-off buffer (partial sums, list of large codes) must be free from here on
        named_bar_sync(kBarFree, kQBlock);

        // ---- sweep 3: interval sums
        float ps[5] = { 0.f, 0.f, 0.f, 0.f, 0.f };
        const float c0 = z * inv_n, th = rc.theta_p * z;
        if (!status && rc.series) {
            // power sums of (e - c0) from the exponentials in registers; codes above th are clamped and listed
            float2 T2 = f2(0.f), T3 = f2(0.f), T4 = f2(0.f);
            const float2 nc0 = f2(-c0);
            const float e_tm = ex2_approx(fmaf(tm, kLog2e, -m2));  // this thread's largest exponential
            if (!__any_sync(0xffffffffu, e_tm > th)) {
#pragma unroll
                for (int i = 0; i < NP; ++i) {
                    if (i / NPV < nj) {
                        const float2 y = __fadd2_rn(e[i], nc0);
                        const float2 y2 = __fmul2_rn(y, y);
                        T2 = __fadd2_rn(T2, y2);
                        T3 = __ffma2_rn(y2, y, T3);
                        T4 = __ffma2_rn(y2, y2, T4);
                    }
                }
            } else {
#pragma unroll
                for (int i = 0; i < NP; ++i) {
                    if (i / NPV < nj) {
                        float2 ev = e[i];
                        if (ev.x > th) {
                            const int slot = atomicAdd(&sh.nlist, 1);
                            if (slot < kListCap) sh.list[slot] = ev.x;
                            ev.x = th;
                        }
                        if (ev.y > th) {
                            const int slot = atomicAdd(&sh.nlist, 1);
                            if (slot < kListCap) sh.list[slot] = ev.y;
                            ev.y = th;
                        }
                        const float2 y = __fadd2_rn(ev, nc0);
                        const float2 y2 = __fmul2_rn(y, y);
                        T2 = __fadd2_rn(T2, y2);
                        T3 = __ffma2_rn(y2, y, T3);
                        T4 = __ffma2_rn(y2, y2, T4);
                    }
                }
            }
            ps[0] = T2.x + T2.y;
            ps[1] = T3.x + T3.y;
            ps[2] = T4.x + T4.y;
        } else if (direct) {
            // both bounds of every code, from the row still sitting in its stage
            const float invz = 1.0f / z;
            float P1 = 0.f, D1 = 0.f, PP = 0.f, PD = 0.f, DD = 0.f;
#pragma unroll 1
            for (int j = 0; j < nj; ++j) {
                const T *v = reinterpret_cast<const T *>(stage + (size_t)(tid + j * kQConsumers) * 16);
                float c[VEC];
                Elem<T>::load(v, c);
#pragma unroll
                for (int q = 0; q < VEC; ++q) {
                    const float ev = ex2_approx(fmaf(c[q], kLog2e, -m2));
                    const float x = ev * invz, sx = fmaf(-ev, invz, 1.0f);
                    const float den_l = fmaf(rc.b1, sx, rc.a1), den_u = fmaf(rc.b1, x, rc.a1);
                    const float xr = x * rcp_approx(den_l * den_u);
                    const float pl = fmaf(xr * den_u, rc.a1, -rc.pl0);  // p^l term minus its centre
                    const float dd = fmaf(xr, sx, -rc.dd0);             // width term minus its centre
                    P1 += pl;
                    D1 += dd;
                    PP = fmaf(pl, pl, PP);
                    PD = fmaf(pl, dd, PD);
                    DD = fmaf(dd, dd, DD);
                }
            }
            ps[0] = P1; ps[1] = D1; ps[2] = PP; ps[3] = PD; ps[4] = DD;
            named_bar_sync(kBarConsumers, kQConsumers);
            if (tid == 0) {
                fence_proxy_async_smem();
                issue(k + kQStages);
            }
        }

        // ---- hand the row to the finalizer warp
        sh.part[0][tid] = ps[0];
        sh.part[1][tid] = ps[1];
        sh.part[2][tid] = ps[2];
        if (direct) {
            sh.part[3][tid] = ps[3];
            sh.part[4][tid] = ps[4];
        }
        if (lane == 0) sh.info.zt[warp].x = zt;
        if (lane == 16) sh.info.zt[warp].y = zt;
        if (tid == 0) {
            sh.info.lr = lr;
            sh.info.pr = pr;
            sh.info.m = m;
            sh.info.e0 = e0;
            sh.info.c0 = c0;
            sh.info.th = th;
            sh.info.argmin = sh.argmin;
            sh.info.nmax = nmax;
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
