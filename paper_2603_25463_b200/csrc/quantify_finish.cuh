// What the streaming quantifiers share: the interval arithmetic's constants, a row whose sweeps are done
// ("parked") and the warp routine that finishes it.  sm_100a only.
#pragma once

#include <climits>

#include "ciar_internal.h"
#include "stream_common.cuh"

namespace ciar {

namespace {

constexpr int kQThreads = 512;           // most threads a CTA of the streaming quantifiers has
constexpr int kQWarps = kQThreads / 32;  // (the parked form is laid out for that many warps)
constexpr int kQStages = 3;
constexpr int kBarRow = 1;                       // named barrier of the row sweeps
constexpr long long kWaitCycles = 2000000000ll;  // bound of a wait for a row (about a second)
constexpr long long kDrainCycles = 20000000ll;   // bound of each wait while leaving after a failure

// The interval arithmetic.  With x = softmax probability, s = 1 - x and beta = e^r - 1 the raw
// InterFuse bounds are
//   p^l = x / (1 + beta s),   p^u = (1 + beta) x / (1 + beta x),
//   p^u - p^l = beta (2 + beta) x s / ((1 + beta s)(1 + beta x)).
// Rows with r <= 1 take the "series" route: every code with x below theta = 2^-8 e^-r enters only
// through the power sums of (e - c0) up to the fourth (e = exp(c - m), c0 = Z / n), from which the
// sums of p^l, of the widths and of their squares are rebuilt by a fourth-order Taylor expansion
// about x0 = 1 / n (terms beyond it are below 1e-7 of the result); the few codes above theta
// (fewer than 256 e^r) are clamped to it in the power sums, listed, and put back exactly.  Rows
// with r > 1 take the "direct" route: both bounds of every code from the formulas above, in the
// scaled form den_l = a1 + b1 s, den_u = a1 + b1 x with (a1, b1) = (1, beta) or (1 / beta, 1) for
// beta > 1, which keeps every term in range for radii up to 80.
struct DirectConst {
    float a1, b1;
    float pl0, dd0;  // the two raw terms at x = 1 / n, about which the direct sums are taken
    int big;
};

constexpr int kPark = 16;      // rows parked before the CTA finishes them, one per warp
constexpr int kListCap = 704;  // > 256 e for r <= 1: more codes than that cannot exceed theta
constexpr int kParkList = 32;  // listed codes a parked row carries itself; the rest of a longer list sits in a shared buffer

// A row whose sweeps are done and whose arithmetic is still to do.
struct Parked {
    // per-warp sums, as lanes 0 and 16 of each warp hold them: [0] exp (terms equal to e0 left out), [4] exp * exponent,
    // route sums in [1] [5] [2] [6] [3] (series: powers 2, 3, 4 of e - c0; direct: pl, dd, pl^2, pl dd, dd^2)
    float wsum[kQWarps][8];
    float list[kParkList];   // series route: exponentials of the codes above theta
    long long lr, pr;
    float m, e0;   // row maximum; the exponential of a code equal to it, as the sweeps computed it
    float c0, th;  // series route: centre of the power sums and clamp level, in units of exp(c - m)
    float rho, r;  // radius as stored, and clamped (after Softplus when raw) as the sweeps used it
    int argmin, nmax, nlist, status, series;
    int par;  // which of the two shared list buffers holds the codes beyond kParkList
};

// Clamped radius of a row from its stored value (Softplus when raw), in float for the sweeps.
__device__ __forceinline__ float row_radius(float rho, int raw, float r_max)
{
    float r = rho;
    if (raw) r = (rho > 0.f) ? rho + log1pf(expf(-rho)) : log1pf(expf(rho));  // Softplus, beta = 1
    return fminf(r, r_max);
}

__device__ __forceinline__ DirectConst make_direct_const(float r, int n)
{
    DirectConst k;
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

// 1 / x for a positive normal double: a float reciprocal refined by two Newton steps (full double accuracy)
__device__ __forceinline__ double fast_rcp(double x)
{
    double r = (double)rcp_approx((float)x);
    r = fma(r, fma(-x, r, 1.0), r);
    return fma(r, fma(-x, r, 1.0), r);
}

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


// Finishes one row whose sums are parked: reduces the per-warp sums, treats the listed codes
// exactly (one per lane), then does the scalar arithmetic (normalisation step, Omega, Sigma, U,
// entropy, the flag) and the stores.  Run by one whole warp.
__device__ __noinline__ void finish_row(const QuantifyArgs &a, const Parked &pk, const float *list, int lane, int nw)
{
    const ciar_quantify_out &o = a.out;
    const long long lr = pk.lr;
    if (pk.status) {
        if (lane == 0) write_unusable(o, lr, pk.status);
        return;
    }
    const bool series = pk.series != 0;
    double v[7];
#pragma unroll
    for (int q = 0; q < 7; ++q) {
        constexpr int kSlot[7] = { 0, 4, 1, 5, 2, 6, 3 };
        v[q] = 0.0;
        if (q < 5 || !series) {
            if (lane < nw) v[q] = (double)pk.wsum[lane][kSlot[q]];
            v[q] = warp_sum_d(v[q]);
        }
    }
    const double nn = (double)a.n, inv_nn = fast_rcp(nn);
    const double e0 = (double)pk.e0;
    const int nmax = pk.nmax;
    const double zpart = v[0], zd = zpart + (double)nmax * e0;  // the row's sum of exponentials
    const double beta = (double)expm1f(pk.r);  // e^r - 1 to float accuracy: the bounds depend on it smoothly
    double S_lo, S_up, omega, ss;
    if (series) {
        const int nlist = pk.nlist < kListCap ? pk.nlist : kListCap;
        const double c0 = (double)pk.c0, th = (double)pk.th;
        const double invz = fast_rcp(zd);
        const double b = 1.0 + beta, kap = beta * (2.0 + beta);
        // listed codes, exactly: sums of e - clamp, p^l, d, p^l^2, p^l d, d^2 (d = p^u - p^l)
        double ls[6] = { 0.0, 0.0, 0.0, 0.0, 0.0, 0.0 };
        for (int i = lane; i < nlist; i += 32) {
            const double e = (double)list[i];
            const double x = e * invz;
            // 1 - x from the other codes' exponentials (no cancellation for a dominant code)
            const double sx = (e == e0 ? zpart + (double)(nmax - 1) * e0 : zd - e) * invz;
            const double den = fast_rcp((1.0 + beta * sx) * (1.0 + beta * x));
            const double pl = x * (1.0 + beta * x) * den, d = kap * x * sx * den;
            ls[0] += e - th;
            ls[1] += pl;
            ls[2] += d;
            ls[3] += pl * pl;
            ls[4] += pl * d;
            ls[5] += d * d;
        }
        if (nlist > 0) {
#pragma unroll
            for (int q = 0; q < 6; ++q) ls[q] = warp_sum_d(ls[q]);
        }
        // Unlisted codes enter through G_k = sum of (x - x0)^k: the power sums over all codes (listed ones
        // clamped to theta) less the clamped codes' share.
        const double nl = (double)nlist, nu = nn - nl;
        const double x0 = c0 * invz, hth = (th - c0) * invz;
        const double iz2 = invz * invz, h2 = hth * hth;
        const double G1 = (zd - ls[0] - nn * c0) * invz - nl * hth;
        const double G2 = v[2] * iz2 - nl * h2, G3 = v[3] * iz2 * invz - nl * h2 * hth, G4 = v[4] * iz2 * iz2 - nl * h2 * h2;
        // Taylor coefficients about x0 of p^l(x) = x / (b - beta x) and of d(x) = p^u - p^l, p^u(x) = b x / (1 + beta x),
        // and what the sums need of them (they do not outlive this block)
        double PL0, DD0, Bd, Ad, Qdd, Qdp, Qpp;
        {
            const double u = b - beta * x0, w = 1.0 + beta * x0;
            const double iuw = fast_rcp(u * w), iu = w * iuw, iw = u * iuw;
            const double rl = beta * iu, ru = -beta * iw;
            PL0 = x0 * iu;
            DD0 = kap * x0 * (1.0 - x0) * iuw;  // p^u - p^l at x0, no cancellation
            const double PL1 = b * iu * iu, PL2 = PL1 * rl, PL3 = PL2 * rl, PL4 = PL3 * rl;
            const double PU2 = b * iw * iw * ru, PU3 = PU2 * ru, PU4 = PU3 * ru;
            const double DD1 = b * beta * (1.0 - 2.0 * x0) * (u + w) * iuw * iuw;  // PU1 - PL1, no cancellation
            const double DD2 = PU2 - PL2, DD3 = PU3 - PL3, DD4 = PU4 - PL4;
            Bd = PL1 * G1 + PL2 * G2 + PL3 * G3 + PL4 * G4;
            Ad = DD1 * G1 + DD2 * G2 + DD3 * G3 + DD4 * G4;
            // sums of products of the first-order-and-up parts, to fourth order
            Qpp = PL1 * PL1 * G2 + 2.0 * PL1 * PL2 * G3 + (2.0 * PL1 * PL3 + PL2 * PL2) * G4;
            Qdd = DD1 * DD1 * G2 + 2.0 * DD1 * DD2 * G3 + (2.0 * DD1 * DD3 + DD2 * DD2) * G4;
            Qdp = DD1 * PL1 * G2 + (DD1 * PL2 + DD2 * PL1) * G3 + (DD1 * PL3 + DD3 * PL1 + DD2 * PL2) * G4;
        }
        const double B = nu * PL0 + Bd + ls[1];  // sum of raw p^l
        const double A = nu * DD0 + Ad + ls[2];  // sum of raw widths
        S_lo = B;
        S_up = A + B;
        const double rs = S_lo > 0.0 && S_up > 0.0 ? fast_rcp(S_lo * S_up) : 0.0;
        double k_lo = (double)a.lo_cap * S_up * rs, k_up = (double)a.hi_cap * S_lo * rs;
        if (!(S_lo > 0.0) || !(k_lo < 1.0)) k_lo = 1.0;
        if (!(S_up > 0.0) || !(k_up > 1.0)) k_up = 1.0;
        const double g = k_up - k_lo;  // delta = k_up d + g p^l
        omega = k_up * A + g * B;
        const double mu = omega * inv_nn;
        const double E0 = k_up * DD0 + g * PL0 - mu;  // delta - mu at x0
        // sum of (delta - mu)^2: unlisted codes from the expansion, listed codes from their five exact sums
        ss = nu * E0 * E0 + 2.0 * E0 * (k_up * Ad + g * Bd) + k_up * k_up * Qdd + 2.0 * k_up * g * Qdp + g * g * Qpp +
             (k_up * k_up * ls[5] + 2.0 * k_up * g * ls[4] + g * g * ls[3] - 2.0 * mu * (k_up * ls[2] + g * ls[1]) + nl * mu * mu);
    } else {
        const DirectConst dc = make_direct_const(pk.r, a.n);  // the same constants as the sweep used
        const double P1 = v[2], D1 = v[3], PP = v[4], PD = v[5], DD = v[6];
        const double a1 = (double)dc.a1, b1 = (double)dc.b1;
        const double kd = dc.big ? 1.0 + 2.0 * a1 : b1 * (2.0 + b1);
        const double B = nn * (double)dc.pl0 + P1;  // sum of the raw lower bounds
        const double Dsum = nn * (double)dc.dd0 + D1;
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
        ss = c1 * c1 * DD + 2.0 * c1 * c2 * PD + c2 * c2 * PP - lin * lin * inv_nn;
    }
    if (lane != 0) return;
    const double sigma = sqrt((ss > 0.0 ? ss : 0.0) * inv_nn);
    const double score = omega * sigma;
    // exponent actually used: c * log2e_f - m2 = (c - m) * log2e_f + off with off = m * log2e_f - m2
    const float m = pk.m;
    const double off = (double)m * (double)kLog2e - (double)(m * kLog2e);
    const double w2 = -off * kLn2D;
    const double unscale = 1.0 + w2 * (1.0 + 0.5 * w2);  // 2^-off: |off| is a rounding error of m * log2e, far below 1e-4
    const double z = zd * unscale;
    const double t = v[1] * unscale - off * z;
    // ln z: z >= 1 up to rounding; log1p keeps the digits of a z just above 1 (a peaked row)
    const double lnz = z < 1.5 ? (double)log1pf((float)(z - 1.0)) : (double)logf((float)z);
    const double p_max = fast_rcp(z);
    const double entropy = lnz - kLn2D * t * p_max;
    int fl;
    switch (a.policy) {
    case CIAR_POLICY_INTERVAL: fl = score > (double)a.tau; break;
    case CIAR_POLICY_ENTROPY: fl = entropy > (double)a.tau; break;
    case CIAR_POLICY_MAXPROB: fl = p_max < (double)a.tau; break;
    case CIAR_POLICY_RANDOM: fl = a.u_flag[pk.pr] < a.tau; break;
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
    if (o.argmax) o.argmax[lr] = pk.argmin + a.vb;
    if (o.flag) o.flag[lr] = (uint8_t)fl;
    if (o.row_status) o.row_status[lr] = 0;
}

}  // namespace

}  // namespace ciar
