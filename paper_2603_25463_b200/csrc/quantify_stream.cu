// Streaming quantifier for rows that fit on chip (2048 .. 16384 codes, scalar or per-row radius).
//
// One persistent CTA walks rows blockIdx.x, blockIdx.x + gridDim.x, ...  Rows arrive through a
// ring of shared-memory stages filled by bulk (TMA) copies that one thread issues several rows
// ahead, so HBM always has requests in flight.  16 consumer warps sweep a landed row twice from
// shared memory (maximum; then one exponential per code, kept in registers: 32 per thread) and
// once more from those registers (interval sums).  A 17th warp, fed through a small hand-off
// buffer, reduces the per-thread sums, works out the interval constants of the rows to come,
// and does the per-row double-precision arithmetic for 16 rows at a time, one row per lane, off
// the consumers' critical path.  Each logit is read from HBM once.
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

// Interval constants of one row.
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
    float theta_p;   // series route: probability above which a code is treated exactly
    float a1, b1;    // direct route
    float pl0, dd0;  // direct route: the two raw terms at x = 1 / n, about which its sums are taken
    int series;
    int big;
};

constexpr int kListCap = 704;  // > 256 (1 + beta) for r <= 1: more codes than that cannot exceed theta
constexpr int kBatch = 16;     // rows finalized together, one per lane (of the first 16)

// What the consumers hand over with one row.
struct RowInfo {
    long long lr, pr;
    float m, e0;   // row maximum; the exponential of a code equal to it, as the consumers computed it
    float c0, th;  // series route: centre of the power sums and clamp level, in units of exp(c - m)
    int argmin, nmax;
    int status;  // CIAR_ROW_* bits found by the consumers (0 = a regular row)
    int cmd;     // 0 = finalize this row, 1 = no more rows, 2 = a skipped row (nothing to finalize)
    float2 zt[kQWarps];  // per-warp sums of exp (terms equal to e0 left out) and of exp * exponent
};

// Rows whose sums are complete and that wait for their scalar arithmetic (struct of arrays, one slot per lane).
struct Batch {
    double v[11][kBatch];  // series: power sums 2..4, zpart, tr, excess, five sums over listed codes; direct: five sums, zpart, tr
    double beta[kBatch];
    long long lr[kBatch], pr[kBatch];
    float m[kBatch], e0[kBatch], c0[kBatch], th[kBatch];
    int argmin[kBatch], nmax[kBatch], nlist[kBatch], status[kBatch];
    RowConst rc[kBatch];
};

struct QShared {
    unsigned long long full[kQStages];
    float wmax[kQWarps];
    float wz[kQWarps];
    int argmin, nmax;  // lowest index holding the row maximum, number of codes whose exponential equals e0
    int bad_nan, bad_finite;
    int abort;
    int nlist;  // codes above theta in the row being swept (reset by the finalizer when it has read them)
    RowInfo info;
    RowConst rc_tab[2][kBatch];  // interval constants of this CTA's rows kBatch b .. kBatch (b + 1) - 1 in rc_tab[b & 1]
    double beta_tab[2][kBatch];  // e^r - 1 of the same rows, in double
    float part[3][kQConsumers];  // series route: per-thread power sums
    float dpart[5][kQWarps];     // direct route: per-warp sums
    float list[kListCap];
    Batch batch;
};
static_assert(sizeof(QShared) + kQStages * 32768 <= 115712, "two CTAs per SM must fit in shared memory");

// Interval constants of a row from its stored radius (float for the consumers, beta in double for the finalizer).
__device__ __forceinline__ RowConst make_row_const(float rho, int raw, float r_max, int n, double &beta_d)
{
    RowConst k;
    k.rho = rho;
    double rd = (double)rho;
    if (raw) rd = (rd > 0.0) ? rd + log1p(exp(-rd)) : log1p(exp(rd));  // Softplus, beta = 1
    if (rd > (double)r_max) rd = (double)r_max;
    beta_d = expm1(rd);
    const float r = (float)rd, beta = (float)beta_d;
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

// A 16-byte vector of a landed row.  fold_max() folds it into a running maximum (bf16: two packed
// halves), pairs() widens it to float2 pairs with -inf floored (a NaN stays a NaN), find() gives the
// position of the first code equal to m.
template <typename T>
struct Vec;

template <>
struct Vec<__nv_bfloat16> {
    static constexpr int kPairs = 4;
    typedef uint32_t Max;
    static __device__ __forceinline__ Max max_init() { return kLogitFloorBf16x2; }
    static __device__ __forceinline__ Max fold_max(Max mx, const uint4 &v)
    {
        return bf16x2_max(mx, bf16x2_max(bf16x2_max(v.x, v.y), bf16x2_max(v.z, v.w)));
    }
    static __device__ __forceinline__ float max_value(Max mx)
    {
        const float2 p = unpack_bf16x2(mx);
        return fmaxf(p.x, p.y);
    }
    static __device__ __forceinline__ void pairs(const uint4 &v, float2 (&c)[4])
    {
        uint32_t w[4] = { v.x, v.y, v.z, v.w };
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            asm("max.NaN.bf16x2 %0, %0, %1;" : "+r"(w[q]) : "r"(kLogitFloorBf16x2));
            c[q] = unpack_bf16x2(w[q]);
        }
    }
    static __device__ __forceinline__ float2 exponent_for_entropy(float2 d) { return d; }  // floored already
};

template <>
struct Vec<float> {
    static constexpr int kPairs = 2;
    typedef float Max;
    static __device__ __forceinline__ Max max_init() { return -INFINITY; }
    static __device__ __forceinline__ Max fold_max(Max mx, const uint4 &v)
    {
        return fmaxf(mx, fmaxf(fmaxf(__uint_as_float(v.x), __uint_as_float(v.y)),
                               fmaxf(__uint_as_float(v.z), __uint_as_float(v.w))));
    }
    static __device__ __forceinline__ float max_value(Max mx) { return mx; }
    static __device__ __forceinline__ void pairs(const uint4 &v, float2 (&c)[2])
    {
        c[0] = make_float2(__uint_as_float(v.x), __uint_as_float(v.y));
        c[1] = make_float2(__uint_as_float(v.z), __uint_as_float(v.w));
    }
    // -inf logit: exp = 0 and the exponent is floored so that the product is 0, not NaN
    static __device__ __forceinline__ float2 exponent_for_entropy(float2 d)
    {
        return make_float2(fmaxf(d.x, kNegHuge), fmaxf(d.y, kNegHuge));
    }
};

__device__ __forceinline__ const uint4 &stage_vec(const unsigned char *stage, int vi)
{
    return *reinterpret_cast<const uint4 *>(stage + (size_t)vi * 16);
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

// Slots of Batch::v.  Both routes: 0 zpart (sum of exponentials without the terms equal to e0), 1 the
// entropy sum.  Series route: 2..4 power sums of (e - c0), 5 sum over listed codes of (e - clamp),
// 6..10 sums over listed codes of p^l, d, p^l^2, p^l d, d^2 (exact, d = p^u - p^l).  Direct route:
// 2..6 the five centred sums.
enum { kVZ = 0, kVT = 1, kVS = 2, kVEx = 5, kVL = 6 };

// Scalar arithmetic of one finished row (normalisation step, Omega, Sigma, U, entropy, the flag)
// and its stores.  Called with one row per lane.
__device__ __forceinline__ void finalize_slot(const QuantifyArgs &a, const Batch &bt, int slot)
{
    const ciar_quantify_out &o = a.out;
    const long long lr = bt.lr[slot], pr = bt.pr[slot];
    const int status = bt.status[slot];
    if (status) {
        write_unusable(o, lr, status);
        return;
    }
    const RowConst rc = bt.rc[slot];
    const double nn = (double)a.n;
    const double e0 = (double)bt.e0[slot];
    const int nmax = bt.nmax[slot];
    const double zd = bt.v[kVZ][slot] + (double)nmax * e0;  // the row's sum of exponentials
    double S_lo, S_up, omega, ss;
    if (rc.series) {
        const double beta = bt.beta[slot];
        const double nl = (double)bt.nlist[slot];
        const double c0 = (double)bt.c0[slot], th = (double)bt.th[slot];
        const double invz = 1.0 / zd;
        const double b = 1.0 + beta, kap = beta * (2.0 + beta);
        const double x0 = c0 * invz, hth = (th - c0) * invz;
        const double iz2 = invz * invz;
        const double H1 = (zd - bt.v[kVEx][slot] - nn * c0) * invz;  // sum of (clamped x - x0)
        const double H2 = bt.v[kVS][slot] * iz2, H3 = bt.v[kVS + 1][slot] * iz2 * invz, H4 = bt.v[kVS + 2][slot] * iz2 * iz2;
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
        // what a code clamped to theta contributed through the power sums
        const double pl_th = PL0 + PL1 * hth + PL2 * h2 + PL3 * h3 + PL4 * h4;
        const double dd_th = DD0 + DD1 * hth + DD2 * h2 + DD3 * h3 + DD4 * h4;
        const double lpl = bt.v[kVL][slot], ld = bt.v[kVL + 1][slot], lpp = bt.v[kVL + 2][slot],
                     lpd = bt.v[kVL + 3][slot], ldd = bt.v[kVL + 4][slot];
        const double B = nn * PL0 + PL1 * H1 + PL2 * H2 + PL3 * H3 + PL4 * H4 + (lpl - nl * pl_th);  // sum of raw p^l
        const double A = nn * DD0 + DD1 * H1 + DD2 * H2 + DD3 * H3 + DD4 * H4 + (ld - nl * dd_th);   // sum of raw widths
        S_lo = B;
        S_up = A + B;
        const double rs = 1.0 / (S_lo * S_up);
        double k_lo = (double)a.lo_cap * S_up * rs, k_up = (double)a.hi_cap * S_lo * rs;
        if (!(S_lo > 0.0) || !(k_lo < 1.0)) k_lo = 1.0;
        if (!(S_up > 0.0) || !(k_up > 1.0)) k_up = 1.0;
        const double g = k_up - k_lo;  // delta = k_up (p^u - p^l) + g p^l
        omega = k_up * A + g * B;
        const double mu = omega / nn;
        const double E0 = k_up * DD0 + g * PL0 - mu, E1 = k_up * DD1 + g * PL1, E2 = k_up * DD2 + g * PL2,
                     E3 = k_up * DD3 + g * PL3, E4 = k_up * DD4 + g * PL4;
        const double q11 = E1 * E1, q12 = 2.0 * E1 * E2, q22 = 2.0 * E1 * E3 + E2 * E2;
        const double sq_th = E0 * E0 + 2.0 * E0 * (E1 * hth + E2 * h2 + E3 * h3 + E4 * h4) + q11 * h2 + q12 * h3 + q22 * h4;
        // listed codes: sum of (delta - mu)^2 from their five exact sums
        const double sl = k_up * k_up * ldd + 2.0 * k_up * g * lpd + g * g * lpp - 2.0 * mu * (k_up * ld + g * lpl) + nl * mu * mu;
        ss = nn * E0 * E0 + 2.0 * E0 * (E1 * H1 + E2 * H2 + E3 * H3 + E4 * H4) + q11 * H2 + q12 * H3 + q22 * H4 +
             (sl - nl * sq_th);
    } else {
        const double P1 = bt.v[kVS][slot], D1 = bt.v[kVS + 1][slot], PP = bt.v[kVS + 2][slot], PD = bt.v[kVS + 3][slot],
                     DD = bt.v[kVS + 4][slot];
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
        ss = c1 * c1 * DD + 2.0 * c1 * c2 * PD + c2 * c2 * PP - lin * lin / nn;
    }
    const double sigma = sqrt((ss > 0.0 ? ss : 0.0) / nn);
    const double score = omega * sigma;
    // exponent actually used: c * log2e_f - m2 = (c - m) * log2e_f + off with off = m * log2e_f - m2
    const float m = bt.m[slot];
    const double off = (double)m * (double)kLog2e - (double)(m * kLog2e);
    const double unscale = exp2(-off);
    const double z = zd * unscale;
    const double t = bt.v[kVT][slot] * unscale - off * z;
    const double lnz = log(z);
    const double p_max = 1.0 / z;
    const double entropy = lnz - kLn2D * t * p_max;
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
    if (o.argmax) o.argmax[lr] = bt.argmin[slot] + a.vb;
    if (o.flag) o.flag[lr] = (uint8_t)fl;
    if (o.row_status) o.row_status[lr] = 0;
}

// Interval constants of this CTA's rows kBatch b .. kBatch b + kBatch - 1, one row per lane of the finalizer warp.
__device__ __forceinline__ void make_rc_batch(const QuantifyArgs &a, QShared &sh, int b, int lane)
{
    const int64_t lr = blockIdx.x + (int64_t)(b * kBatch + lane) * gridDim.x;
    int64_t pr;
    float rho = a.r_scalar;
    if (a.radius_mode == CIAR_RADIUS_PER_ROW) {
        rho = 0.f;
        if (lr < a.rows && map_row(a.rm, lr, pr)) rho = reinterpret_cast<const float *>(a.radius)[pr];
    }
    double beta;
    sh.rc_tab[b & 1][lane] = make_row_const(rho, a.radius_is_raw, a.r_max, a.n, beta);
    sh.beta_tab[b & 1][lane] = beta;
}

// The finalizer warp.  Per row: take the consumers' partial sums out of the hand-off buffer, give
// the buffer back, reduce in double, treat the listed codes exactly (one per lane), and park the
// row in a batch slot.  Per kBatch rows: the scalar arithmetic and the stores, one row per lane.
__device__ __noinline__ void finalize_rows(const QuantifyArgs &a, QShared &sh, int lane)
{
    Batch &bt = sh.batch;
    if (lane < kBatch) {
        make_rc_batch(a, sh, 0, lane);
        make_rc_batch(a, sh, 1, lane);
    }
    __syncwarp();
    named_bar_arrive(kBarFree, kQBlock);
    int filled = 0;
    for (int k = 0;; ++k) {
        named_bar_sync(kBarFull, kQBlock);
        const int cmd = sh.info.cmd;
        if (cmd == 1) break;
        // Every row before k has been handed over, so the table half of the batch before this one
        // is idle: fill it with the constants of the batch after this one.  The consumers see them
        // after their next wait on the free barrier.
        if ((k % kBatch) == 0 && k > 0 && lane < kBatch) make_rc_batch(a, sh, k / kBatch + 1, lane);
        if (cmd == 2) {  // a row the consumers skipped
            __syncwarp();
            named_bar_arrive(kBarFree, kQBlock);
            continue;
        }
        const RowConst rc = sh.rc_tab[(k / kBatch) & 1][k % kBatch];
        const double beta = sh.beta_tab[(k / kBatch) & 1][k % kBatch];
        const int status = sh.info.status;
        const bool series = !status && rc.series;
        double s[5] = { 0.0, 0.0, 0.0, 0.0, 0.0 };
        if (series) {
#pragma unroll
            for (int q = 0; q < 3; ++q) {
                double acc = 0.0;
#pragma unroll
                for (int i = 0; i < kQConsumers / 32; ++i) acc += (double)sh.part[q][lane + 32 * i];
                s[q] = acc;
            }
        } else if (!status && lane < kQWarps) {
#pragma unroll
            for (int q = 0; q < 5; ++q) s[q] = (double)sh.dpart[q][lane];
        }
        double zpart = 0.0, tr = 0.0;
        if (lane < kQWarps) {
            zpart = (double)sh.info.zt[lane].x;
            tr = (double)sh.info.zt[lane].y;
        }
        const float e0 = sh.info.e0, th = sh.info.th;
        const int nmax = sh.info.nmax;
        int nlist = series ? sh.nlist : 0;
        nlist = nlist > kListCap ? kListCap : nlist;
        if (lane == 0) {
            bt.lr[filled] = sh.info.lr;
            bt.pr[filled] = sh.info.pr;
            bt.m[filled] = sh.info.m;
            bt.e0[filled] = e0;
            bt.c0[filled] = sh.info.c0;
            bt.th[filled] = th;
            bt.argmin[filled] = sh.info.argmin;
            bt.nmax[filled] = nmax;
            bt.nlist[filled] = nlist;
            bt.status[filled] = status;
            bt.rc[filled] = rc;
            bt.beta[filled] = beta;
        }
        const float e_first = lane < nlist ? sh.list[lane] : 0.f;  // this lane's listed code among the first 32
        // Up to 32 listed codes travel in registers and the buffer goes back to the consumers at
        // once; a longer list is read in place, so the buffer is held until it has been read.
        const bool hold = nlist > 32;
        if (!hold) {
            __syncwarp();
            if (lane == 0) sh.nlist = 0;
            named_bar_arrive(kBarFree, kQBlock);
        }
        zpart = warp_sum_d(zpart);
        tr = warp_sum_d(tr);
        const int ns = series ? 3 : 5;
#pragma unroll
        for (int q = 0; q < 5; ++q)
            if (q < ns) s[q] = warp_sum_d(s[q]);
        double ls[6] = { 0.0, 0.0, 0.0, 0.0, 0.0, 0.0 };  // over listed codes: e - clamp, p^l, d, p^l^2, p^l d, d^2
        if (nlist > 0) {
            const double e0d = (double)e0, zd = zpart + (double)nmax * e0d, invz = 1.0 / zd;
            const double kap = beta * (2.0 + beta);
            for (int i = lane; i < nlist; i += 32) {
                const double e = i < 32 ? (double)e_first : (double)sh.list[i];
                const double x = e * invz;
                // 1 - x from the other codes' exponentials (no cancellation for a dominant code)
                const double sx = (e == e0d ? zpart + (double)(nmax - 1) * e0d : zd - e) * invz;
                const double den = 1.0 / ((1.0 + beta * sx) * (1.0 + beta * x));
                const double pl = x * (1.0 + beta * x) * den, d = kap * x * sx * den;
                ls[0] += e - (double)th;
                ls[1] += pl;
                ls[2] += d;
                ls[3] += pl * pl;
                ls[4] += pl * d;
                ls[5] += d * d;
            }
            if (hold) {
                __syncwarp();
                if (lane == 0) sh.nlist = 0;
                named_bar_arrive(kBarFree, kQBlock);
            }
#pragma unroll
            for (int q = 0; q < 6; ++q) ls[q] = warp_sum_d(ls[q]);
        }
        if (lane == 0) {
            bt.v[kVZ][filled] = zpart;
            bt.v[kVT][filled] = tr;
#pragma unroll
            for (int q = 0; q < 5; ++q) bt.v[kVS + q][filled] = s[q];
            if (series) {
                bt.v[kVEx][filled] = ls[0];
#pragma unroll
                for (int q = 0; q < 5; ++q) bt.v[kVL + q][filled] = ls[1 + q];
            }
        }
        __syncwarp();
        if (++filled == kBatch) {
            if (lane < kBatch) finalize_slot(a, bt, lane);
            filled = 0;
            __syncwarp();
        }
    }
    if (lane < filled) finalize_slot(a, bt, lane);
}

// FULL: every consumer thread owns exactly JV vectors (the row has 512 * JV of them).
template <typename T, int JV, int MINB, bool FULL>
__global__ void __launch_bounds__(kQBlock, MINB) quantify_stream_kernel(const __grid_constant__ QuantifyArgs a)
{
    typedef Vec<T> V;
    constexpr int VEC = Elem<T>::kVec;
    constexpr int NPV = V::kPairs;  // float2 pairs per 16-byte vector
    constexpr int NP = JV * NPV;    // pairs per thread
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
    int nj = JV;
    if (!FULL) {
        nj = (nvec - tid + kQConsumers - 1) / kQConsumers;
        nj = nj < 0 ? 0 : (nj > JV ? JV : nj);
    }
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

    uint32_t phases = 0;
    int k = 0;
    bool aborted = false;
    for (;; ++k) {
        const int64_t lr = blockIdx.x + (int64_t)k * stride_rows;
        if (lr >= a.rows) break;
        const int s = k % kQStages;
        int64_t pr;
        if (!map_row(a.rm, lr, pr)) {  // a position past the end of the sequence: nothing to quantify
            if (tid == 0) {
                if (o.flag) o.flag[lr] = 0;
                if (o.row_status) o.row_status[lr] = 0;
                issue(k + kQStages);
            }
            named_bar_sync(kBarFree, kQBlock);
            if (tid == 0) sh.info.cmd = 2;
            __syncwarp();
            named_bar_arrive(kBarFull, kQBlock);
            continue;
        }
        const unsigned char *stage = smem + (size_t)s * kStageBytes;
        if (mbar_wait_bounded(&sh.full[s], (phases >> s) & 1u, kWaitCycles)) phases ^= 1u << s;
        else sh.abort = 1;

        // ---- sweep 1: the row's maximum
        typename V::Max mx = V::max_init();
#pragma unroll
        for (int j = 0; j < JV; ++j)
            if (FULL || j < nj) mx = V::fold_max(mx, stage_vec(stage, tid + j * kQConsumers));
        const float tm = V::max_value(mx);
        const float wm = warp_redux_max(tm);
        if (lane == 0) sh.wmax[warp] = wm;
        if (tid == 0) {
            sh.argmin = INT_MAX;
            sh.nmax = 0;
        }
        __syncwarp();
        named_bar_sync(kBarConsumers, kQConsumers);
        if (sh.abort) {
            aborted = true;
            break;
        }
        const float m = warp_redux_max(sh.wmax[lane & (kQWarps - 1)]);
        if (tm == m) {  // this thread holds a maximum: its lowest index competes for the arg-max
            int best = INT_MAX;
            for (int j = nj - 1; j >= 0; --j) {
                const T *v = reinterpret_cast<const T *>(stage + (size_t)(tid + j * kQConsumers) * 16);
#pragma unroll
                for (int q = VEC - 1; q >= 0; --q)
                    if (Elem<T>::widen(v[q]) == m) best = (tid + j * kQConsumers) * VEC + q;
            }
            if (best != INT_MAX) atomicMin(&sh.argmin, best);
        }

        // ---- sweep 2: exponentials (kept in registers), their sum and the entropy sum
        const float m2 = m * kLog2e;
        float2 e[NP];
        float2 z2 = f2(0.f), t2 = f2(0.f);
        {
            const float2 L2 = f2(kLog2e), nm2 = f2(-m2);
#pragma unroll
            for (int j = 0; j < JV; ++j) {
                if (FULL || j < nj) {
                    float2 c[NPV];
                    V::pairs(stage_vec(stage, tid + j * kQConsumers), c);
#pragma unroll
                    for (int q = 0; q < NPV; ++q) {
                        const float2 d = __ffma2_rn(c[q], L2, nm2);
                        const float2 ev = make_float2(ex2_approx(d.x), ex2_approx(d.y));  // a NaN logit poisons the sums on purpose
                        z2 = __fadd2_rn(z2, ev);
                        t2 = __ffma2_rn(ev, V::exponent_for_entropy(d), t2);
                        e[j * NPV + q] = ev;
                    }
                } else {
#pragma unroll
                    for (int q = 0; q < NPV; ++q) e[j * NPV + q] = f2(0.f);
                }
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
                if (FULL || i / NPV < nj) {
                    if (e[i].x == e0) ++cnt; else zz += e[i].x;
                    if (e[i].y == e0) ++cnt; else zz += e[i].y;
                }
            }
            zs = zz;
            atomicAdd(&sh.nmax, cnt);
        }
        const float zt = warp_sum_pair(zs, t2.x + t2.y, lane);  // lanes 0..15: z, lanes 16..31: t
        if (lane == 0) sh.wz[warp] = zt;
        __syncwarp();
        named_bar_sync(kBarConsumers, kQConsumers);
        float z = sh.wz[lane & (kQWarps - 1)];
#pragma unroll
        for (int ofs = 8; ofs > 0; ofs >>= 1) z += __shfl_xor_sync(0xffffffffu, z, ofs);
        const int nmax = sh.nmax;
        z = fmaf((float)nmax, e0, z);

        int status = 0;
        if (!(m > kLogitFloor) || !(z > 0.f) || !(z < INFINITY)) {
            // an unusable row (NaN / +inf logit, no finite logit): classify it from the landed bytes
            // exactly as the row-status bits are defined
            if (tid == 0) sh.bad_nan = sh.bad_finite = 0;
            named_bar_sync(kBarConsumers, kQConsumers);
            int has_nan = 0, has_finite = 0;
            for (int j = 0; j < nj; ++j) {
                const T *v = reinterpret_cast<const T *>(stage + (size_t)(tid + j * kQConsumers) * 16);
#pragma unroll
                for (int q = 0; q < VEC; ++q) {
                    const float c = Elem<T>::widen(v[q]);
                    if (!(c == c) || c == INFINITY) has_nan = 1;
                    if (c == c && fabsf(c) != INFINITY) has_finite = 1;
                }
            }
            if (has_nan) sh.bad_nan = 1;
            if (has_finite) sh.bad_finite = 1;
            named_bar_sync(kBarConsumers, kQConsumers);
            if (sh.bad_nan) status |= CIAR_ROW_NAN;
            if (!sh.bad_finite) status |= CIAR_ROW_NO_FINITE;
            if (!status) status = CIAR_ROW_NAN;  // sums overflowed without any single bad logit
        }
        // the hand-off buffer (partial sums, list of large codes) and this row's constants are ours from here on
        named_bar_sync(kBarFree, kQBlock);
        const RowConst rc = sh.rc_tab[(k / kBatch) & 1][k % kBatch];
        if (!(rc.rho == rc.rho)) status |= CIAR_ROW_NAN;
        const bool direct = !status && !rc.series;
        if (tid == 0 && !direct) {  // every consumer has read the stage: refill it
            fence_proxy_async_smem();
            issue(k + kQStages);
        }

        // ---- sweep 3: interval sums
        const float c0 = z * inv_n, th = rc.theta_p * z;
        if (!status && rc.series) {
            // Codes above th are listed and clamped to th.  Most threads hold none, and a vector
            // holding none is skipped on one comparison of its maximum.
            const float e_tm = ex2_approx(fmaf(tm, kLog2e, -m2));  // this thread's largest exponential
            if (__any_sync(0xffffffffu, e_tm > th)) {
#pragma unroll
                for (int j = 0; j < JV; ++j) {
                    float2 g = e[j * NPV];
#pragma unroll
                    for (int q = 1; q < NPV; ++q) g = make_float2(fmaxf(g.x, e[j * NPV + q].x), fmaxf(g.y, e[j * NPV + q].y));
                    if (fmaxf(g.x, g.y) > th) {
#pragma unroll
                        for (int q = 0; q < NPV; ++q) {
                            float2 ev = e[j * NPV + q];
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
                            e[j * NPV + q] = ev;
                        }
                    }
                }
            }
            // power sums of (e - c0)
            float2 T2 = f2(0.f), T3 = f2(0.f), T4 = f2(0.f);
            const float2 nc0 = f2(-c0);
#pragma unroll
            for (int i = 0; i < NP; ++i) {
                if (FULL || i / NPV < nj) {
                    const float2 y = __fadd2_rn(e[i], nc0);
                    const float2 y2 = __fmul2_rn(y, y);
                    T2 = __fadd2_rn(T2, y2);
                    T3 = __ffma2_rn(y2, y, T3);
                    T4 = __ffma2_rn(y2, y2, T4);
                }
            }
            sh.part[0][tid] = T2.x + T2.y;
            sh.part[1][tid] = T3.x + T3.y;
            sh.part[2][tid] = T4.x + T4.y;
        } else if (direct) {
            // both bounds of every code, from the row still sitting in its stage
            const float invz = 1.0f / z;
            float ps[5] = { 0.f, 0.f, 0.f, 0.f, 0.f };
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
                    ps[0] += pl;
                    ps[1] += dd;
                    ps[2] = fmaf(pl, pl, ps[2]);
                    ps[3] = fmaf(pl, dd, ps[3]);
                    ps[4] = fmaf(dd, dd, ps[4]);
                }
            }
#pragma unroll
            for (int q = 0; q < 5; ++q) {
                const float w = warp_sum_f(ps[q]);
                if (lane == 0) sh.dpart[q][warp] = w;
            }
            named_bar_sync(kBarConsumers, kQConsumers);
            if (tid == 0) {
                fence_proxy_async_smem();
                issue(k + kQStages);
            }
        }

        // ---- hand the row to the finalizer warp
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
            sh.info.cmd = 0;
        }
        __syncwarp();
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
    __syncwarp();
    named_bar_arrive(kBarFull, kQBlock);
}

template <typename T, int JV, int MINB, bool FULL>
cudaError_t launch_one(const QuantifyArgs &a, cudaStream_t stream)
{
    constexpr size_t smem = (size_t)kQStages * kQConsumers * JV * 16 + sizeof(QShared);
    static bool configured[64] = {};
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!configured[dev]) {
        err = cudaFuncSetAttribute(quantify_stream_kernel<T, JV, MINB, FULL>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   (int)smem);
        if (err != cudaSuccess) return err;
        configured[dev] = true;
    }
    const int64_t cap = (int64_t)sm_count() * MINB;
    const unsigned grid = (unsigned)(a.rows < cap ? a.rows : cap);
    quantify_stream_kernel<T, JV, MINB, FULL><<<grid, kQBlock, smem, stream>>>(a);
    count_launch();
    return cudaGetLastError();
}

template <typename T, int JV, int MINB>
cudaError_t launch_jv(const QuantifyArgs &a, cudaStream_t stream)
{
    const int nvec = a.n / Elem<T>::kVec;
    if (nvec == kQConsumers * JV) return launch_one<T, JV, MINB, true>(a, stream);
    return launch_one<T, JV, MINB, false>(a, stream);
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
        if (a.n <= 4096) return launch_jv<float, 2, 2>(a, stream);
        if (a.n <= 8192) return launch_jv<float, 4, 2>(a, stream);
        return launch_jv<float, 8, 1>(a, stream);
    }
    if (a.n <= 4096) return launch_jv<__nv_bfloat16, 1, 2>(a, stream);
    if (a.n <= 8192) return launch_jv<__nv_bfloat16, 2, 2>(a, stream);
    return launch_jv<__nv_bfloat16, 4, 2>(a, stream);
}

}  // namespace ciar
