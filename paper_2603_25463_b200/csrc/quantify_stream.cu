// Streaming quantifier for rows that fit a shared-memory stage (2048 .. 16384 codes, scalar or per-row radius).
//
// One persistent CTA per SM walks rows blockIdx.x, blockIdx.x + gridDim.x, ...  Its warps have three roles that
// meet only on mbarriers (there is no CTA-wide barrier inside the row loop):
//   * one producer thread copies each row into the next free stage of a shared-memory ring with one bulk (TMA)
//     copy, several rows ahead, so HBM always has requests in flight;
//   * 16 sweep warps, in groups of WPR warps that share a row (the groups take alternate rows).  A warp works on
//     its share of the landed row alone: a sweep for the maximum of the share, which becomes the reference of the
//     share's exponentials; the codes equal to that maximum are taken out of the stage (a term near 1 would cost
//     the small terms added to it their low bits; they come back exactly, as a logit and a count); a second
//     sweep with one exponential per code and the sums of exp, exp * exponent, exp^2, exp^3, exp^4 in packed
//     fp32x2, nothing kept per code.  The warp's sums, maximum and count go to the stage's slot;
//   * a few finishing warps, a row each in turn.  While the stage is held: the warps' sums are brought to the
//     row maximum and joined, and the few codes whose probability exceeds theta = 2^-8 / (e^r - 1) are looked up in
//     the stage (only lanes whose own maximum could be that high are looked at).  Then the stage goes back to
//     the producer and the row is filed in a batch.  Every 32 rows the warp does the batch's scalar arithmetic, a
//     row per lane, in double: the listed codes exactly, the series for the rest, the normalisation step,
//     Omega, Sigma, U, the entropy, the flag, and the stores.
// Rows with r > 1 take the direct route: the sweep warps exchange their sums of exponentials, then form both
// bounds of every code.  Each logit is read from HBM once.
#include "quantify_finish.cuh"

namespace ciar {

namespace {

constexpr int kCW = 16;         // sweep warps of a CTA
constexpr int kJV = 8;          // 16-byte vectors of a row one lane owns (at most)
constexpr int kMaxStages = 16;
constexpr int kSmemBudget = 227 * 1024;
constexpr int kBatch = 32;      // rows a finishing warp collects before it does their scalar arithmetic
constexpr int kHitCap = 16;     // codes above theta (other than the warps' maxima) a batched row can carry
constexpr int kLaneHits = 4;    // ... and one lane of the collecting warp can note
constexpr int kSums = 9;        // sums a sweep warp leaves (series route: the first five)

// What travels with a stage: its barriers, the row's place, and what the sweep warps leave for the finisher.
template <int WPR>
struct RowSlot {
    unsigned long long full;   // the row has landed (producer: 1 arrival + the copy's bytes)
    unsigned long long swept;  // every warp of the group has published its sums
    unsigned long long empty;  // the finisher no longer needs the stage
    long long lr, pr;          // logical row; physical row, -1 for a position past the end of its sequence
    float rho;                 // the row's radius as stored
    float wmax[WPR];           // per warp: maximum logit of its share, the reference of its exponentials
    int wcnt[WPR];             // per warp: codes equal to that maximum (taken out of the stage and of the sums)
    int wfirst[WPR];           // per warp: lowest index among them
    float wsum[WPR][12];       // per warp: [0] sum exp, [1] sum exp * exponent, [2..] route sums (series: exp^2, exp^3, exp^4
                               // about the warp's maximum; direct: pl, dd, then about the row's centres pl^2, pl dd, dd^2, pl, dd)
    __align__(16) float lmax[WPR * 32];  // per sweep lane: the maximum logit among its codes (after the share's maxima were taken out)
};

// Rows whose stage has been handed back, waiting for their scalar arithmetic; one row per column.
template <int WPR>
struct RowBatch {
    static constexpr int E = WPR + kHitCap;
    float v[kSums][kBatch]; // the warps' sums joined, in units of the row maximum (the warps' maxima are not in them)
    float zf[kBatch];       // the row's sum of exponentials as the collecting warp formed it: theta is taken from it
    float plc[kBatch], ddc[kBatch];  // direct route: the centres the sweep warps used
    double cen[4][kBatch];  // nearly uniform rows: centre and central power sums (orders 2..4) taken from the codes themselves
    long long lr[kBatch], pr[kBatch];
    float m[kBatch], rho[kBatch];
    int argmin[kBatch], status[kBatch], nent[kBatch];
    float ec[E][kBatch];    // entries: logit of a code that is treated on its own
    short mult[E][kBatch];  // > 0: a warp's maximum, that many codes, not in the sums; -1: a code above theta, in the sums
};
constexpr int kStatusCentral = 256;  // internal status bit: `cen` holds the row's central sums

template <int S, int GROUPS, int NFIN, int WPR>
struct Control {
    RowSlot<WPR> slot[S];
    unsigned long long zdone[GROUPS];  // direct route: the group's warps have published their sums of exponentials
    int abort;                         // a wait ran out somewhere: everybody leaves
    int issued;                        // rows the producer has dealt with
    int fin_next[NFIN];                // first row each finisher has not finished
    int pairs[NFIN][32];               // scratch of the collecting warps
    RowBatch<WPR> batch[NFIN];
};

__host__ __device__ constexpr int stages_for(int stage_bytes, int nfin, int wpr)
{
    const int batch = wpr == 2 ? (int)sizeof(RowBatch<2>) : wpr == 4 ? (int)sizeof(RowBatch<4>) : wpr == 8 ? (int)sizeof(RowBatch<8>) : (int)sizeof(RowBatch<16>);
    const int slot = wpr == 2 ? (int)sizeof(RowSlot<2>) : wpr == 4 ? (int)sizeof(RowSlot<4>) : wpr == 8 ? (int)sizeof(RowSlot<8>) : (int)sizeof(RowSlot<16>);
    int s = (kSmemBudget - 1024 - nfin * (batch + 128)) / (stage_bytes + slot);
    s = s > kMaxStages ? kMaxStages : s;
    // a whole number of rounds of the groups: a group then meets each stage's uses in order (a warp must never wait
    // for a phase of a barrier before it has seen the phase before it)
    return s - s % (kCW / wpr);
}

// Sums four values over the warp with six shuffles: on return lanes 0..7 hold the sum of v0, 8..15 of v1,
// 16..23 of v2, 24..31 of v3.
__device__ __forceinline__ float warp_sum4(float v0, float v1, float v2, float v3, int lane)
{
    const bool hi = (lane & 16) != 0;
    float k0 = hi ? v2 : v0, k1 = hi ? v3 : v1;
    k0 += __shfl_xor_sync(0xffffffffu, hi ? v0 : v2, 16);
    k1 += __shfl_xor_sync(0xffffffffu, hi ? v1 : v3, 16);
    const bool mid = (lane & 8) != 0;
    float k = mid ? k1 : k0;
    k += __shfl_xor_sync(0xffffffffu, mid ? k0 : k1, 8);
    k += __shfl_xor_sync(0xffffffffu, k, 4);
    k += __shfl_xor_sync(0xffffffffu, k, 2);
    k += __shfl_xor_sync(0xffffffffu, k, 1);
    return k;
}

// One lane's sum of exp * exponent with the product of a -inf logit (exponential 0) taken as 0.
template <typename T>
__device__ __noinline__ float lane_entropy_sum(const unsigned char *stage, int v0, int nj, int rowl, float m2)
{
    constexpr int VEC = Elem<T>::kVec;
    float ts = 0.f;
    for (int j = 0; j < nj; ++j) {
        const T *v = reinterpret_cast<const T *>(stage + (size_t)(v0 + j * rowl) * 16);
#pragma unroll
        for (int q = 0; q < VEC; ++q) {
            const float d = fmaf(Elem<T>::widen(v[q]), kLog2e, -m2);
            ts = fmaf(ex2_approx(d), fmaxf(d, kNegHuge), ts);
        }
    }
    return ts;
}

// Largest probability a code may have and still enter through the series (as a fraction of the row's mass): the
// expansions run in powers of beta (x - x0), beta = e^r - 1, and are cut after the fourth order, so what counts is
// beta x <= 2^-8 (the error of the sums of squares is of relative order (beta x)^3); no code but a maximum exceeds 1/2.
__device__ __forceinline__ float theta_of(float r)
{
    return fminf(0.5f, 0.00390625f / expm1f(r));
}

template <typename T>
__device__ __forceinline__ T narrow(float x);
template <>
__device__ __forceinline__ float narrow<float>(float x) { return x; }
template <>
__device__ __forceinline__ __nv_bfloat16 narrow<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

// The logit that stands in for a maximum taken out of a share whose maximum is mw: so far below mw that its
// exponential is 0 and its product with the exponent is 0 too.
template <typename T>
__device__ __forceinline__ T low_logit(float mw)
{
    return narrow<T>(mw - fmaxf(139.f, 0.5f * fabsf(mw)));
}

// Takes the codes equal to the share's maximum mw out of the stage: each becomes a logit so far below mw that its
// exponential is 0 and its product with the exponent is 0 too.  The whole warp looks at one holding lane's
// codes at a time, a code per lane.  cnt / first: how many such codes, lowest index among them; lm: the lane's
// own maximum, which for a holding lane becomes the largest of its other codes.
template <typename T>
__device__ __noinline__ void remove_maxima(unsigned char *stage, unsigned holders, int w, int rowl, int nj_full, int nj, float mw,
                                           int lane, int &cnt, int &first, float &lm)
{
    constexpr int VEC = Elem<T>::kVec;
    const T low = low_logit<T>(mw);
    int c = 0, f = INT_MAX;
    for (; holders != 0; holders &= holders - 1) {
        const int h = __ffs((int)holders) - 1;
        const int hn = (nj_full >= 0 ? nj_full : __shfl_sync(0xffffffffu, nj, h)) * VEC;  // the lane's codes
        float rest = -INFINITY;
        for (int i = lane; i < hn; i += 32) {
            const int vi = w * 32 + h + (i / VEC) * rowl;
            T *p = reinterpret_cast<T *>(stage + (size_t)vi * 16) + i % VEC;
            const float x = Elem<T>::widen(*p);
            if (x == mw) {
                *p = low;
                ++c;
                f = min(f, vi * VEC + i % VEC);
            } else {
                rest = fmaxf(rest, x);
            }
        }
        rest = warp_redux_max(rest);
        if (lane == h) lm = rest;
    }
    cnt = __reduce_add_sync(0xffffffffu, c);
    first = __reduce_min_sync(0xffffffffu, f);
    __syncwarp();
}

// 2^d for d in (-0.03, 0]: the exponential series to the fourth order (its error there is below 3e-11).
__device__ __forceinline__ float exp2_near_zero(float d)
{
    const float t = d * 0.69314718f;
    return fmaf(t, fmaf(t, fmaf(t, fmaf(t, 0.041666668f, 0.16666667f), 0.5f), 1.0f), 1.0f);
}

// 1 / y to float accuracy: the approximate reciprocal and one Newton step.  (The approximation's error is a
// saw-tooth in y; on a row of nearly equal codes it would tilt the small differences between their terms.)
__device__ __forceinline__ float rcp_refined(float y)
{
    const float r = rcp_approx(y);
    return fmaf(r, fmaf(-y, r, 1.0f), r);
}

// Direct route: what every lane needs of the row once all the warps of its group have published their share's
// maximum, count and sum of exponentials -- the row maximum m, the row's sum of exponentials z, and the centres
// about which the squares of the two raw terms are summed: the terms at the mean probability of the codes that
// are swept (the maxima have been taken out).  The sweep warps and the finisher call this on the same slot
// and get the same floats.
template <int WPR>
struct DirectRow {
    float m, z, plc, ddc;
};

template <int WPR>
__device__ __forceinline__ DirectRow<WPR> direct_row(const RowSlot<WPR> &sl, const DirectConst &dc, int n, int lane)
{
    DirectRow<WPR> d;
    const float wmo = lane < WPR ? sl.wmax[lane] : -INFINITY;
    d.m = warp_redux_max(wmo);
    const float m2r = d.m * kLog2e;
    float zr = 0.f, zc = 0.f;
    if (lane < WPR && wmo > -INFINITY && wmo < INFINITY) {
        zr = ex2_approx(wmo * kLog2e - m2r) * sl.wsum[lane][0];
        zc = fmaf((float)sl.wcnt[lane], ex2_approx(fmaf(wmo, kLog2e, -m2r)), zr);
    }
    const float zrest = warp_sum_f(zr);
    d.z = warp_sum_f(zc);
    const float xc = zrest / ((float)n * d.z), sx = 1.0f - xc;
    const float den_l = fmaf(dc.b1, sx, dc.a1), den_u = fmaf(dc.b1, xc, dc.a1);
    const float xr = xc * rcp_refined(den_l * den_u);
    d.plc = xr * den_u * dc.a1;
    d.ddc = xr * sx;
    if (!(d.plc == d.plc) || !(d.ddc == d.ddc)) d.plc = d.ddc = 0.f;  // (an unusable row: anything finite will do)
    return d;
}

// ---------------------------------------------------------------- the sweep warps

template <typename T, int WPR, int S, bool FULL, typename Ctl>
__device__ __forceinline__ void sweep_rows(const QuantifyArgs &a, unsigned char *smem, Ctl &sh, int cw, int lane, int nk)
{
    typedef Vec<T> V;
    constexpr int VEC = Elem<T>::kVec;
    constexpr int NPV = V::kPairs;
    constexpr int GROUPS = kCW / WPR;
    constexpr int ROWL = WPR * 32;  // lanes that share a row
    constexpr int SB = ROWL * kJV * 16;
    const int g = cw / WPR, w = cw % WPR;
    const int v0 = w * 32 + lane;  // the lane's first vector of a row; the others follow at ROWL
    int nj = kJV;
    if (!FULL) {
        nj = (a.n / VEC - v0 + ROWL - 1) / ROWL;
        nj = nj < 0 ? 0 : (nj > kJV ? kJV : nj);
    }
    const long long limit = a.wait_cycles;
    uint32_t zphase = 0;

    for (int k = g; k < nk; k += GROUPS) {
        const int s = k % S;
        const uint32_t par = (uint32_t)(k / S) & 1u;
        RowSlot<WPR> &sl = sh.slot[s];
        unsigned char *stage = smem + (size_t)s * SB;
        if (!wait_phase(&sl.full, par, &sh.abort, limit)) break;
        if (sl.pr < 0) {  // nothing to quantify: pass the stage on
            if (lane == 0) mbar_arrive(&sl.swept);
            continue;
        }
        const float r = row_radius(sl.rho, a.radius_is_raw, a.r_max);
        const bool series = r <= 1.0f;

        // ---- sweep 1: the maximum of this warp's share, taken out of the stage
        typename V::Max mx = V::max_init();
#pragma unroll
        for (int j = 0; j < kJV; ++j)
            if (FULL || j < nj) mx = V::fold_max(mx, stage_vec(stage, v0 + j * ROWL));
        float lm = V::max_value(mx);
        const float mw = warp_redux_max(lm);
        const bool live = mw > -INFINITY && mw < INFINITY;  // the share holds a finite code and no +inf
        const float m2 = mw * kLog2e;
        int cnt = 0, first = INT_MAX;
        if (live) remove_maxima<T>(stage, __ballot_sync(0xffffffffu, lm == mw), w, ROWL, FULL ? kJV : -1, nj, mw, lane, cnt, first, lm);
        if (lane == 0) {
            sl.wmax[w] = mw;
            sl.wcnt[w] = cnt;
            sl.wfirst[w] = first;
        }
        const float2 L2 = f2(kLog2e), nm2 = f2(-m2);

        if (series) {
            // ---- sweep 2, series route: one exponential per code; sums of exp, exp * exponent, exp^2, exp^3, exp^4
            float2 z2 = f2(0.f), t2 = f2(0.f), s2 = f2(0.f), s3 = f2(0.f), s4 = f2(0.f);
            if (live) {
#pragma unroll
                for (int j = 0; j < kJV; ++j) {
                    if (FULL || j < nj) {
                        float2 c[NPV];
                        V::pairs(stage_vec(stage, v0 + j * ROWL), c);
#pragma unroll
                        for (int q = 0; q < NPV; ++q) {
                            const float2 d = __ffma2_rn(c[q], L2, nm2);
                            const float2 e = make_float2(ex2_approx(d.x), ex2_approx(d.y));  // a NaN logit poisons the sums on purpose
                            z2 = __fadd2_rn(z2, e);
                            t2 = __ffma2_rn(e, d, t2);  // 0 * -inf = NaN for a -inf logit: redone below
                            const float2 ee = __fmul2_rn(e, e);
                            s2 = __fadd2_rn(s2, ee);
                            s3 = __ffma2_rn(ee, e, s3);
                            s4 = __ffma2_rn(ee, ee, s4);
                        }
                    }
                }
            }
            float ts = t2.x + t2.y;
            if (!(ts == ts)) ts = lane_entropy_sum<T>(stage, v0, nj, ROWL, m2);
            const float r4 = warp_sum4(z2.x + z2.y, ts, s2.x + s2.y, s3.x + s3.y, lane);
            const float r5 = warp_sum_f(s4.x + s4.y);
            if ((lane & 7) == 0) sl.wsum[w][lane >> 3] = r4;
            if (lane == 0) sl.wsum[w][4] = r5;
            sl.lmax[v0] = lm;  // tells the finisher where to look for codes above theta
        } else {
            // ---- direct route (r > 1): the sum of exponentials first, exchanged within the group ...
            float2 z2 = f2(0.f), t2 = f2(0.f);
            if (live) {
#pragma unroll
                for (int j = 0; j < kJV; ++j) {
                    if (FULL || j < nj) {
                        float2 c[NPV];
                        V::pairs(stage_vec(stage, v0 + j * ROWL), c);
#pragma unroll
                        for (int q = 0; q < NPV; ++q) {
                            const float2 d = __ffma2_rn(c[q], L2, nm2);
                            const float2 e = make_float2(ex2_approx(d.x), ex2_approx(d.y));
                            z2 = __fadd2_rn(z2, e);
                            t2 = __ffma2_rn(e, d, t2);
                        }
                    }
                }
            }
            float ts = t2.x + t2.y;
            if (!(ts == ts)) ts = lane_entropy_sum<T>(stage, v0, nj, ROWL, m2);
            const float zt = warp_sum_pair(z2.x + z2.y, ts, lane);  // lanes 0..15: z, lanes 16..31: t
            if ((lane & 15) == 0) sl.wsum[w][lane >> 4] = zt;
            __syncwarp();
            if (WPR > 1) {
                if (lane == 0) mbar_arrive(&sh.zdone[g]);
                if (!wait_phase<false>(&sh.zdone[g], zphase, &sh.abort, limit)) break;
                zphase ^= 1u;
            }
            // ... then both bounds of every code, from the row still sitting in its stage (the maxima that were
            // taken out are left out here; the finisher brings them in): sums of the two raw terms, and of their
            // deviations from the row's centres, squares and product
            const DirectConst dc = make_direct_const(r, a.n);
            const DirectRow<WPR> dr = direct_row<WPR>(sl, dc, a.n, lane);
            const float m2r = dr.m * kLog2e;
            const float invz = 1.0f / dr.z;
            // A row whose exponentials are nearly all close to the maximum's: its widths differ so little that the
            // approximate exponential's error (a saw-tooth in the exponent) would tilt the differences.
            const bool tight = dr.z > 0.9f * (float)a.n;
            float ps[7] = { 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f };
            const float lowf = Elem<T>::widen(low_logit<T>(mw));  // what stands where a maximum was: left out of the sums
            int nskip = 0;
#pragma unroll 1
            for (int j = 0; j < nj; ++j) {
                const T *v = reinterpret_cast<const T *>(stage + (size_t)(v0 + j * ROWL) * 16);
                float c[VEC];
                Elem<T>::load(v, c);
#pragma unroll
                for (int q = 0; q < VEC; ++q) {
                    if (live && c[q] == lowf) {
                        ++nskip;
                        continue;
                    }
                    const float dq = fmaf(c[q], kLog2e, -m2r);
                    float ev = ex2_approx(dq);
                    if (tight && dq > -0.03f) ev = exp2_near_zero(dq);
                    const float x = ev * invz, sx = fmaf(-ev, invz, 1.0f);
                    const float den_l = fmaf(dc.b1, sx, dc.a1), den_u = fmaf(dc.b1, x, dc.a1);
                    const float xr = x * rcp_refined(den_l * den_u);
                    const float pl = xr * den_u * dc.a1, dd = xr * sx;  // p^l term, width term
                    const float pc = pl - dr.plc, dcn = dd - dr.ddc;
                    ps[0] += pl;
                    ps[1] += dd;
                    ps[2] = fmaf(pc, pc, ps[2]);
                    ps[3] = fmaf(pc, dcn, ps[3]);
                    ps[4] = fmaf(dcn, dcn, ps[4]);
                    ps[5] += pc;
                    ps[6] += dcn;
                }
            }
            // a code of the row that happened to hold that very logit was left out too: it has probability 0
            const int extra = __reduce_add_sync(0xffffffffu, nskip) - cnt;
            if (lane == 0 && extra > 0) {
                const float x = (float)extra;
                ps[2] = fmaf(x * dr.plc, dr.plc, ps[2]);
                ps[3] = fmaf(x * dr.plc, dr.ddc, ps[3]);
                ps[4] = fmaf(x * dr.ddc, dr.ddc, ps[4]);
                ps[5] = fmaf(-x, dr.plc, ps[5]);
                ps[6] = fmaf(-x, dr.ddc, ps[6]);
            }
            const float r4 = warp_sum4(ps[0], ps[1], ps[2], ps[3], lane);
            const float r3 = warp_sum4(ps[4], ps[5], ps[6], 0.f, lane);
            if ((lane & 7) == 0) {
                sl.wsum[w][2 + (lane >> 3)] = r4;
                if (lane < 24) sl.wsum[w][6 + (lane >> 3)] = r3;
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&sl.swept);
    }
}

// ---------------------------------------------------------------- the finishing warps

// The sums a row's scalar arithmetic starts from (series route), however they were gathered.
struct SeriesSums {
    double zd;        // the row's sum of exponentials (units of the row maximum)
    double P[4];      // power sums (orders 1..4) of the exponentials of the codes that enter through the series
    double nu, nl;    // how many those are; how many codes are treated exactly
    double ls[5];     // exact sums over the latter: p^l, d, p^l^2, p^l d, d^2 (d = p^u - p^l)
};

// One code treated exactly: x = e / Z, 1 - x from the other codes' exponentials.
__device__ __forceinline__ void add_listed(SeriesSums &q, double e, double mult, double invz, double beta, double kap)
{
    const double x = e * invz, sx = (q.zd - e) * invz;
    const double den = fast_rcp((1.0 + beta * sx) * (1.0 + beta * x));
    const double pl = x * (1.0 + beta * x) * den, d = kap * x * sx * den;
    q.ls[0] += mult * pl;
    q.ls[1] += mult * d;
    q.ls[2] += mult * pl * pl;
    q.ls[3] += mult * pl * d;
    q.ls[4] += mult * d * d;
    q.nl += mult;
    q.nu -= mult;
}

// The end of a row's arithmetic, from the sums of the raw bounds on: normalisation step done, Sigma, U, entropy,
// flag, stores.  zd, t_raw: sum of exp and of exp * exponent over all codes, in units of the row maximum.
__device__ __forceinline__ void store_row(const QuantifyArgs &a, long long lr, long long pr, float m, int argmin, double zd, double t_raw,
                                          double S_lo, double S_up, double omega, double ss)
{
    const ciar_quantify_out &o = a.out;
    const double inv_nn = fast_rcp((double)a.n);
    const double sigma = sqrt((ss > 0.0 ? ss : 0.0) * inv_nn);
    const double score = omega * sigma;
    // exponent actually used: c * log2e_f - m2 = (c - m) * log2e_f + off with off = m * log2e_f - m2
    const float m2 = m * kLog2e;
    const double off = (double)m * (double)kLog2e - (double)m2;
    const double w2 = -off * kLn2D;
    const double unscale = 1.0 + w2 * (1.0 + 0.5 * w2);  // 2^-off: |off| is a rounding error of m * log2e, far below 1e-4
    const double z = zd * unscale;
    const double t = t_raw * unscale - off * z;
    // ln z: z >= 1 up to rounding; log1p keeps the digits of a z just above 1 (a peaked row)
    const double lnz = z < 1.5 ? (double)log1pf((float)(z - 1.0)) : (double)logf((float)z);
    const double p_max = fast_rcp(z);
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
    if (o.argmax) o.argmax[lr] = argmin + a.vb;
    if (o.flag) o.flag[lr] = (uint8_t)fl;
    if (o.row_status) o.row_status[lr] = 0;
}

// Series route: from the sums to the sums of the raw bounds and of the squared widths.  `central`: the centre c0 and
// the central power sums C2..C4 of the series codes, when they were taken from the codes themselves.
__device__ __forceinline__ void series_tail(const QuantifyArgs &a, const SeriesSums &q, float r, const double *central, double &S_lo,
                                            double &S_up, double &omega, double &ss)
{
    const double beta = (double)expm1f(r);  // e^r - 1 to float accuracy: the bounds depend on it smoothly
    const double b = 1.0 + beta, kap = beta * (2.0 + beta);
    const double invz = fast_rcp(q.zd), nu = q.nu;
    double c0, C2, C3, C4;
    if (central) {
        c0 = central[0];
        C2 = central[1];
        C3 = central[2];
        C4 = central[3];
    } else {
        // central power sums about the mean exponential of those codes
        c0 = nu > 0.0 ? q.P[0] * fast_rcp(nu) : 0.0;
        C2 = q.P[1] - nu * c0 * c0;
        C3 = q.P[2] - 3.0 * c0 * q.P[1] + 2.0 * nu * c0 * c0 * c0;
        C4 = q.P[3] - 4.0 * c0 * q.P[2] + 6.0 * c0 * c0 * q.P[1] - 3.0 * nu * c0 * c0 * c0 * c0;
    }
    // Series about x0 = c0 / Z for those codes: G_k = sum of (x - x0)^k (G_1 is 0 up to rounding by the choice of c0)
    const double x0 = c0 * invz;
    const double iz2 = invz * invz;
    const double G1 = (q.P[0] - nu * c0) * invz;
    const double G2 = C2 * iz2, G3 = C3 * iz2 * invz, G4 = C4 * iz2 * iz2;
    // Taylor coefficients about x0 of p^l(x) = x / (b - beta x) and of d(x) = p^u - p^l, p^u(x) = b x / (1 + beta x),
    // and what the sums need of them
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
    const double *ls = q.ls;
    const double B = nu * PL0 + Bd + ls[0];  // sum of raw p^l
    const double A = nu * DD0 + Ad + ls[1];  // sum of raw widths
    S_lo = B;
    S_up = A + B;
    const double rs = S_lo > 0.0 && S_up > 0.0 ? fast_rcp(S_lo * S_up) : 0.0;
    double k_lo = (double)a.lo_cap * S_up * rs, k_up = (double)a.hi_cap * S_lo * rs;
    if (!(S_lo > 0.0) || !(k_lo < 1.0)) k_lo = 1.0;
    if (!(S_up > 0.0) || !(k_up > 1.0)) k_up = 1.0;
    const double g = k_up - k_lo;  // delta = k_up d + g p^l
    omega = k_up * A + g * B;
    const double mu = omega * fast_rcp((double)a.n);
    const double E0 = k_up * DD0 + g * PL0 - mu;  // delta - mu at x0
    // sum of (delta - mu)^2: series codes from the expansion, listed codes from their five exact sums
    ss = nu * E0 * E0 + 2.0 * E0 * (k_up * Ad + g * Bd) + k_up * k_up * Qdd + 2.0 * k_up * g * Qdp + g * g * Qpp +
         (k_up * k_up * ls[4] + 2.0 * k_up * g * ls[3] + g * g * ls[2] - 2.0 * mu * (k_up * ls[1] + g * ls[0]) + q.nl * mu * mu);
}

// The scalar arithmetic of the collected rows, a row per lane.
template <int WPR>
__device__ __noinline__ void finish_batch(const QuantifyArgs &a, const RowBatch<WPR> &bt, int count, int lane)
{
    if (lane >= count) return;
    const long long lr = bt.lr[lane], pr = bt.pr[lane];
    const int status = bt.status[lane];
    if (status & 255) {
        write_unusable(a.out, lr, status & 255);
        return;
    }
    const float m = bt.m[lane];
    const float r = row_radius(bt.rho[lane], a.radius_is_raw, a.r_max);
    const float m2 = m * kLog2e;
    const int nent = bt.nent[lane];
    double S_lo, S_up, omega, ss;
    // the warps' maxima come back: sum of exponentials and of exp * exponent over all codes
    double zd = (double)bt.v[0][lane], t = (double)bt.v[1][lane];
    for (int i = 0; i < nent; ++i) {
        const int mu = bt.mult[i][lane];
        if (mu <= 0) continue;
        const float d = fmaf(bt.ec[i][lane], kLog2e, -m2);
        const double e = (double)ex2_approx(d);
        zd += (double)mu * e;
        t += (double)mu * e * (double)fmaxf(d, kNegHuge);
    }
    if (r <= 1.0f) {
        const float th = theta_of(r) * bt.zf[lane];  // theta in units of exp(c - m)
        const double beta = (double)expm1f(r), kap = beta * (2.0 + beta), invz = fast_rcp(zd);
        SeriesSums q;
        q.zd = zd;
        q.P[0] = (double)bt.v[0][lane];
        q.P[1] = (double)bt.v[2][lane];
        q.P[2] = (double)bt.v[3][lane];
        q.P[3] = (double)bt.v[4][lane];
        q.nu = (double)a.n;
        q.nl = 0.0;
#pragma unroll
        for (int i = 0; i < 5; ++i) q.ls[i] = 0.0;
        for (int i = 0; i < nent; ++i) {
            const int mu = bt.mult[i][lane];
            if (mu == 0) continue;
            const float ef = ex2_approx(fmaf(bt.ec[i][lane], kLog2e, -m2));
            const double e = (double)ef, e2 = e * e;
            if (mu < 0) {  // a code above theta that the sweeps summed: out of the power sums, in exactly
                q.P[0] -= e;
                q.P[1] -= e2;
                q.P[2] -= e2 * e;
                q.P[3] -= e2 * e2;
                add_listed(q, e, 1.0, invz, beta, kap);
            } else if (ef > th) {  // a warp's maxima above theta: exactly
                add_listed(q, e, (double)mu, invz, beta, kap);
            } else {  // a warp's maxima below theta: into the power sums
                const double c = (double)mu;
                q.P[0] += c * e;
                q.P[1] += c * e2;
                q.P[2] += c * e2 * e;
                q.P[3] += c * e2 * e2;
            }
        }
        double cen[4];
        const bool central = (status & kStatusCentral) != 0;
        if (central) {
#pragma unroll
            for (int i = 0; i < 4; ++i) cen[i] = bt.cen[i][lane];
        }
        series_tail(a, q, r, central ? cen : nullptr, S_lo, S_up, omega, ss);
    } else {
        const DirectConst dc = make_direct_const(r, a.n);  // the same constants as the sweep used
        double P1 = (double)bt.v[2][lane], D1 = (double)bt.v[3][lane], PP = (double)bt.v[4][lane], PD = (double)bt.v[5][lane],
               DD = (double)bt.v[6][lane], P1c = (double)bt.v[7][lane], D1c = (double)bt.v[8][lane];
        const double a1 = (double)dc.a1, b1 = (double)dc.b1, plc = (double)bt.plc[lane], ddc = (double)bt.ddc[lane];
        // the warps' maxima were left out of the sweep's sums: their raw terms come in here
        const double invz = fast_rcp(zd);
        double nswept = (double)a.n;
        for (int i = 0; i < nent; ++i) {
            const int mu = bt.mult[i][lane];
            if (mu <= 0) continue;
            const double e = (double)ex2_approx(fmaf(bt.ec[i][lane], kLog2e, -m2));
            const double x = e * invz, sx = (zd - e) * invz;
            const double xr = x * fast_rcp((a1 + b1 * sx) * (a1 + b1 * x));
            P1 += (double)mu * xr * (a1 + b1 * x) * a1;
            D1 += (double)mu * xr * sx;
            nswept -= (double)mu;
        }
        const double nn = (double)a.n;
        const double kd = dc.big ? 1.0 + 2.0 * a1 : b1 * (2.0 + b1);
        const double B = P1;        // sum of the raw lower bounds
        const double A = kd * D1;   // sum of the raw widths
        S_lo = B;
        S_up = A + B;
        double k_lo = 1.0, k_up = 1.0;
        if (S_lo > 0.0 && (double)a.lo_cap / S_lo < 1.0) k_lo = (double)a.lo_cap / S_lo;
        if (S_up > 0.0 && (double)a.hi_cap / S_up > 1.0) k_up = (double)a.hi_cap / S_up;
        // delta_i = k_up d_i + (k_up - k_lo) p^l_i = c1 dd_i + c2 pl_i.  The swept codes' deviations were summed about
        // delta at the centres: they are moved to the mean mu; the maxima's deviations from mu are formed one by one
        // (a row of equal codes is all maxima: its sum of squares must come out as 0, not as a difference of equals)
        const double c1 = k_up * kd, c2 = k_up - k_lo;
        omega = c1 * D1 + c2 * B;
        const double shift = omega * fast_rcp(nn) - (c1 * ddc + c2 * plc);  // mu - delta(centres)
        const double lin = c1 * D1c + c2 * P1c;
        ss = c1 * c1 * DD + 2.0 * c1 * c2 * PD + c2 * c2 * PP - 2.0 * shift * lin + nswept * shift * shift;
        for (int i = 0; i < nent; ++i) {
            const int mu = bt.mult[i][lane];
            if (mu <= 0) continue;
            const double e = (double)ex2_approx(fmaf(bt.ec[i][lane], kLog2e, -m2));
            const double x = e * invz, sx = (zd - e) * invz;
            const double xr = x * fast_rcp((a1 + b1 * sx) * (a1 + b1 * x));
            const double dev = c1 * (xr * sx - ddc) + c2 * (xr * (a1 + b1 * x) * a1 - plc) - shift;
            ss += (double)mu * dev * dev;
        }
    }
    store_row(a, lr, pr, m, bt.argmin[lane], zd, t, S_lo, S_up, omega, ss);
}

// A row with more codes above theta than a batch column carries: everything is done here, by the whole warp,
// while the stage is held.  v: the joined sums without the warps' maxima.
template <typename T, int WPR>
__device__ __noinline__ void finish_crowded_row(const QuantifyArgs &a, RowSlot<WPR> &sl, const unsigned char *stage, int lane, float m, float r,
                                                float th, const float (&v)[5], int argmin)
{
    constexpr int VEC = Elem<T>::kVec;
    const int nvec = a.n / VEC;
    const float m2 = m * kLog2e;
    const int w = lane % WPR;
    const float wm = sl.wmax[w];
    const int wc = lane < WPR && wm > -INFINITY && wm < INFINITY ? sl.wcnt[w] : 0;
    const float dwm = fmaf(wm, kLog2e, -m2);
    const float ewf = wc > 0 ? ex2_approx(dwm) : 0.f;
    const double ew = (double)ewf;
    SeriesSums q;
    q.zd = (double)v[0] + warp_sum_d((double)wc * ew);
    const double t = (double)v[1] + warp_sum_d(wc > 0 ? (double)wc * ew * (double)fmaxf(dwm, kNegHuge) : 0.0);
    const double beta = (double)expm1f(r), kap = beta * (2.0 + beta), invz = fast_rcp(q.zd);
    q.nu = 0.0;
    q.nl = 0.0;
#pragma unroll
    for (int i = 0; i < 5; ++i) q.ls[i] = 0.0;
    double rm[4] = { 0.0, 0.0, 0.0, 0.0 };
    // this lane's share of the codes above theta: a warp's maxima (lanes below WPR), then its part of the stage
    if (wc > 0) {
        if (ewf > th) {
            add_listed(q, ew, (double)wc, invz, beta, kap);
        } else {
            const double c = (double)wc, e2 = ew * ew;
            rm[0] -= c * ew;
            rm[1] -= c * e2;
            rm[2] -= c * e2 * ew;
            rm[3] -= c * e2 * e2;
        }
    }
    for (int vi = lane; vi < nvec; vi += 32) {
        const T *p = reinterpret_cast<const T *>(stage + (size_t)vi * 16);
        for (int i = 0; i < VEC; ++i) {
            const float ef = ex2_approx(fmaf(Elem<T>::widen(p[i]), kLog2e, -m2));
            if (ef > th) {
                const double e = (double)ef, e2 = e * e;
                rm[0] += e;
                rm[1] += e2;
                rm[2] += e2 * e;
                rm[3] += e2 * e2;
                add_listed(q, e, 1.0, invz, beta, kap);
            }
        }
    }
    const long long lr = sl.lr, pr = sl.pr;  // (the slot goes back with the stage)
    __syncwarp();
    if (lane == 0) mbar_arrive(&sl.empty);
#pragma unroll
    for (int i = 0; i < 5; ++i) q.ls[i] = warp_sum_d(q.ls[i]);
#pragma unroll
    for (int i = 0; i < 4; ++i) rm[i] = warp_sum_d(rm[i]);
    q.nl = warp_sum_d(q.nl);
    q.nu = (double)a.n - q.nl;
    q.P[0] = (double)v[0] - rm[0];
    q.P[1] = (double)v[2] - rm[1];
    q.P[2] = (double)v[3] - rm[2];
    q.P[3] = (double)v[4] - rm[3];
    if (lane != 0) return;
    double S_lo, S_up, omega, ss;
    series_tail(a, q, r, nullptr, S_lo, S_up, omega, ss);
    store_row(a, lr, pr, m, argmin, q.zd, t, S_lo, S_up, omega, ss);
}

// Says what is wrong with an unusable row (NaN / +inf logit, no finite logit) from the landed bytes, exactly as the
// row-status bits are defined (a maximum that was taken out left a finite logit in its place).
template <typename T>
__device__ __noinline__ int classify_row(const unsigned char *stage, int nvec, int lane)
{
    constexpr int VEC = Elem<T>::kVec;
    int has_nan = 0, has_finite = 0;
    for (int vi = lane; vi < nvec; vi += 32) {
        const T *p = reinterpret_cast<const T *>(stage + (size_t)vi * 16);
#pragma unroll
        for (int q = 0; q < VEC; ++q) {
            const float c = Elem<T>::widen(p[q]);
            if (!(c == c) || c == INFINITY) has_nan = 1;
            if (c == c && fabsf(c) != INFINITY) has_finite = 1;
        }
    }
    int status = 0;
    if (__any_sync(0xffffffffu, has_nan)) status |= CIAR_ROW_NAN;
    if (!__any_sync(0xffffffffu, has_finite)) status |= CIAR_ROW_NO_FINITE;
    return status ? status : CIAR_ROW_NAN;  // sums overflowed without any single bad logit
}

// Nearly equal exponentials: the central power sums of the codes that enter through the series, taken from the
// codes themselves about the float c0f, into column `col` of the batch.  wc, ew: this lane's warp's maxima
// (lanes below WPR), which sit in the stage as codes of exponential 0.
template <typename T, int WPR>
__device__ __noinline__ void central_sums(const unsigned char *stage, int nvec, int lane, float m2, float th, float c0f, int wc, float ew,
                                          RowBatch<WPR> &bt, int col)
{
    constexpr int VEC = Elem<T>::kVec;
    double y[4] = { 0.0, 0.0, 0.0, 0.0 };
    for (int vi = lane; vi < nvec; vi += 32) {
        const T *p = reinterpret_cast<const T *>(stage + (size_t)vi * 16);
        float b1 = 0.f, b2 = 0.f, b3 = 0.f, b4 = 0.f;
#pragma unroll
        for (int q = 0; q < VEC; ++q) {
            const float ef = ex2_approx(fmaf(Elem<T>::widen(p[q]), kLog2e, -m2));
            if (ef > th) continue;
            const float yy = ef - c0f, y2 = yy * yy;
            b1 += yy;
            b2 += y2;
            b3 = fmaf(y2, yy, b3);
            b4 = fmaf(y2, y2, b4);
        }
        y[0] += (double)b1;
        y[1] += (double)b2;
        y[2] += (double)b3;
        y[3] += (double)b4;
    }
    if (lane < WPR && wc > 0) {  // the maxima that were taken out: their terms are put right
        const double c = (double)wc, y0 = -(double)c0f;
        double yk = y0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            y[i] -= c * yk;
            yk *= y0;
        }
        if (!(ew > th)) {
            const double y1 = (double)ew - (double)c0f;
            yk = y1;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                y[i] += c * yk;
                yk *= y1;
            }
        }
    }
#pragma unroll
    for (int q = 1; q < 4; ++q) y[q] = warp_sum_d(y[q]);
    if (lane == 0) {
        // (the first-order sum about the centre is formed again from the power sum and the centre when the series is evaluated)
        bt.cen[0][col] = (double)c0f;
        bt.cen[1][col] = y[1];
        bt.cen[2][col] = y[2];
        bt.cen[3][col] = y[3];
    }
}

// Exclusive prefix over the lanes of a small per-lane count (below 32), and the total, from five ballots.
__device__ __forceinline__ int lane_prefix(int cnt, int lane, int &total)
{
    const unsigned lt = (1u << lane) - 1u;
    int pre = 0;
    total = 0;
#pragma unroll
    for (int b = 0; b < 5; ++b) {
        const unsigned v = __ballot_sync(0xffffffffu, (cnt >> b) & 1);
        pre += __popc(v & lt) << b;
        total += __popc(v) << b;
    }
    return pre;
}

// Collects one row while its stage is held: brings the warps' sums to the row maximum and joins them, finds the
// codes above theta in the stage, hands the stage back (lane 0 arrives on the slot's `empty` barrier) and files
// the row in column `col` of the batch.  Returns false when the row was finished on the spot instead (it has more
// such codes than a column carries).  Run by one whole warp.  The order of the steps is the shortest way to the
// moment the stage can go back; what does not need the stage comes after it.
template <typename T, int WPR>
__device__ __noinline__ bool collect_row(const QuantifyArgs &a, RowSlot<WPR> &sl, const unsigned char *stage, RowBatch<WPR> &bt, int col,
                                         int lane, int *pairs)
{
    typedef Vec<T> V;
    constexpr int VEC = Elem<T>::kVec;
    constexpr int ROWL = WPR * 32;
    constexpr int PER = 32 / WPR;             // sums joined at a time
    constexpr int NPASS = (kSums + PER - 1) / PER;
    const int nvec = a.n / VEC;
    const int w = lane % WPR;

    const float wm = sl.wmax[w];
    const bool live = wm > -INFINITY && wm < INFINITY;
    const int wc = live ? sl.wcnt[w] : 0;
    const float m = warp_redux_max(wm);
    const float m2 = m * kLog2e;
    const float rho = sl.rho;
    const float r = row_radius(rho, a.radius_is_raw, a.r_max);
    const bool series = r <= 1.0f;
    const float dw = live ? wm * kLog2e - m2 : 0.f;  // what the warp's exponents lack of the row's
    const float sc = live ? ex2_approx(dw) : 0.f;    // scale of the warp's exponentials in units of the row maximum
    const float ew = live ? ex2_approx(fmaf(wm, kLog2e, -m2)) : 0.f;  // the warp's maximum itself, in those units

    // the warps' sums joined, 32 / WPR of the seven at a time, one (sum, warp) pair per lane: after the loop the
    // first lane of each group of WPR holds a total in xs[pass]
    float xs[NPASS];
#pragma unroll
    for (int ps = 0; ps < NPASS; ++ps) {
        if (series && ps * PER >= 5) {  // the series route leaves five sums
            xs[ps] = 0.f;
            continue;
        }
        const int q = ps * PER + lane / WPR;
        float x = 0.f;
        if (q < kSums) {  // (a share without a finite code has scale 0; its direct-route sums still count)
            float f = sc;
            if (q >= 2) {
                const float sc2 = sc * sc;
                f = !series ? 1.0f : q == 2 ? sc2 : q == 3 ? sc2 * sc : sc2 * sc2;
            }
            x = sl.wsum[w][q] * f;
            if (q == 1) x = fmaf(sc * dw, sl.wsum[w][0], x);
        }
#pragma unroll
        for (int o = WPR / 2; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
        xs[ps] = x;
    }
    const float v0 = __shfl_sync(0xffffffffu, xs[0], 0);
    const float v2 = __shfl_sync(0xffffffffu, xs[2 / PER], (2 % PER) * WPR);
    const float zf = v0 + warp_sum_f(lane < WPR ? (float)wc * ew : 0.f);  // the row's sum of exponentials

    int status = 0;
    if (!(m > -INFINITY) || !(m < INFINITY) || !(zf > 0.f) || !(zf < INFINITY)) status = classify_row<T>(stage, nvec, lane);
    if (!(rho == rho)) status |= CIAR_ROW_NAN;

    float h[kLaneHits];
#pragma unroll
    for (int i = 0; i < kLaneHits; ++i) h[i] = 0.f;
    int cnt = 0, below = 0, nhit = 0;
    bool crowded = false;
    const float th = theta_of(r) * zf;  // theta in units of exp(c - m)
    if (!status && series) {
        const float dlo = __log2f(th) - 1e-3f;  // a slightly low stand-in for log2(th): no exponent below it gives more than th
        // The sweep lanes whose own maximum exceeds theta, WPR of them looked up per lane here ...
        unsigned mine = 0;
#pragma unroll
        for (int i = 0; i < WPR; ++i)
            if (fmaf(sl.lmax[lane * WPR + i], kLog2e, -m2) > dlo) mine |= 1u << i;
        int total;
        int pos = lane_prefix(__popc(mine), lane, total);
        crowded = total > 32;
        if (!crowded && total > 0) {  // (most rows have no such lane)
            for (; mine != 0; mine &= mine - 1) pairs[pos++] = lane * WPR + __ffs((int)mine) - 1;
            __syncwarp();
            // ... each is looked at by one lane: which of its kJV vectors hold such a code ...
            unsigned vmask = 0;
            const int sv = lane < total ? pairs[lane] : 0;  // the sweep lane's first vector
            if (lane < total) {
#pragma unroll
                for (int j = 0; j < kJV; ++j) {
                    const int vi = j * ROWL + sv;
                    if (vi < nvec && fmaf(V::max_value(V::fold_max(V::max_init(), stage_vec(stage, vi))), kLog2e, -m2) > dlo) vmask |= 1u << j;
                }
            }
            pos = lane_prefix(__popc(vmask), lane, total);
            crowded = total > 32;
            __syncwarp();
            if (!crowded && total > 0) {
                for (; vmask != 0; vmask &= vmask - 1) pairs[pos++] = (__ffs((int)vmask) - 1) * ROWL + sv;
                __syncwarp();
                // ... and each of those vectors by one lane, which notes the logits of the codes it finds
                if (lane < total) {
                    const T *p = reinterpret_cast<const T *>(stage + (size_t)pairs[lane] * 16);
                    float c[VEC];
                    Elem<T>::load(p, c);
#pragma unroll
                    for (int q = 0; q < VEC; ++q) {
                        if (ex2_approx(fmaf(c[q], kLog2e, -m2)) > th) {
#pragma unroll
                            for (int i = 0; i < kLaneHits; ++i)
                                if (cnt == i) h[i] = c[q];
                            ++cnt;
                        }
                    }
                }
                below = lane_prefix(cnt > kLaneHits ? kLaneHits : cnt, lane, nhit);
                crowded = nhit > kHitCap || __any_sync(0xffffffffu, cnt > kLaneHits);
            }
        }
        if (crowded) {
            float v[5];
#pragma unroll
            for (int i = 0; i < 5; ++i) v[i] = __shfl_sync(0xffffffffu, xs[i / PER], (i % PER) * WPR);
            const bool top = lane < WPR && live && wm == m;
            finish_crowded_row<T, WPR>(a, sl, stage, lane, m, r, th, v, __reduce_min_sync(0xffffffffu, top ? sl.wfirst[w] : INT_MAX));
            return false;
        }
        // Nearly equal exponentials?  Then the central power sums, as differences of raw ones, would have lost their
        // digits: a look in float at the raw sums of the codes that enter through the series tells.
        float P1f = v0, P2f = v2, nuf;
        const bool max_in_series = lane < WPR && wc > 0 && !(ew > th);
        if (nhit == 0 && !__any_sync(0xffffffffu, max_in_series)) {
            // (the usual case: nothing but the warps' maxima is treated exactly)
            nuf = (float)(a.n - __reduce_add_sync(0xffffffffu, lane < WPR ? wc : 0));
        } else {
            float a1 = 0.f, a2 = 0.f, an = 0.f;
#pragma unroll
            for (int i = 0; i < kLaneHits; ++i) {
                if (cnt > i) {
                    const float e = ex2_approx(fmaf(h[i], kLog2e, -m2));
                    a1 -= e;
                    a2 = fmaf(-e, e, a2);
                    an -= 1.f;
                }
            }
            if (lane < WPR && wc > 0) {
                if (ew > th) {
                    an -= (float)wc;
                } else {
                    a1 = fmaf((float)wc, ew, a1);
                    a2 = fmaf((float)wc * ew, ew, a2);
                }
            }
            const float s4 = warp_sum4(a1, a2, an, 0.f, lane);
            P1f += __shfl_sync(0xffffffffu, s4, 0);
            P2f += __shfl_sync(0xffffffffu, s4, 8);
            nuf = (float)a.n + __shfl_sync(0xffffffffu, s4, 16);
        }
        if (P1f > 0.f && !(P2f * nuf > 1.05f * P1f * P1f)) {
            central_sums<T, WPR>(stage, nvec, lane, m2, th, P1f / nuf, wc, ew, bt, col);
            status = kStatusCentral;
        }
    }
    const bool top = lane < WPR && live && wm == m;
    const int argmin = __reduce_min_sync(0xffffffffu, top ? sl.wfirst[w] : INT_MAX);
    const long long lr = sl.lr, pr = sl.pr;
    float plc = 0.f, ddc = 0.f;
    if (!series) {
        const DirectRow<WPR> dr = direct_row<WPR>(sl, make_direct_const(r, a.n), a.n, lane);
        plc = dr.plc;
        ddc = dr.ddc;
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&sl.empty);  // nothing more is read from the stage or its slot

    // ---- the row is filed
    if (lane == 0) {
        bt.lr[col] = lr;
        bt.pr[col] = pr;
        bt.m[col] = m;
        bt.rho[col] = rho;
        bt.argmin[col] = argmin;
        bt.zf[col] = zf;
        bt.plc[col] = plc;
        bt.ddc[col] = ddc;
        bt.status[col] = status;
        bt.nent[col] = WPR + nhit;
    }
    if (w == 0) {
#pragma unroll
        for (int ps = 0; ps < NPASS; ++ps)
            if (ps * PER + lane / WPR < kSums) bt.v[ps * PER + lane / WPR][col] = xs[ps];
    }
    if (lane < WPR) {  // the warps' maxima: entries 0 .. WPR-1 (a share has at most 2048 codes)
        bt.ec[lane][col] = wm;
        bt.mult[lane][col] = (short)wc;
    }
#pragma unroll
    for (int i = 0; i < kLaneHits; ++i) {
        if (cnt > i) {
            bt.ec[WPR + below + i][col] = h[i];
            bt.mult[WPR + below + i][col] = -1;
        }
    }
    return true;
}

template <typename T, int WPR, int S, int NFIN, typename Ctl>
__device__ __forceinline__ void finish_rows(const QuantifyArgs &a, const unsigned char *smem, Ctl &sh, int f, int lane, int nk)
{
    constexpr int SB = WPR * 32 * kJV * 16;
    const long long limit = a.wait_cycles;
    RowBatch<WPR> &bt = sh.batch[f];
    int filled = 0;
    int k = 0;
    // Each stage is always served by the same finishing warp (stage s by warp s % NFIN), which takes its rows in the
    // order of the walk: a warp then never waits for a phase of a barrier before it has seen the phase before it.
    for (; k < nk; ++k) {
        const int s = k % S;
        if (s % NFIN != f) continue;
        const uint32_t par = (uint32_t)(k / S) & 1u;
        RowSlot<WPR> &sl = sh.slot[s];
        if (!wait_phase(&sl.swept, par, &sh.abort, limit)) break;
        if (sl.pr < 0) {  // a position past the end of its sequence: nothing to send to the cloud
            if (lane == 0) {
                const long long lr = sl.lr;
                if (a.out.flag) a.out.flag[lr] = 0;
                if (a.out.row_status) a.out.row_status[lr] = 0;
                mbar_arrive(&sl.empty);
            }
            continue;
        }
        if (collect_row<T, WPR>(a, sl, smem + (size_t)s * SB, bt, filled, lane, sh.pairs[f]) && ++filled == kBatch) {
            __syncwarp();
            finish_batch<WPR>(a, bt, filled, lane);
            __syncwarp();
            filled = 0;
        }
    }
    __syncwarp();
    if (filled > 0) finish_batch<WPR>(a, bt, filled, lane);
    if (lane == 0) sh.fin_next[f] = k;
}

// ---------------------------------------------------------------- the kernel

// WPR: sweep warps that share a row (a row has up to WPR * 32 * 8 vectors of 16 bytes).  FULL: exactly that many.
template <typename T, int WPR, int NFIN, bool FULL>
__global__ void __launch_bounds__((kCW + NFIN + 1) * 32, 1) quantify_stream_kernel(const __grid_constant__ QuantifyArgs a)
{
    constexpr int GROUPS = kCW / WPR;
    constexpr int SB = WPR * 32 * kJV * 16;
    constexpr int S = stages_for(SB, NFIN, WPR);
    typedef Control<S, GROUPS, NFIN, WPR> Ctl;
    static_assert(S >= 3 && S % GROUPS == 0 && (size_t)S * SB + sizeof(Ctl) <= (size_t)kSmemBudget, "the ring and its slots must fit in shared memory");
    extern __shared__ __align__(128) unsigned char smem[];
    Ctl &sh = *reinterpret_cast<Ctl *>(smem + (size_t)S * SB);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nk = (int)((a.rows - blockIdx.x + gridDim.x - 1) / gridDim.x);  // rows this CTA walks (the grid never exceeds the rows)

    if (tid == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(&sh.slot[s].full, 1);
            mbar_init(&sh.slot[s].swept, WPR);
            mbar_init(&sh.slot[s].empty, 1);
        }
        for (int g = 0; g < GROUPS; ++g) mbar_init(&sh.zdone[g], WPR);
        sh.abort = 0;
        sh.issued = 0;
        for (int f = 0; f < NFIN; ++f) sh.fin_next[f] = f;
        mbar_init_fence();
    }
    __syncthreads();

    // (the finishing warps and the producer take the lowest warp numbers)
    if (warp > NFIN) {
        sweep_rows<T, WPR, S, FULL>(a, smem, sh, warp - NFIN - 1, lane, nk);
    } else if (warp < NFIN) {
        finish_rows<T, WPR, S, NFIN>(a, smem, sh, warp, lane, nk);
    } else if (lane == 0) {
        // ---- the producer: one bulk copy per row, as soon as the stage's previous row has been handed back.
        // A row's place and stored radius are fetched one row early, so that their latency hides behind that wait.
        const uint32_t row_bytes = (uint32_t)(a.n / Elem<T>::kVec) * 16u;
        const bool per_row = a.radius_mode == CIAR_RADIUS_PER_ROW;
        int64_t lr_n = blockIdx.x, pr_n = -1;
        float rho_n = a.r_scalar;
        auto look = [&](int k) {
            lr_n = blockIdx.x + (int64_t)k * gridDim.x;
            pr_n = -1;
            if (k < nk) {
                int64_t pr;
                if (map_row(a.rm, lr_n, pr)) {
                    pr_n = pr;
                    if (per_row) rho_n = __ldg(reinterpret_cast<const float *>(a.radius) + pr);
                }
            }
        };
        look(0);
        for (int k = 0; k < nk; ++k) {
            const int s = k % S;
            RowSlot<WPR> &sl = sh.slot[s];
            const int64_t lr = lr_n, pr = pr_n;
            const float rho = rho_n;
            look(k + 1);
            if (k >= S && !wait_phase(&sl.empty, (uint32_t)(k / S - 1) & 1u, &sh.abort, a.wait_cycles)) break;
            sl.lr = lr;
            sl.pr = pr;
            sl.rho = rho;
            if (pr < 0) {
                mbar_arrive(&sl.full);
            } else if (!(a.drop_cta == (int)blockIdx.x && a.drop_k == k)) {
                fence_proxy_async_smem();  // the stage's earlier reads and writes are done before the copy writes it
                mbar_arrive_expect_tx(&sl.full, row_bytes);
                bulk_copy_g2s(smem + (size_t)s * SB, reinterpret_cast<const T *>(a.logits) + a.vb + pr * a.row_stride, row_bytes,
                              &sl.full);
            }
            sh.issued = k + 1;
        }
    }
    __syncthreads();

    if (sh.abort && tid == 0) {
        // A wait ran out (a copy never arrived).  The rows from the first unfinished one on are marked, and the
        // copies still in flight get a last bounded chance to land before the CTA leaves.
        int kmin = nk;
        for (int f = 0; f < NFIN; ++f) kmin = min(kmin, sh.fin_next[f]);
        for (int k = kmin; k < nk; ++k) write_unusable(a.out, blockIdx.x + (long long)k * gridDim.x, CIAR_ROW_TIMEOUT);
        const int issued = sh.issued;
        for (int k = max(0, issued - S); k < issued; ++k)
            mbar_wait_bounded(&sh.slot[k % S].full, (uint32_t)(k / S) & 1u, kDrainCycles);
    }
}

template <typename T, int WPR, int NFIN, bool FULL>
cudaError_t launch_one(const QuantifyArgs &a, cudaStream_t stream)
{
    constexpr int SB = WPR * 32 * kJV * 16;
    constexpr int S = stages_for(SB, NFIN, WPR);
    constexpr size_t smem = (size_t)S * SB + sizeof(Control<S, kCW / WPR, NFIN, WPR>);
    static_assert(smem <= (size_t)kSmemBudget, "the ring, its slots and the finishers' batches must fit in shared memory");
    static bool configured[64] = {};
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!configured[dev]) {
        err = cudaFuncSetAttribute(quantify_stream_kernel<T, WPR, NFIN, FULL>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (err != cudaSuccess) return err;
        configured[dev] = true;
    }
    const int64_t cap = sm_count();
    const unsigned grid = (unsigned)(a.rows < cap ? a.rows : cap);
    quantify_stream_kernel<T, WPR, NFIN, FULL><<<grid, (kCW + NFIN + 1) * 32, smem, stream>>>(a);
    count_launch();
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_typed(const QuantifyArgs &a, cudaStream_t stream)
{
    const int nvec = a.n / Elem<T>::kVec;
    const int per_warp = 32 * kJV;  // vectors one warp takes
    if (nvec <= 2 * per_warp) return nvec == 2 * per_warp ? launch_one<T, 2, 3, true>(a, stream) : launch_one<T, 2, 3, false>(a, stream);
    if (nvec <= 4 * per_warp) return nvec == 4 * per_warp ? launch_one<T, 4, 4, true>(a, stream) : launch_one<T, 4, 4, false>(a, stream);
    if (nvec <= 8 * per_warp) return nvec == 8 * per_warp ? launch_one<T, 8, 3, true>(a, stream) : launch_one<T, 8, 3, false>(a, stream);
    return nvec == 16 * per_warp ? launch_one<T, 16, 2, true>(a, stream) : launch_one<T, 16, 2, false>(a, stream);
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
    if (dtype == CIAR_F32) return launch_typed<float>(a, stream);
    return launch_typed<__nv_bfloat16>(a, stream);
}

}  // namespace ciar
