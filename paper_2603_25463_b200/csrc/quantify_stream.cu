// Streaming quantifier for rows that fit on chip (2048 .. 16384 codes, scalar or per-row radius).
//
// One persistent CTA of 16 warps walks rows blockIdx.x, blockIdx.x + gridDim.x, ...  Rows arrive
// through a ring of shared-memory stages filled by bulk (TMA) copies that one thread issues
// several rows ahead, so HBM always has requests in flight.  The warps sweep a landed row twice
// from shared memory (maximum; then one exponential per code, kept in registers: 32 per thread)
// and once more from those registers (interval sums), reduce their sums with shuffles and park
// them in shared memory.  Every 16 rows the CTA stops for a moment and each warp finishes one
// parked row: the handful of large codes exactly, one per lane, then the row's double-precision
// scalar arithmetic and its stores.  Each logit is read from HBM once.
#include <climits>

#include "ciar_internal.h"
#include "stream_common.cuh"

namespace ciar {

namespace {

constexpr int kQThreads = 512;
constexpr int kQWarps = kQThreads / 32;
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

struct QShared {
    unsigned long long full[kQStages];
    // by the row's turn (rows swept so far, low bits): a row's first sweep runs while the row before it is still in use
    float wmax[2][kQWarps];
    int argmin[2], nmax[4];  // lowest index holding the row maximum, number of codes whose exponential equals e0
    int bad_nan, bad_finite;
    int abort;
    int nlist;  // codes above theta in the row being swept
    float list[2][kListCap];  // by row parity: a long list must outlive the next row's sweeps
    Parked park[kPark];
};
static_assert(sizeof(QShared) + kQStages * 32768 <= 115712, "two CTAs per SM must fit in shared memory");

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
__device__ __noinline__ void finish_row(const QuantifyArgs &a, const Parked &pk, const float *list, int lane)
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
            if (lane < kQWarps) v[q] = (double)pk.wsum[lane][kSlot[q]];
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

// FULL: every thread owns exactly JV vectors (the row has 512 * JV of them).  MAPPED: the rows go through a
// position map (decode mode), so some of them hold nothing to quantify.
template <typename T, int JV, int MINB, bool FULL, bool MAPPED>
__global__ void __launch_bounds__(kQThreads, MINB) quantify_stream_kernel(const __grid_constant__ QuantifyArgs a)
{
    typedef Vec<T> V;
    constexpr int VEC = Elem<T>::kVec;
    constexpr int NPV = V::kPairs;  // float2 pairs per 16-byte vector
    constexpr int NP = JV * NPV;    // pairs per thread
    constexpr int kStageBytes = kQThreads * JV * 16;
    extern __shared__ __align__(128) unsigned char smem[];
    QShared &sh = *reinterpret_cast<QShared *>(smem + (size_t)kQStages * kStageBytes);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    if (tid == 0) {
#pragma unroll
        for (int s = 0; s < kQStages; ++s) mbar_init(&sh.full[s], 1);
        sh.abort = 0;
        sh.nlist = 0;
        mbar_init_fence();
    }
    __syncthreads();

    const int nvec = a.n / VEC;
    int nj = JV;
    if (!FULL) {
        nj = (nvec - tid + kQThreads - 1) / kQThreads;
        nj = nj < 0 ? 0 : (nj > JV ? JV : nj);
    }
    const ciar_quantify_out &o = a.out;
    // (row indices, pointers and sizes are formed from the kernel arguments where they are used: nothing
    // that can be recomputed in an instruction or two is kept in a register across the sweeps)
    auto row_of = [&](int k) -> int64_t { return blockIdx.x + (int64_t)k * gridDim.x; };

    // issues the copy of this CTA's k-th row into its stage (thread 0 only)
    auto issue = [&](int k) {
        const int64_t lr = row_of(k);
        int64_t pr;
        if (lr < a.rows && map_row(a.rm, lr, pr)) {
            const int s = k % kQStages;
            const uint32_t row_bytes = (uint32_t)(a.n / VEC) * 16u;
            mbar_arrive_expect_tx(&sh.full[s], row_bytes);
            bulk_copy_g2s(smem + (size_t)s * kStageBytes, reinterpret_cast<const T *>(a.logits) + a.vb + pr * a.row_stride,
                          row_bytes, &sh.full[s]);
        }
    };
    // Every warp finishes one parked row.  A row whose list outgrew its slot first moves the slot's
    // part next to the rest, which waits in the shared buffer of the row's parity.
    auto finish_parked = [&](int count) {
        __syncthreads();
        if (warp < count) {
            Parked &p = sh.park[warp];
            const float *list = p.list;
            if (p.nlist > kParkList) {
                float *big = sh.list[p.par];
                for (int i = lane; i < kParkList; i += 32) big[i] = p.list[i];
                __syncwarp();
                list = big;
            }
            finish_row(a, p, list, lane);
        }
        __syncthreads();
    };
    if (tid == 0) {
#pragma unroll
        for (int s = 0; s < kQStages; ++s) issue(s);
    }

    uint32_t phases = 0;
    int filled = 0;
    int it = 0;  // rows swept so far: its low bits pick the slot of everything that is double-buffered by row
    bool aborted = false;

    const int nk = (int)((a.rows - blockIdx.x + gridDim.x - 1) / gridDim.x);  // rows this CTA walks (the grid never exceeds the rows)
    // The next row at or after `from` that has something to quantify (-1: none left).
    auto next_active = [&](int from) -> int {
        if (!MAPPED) return from < nk ? from : -1;
        for (int kk = from; kk < nk; ++kk) {
            int64_t pr;
            if (map_row(a.rm, row_of(kk), pr)) return kk;
        }
        return -1;
    };
    // Thread 0: the positions past the end of a sequence among rows [from, to) get their outputs, and each hands
    // its stage's turn to the row three further on.  Only called when the stages of those rows are free.
    auto retire_skipped = [&](int from, int to) {
        if (!MAPPED) return;
        for (int kk = from; kk < (to < 0 ? nk : to); ++kk) {
            const int64_t lr = row_of(kk);
            if (o.flag) o.flag[lr] = 0;
            if (o.row_status) o.row_status[lr] = 0;
            issue(kk + kQStages);
        }
    };
    // Waits for row kk to land and takes the maximum over it (sweep 1): each warp's maximum goes to the slot
    // of the row's turn, and only that is kept.  Thread 0 also clears the row's arg-max and maximum-count slots.
    auto first_sweep = [&](int kk, int turn) {
        const int s = kk % kQStages;
        const unsigned char *stage = smem + (size_t)s * kStageBytes;
        if (mbar_wait_bounded(&sh.full[s], (phases >> s) & 1u, kWaitCycles)) phases ^= 1u << s;
        else sh.abort = 1;
        typename V::Max mx = V::max_init();
#pragma unroll
        for (int j = 0; j < JV; ++j)
            if (FULL || j < nj) mx = V::fold_max(mx, stage_vec(stage, tid + j * kQThreads));
        const float wm = warp_redux_max(V::max_value(mx));
        if (lane == 0) sh.wmax[turn & 1][warp] = wm;
        if (tid == 0) {
            sh.argmin[turn & 1] = INT_MAX;
            sh.nmax[turn & 3] = 0;
        }
    };

    int k = next_active(0);
    if (tid == 0) retire_skipped(0, k);
    if (k >= 0) {
        first_sweep(k, 0);
        __syncwarp();
        named_bar_sync(kBarRow, kQThreads);
        if (sh.abort) aborted = true;
    }
    while (k >= 0 && !aborted) {
        const int s = k % kQStages;
        const int par = it & 1;
        const unsigned char *stage = smem + (size_t)s * kStageBytes;
        Parked &pk = sh.park[filled];
        if (tid == 0) {  // the row's place and stored radius: the others read the radius after the barrier
            const int64_t lr = row_of(k);
            int64_t pr;
            map_row(a.rm, lr, pr);
            pk.nlist = 0;
            pk.lr = lr;
            pk.pr = pr;
            pk.rho = a.radius_mode == CIAR_RADIUS_PER_ROW ? reinterpret_cast<const float *>(a.radius)[pr] : a.r_scalar;
        }
        const float m = warp_redux_max(sh.wmax[par][lane & (kQWarps - 1)]);
        // ---- sweep 1 of the row after this one, so that one barrier per row serves both
        // (a row three or more further on has not been asked for yet: its sweep waits until this row is done)
        const int kn = next_active(k + 1);
        const bool ahead = kn >= 0 && (!MAPPED || kn - k < kQStages);
        if (ahead) first_sweep(kn, it + 1);

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
                    V::pairs(stage_vec(stage, tid + j * kQThreads), c);
#pragma unroll
                    for (int q = 0; q < NPV; ++q) {
                        const float2 d = __ffma2_rn(c[q], L2, nm2);
                        const float2 ev = make_float2(ex2_once(d.x), ex2_once(d.y));  // a NaN logit poisons the sums on purpose
                        z2 = __fadd2_rn(z2, ev);
                        t2 = __ffma2_rn(ev, d, t2);  // 0 * -inf = NaN for a -inf logit: redone below
                        e[j * NPV + q] = ev;
                    }
                } else {
#pragma unroll
                    for (int q = 0; q < NPV; ++q) e[j * NPV + q] = f2(0.f);
                }
            }
        }
        float zs = z2.x + z2.y, ts = t2.x + t2.y;
        if (!(ts == ts)) {
            // A -inf logit (exponential 0, exponent -inf) or a real NaN: form this thread's entropy sum
            // again with the product of such a code taken as 0.  A real NaN still shows in the sum of exponentials.
            ts = 0.f;
            for (int j = 0; j < nj; ++j) {
                const T *v = reinterpret_cast<const T *>(stage + (size_t)(tid + j * kQThreads) * 16);
#pragma unroll
                for (int q = 0; q < VEC; ++q) {
                    const float d = fmaf(Elem<T>::widen(v[q]), kLog2e, -m2);
                    ts = fmaf(ex2_approx(d), fmaxf(d, kNegHuge), ts);
                }
            }
        }
        const float e0 = ex2_approx(fmaf(m, kLog2e, -m2));  // the exponential every maximum got
        if (sh.wmax[par][warp] == m) {
            // This warp owns a maximum.  A term near 1 would cost the small terms their low bits, so its threads
            // form their partial sums again without the terms equal to e0; they come back exactly, as a count.
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
            if (cnt > 0) {
                atomicAdd(&sh.nmax[it & 3], cnt);
                // the thread's lowest index holding the maximum competes for the arg-max
                int best = INT_MAX;
                for (int j = nj - 1; j >= 0; --j) {
                    const T *v = reinterpret_cast<const T *>(stage + (size_t)(tid + j * kQThreads) * 16);
#pragma unroll
                    for (int q = VEC - 1; q >= 0; --q)
                        if (Elem<T>::widen(v[q]) == m) best = (tid + j * kQThreads) * VEC + q;
                }
                if (best != INT_MAX) atomicMin(&sh.argmin[par], best);
            }
        }
        {
            const float zt = warp_sum_pair(zs, ts, lane);  // lanes 0..15: z, lanes 16..31: t
            if ((lane & 15) == 0) pk.wsum[warp][lane >> 2] = zt;
        }
        __syncwarp();
        named_bar_sync(kBarRow, kQThreads);
        if (sh.abort) {
            aborted = true;
            break;
        }
        float z = pk.wsum[lane & (kQWarps - 1)][0];
#pragma unroll
        for (int ofs = 8; ofs > 0; ofs >>= 1) z += __shfl_xor_sync(0xffffffffu, z, ofs);
        const int nmax = sh.nmax[it & 3];
        z = fmaf((float)nmax, e0, z);
        const float rho = pk.rho;

        int status = 0;
        if (!(m > -INFINITY) || !(z > 0.f) || !(z < INFINITY)) {
            // an unusable row (NaN / +inf logit, no finite logit): classify it from the landed bytes
            // exactly as the row-status bits are defined
            if (tid == 0) sh.bad_nan = sh.bad_finite = 0;
            named_bar_sync(kBarRow, kQThreads);
            int has_nan = 0, has_finite = 0;
            for (int j = 0; j < nj; ++j) {
                const T *v = reinterpret_cast<const T *>(stage + (size_t)(tid + j * kQThreads) * 16);
#pragma unroll
                for (int q = 0; q < VEC; ++q) {
                    const float c = Elem<T>::widen(v[q]);
                    if (!(c == c) || c == INFINITY) has_nan = 1;
                    if (c == c && fabsf(c) != INFINITY) has_finite = 1;
                }
            }
            if (has_nan) sh.bad_nan = 1;
            if (has_finite) sh.bad_finite = 1;
            named_bar_sync(kBarRow, kQThreads);
            if (sh.bad_nan) status |= CIAR_ROW_NAN;
            if (!sh.bad_finite) status |= CIAR_ROW_NO_FINITE;
            if (!status) status = CIAR_ROW_NAN;  // sums overflowed without any single bad logit
        }
        if (!(rho == rho)) status |= CIAR_ROW_NAN;
        const float r = row_radius(rho, a.radius_is_raw, a.r_max);
        const bool series = r <= 1.0f;
        const bool direct = !status && !series;
        const float c0 = z * rcp_approx((float)a.n), th = 0.00390625f * ex2_approx(-r * kLog2e) * z;  // clamp level: theta = 2^-8 e^-r
        if (tid == 0) {
            if (!direct) {  // every thread has read the stage: refill it
                fence_proxy_async_smem();
                issue(k + kQStages);
                retire_skipped(k + 1, kn);
            }
            // the row's scalars, parked as soon as they exist
            pk.m = m;
            pk.e0 = e0;
            pk.c0 = c0;
            pk.th = th;
            pk.r = r;
            pk.argmin = sh.argmin[par];
            pk.nmax = nmax;
            pk.status = status;
            pk.series = series;
            pk.par = par;
        }
        // ---- sweep 3: interval sums
        float r0 = 0.f, r1 = 0.f, r2 = 0.f;  // warp sums: r0, r1 hold two sums each (lanes 0..15 / 16..31)
        if (!status && series) {
            // Codes above th are listed and clamped to th.  Most warps hold none (seen from the warp's maximum
            // logit), and a vector holding none is skipped on one comparison of its maximum.
            // (th_log is a slightly low stand-in for log2(th), so the test on the warp's maximum errs on the safe side)
            const float th_log = __log2f(th) - 1e-3f;
            if (__builtin_expect(fmaf(sh.wmax[par][warp], kLog2e, -m2) > th_log, 0)) {  // warps whose maximum is below theta hold no such code
#pragma unroll
                for (int j = 0; j < JV; ++j) {
                    float2 g = e[j * NPV];
#pragma unroll
                    for (int q = 1; q < NPV; ++q) g = make_float2(fmaxf(g.x, e[j * NPV + q].x), fmaxf(g.y, e[j * NPV + q].y));
                    if (fmaxf(g.x, g.y) > th) {
#pragma unroll
                        for (int q = 0; q < 2 * NPV; ++q) {
                            float &ev = (q & 1) ? e[j * NPV + q / 2].y : e[j * NPV + q / 2].x;
                            if (ev > th) {
                                const int slot = atomicAdd(&pk.nlist, 1);
                                if (slot < kParkList) pk.list[slot] = ev;
                                else if (slot < kListCap) sh.list[par][slot] = ev;
                                ev = th;
                            }
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
            r0 = warp_sum_pair(T2.x + T2.y, T3.x + T3.y, lane);
            r1 = warp_sum_f(T4.x + T4.y);
        } else if (direct) {
            // both bounds of every code, from the row still sitting in its stage
            const DirectConst dc = make_direct_const(r, a.n);
            const float invz = 1.0f / z;
            float ps[5] = { 0.f, 0.f, 0.f, 0.f, 0.f };
#pragma unroll 1
            for (int j = 0; j < nj; ++j) {
                const T *v = reinterpret_cast<const T *>(stage + (size_t)(tid + j * kQThreads) * 16);
                float c[VEC];
                Elem<T>::load(v, c);
#pragma unroll
                for (int q = 0; q < VEC; ++q) {
                    const float ev = ex2_approx(fmaf(c[q], kLog2e, -m2));
                    const float x = ev * invz, sx = fmaf(-ev, invz, 1.0f);
                    const float den_l = fmaf(dc.b1, sx, dc.a1), den_u = fmaf(dc.b1, x, dc.a1);
                    const float xr = x * rcp_approx(den_l * den_u);
                    const float pl = fmaf(xr * den_u, dc.a1, -dc.pl0);  // p^l term minus its centre
                    const float dd = fmaf(xr, sx, -dc.dd0);             // width term minus its centre
                    ps[0] += pl;
                    ps[1] += dd;
                    ps[2] = fmaf(pl, pl, ps[2]);
                    ps[3] = fmaf(pl, dd, ps[3]);
                    ps[4] = fmaf(dd, dd, ps[4]);
                }
            }
            r0 = warp_sum_pair(ps[0], ps[1], lane);
            r1 = warp_sum_pair(ps[2], ps[3], lane);
            r2 = warp_sum_f(ps[4]);
            named_bar_sync(kBarRow, kQThreads);
            if (tid == 0) {
                fence_proxy_async_smem();
                issue(k + kQStages);
                retire_skipped(k + 1, kn);
            }
        }

        // ---- park the row's sums
        if ((lane & 15) == 0) {
            float *w = &pk.wsum[warp][lane >> 2];
            w[1] = r0;
            w[2] = r1;
            w[3] = r2;
        }
        // A row parked before this one may have listed more codes than its slot holds; the rest sits in the
        // shared buffer of its parity, which the row after this one reuses: finish the parked rows now.
        const bool long_pending = filled > 0 && sh.park[filled - 1].nlist > kParkList;
        if (++filled == kPark || long_pending) {
            finish_parked(filled);
            filled = 0;
        }
        k = kn;
        ++it;
        if (MAPPED && k >= 0 && !ahead) {  // the next row's first sweep could not run ahead: it runs here, with a barrier of its own
            first_sweep(k, it);
            __syncwarp();
            named_bar_sync(kBarRow, kQThreads);
            if (sh.abort) aborted = true;
        }
    }
    if (filled > 0) finish_parked(filled);

    if (aborted && tid == 0) {
        // A copy never arrived.  Mark this row and the rest of this CTA's rows, then give the
        // copies still in flight a last bounded chance to land before the CTA leaves.
        for (int k2 = k;; ++k2) {
            const int64_t lr = row_of(k2);
            if (lr >= a.rows) break;
            write_unusable(o, lr, CIAR_ROW_TIMEOUT);
        }
        for (int s = 0; s < kQStages; ++s) mbar_wait_bounded(&sh.full[s], (phases >> s) & 1u, kDrainCycles);
    }
}

template <typename T, int JV, int MINB, bool FULL, bool MAPPED>
cudaError_t launch_one(const QuantifyArgs &a, cudaStream_t stream)
{
    constexpr size_t smem = (size_t)kQStages * kQThreads * JV * 16 + sizeof(QShared);
    static bool configured[64] = {};
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!configured[dev]) {
        err = cudaFuncSetAttribute(quantify_stream_kernel<T, JV, MINB, FULL, MAPPED>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   (int)smem);
        if (err != cudaSuccess) return err;
        configured[dev] = true;
    }
    const int64_t cap = (int64_t)sm_count() * MINB;
    const unsigned grid = (unsigned)(a.rows < cap ? a.rows : cap);
    quantify_stream_kernel<T, JV, MINB, FULL, MAPPED><<<grid, kQThreads, smem, stream>>>(a);
    count_launch();
    return cudaGetLastError();
}

template <typename T, int JV, int MINB>
cudaError_t launch_jv(const QuantifyArgs &a, cudaStream_t stream)
{
    const int nvec = a.n / Elem<T>::kVec;
    const bool mapped = a.rm.pos != nullptr;
    if (nvec == kQThreads * JV) return mapped ? launch_one<T, JV, MINB, true, true>(a, stream) : launch_one<T, JV, MINB, true, false>(a, stream);
    return mapped ? launch_one<T, JV, MINB, false, true>(a, stream) : launch_one<T, JV, MINB, false, false>(a, stream);
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
