// Streaming verifier for rows that fit on chip (2048 .. 16384 codes) when the draft rows' softmax
// statistics come with the call.  Three launches, none of which waits for another CTA:
//   plan    one thread per window: the first flagged row and which rows the cloud tests; the tested
//           rows are written out as one compact list, so that the next kernel's CTAs get equal shares.
//   accept  persistent CTAs walk the list; target rows arrive through a ring of shared-memory
//           stages filled by bulk (TMA) copies; two sweeps (maximum, sum of exponentials); every 16
//           rows each warp finishes one row: the accept test on the drafted token, in double.
//   window  one CTA per window: accepted length, and for a rejected window the residual sample.
#include <climits>

#include "ciar_internal.h"
#include "online_stats.cuh"
#include "stream_common.cuh"
#include "verify_resample.cuh"

namespace ciar {

namespace {

constexpr int kVThreads = 512;
constexpr int kVWarps = kVThreads / 32;
constexpr int kVStages = 3;
constexpr int kVPark = 16;
constexpr int kPlanThreads = 128;
constexpr int kWinThreads = 512;  // threads that resample one rejected window
constexpr long long kWaitCycles = 2000000000ll;
constexpr long long kDrainCycles = 20000000ll;

__device__ __forceinline__ bool tested_row(int mode, int32_t j, int32_t f, int32_t wlen, const uint8_t *flag, int64_t lr)
{
    if (j >= wlen) return false;
    if (mode == CIAR_VERIFY_ALL) return true;
    if (mode == CIAR_VERIFY_ANCHORED) return j >= f;
    return flag[lr] != 0;
}

// ---- plan
// One thread per window.  A warp reserves room for its windows' tested rows with one atomic add on
// the list's counter (tested[rows], zeroed before the launch); the order of the list is not fixed
// from run to run, and nothing depends on it.
__global__ void __launch_bounds__(kPlanThreads) verify_plan_kernel(VerifyArgs a)
{
    const int lane = threadIdx.x & 31;
    const int64_t nw = a.rows / a.window;
    const int64_t w = (int64_t)blockIdx.x * kPlanThreads + threadIdx.x;
    uint8_t *accept_arr = a.out.accept ? a.out.accept : a.ws.accept;
    int cnt = 0;
    int32_t f = 0, wlen = 0;
    const int64_t row0 = w * a.window;
    if (w < nw) {
        wlen = window_len(a.rm, w);
        if (a.mode != CIAR_VERIFY_ALL) {
            f = wlen;
            for (int32_t j = wlen - 1; j >= 0; --j)  // independent loads, lowest flagged row wins
                if (a.flag[row0 + j]) f = j;
        }
        if (a.out.first_flag) a.out.first_flag[w] = f;
        if (a.out.cloud_call) a.out.cloud_call[w] = (uint8_t)(f < wlen);
        for (int32_t j = 0; j < a.window; ++j) {
            const int64_t lr = row0 + j;
            if (tested_row(a.mode, j, f, wlen, a.flag, lr)) {
                ++cnt;
            } else {  // rows the cloud does not test count as kept
                accept_arr[lr] = 1;
                if (a.out.p_draft_tok) a.out.p_draft_tok[lr] = 0.f;
                if (a.out.p_target_tok) a.out.p_target_tok[lr] = 0.f;
                if (a.out.row_status) a.out.row_status[lr] = 0;
            }
        }
    }
    int incl = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += up;
    }
    int base = 0;
    if (lane == 31 && incl > 0) base = atomicAdd(&a.ws.tested[a.rows], incl);
    base = __shfl_sync(0xffffffffu, base, 31);
    int pos = base + incl - cnt;
    if (w < nw)
        for (int32_t j = 0; j < a.window; ++j)
            if (tested_row(a.mode, j, f, wlen, a.flag, row0 + j)) a.ws.tested[pos++] = (int32_t)(row0 + j);
}

// ---- accept

// Softmax statistics and status bits of one row straight from global memory, by one warp (the
// slow way: only rows whose streamed statistics came out unusable take it).
template <typename T>
__device__ __noinline__ int warp_row_stats(const T *row, int32_t n, int lane, float &m_out, double &z_out)
{
    float m = -INFINITY;
    int has_nan = 0, has_finite = 0;
    for (int32_t i = lane; i < n; i += 32) {
        const float c = Elem<T>::widen(row[i]);
        if (!(c == c) || c == INFINITY) has_nan = 1;
        if (c == c && fabsf(c) != INFINITY) has_finite = 1;
        m = fmaxf(m, c);
    }
    m = warp_redux_max(m);
    has_nan = __any_sync(0xffffffffu, has_nan);
    has_finite = __any_sync(0xffffffffu, has_finite);
    int status = 0;
    if (has_nan) status |= CIAR_ROW_NAN;
    if (!has_finite) status |= CIAR_ROW_NO_FINITE;
    double z = 0.0;
    if (!status) {
        for (int32_t i = lane; i < n; i += 32) z += (double)ex2_approx((Elem<T>::widen(row[i]) - m) * kLog2e);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
    }
    m_out = m;
    z_out = z;
    return status;
}

struct VParked {
    float wz[kVWarps];  // per-warp sums of exp(t - m) (terms equal to e0 left out)
    int64_t lr;
    float m, e0;
    int nmax;
};

struct VShared {
    unsigned long long full[kVStages];
    float wmax[2][kVWarps];  // by row parity
    int nmax[4], abort;       // count of maxima, by row index mod 4
    VParked park[kVPark];
};

// The accept test of one tested row from the two rows' softmax statistics, by one thread: u * p_x < q_x in double, p and q
// the draft's and the target's probability of the drafted token.  status: what is already known to be wrong with the row.
template <typename T>
__device__ __forceinline__ void accept_decide(const VerifyArgs &a, int64_t lr, int64_t pr, float mq, double zq, float mp, double zp,
                                              int status)
{
    const T *drow = reinterpret_cast<const T *>(a.draft) + pr * a.row_stride + a.vb;
    const T *trow = reinterpret_cast<const T *>(a.target) + pr * a.row_stride + a.vb;
    const int32_t x = a.tokens[pr];
    const bool bad_token = (x < 0 || x >= a.vocab);
    if (bad_token) status |= CIAR_ROW_BAD_TOKEN;
    int acc = 0;
    float px_out = __int_as_float(0x7fc00000), qx_out = px_out;
    if (!(status & (CIAR_ROW_NAN | CIAR_ROW_NO_FINITE))) {
        double px = 0.0, qx = 0.0;
        if (x >= a.vb && x < a.vb + a.n) {  // a code outside the valid slice has probability 0
            const double cx = (double)Elem<T>::widen(drow[x - a.vb]);
            const double tx = (double)Elem<T>::widen(trow[x - a.vb]);
            px = exp(cx - (double)mp) / zp;
            qx = exp(tx - (double)mq) / zq;
        }
        acc = (!bad_token && (double)a.u_accept[pr] * px < qx) ? 1 : 0;
        if (!bad_token) {
            px_out = (float)px;
            qx_out = (float)qx;
        }
        a.ws.tq_max[lr] = mq;
        a.ws.tq_sum[lr] = (float)zq;
    } else {
        a.ws.tq_max[lr] = mq;
        a.ws.tq_sum[lr] = __int_as_float(0x7fc00000);  // tells the window kernel that there is nothing to resample from
    }
    uint8_t *accept_arr = a.out.accept ? a.out.accept : a.ws.accept;
    accept_arr[lr] = (uint8_t)acc;
    if (a.out.p_draft_tok) a.out.p_draft_tok[lr] = px_out;
    if (a.out.p_target_tok) a.out.p_target_tok[lr] = qx_out;
    if (a.out.row_status) a.out.row_status[lr] = (uint8_t)status;
}

// The accept test of one tested row whose target statistics are parked, by one warp.
template <typename T>
__device__ __noinline__ void accept_row(const VerifyArgs &a, const VParked &pk, int lane)
{
    const int64_t lr = pk.lr;
    int64_t pr;
    map_row(a.rm, lr, pr);
    const T *drow = reinterpret_cast<const T *>(a.draft) + pr * a.row_stride + a.vb;
    const T *trow = reinterpret_cast<const T *>(a.target) + pr * a.row_stride + a.vb;
    // target statistics from the sweeps
    double zq = lane < kVWarps ? (double)pk.wz[lane] : 0.0;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) zq += __shfl_xor_sync(0xffffffffu, zq, o);
    zq += (double)pk.nmax * (double)pk.e0;
    float mq = pk.m;
    // the exponent used was c * log2e_f - fl(m * log2e_f): take the common offset out again
    const double off = (double)mq * (double)kLog2e - (double)(mq * kLog2e);
    zq *= exp2(-off);
    int status = 0;
    if (!(mq > -INFINITY) || !(zq > 0.0) || !(zq < INFINITY)) status |= warp_row_stats(trow, a.n, lane, mq, zq);
    // draft statistics from the quantifier; unusable ones are recomputed to learn what is wrong with the row
    float mp = a.draft_row_max[lr];
    double zp = (double)a.draft_sum_exp[lr];
    if (!(zp > 0.0) || !(zp < INFINITY) || !(mp == mp)) status |= warp_row_stats(drow, a.n, lane, mp, zp);
    if (lane != 0) return;
    accept_decide<T>(a, lr, pr, mq, zq, mp, zp, status);
}

// ---- accept, rows that fit a shared-memory stage.  One persistent CTA per SM walks its share of the list; its warps
// have three roles that meet on mbarriers only: a producer thread that copies each target row into the next free stage
// with one bulk (TMA) copy, several rows ahead; 16 sweep warps, in groups of WPR warps that share a row (the groups take
// alternate rows), each warp summing exp(t - its own share's maximum) over its share; and a few finishing warps that bring
// the warps' sums to the row maximum, join them, hand the stage back and file the row; every 32 rows a finishing warp does
// the accept tests of its batch, a row per lane (the drafted token's two logits come from global memory).
constexpr int kACW = 16;     // sweep warps
constexpr int kAJV = 8;      // 16-byte vectors of a row one lane owns (at most)
constexpr int kAFin = 3;     // finishing warps
constexpr int kABatch = 32;  // rows per batch of accept tests
constexpr int kAMaxStages = 16;
constexpr int kASmem = 227 * 1024;

template <int WPR>
struct ASlot {
    unsigned long long full, swept, empty;  // the row has landed / every warp has published its sum / the stage may be refilled
    int64_t lr;                             // logical row (-1: nothing to do)
    float wmax[WPR], wz[WPR];               // per warp: maximum of its share, sum of exp(t - that maximum)
};

struct ABatch {
    int64_t lr[kABatch];
    float m[kABatch], z[kABatch];  // row maximum, sum of exp(t - m) as computed (offset of the exponent still in it)
};

template <int S, int WPR>
struct AControl {
    ASlot<WPR> slot[S];
    int abort, issued;
    int fin_next[kAFin];
    ABatch batch[kAFin];
};

// (a whole number of rounds of the groups, so that a group meets each stage's uses in order: a warp must never wait for
// a phase of a barrier before it has seen the phase before it)
__host__ __device__ constexpr int accept_stages(int stage_bytes, int groups)
{
    int s = (kASmem - 4096) / (stage_bytes + 256);
    s = s > kAMaxStages ? kAMaxStages : s;
    return s - s % groups;
}

// The accept tests of a batch, a row per lane; rows whose statistics came out unusable are then redone one by one by the
// whole warp, which learns from the rows themselves what is wrong with them.
template <typename T>
__device__ __noinline__ void accept_batch(const VerifyArgs &a, const ABatch &bt, int count, int lane)
{
    int64_t lr = 0, pr = 0;
    bool slow = false;
    if (lane < count) {
        lr = bt.lr[lane];
        map_row(a.rm, lr, pr);
        float mq = bt.m[lane];
        // the exponent used was c * log2e_f - fl(m * log2e_f): take the common offset out again
        const double off = (double)mq * (double)kLog2e - (double)(mq * kLog2e);
        const double w2 = -off * kLn2D;
        const double zq = (double)bt.z[lane] * (1.0 + w2 * (1.0 + 0.5 * w2));  // 2^-off, |off| far below 1e-4
        const float mp = a.draft_row_max[lr];
        const double zp = (double)a.draft_sum_exp[lr];
        slow = !(mq > -INFINITY) || !(mq < INFINITY) || !(zq > 0.0) || !(zq < (double)INFINITY) || !(zp > 0.0) ||
               !(zp < (double)INFINITY) || !(mp == mp);
        if (!slow) accept_decide<T>(a, lr, pr, mq, zq, mp, zp, 0);
    }
    for (unsigned todo = __ballot_sync(0xffffffffu, slow); todo != 0; todo &= todo - 1) {
        const int h = __ffs((int)todo) - 1;
        const int64_t lr_h = __shfl_sync(0xffffffffu, lr, h), pr_h = __shfl_sync(0xffffffffu, pr, h);
        const T *drow = reinterpret_cast<const T *>(a.draft) + pr_h * a.row_stride + a.vb;
        const T *trow = reinterpret_cast<const T *>(a.target) + pr_h * a.row_stride + a.vb;
        float mq, mp = a.draft_row_max[lr_h];
        double zq, zp = (double)a.draft_sum_exp[lr_h];
        int status = warp_row_stats(trow, a.n, lane, mq, zq);
        if (!(zp > 0.0) || !(zp < (double)INFINITY) || !(mp == mp)) status |= warp_row_stats(drow, a.n, lane, mp, zp);
        if (lane == 0) accept_decide<T>(a, lr_h, pr_h, mq, zq, mp, zp, status);
    }
}

// WPR: sweep warps that share a row (a row has up to WPR * 32 * 8 vectors of 16 bytes).  FULL: exactly that many.
template <typename T, int WPR, bool FULL>
__global__ void __launch_bounds__((kACW + kAFin + 1) * 32, 1) verify_accept_kernel(const __grid_constant__ VerifyArgs a)
{
    typedef Vec<T> V;
    constexpr int VEC = Elem<T>::kVec;
    constexpr int NPV = V::kPairs;
    constexpr int GROUPS = kACW / WPR;
    constexpr int ROWL = WPR * 32;
    constexpr int SB = ROWL * kAJV * 16;
    constexpr int S = accept_stages(SB, GROUPS);
    typedef AControl<S, WPR> Ctl;
    static_assert(S >= 3 && S % GROUPS == 0 && (size_t)S * SB + sizeof(Ctl) <= (size_t)kASmem, "the ring and its slots must fit in shared memory");
    extern __shared__ __align__(128) unsigned char smem[];
    Ctl &sh = *reinterpret_cast<Ctl *>(smem + (size_t)S * SB);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int total = a.ws.tested[a.rows];  // written by the plan kernel
    const int stride = gridDim.x;
    const int nk = blockIdx.x < total ? (total - 1 - (int)blockIdx.x) / stride + 1 : 0;  // rows this CTA walks
    const long long limit = kWaitCycles;

    if (tid == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(&sh.slot[s].full, 1);
            mbar_init(&sh.slot[s].swept, WPR);
            mbar_init(&sh.slot[s].empty, 1);
        }
        sh.abort = 0;
        sh.issued = 0;
        for (int f = 0; f < kAFin; ++f) sh.fin_next[f] = f;
        mbar_init_fence();
    }
    __syncthreads();

    if (warp > kAFin) {
        // ---- a sweep warp: the maximum of its share, then the sum of exponentials about it
        const int cw = warp - kAFin - 1, g = cw / WPR, w = cw % WPR;
        const int v0 = w * 32 + lane;
        int nj = kAJV;
        if (!FULL) {
            nj = (a.n / VEC - v0 + ROWL - 1) / ROWL;
            nj = nj < 0 ? 0 : (nj > kAJV ? kAJV : nj);
        }
        for (int k = g; k < nk; k += GROUPS) {
            const int s = k % S;
            ASlot<WPR> &sl = sh.slot[s];
            const unsigned char *stage = smem + (size_t)s * SB;
            if (!wait_phase(&sl.full, (uint32_t)(k / S) & 1u, &sh.abort, limit)) break;
            typename V::Max mx = V::max_init();
#pragma unroll
            for (int j = 0; j < kAJV; ++j)
                if (FULL || j < nj) mx = V::fold_max(mx, stage_vec(stage, v0 + j * ROWL));
            const float mw = warp_redux_max(V::max_value(mx));
            float2 z2 = f2(0.f);
            if (mw > -INFINITY && mw < INFINITY) {
                const float2 L2 = f2(kLog2e), nm2 = f2(-(mw * kLog2e));
#pragma unroll
                for (int j = 0; j < kAJV; ++j) {
                    if (FULL || j < nj) {
                        float2 c[NPV];
                        V::pairs(stage_vec(stage, v0 + j * ROWL), c);
#pragma unroll
                        for (int q = 0; q < NPV; ++q) {
                            const float2 d = __ffma2_rn(c[q], L2, nm2);
                            z2 = __fadd2_rn(z2, make_float2(ex2_approx(d.x), ex2_approx(d.y)));  // a NaN logit poisons the sum on purpose
                        }
                    }
                }
            }
            const float wz = warp_sum_f(z2.x + z2.y);
            if (lane == 0) {
                sl.wmax[w] = mw;
                sl.wz[w] = wz;
                mbar_arrive(&sl.swept);
            }
        }
    } else if (warp < kAFin) {
        // ---- a finishing warp: joins the warps' sums, hands the stage back, files the row; accept tests by the batch
        ABatch &bt = sh.batch[warp];
        // (stage s is always served by finishing warp s % kAFin, in the order of the walk: a warp never waits for a
        // phase of a barrier before it has seen the phase before it)
        int filled = 0, k = 0;
        for (; k < nk; ++k) {
            const int s = k % S;
            if (s % kAFin != warp) continue;
            ASlot<WPR> &sl = sh.slot[s];
            if (!wait_phase(&sl.swept, (uint32_t)(k / S) & 1u, &sh.abort, limit)) break;
            const float wm = sl.wmax[lane % WPR];
            const float m = warp_redux_max(wm);
            // a share without a finite code adds nothing; a +inf or NaN anywhere makes the sum unusable, as it must be
            float x = 0.f;
            if (lane < WPR && wm > -INFINITY) x = ex2_approx(wm * kLog2e - m * kLog2e) * sl.wz[lane];
#pragma unroll
            for (int o = WPR / 2; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
            if (lane == 0) {
                bt.lr[filled] = sl.lr;
                bt.m[filled] = m;
                bt.z[filled] = x;
                mbar_arrive(&sl.empty);
            }
            if (++filled == kABatch) {
                __syncwarp();
                accept_batch<T>(a, bt, filled, lane);
                __syncwarp();
                filled = 0;
            }
        }
        __syncwarp();
        if (filled > 0) accept_batch<T>(a, bt, filled, lane);
        if (lane == 0) sh.fin_next[warp] = k;
    } else if (lane == 0) {
        // ---- the producer
        const uint32_t row_bytes = (uint32_t)(a.n / VEC) * 16u;
        const T *tbase = reinterpret_cast<const T *>(a.target) + a.vb;
        int64_t lr_n = nk > 0 ? a.ws.tested[blockIdx.x] : -1, pr_n = 0;
        if (nk > 0) map_row(a.rm, lr_n, pr_n);
        for (int k = 0; k < nk; ++k) {
            const int s = k % S;
            ASlot<WPR> &sl = sh.slot[s];
            const int64_t lr = lr_n, pr = pr_n;
            if (k + 1 < nk) {  // the next row's place, fetched early
                lr_n = a.ws.tested[blockIdx.x + (k + 1) * stride];
                map_row(a.rm, lr_n, pr_n);
            }
            if (k >= S && !wait_phase(&sl.empty, (uint32_t)(k / S - 1) & 1u, &sh.abort, limit)) break;
            sl.lr = lr;
            fence_proxy_async_smem();
            mbar_arrive_expect_tx(&sl.full, row_bytes);
            bulk_copy_g2s(smem + (size_t)s * SB, tbase + pr * a.row_stride, row_bytes, &sl.full);
            sh.issued = k + 1;
        }
    }
    __syncthreads();

    if (sh.abort && tid == 0) {
        // A copy never arrived: the rows this CTA still owed are marked, and the copies in flight get a last bounded
        // chance to land before the CTA leaves.
        uint8_t *accept_arr = a.out.accept ? a.out.accept : a.ws.accept;
        int kmin = nk;
        for (int f = 0; f < kAFin; ++f) kmin = min(kmin, sh.fin_next[f]);
        for (int k = kmin; k < nk; ++k) {
            const int64_t lr = a.ws.tested[blockIdx.x + k * stride];
            accept_arr[lr] = 0;
            a.ws.tq_sum[lr] = __int_as_float(0x7fc00000);
            if (a.out.row_status) a.out.row_status[lr] = CIAR_ROW_TIMEOUT;
        }
        const int issued = sh.issued;
        for (int k = max(0, issued - S); k < issued; ++k)
            mbar_wait_bounded(&sh.slot[k % S].full, (uint32_t)(k / S) & 1u, kDrainCycles);
    }
}

// ---- accept, rows wider than the on-chip sweep takes: one pass over a row, 32 KB at a time ("chunks") through
// the same ring, the statistics kept on line by every warp and joined once per row.
constexpr int kVWJ = 4;
constexpr int kVChunkVecs = kVThreads * kVWJ;
constexpr int kVChunkBytes = kVChunkVecs * 16;

struct VWShared {
    unsigned long long full[kVStages];
    float wm[kVWarps];  // per warp: running maximum, sum relative to it, number of codes equal to it
    double wz[kVWarps];
    int wcnt[kVWarps];
    int abort;
    VParked park[kVPark];
};

template <typename T>
__global__ void __launch_bounds__(kVThreads, 2) verify_accept_wide_kernel(const __grid_constant__ VerifyArgs a)
{
    constexpr int VEC = Elem<T>::kVec;
    extern __shared__ __align__(128) unsigned char smem[];
    VWShared &sh = *reinterpret_cast<VWShared *>(smem + (size_t)kVStages * kVChunkBytes);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) {
#pragma unroll
        for (int s = 0; s < kVStages; ++s) mbar_init(&sh.full[s], 1);
        sh.abort = 0;
        mbar_init_fence();
    }
    __syncthreads();
    const int nvec = a.n / VEC;
    const int nch = (nvec + kVChunkVecs - 1) / kVChunkVecs;
    const T *tbase = reinterpret_cast<const T *>(a.target) + a.vb;
    const int total = a.ws.tested[a.rows];  // written by the plan kernel
    const int stride = gridDim.x;
    const int mine = blockIdx.x < total ? (total - 1 - (int)blockIdx.x) / stride + 1 : 0;  // rows this CTA walks

    // thread 0: asks for chunk c of this CTA's kr-th row, the g-th chunk of its walk, into stage g mod 3
    auto issue = [&](int kr, int c, int g) {
        if (kr >= mine) return;
        int64_t pr;
        map_row(a.rm, a.ws.tested[blockIdx.x + kr * stride], pr);
        const int v0 = c * kVChunkVecs;
        const uint32_t bytes = (uint32_t)min(kVChunkVecs, nvec - v0) * 16u;
        const int s = g % kVStages;
        mbar_arrive_expect_tx(&sh.full[s], bytes);
        bulk_copy_g2s(smem + (size_t)s * kVChunkBytes, tbase + pr * a.row_stride + (int64_t)v0 * VEC, bytes, &sh.full[s]);
    };
    auto finish_parked = [&](int count) {
        __syncthreads();
        if (warp < count) accept_row<T>(a, sh.park[warp], lane);
        __syncthreads();
    };
    int pr_k = 0, pr_c = 0;  // the chunk to ask for next, three ahead of the sweep
    auto advance = [&]() {
        if (++pr_c == nch) {
            pr_c = 0;
            ++pr_k;
        }
    };
#pragma unroll 1
    for (int i = 0; i < kVStages; ++i) {
        if (tid == 0) issue(pr_k, pr_c, i);
        advance();
    }
    int k = 0, g = 0, filled = 0;
    bool aborted = false;
    for (; k < mine; ++k) {
        OnlineStats st;
        st.reset();
#pragma unroll 1
        for (int c = 0; c < nch; ++c) {
            const int s = g % kVStages;
            const unsigned char *stage = smem + (size_t)s * kVChunkBytes;
            const int v0 = c * kVChunkVecs;
            // once a copy has failed to arrive nothing is waited for any more; the CTA leaves after this row's barrier
            if (!sh.abort && !mbar_wait_bounded(&sh.full[s], (uint32_t)(g / kVStages) & 1u, kWaitCycles)) sh.abort = 1;
            if (nvec - v0 >= kVChunkVecs) {
                online_sweep<T, kVThreads, kVWJ, true, false>(st, stage, tid, kVWJ, c);
            } else {
                int nj = (nvec - v0 - tid + kVThreads - 1) / kVThreads;
                nj = nj < 0 ? 0 : nj;
                online_sweep<T, kVThreads, kVWJ, false, false>(st, stage, tid, nj, c);
            }
            __syncwarp();
            __syncthreads();  // every thread has read the stage
            if (tid == 0 && !sh.abort) {
                fence_proxy_async_smem();
                issue(pr_k, pr_c, g + kVStages);
            }
            advance();
            ++g;
        }
        {
            double zw, tw;
            int cw;
            online_warp_totals(st, zw, tw, cw);
            if (lane == 0) {
                sh.wm[warp] = st.m_w;
                sh.wz[warp] = zw;
                sh.wcnt[warp] = cw;
            }
        }
        __syncthreads();  // the warps' shares are out
        if (sh.abort) {
            aborted = true;
            break;
        }
        if (warp == 0) {
            // Park the row in the form the finishing routine reads: the sum as a float pair (high part in warp
            // 0's place, the remainder in warp 1's, zeros in the others), so that its double sum is the sum.
            float m;
            double zc, tc;
            int nc;
            online_join<kVWarps>(sh.wm, sh.wz, nullptr, sh.wcnt, lane, m, zc, tc, nc);
            VParked &pk = sh.park[filled];
            const float hi = (float)zc;
            if (lane < kVWarps) pk.wz[lane] = lane == 0 ? hi : (lane == 1 ? (float)(zc - (double)hi) : 0.f);
            if (lane == 0) {
                pk.lr = a.ws.tested[blockIdx.x + k * stride];
                pk.m = m;
                pk.e0 = ex2_approx(fmaf(m, kLog2e, -(m * kLog2e)));
                pk.nmax = nc;
            }
        }
        if (++filled == kVPark) {
            finish_parked(filled);
            filled = 0;
        }
    }
    if (filled > 0) finish_parked(filled);
    if (aborted && tid == 0) {
        // A copy never arrived: the rows this CTA still owed are marked, and the copies in flight
        // get a last bounded chance to land before the CTA leaves.
        uint8_t *accept_arr = a.out.accept ? a.out.accept : a.ws.accept;
        for (int k2 = k; k2 < mine; ++k2) {
            const int64_t lr = a.ws.tested[blockIdx.x + k2 * stride];
            accept_arr[lr] = 0;
            a.ws.tq_sum[lr] = __int_as_float(0x7fc00000);
            if (a.out.row_status) a.out.row_status[lr] = CIAR_ROW_TIMEOUT;
        }
        for (int i = 0; i < kVStages; ++i)
            mbar_wait_bounded(&sh.full[(g + i) % kVStages], (uint32_t)((g + i) / kVStages) & 1u, kDrainCycles);
    }
}

// ---- window: accepted length and, for a rejected window, the residual sample of its first rejected row
template <typename T>
__global__ void __launch_bounds__(kWinThreads) verify_window_kernel(VerifyArgs a)
{
    __shared__ double scan_warp[kWinThreads / 32];
    __shared__ int sh_i[2];
    __shared__ int sh_a;
    __shared__ float sh_f[5];  // of the first rejected row: target max / sum, draft max / sum, the uniform of its resampling
    const T *dbase = reinterpret_cast<const T *>(a.draft);
    const T *tbase = reinterpret_cast<const T *>(a.target);
    const uint8_t *accept_arr = a.out.accept ? a.out.accept : a.ws.accept;
    const int64_t nw = a.rows / a.window;
    for (int64_t w = blockIdx.x; w < nw; w += gridDim.x) {
        const int32_t wlen = window_len(a.rm, w);
        const int64_t row0 = w * a.window;
        if (threadIdx.x < 32) {
            // The first warp scans the window, a row per lane.  Every load a lane may need goes out at once: its row's flag
            // and accept bit, and the statistics and the uniform the resampling would use if this row is the first rejected.
            const int lane = threadIdx.x;
            int32_t f = 0, acc_len = wlen;
            if (a.mode != CIAR_VERIFY_ALL) f = wlen;
            for (int32_t base = 0; base < wlen; base += 32) {
                const int32_t j = base + lane;
                const bool in = j < wlen;
                const int64_t lr = row0 + j;
                const uint8_t fl = in && a.flag ? a.flag[lr] : 0, ac = in ? accept_arr[lr] : 1;
                float s_mq = 0.f, s_zq = 0.f, s_mp = 0.f, s_zp = 0.f, s_u = 0.f;
                if (in) {
                    int64_t pr;
                    map_row(a.rm, lr, pr);
                    s_mq = a.ws.tq_max[lr];
                    s_zq = a.ws.tq_sum[lr];
                    s_mp = a.draft_row_max[lr];
                    s_zp = a.draft_sum_exp[lr];
                    s_u = a.u_resample[pr];
                }
                if (a.mode != CIAR_VERIFY_ALL && f == wlen) {
                    const unsigned mk = __ballot_sync(0xffffffffu, in && fl != 0);
                    if (mk) f = base + __ffs((int)mk) - 1;
                }
                bool tested = in;
                if (a.mode == CIAR_VERIFY_ANCHORED) tested = in && j >= f;
                else if (a.mode == CIAR_VERIFY_PER_TOKEN) tested = in && fl != 0;
                const unsigned rej = __ballot_sync(0xffffffffu, tested && ac == 0);
                if (rej && acc_len == wlen) {
                    const int src = __ffs((int)rej) - 1;
                    acc_len = base + src;
                    if (lane == src) {
                        sh_f[0] = s_mq;
                        sh_f[1] = s_zq;
                        sh_f[2] = s_mp;
                        sh_f[3] = s_zp;
                        sh_f[4] = s_u;
                    }
                }
            }
            if (lane == 0) {
                sh_a = acc_len;
                if (a.out.accepted_len) a.out.accepted_len[w] = acc_len;
            }
        }
        __syncthreads();
        const int32_t acc_len = sh_a;
        int32_t tok = -1;
        if (acc_len < wlen) {
            const int64_t lr = row0 + acc_len;
            int64_t pr;
            map_row(a.rm, lr, pr);
            const float mq = sh_f[0], mp = sh_f[2];
            const double zq = (double)sh_f[1], zp = (double)sh_f[3];
            // unusable logits on either side (their statistics are NaN): nothing to resample from
            if (zq > 0.0 && zq < INFINITY && zp > 0.0 && zp < INFINITY && mp == mp) {
                const RowView<T> rd(dbase + pr * a.row_stride, a.vb, a.n);
                const RowView<T> rt(tbase + pr * a.row_stride, a.vb, a.n);
                tok = resample_row<T, kWinThreads>(rd, rt, mp, zp, mq, zq, sh_f[4], a.vb, scan_warp, sh_i);
            }
        }
        if (threadIdx.x == 0) {
            if (a.out.resampled_token) a.out.resampled_token[w] = tok;
            a.ws.candidate[row0] = tok;  // kept for the decode step, which reads its result here
        }
        __syncthreads();
    }
}

template <typename T, int WPR, bool FULL>
cudaError_t launch_accept_one(const VerifyArgs &a, cudaStream_t stream)
{
    constexpr int SB = WPR * 32 * kAJV * 16;
    constexpr int S = accept_stages(SB, kACW / WPR);
    constexpr size_t smem = (size_t)S * SB + sizeof(AControl<S, WPR>);
    static bool configured[64] = {};
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!configured[dev]) {
        err = cudaFuncSetAttribute(verify_accept_kernel<T, WPR, FULL>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (err != cudaSuccess) return err;
        configured[dev] = true;
    }
    const int64_t cap = sm_count();
    const unsigned grid = (unsigned)(a.rows < cap ? a.rows : cap);
    verify_accept_kernel<T, WPR, FULL><<<grid, (kACW + kAFin + 1) * 32, smem, stream>>>(a);
    count_launch();
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_accept(const VerifyArgs &a, cudaStream_t stream)
{
    const int nvec = a.n / Elem<T>::kVec;
    const int per_warp = 32 * kAJV;  // vectors one warp takes
    if (nvec <= 2 * per_warp) return nvec == 2 * per_warp ? launch_accept_one<T, 2, true>(a, stream) : launch_accept_one<T, 2, false>(a, stream);
    if (nvec <= 4 * per_warp) return nvec == 4 * per_warp ? launch_accept_one<T, 4, true>(a, stream) : launch_accept_one<T, 4, false>(a, stream);
    if (nvec <= 8 * per_warp) return nvec == 8 * per_warp ? launch_accept_one<T, 8, true>(a, stream) : launch_accept_one<T, 8, false>(a, stream);
    return nvec == 16 * per_warp ? launch_accept_one<T, 16, true>(a, stream) : launch_accept_one<T, 16, false>(a, stream);
}

template <typename T>
cudaError_t launch_accept_wide(const VerifyArgs &a, cudaStream_t stream)
{
    constexpr size_t smem = (size_t)kVStages * kVChunkBytes + sizeof(VWShared);
    static bool configured[64] = {};
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!configured[dev]) {
        err = cudaFuncSetAttribute(verify_accept_wide_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (err != cudaSuccess) return err;
        configured[dev] = true;
    }
    const int64_t cap = (int64_t)sm_count() * 2;
    const unsigned grid = (unsigned)(a.rows < cap ? a.rows : cap);
    verify_accept_wide_kernel<T><<<grid, kVThreads, smem, stream>>>(a);
    count_launch();
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_all(const VerifyArgs &a, cudaStream_t stream)
{
    cudaError_t err = cudaMemsetAsync(a.ws.tested + a.rows, 0, sizeof(int32_t), stream);
    if (err != cudaSuccess) return err;
    const int64_t nwin = a.rows / a.window;
    verify_plan_kernel<<<(unsigned)((nwin + kPlanThreads - 1) / kPlanThreads), kPlanThreads, 0, stream>>>(a);
    count_launch();
    err = cudaGetLastError();
    if (err != cudaSuccess) return err;
    err = a.n > 16384 ? launch_accept_wide<T>(a, stream) : launch_accept<T>(a, stream);
    if (err != cudaSuccess) return err;
    const int64_t nw = a.rows / a.window;
    const int64_t cap = (int64_t)sm_count() * 4;
    const unsigned grid = (unsigned)(nw < cap ? nw : cap);
    verify_window_kernel<T><<<grid, kWinThreads, 0, stream>>>(a);
    count_launch();
    return cudaGetLastError();
}

}  // namespace

bool verify_stream_eligible(const VerifyArgs &a, int dtype)
{
    const int vec = dtype == CIAR_F32 ? 4 : 8;
    if (!a.draft_row_max || !a.draft_sum_exp) return false;
    if (a.vb % vec != 0 || a.n % vec != 0) return false;
    if (a.rows >= INT_MAX) return false;
    return a.n >= 2048 && a.n <= (1 << 28);
}

cudaError_t launch_verify_stream(const VerifyArgs &a, int dtype, cudaStream_t stream)
{
    if (a.rows == 0) return cudaSuccess;
    return dtype == CIAR_F32 ? launch_all<float>(a, stream) : launch_all<__nv_bfloat16>(a, stream);
}

}  // namespace ciar
