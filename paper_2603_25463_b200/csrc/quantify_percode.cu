// Streaming quantifier for rows with one interval radius per code (the form in which the interval head emits it):
// a row's logits AND its radii arrive together through a ring of shared-memory stages filled by bulk (TMA) copies,
// so both tensors are read from HBM exactly once.
//
// One persistent CTA per SM walks rows blockIdx.x, blockIdx.x + gridDim.x, ...  Its 32 warps form two groups of 16
// that take these rows in turn, each group with its own named barrier and scratch, so that while one group stands
// at a barrier or in a reduction the other keeps the pipes busy.  A group sweeps its landed row three times from
// shared memory: the maximum; one exponential per code with the softmax and entropy sums; then both InterFuse
// bounds of every code from its own radius (the exponential formed again: nothing per code is kept in registers),
// with the five sums Omega and Sigma are built from.  The second and third sweep end in a group barrier that
// publishes the per-warp sums (the first sweep of a row runs before the last barrier of the group's row before it);
// every thread of the group then holds the row's totals in float.  A row whose widths are nearly uniform gets a
// fourth sweep that sums (delta - mu)^2 directly (the moment form would cancel).  The sweeps leave their per-warp
// sums in the row's parking slot; every 16 rows each warp of the group joins one parked row's sums in double and
// finishes it (logarithm, square root, flag, stores).  The thread that ends a row's last sweep issues the copies of
// the row three further on.
#include <type_traits>

#include "quantify_finish.cuh"

namespace ciar {

namespace {

constexpr int kPcThreads = 1024;
constexpr int kPcGroups = 2;
constexpr int kPcGT = kPcThreads / kPcGroups;  // threads of a group
constexpr int kPcGW = kPcGT / 32;              // warps of a group; as many rows are parked before they are finished
constexpr int kPcStages = 3;
constexpr int kPcJV = 4;            // 16-byte vectors of a row per thread, at most
constexpr int kPcRowBytes = 32768;  // widest row of one tensor a stage takes (16384 bf16 / 8192 fp32 codes)
constexpr int kBarPc = 1;           // named barriers kBarPc + group
constexpr int kPcListCap = 1024;    // rows a CTA may walk when the rows go through a position map (decode mode)

// A row's totals in double: the softmax sums as computed (relative to m2 = fl(m * log2e)) and the five interval sums.
struct PcTotals {
    double z_raw, t_raw, A, B, AA, AB, BB;
};

// A row whose sweeps are done: the per-warp sums as the sweeps left them (joined in double when the row is finished)
// and the row's scalars.
struct PcParked {
    float zs[kPcGW], ts[kPcGW];  // sum of exponentials (maximum codes left out), entropy sum
    float sums[5][kPcGW];        // d, p^l, d^2, d p^l, p^l^2 (a dominant code's p^l terms less 1)
    float dev[kPcGW];            // sum of (delta - mu)^2 from the fourth sweep, when low_cv
    long long lr;
    float m;
    int first, nmax, dominant, low_cv;
};

// Scratch of one group.
struct PcGroup {
    PcParked park[kPcGW];
    float wmax[2][kPcGW];  // by the row's turn: a row's maxima are written while the row before it is still in use
    int cnt, first;  // codes counted as the row maximum, and the lowest code equal to it
    int abort;       // a wait of this group ran out (set before the group's barrier, read after it: uniform)
};

struct PcShared {
    unsigned long long full[kPcStages];
    PcGroup grp[kPcGroups];
    // decode mode: which of this CTA's rows (as multiples of the grid) hold something to quantify
    int nlist;
    int list[kPcListCap];
};

// Sum over the 16 per-warp values of a group (every lane gets it).
__device__ __forceinline__ float group_sum_f(const float *v, int lane)
{
    float x = v[lane & (kPcGW - 1)];
#pragma unroll
    for (int o = kPcGW / 2; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

__device__ __forceinline__ double group_sum_d(const float *v, int lane)
{
    double x = (double)v[lane & (kPcGW - 1)];
#pragma unroll
    for (int o = kPcGW / 2; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

// The per-warp sums of a row joined in double (a warp; every lane gets the totals).  The exponent actually used is
// c * log2e_f - m2 = (c - m) * log2e_f + off with off = m * log2e_f - m2; a code counted as the maximum, left out of
// the sweeps' sums, contributes exactly 2^off to z_raw and 2^off off to t_raw.  A dominant code (see the kernel) entered
// the sums of p^l and p^l^2 less 1.
__device__ __forceinline__ PcTotals row_totals(const PcParked &gs, int lane, float m, int nmax, int dominant)
{
    const double off = (double)m * (double)kLog2e - (double)(m * kLog2e);
    const double scale = exp2(off);
    PcTotals t;
    t.z_raw = group_sum_d(gs.zs, lane) + (double)nmax * scale;
    t.t_raw = group_sum_d(gs.ts, lane) + (double)nmax * scale * off;
    t.A = group_sum_d(gs.sums[0], lane);
    t.B = group_sum_d(gs.sums[1], lane) + (double)dominant;
    t.AA = group_sum_d(gs.sums[2], lane);
    t.AB = group_sum_d(gs.sums[3], lane);
    t.BB = group_sum_d(gs.sums[4], lane) + (double)dominant;
    return t;
}

// The normalisation step's scales and what follows from them: delta_i = k_up d_i + g p^l_i, every term >= 0.
struct PcScales {
    double k_up, g, omega, mu;
};

__device__ __forceinline__ PcScales row_scales(const PcTotals &t, float lo_cap, float hi_cap, double nn)
{
    const double S_lo = t.B, S_up = t.A + t.B;
    double k_lo = 1.0, k_up = 1.0;
    if (S_lo > 0.0 && (double)lo_cap / S_lo < 1.0) k_lo = (double)lo_cap / S_lo;
    if (S_up > 0.0 && (double)hi_cap / S_up > 1.0) k_up = (double)hi_cap / S_up;
    PcScales s;
    s.k_up = k_up;
    s.g = k_up - k_lo;
    s.omega = k_up * t.A + s.g * t.B;
    s.mu = s.omega / nn;
    return s;
}

// e^r - 1 for a stored (not raw) radius: a short series below 1/2, the exponential itself above.
__device__ __forceinline__ float expm1_fast(float r)
{
    float s = fmaf(r, 1.0f / 7.0f, 1.0f);
    s = fmaf(r * (1.0f / 6.0f), s, 1.0f);
    s = fmaf(r * (1.0f / 5.0f), s, 1.0f);
    s = fmaf(r * (1.0f / 4.0f), s, 1.0f);
    s = fmaf(r * (1.0f / 3.0f), s, 1.0f);
    s = fmaf(r * 0.5f, s, 1.0f);
    const float big = ex2_approx(r * kLog2e) - 1.0f;
    return fabsf(r) < 0.5f ? r * s : big;
}

// beta = e^r - 1 of one code, r clamped to r_max.  RAW: the stored value is rho and r = Softplus(rho) = ln(1 + e^rho),
// so beta = e^rho with no logarithm at all, and the clamp becomes beta <= e^r_max - 1.  (The selects keep a NaN
// radius, which must poison its row.)
template <bool RAW>
__device__ __forceinline__ float code_beta(float rho, float r_max, float beta_max)
{
    if (RAW) {
        const float u = ex2_approx(rho * kLog2e);
        return !(u > beta_max) ? u : beta_max;
    }
    return expm1_fast(!(rho > r_max) ? rho : r_max);
}

// code_beta for two codes: the scaling of the exponent is packed, the rest is per code
template <bool RAW>
__device__ __forceinline__ float2 code_beta2(float2 rho, float r_max, float beta_max)
{
    if (RAW) {
        const float2 x = __fmul2_rn(rho, make_float2(kLog2e, kLog2e));
        const float ux = ex2_approx(x.x), uy = ex2_approx(x.y);
        return make_float2(!(ux > beta_max) ? ux : beta_max, !(uy > beta_max) ? uy : beta_max);
    }
    return make_float2(code_beta<false>(rho.x, r_max, beta_max), code_beta<false>(rho.y, r_max, beta_max));
}

// One code's raw bounds from its exponential e (any common scale), the row's sum z of them and w = z - e:
//   p^l = e / (z + beta w),   p^u = (1 + beta) e / (z + beta e),
//   d = p^u - p^l = beta (2 + beta) e w / ((z + beta w)(z + beta e))   -- no cancellation for small radii.
// (e * rd alone may underflow for a large beta, hence the grouping.)
__device__ __forceinline__ void code_bounds(float e, float w, float z, float beta, float &pl, float &d)
{
    const float den_l = fmaf(beta, w, z), den_u = fmaf(beta, e, z);
    const float rd = rcp_approx(den_l * den_u);
    pl = e * (rd * den_u);
    d = (fmaf(beta, beta, beta + beta) * rd) * (e * w);
}

// MAPPED: the rows go through a position map (decode mode).
template <typename T, bool RAW, bool MAPPED>
__global__ void __launch_bounds__(kPcThreads, 1) quantify_percode_kernel(const __grid_constant__ QuantifyArgs a)
{
    constexpr int GT = kPcGT, GW = kPcGW, JV = kPcJV;
    constexpr int VEC = Elem<T>::kVec;
    constexpr int NPV = Vec<T>::kPairs;  // float2 pairs per 16-byte vector
    extern __shared__ __align__(128) unsigned char smem[];
    const int nvec = a.n / VEC;
    const uint32_t row_bytes = (uint32_t)nvec * 16u;
    const size_t stage_bytes = 2 * (size_t)row_bytes;  // logits, then radii
    PcShared &sh = *reinterpret_cast<PcShared *>(smem + kPcStages * stage_bytes);
    const int grp = threadIdx.x / GT, gtid = threadIdx.x % GT, lane = gtid & 31, gwarp = gtid >> 5;
    const int bar = kBarPc + grp;
    PcGroup &gs = sh.grp[grp];
    const ciar_quantify_out &o = a.out;

    if (threadIdx.x == 0) {
#pragma unroll
        for (int s = 0; s < kPcStages; ++s) mbar_init(&sh.full[s], 1);
        sh.nlist = 0;
        mbar_init_fence();
    }
    if (gtid == 0) {
        gs.abort = 0;
        gs.cnt = 0;
        gs.first = INT_MAX;
    }
    __syncthreads();
    // Decode mode: the rows go through a position map, and a position past the end of its sequence holds nothing to
    // quantify.  Such rows get their outputs here; the others are listed (in any order: rows are independent), and
    // the CTA walks the list.
    constexpr bool mapped = MAPPED;
    if (mapped) {
        const int nk = (int)((a.rows - blockIdx.x + gridDim.x - 1) / gridDim.x);  // at most kPcListCap (checked by the host)
        for (int i = threadIdx.x; i < nk; i += kPcThreads) {
            const int64_t lr = blockIdx.x + (int64_t)i * gridDim.x;
            int64_t pr;
            if (map_row(a.rm, lr, pr)) {
                sh.list[atomicAdd(&sh.nlist, 1)] = i;
            } else {
                if (o.flag) o.flag[lr] = 0;
                if (o.row_status) o.row_status[lr] = 0;
            }
        }
        __syncthreads();
    }
    const int nlist = mapped ? sh.nlist : 0;

    // The CTA's k-th row (a.rows when it has no more); the groups take k = 0, 1, 2, ... in turn, row k lands in
    // stage k % kPcStages.
    auto row_of = [&](int k) -> int64_t {
        if (mapped) return k < nlist ? blockIdx.x + (int64_t)sh.list[k] * gridDim.x : a.rows;
        return blockIdx.x + (int64_t)k * gridDim.x;
    };
    auto phys_row = [&](int64_t lr) -> int64_t {
        int64_t pr = lr;
        if (mapped) map_row(a.rm, lr, pr);
        return pr;
    };
    auto issue = [&](int k) {  // one thread
        const int64_t lr = row_of(k);
        if (lr < a.rows) {
            const int s = k % kPcStages;
            unsigned char *stage = smem + s * stage_bytes;
            const size_t at = (size_t)(a.vb + phys_row(lr) * a.row_stride);
            mbar_arrive_expect_tx(&sh.full[s], 2 * row_bytes);
            bulk_copy_g2s(stage, reinterpret_cast<const T *>(a.logits) + at, row_bytes, &sh.full[s]);
            bulk_copy_g2s(stage + row_bytes, reinterpret_cast<const T *>(a.radius) + at, row_bytes, &sh.full[s]);
        }
    };
    if (threadIdx.x == 0) {
#pragma unroll
        for (int s = 0; s < kPcStages; ++s) issue(s);
    }

    const double nn = (double)a.n;
    // Every warp of the group finishes one parked row: it joins the per-warp sums in double, lane 0 does the rest.
    auto finish_parked = [&](int count) {
        named_bar_sync(bar, GT);
        if (gwarp < count) {
            const PcParked &p = gs.park[gwarp];
            const PcTotals tt = row_totals(p, lane, p.m, p.nmax, p.dominant);
            const double dev = group_sum_d(p.dev, lane);
            if (lane != 0) return;
            if (!(tt.A == tt.A) || !(tt.B == tt.B)) {  // a NaN radius among the row's codes (it went through every sum)
                write_unusable(o, p.lr, CIAR_ROW_NAN);
                return;
            }
            const PcScales sc = row_scales(tt, a.lo_cap, a.hi_cap, nn);
            double var = (sc.k_up * sc.k_up * tt.AA + 2.0 * sc.k_up * sc.g * tt.AB + sc.g * sc.g * tt.BB) / nn - sc.mu * sc.mu;
            if (p.low_cv) var = dev / nn;
            const float m = p.m;
            const double off = (double)m * (double)kLog2e - (double)(m * kLog2e);
            const double unscale = exp2(-off);
            const double z = tt.z_raw * unscale;
            const double t = tt.t_raw * unscale - off * z;
            const double sigma = sqrt(var > 0.0 ? var : 0.0);
            const double score = sc.omega * sigma;
            const double lnz = z < 1.5 ? log1p(z - 1.0) : log(z);  // a peaked row: z just above 1
            const double p_max = 1.0 / z;
            const double entropy = lnz - kLn2D * t * p_max;
            const long long lr = p.lr;
            int fl;
            switch (a.policy) {
            case CIAR_POLICY_INTERVAL: fl = score > (double)a.tau; break;
            case CIAR_POLICY_ENTROPY: fl = entropy > (double)a.tau; break;
            case CIAR_POLICY_MAXPROB: fl = p_max < (double)a.tau; break;
            case CIAR_POLICY_RANDOM: fl = a.u_flag[phys_row(lr)] < a.tau; break;
            default: fl = 1; break;
            }
            if (o.row_max) o.row_max[lr] = m;
            if (o.sum_exp) o.sum_exp[lr] = (float)z;
            if (o.lse) o.lse[lr] = (float)((double)m + lnz);
            if (o.p_max) o.p_max[lr] = (float)p_max;
            if (o.entropy) o.entropy[lr] = (float)entropy;
            if (o.S_lo) o.S_lo[lr] = (float)tt.B;
            if (o.S_up) o.S_up[lr] = (float)(tt.A + tt.B);
            if (o.omega) o.omega[lr] = (float)sc.omega;
            if (o.sigma) o.sigma[lr] = (float)sigma;
            if (o.score) o.score[lr] = (float)score;
            if (o.argmax) o.argmax[lr] = p.first + a.vb;
            if (o.flag) o.flag[lr] = (uint8_t)fl;
            if (o.row_status) o.row_status[lr] = 0;
        }
    };

    const float beta_max = (float)expm1((double)a.r_max);
    const float inv_n = 1.0f / (float)a.n;
    int filled = 0;
    bool aborted = false;
    int k = grp;
    // Waits for the CTA's kk-th row to land and takes the maximum over it (sweep 1); each warp's maximum goes to the
    // given slot.  It runs one row ahead, before the last barrier of the group's row before, so that barrier also
    // publishes these maxima.  (The stage's phases complete in the order of its rows kk, kk + 3, kk + 6, ...: this
    // row's has parity (kk / 3) & 1.)
    auto first_sweep = [&](int kk, int slot) {
        const int s = kk % kPcStages;
        const unsigned char *stage = smem + s * stage_bytes;
        if (!mbar_wait_bounded(&sh.full[s], (uint32_t)(kk / kPcStages) & 1u, kWaitCycles)) gs.abort = 1;
        typename Vec<T>::Max mx = Vec<T>::max_init();
#pragma unroll
        for (int j = 0; j < JV; ++j) {
            const int vi = gtid + j * GT;
            if (vi < nvec) mx = Vec<T>::fold_max(mx, stage_vec(stage, vi));
        }
        const float wm = warp_redux_max(Vec<T>::max_value(mx));
        if (lane == 0) gs.wmax[slot][gwarp] = wm;
    };
    int it = 0;  // rows this group has started: its low bit picks the slot of the per-warp maxima
    if (row_of(k) < a.rows) {
        first_sweep(k, 0);
        named_bar_sync(bar, GT);
        if (gs.abort) aborted = true;
    }
    for (; row_of(k) < a.rows && !aborted; k += kPcGroups, ++it) {
        const int s = k % kPcStages;
        const unsigned char *stage = smem + s * stage_bytes;
        const unsigned char *rstage = stage + row_bytes;
        PcParked &pk = gs.park[filled];  // the sweeps leave their per-warp sums in the row's parking slot
        const bool more = row_of(k + kPcGroups) < a.rows;  // the group has a row after this one
        const float m = warp_redux_max(gs.wmax[it & 1][lane & (GW - 1)]);
        const float m2 = m * kLog2e;

        // ---- sweep 2: the sum of the exponentials and the entropy sum.  Codes whose exponential equals the
        // maximum's are counted: their terms, 2^off each, enter exactly when the totals are formed.
        const float e0f = ex2_approx(fmaf(m, kLog2e, -m2));
        bool has_max;  // this thread holds a code counted as a maximum
        {
            float2 z2 = f2(0.f), t2 = f2(0.f);
            int cnt = 0;
            const float2 L2 = f2(kLog2e), nm2 = f2(-m2);
#pragma unroll
            for (int j = 0; j < JV; ++j) {
                const int vi = gtid + j * GT;
                if (vi < nvec) {
                    float2 c[NPV];
                    Vec<T>::pairs(stage_vec(stage, vi), c);
#pragma unroll
                    for (int q = 0; q < NPV; ++q) {
                        const float2 d = __ffma2_rn(c[q], L2, nm2);
                        float2 ev = make_float2(ex2_approx(d.x), ex2_approx(d.y));  // a NaN logit poisons z on purpose
                        if (ev.x == e0f) {
                            ++cnt;
                            ev.x = 0.f;
                        }
                        if (ev.y == e0f) {
                            ++cnt;
                            ev.y = 0.f;
                        }
                        z2 = __fadd2_rn(z2, ev);
                        t2 = __ffma2_rn(ev, d, t2);  // 0 * -inf = NaN for a -inf logit: redone below
                    }
                }
            }
            float z = z2.x + z2.y, t = t2.x + t2.y;
            has_max = cnt > 0;
            int first = INT_MAX;
            if (has_max) {  // the lowest code of this thread equal to the maximum
#pragma unroll
                for (int j = 0; j < JV; ++j) {
                    const int vi = gtid + j * GT;
                    if (vi < nvec) {
                        float c[VEC];
                        Elem<T>::load(reinterpret_cast<const T *>(stage + (size_t)vi * 16), c);
#pragma unroll
                        for (int q = VEC - 1; q >= 0; --q)
                            if (c[q] == m) first = min(first, vi * VEC + q);
                    }
                }
            }
            if (!(t == t)) {
                // The entropy sum met a -inf logit (exponential 0, exponent -inf) or a real NaN: it is formed again with
                // such products taken as 0 (a real NaN still shows in the sum of exponentials).
                t = 0.f;
                for (int vi = gtid; vi < nvec; vi += GT) {
                    const T *cp = reinterpret_cast<const T *>(stage + (size_t)vi * 16);
#pragma unroll 1
                    for (int q = 0; q < VEC; ++q) {
                        const float d = fmaf(Elem<T>::widen(cp[q]), kLog2e, -m2), ev = ex2_approx(d);
                        if (ev != e0f) t = fmaf(ev, fmaxf(d, kNegHuge), t);
                    }
                }
            }
            const float zt = warp_sum_pair(z, t, lane);  // lanes 0..15: z, lanes 16..31: t
            if (lane == 0) pk.zs[gwarp] = zt;
            if (lane == 16) pk.ts[gwarp] = zt;
            if (__any_sync(0xffffffffu, has_max)) {
                cnt = __reduce_add_sync(0xffffffffu, cnt);
                first = __reduce_min_sync(0xffffffffu, first);
                if (lane == 0) {
                    atomicAdd(&gs.cnt, cnt);
                    atomicMin(&gs.first, first);
                }
            }
        }
        named_bar_sync(bar, GT);
        // Every thread needs the row's sum only in float; the totals in double are formed when the row is finished.
        const int nmax = gs.cnt, first = gs.first;
        const float z_others = group_sum_f(pk.zs, lane);
        const float zf = z_others + (float)nmax * e0f;

        int status = 0;
        if (m == -INFINITY) status |= CIAR_ROW_NO_FINITE;
        else if (!(zf < INFINITY) || !(zf > 0.f)) status |= CIAR_ROW_NAN;  // NaN or +inf logit
        if (status) {
            // nothing more is read from the stage: hand it to the row three further on
            if (more) first_sweep(k + kPcGroups, (it + 1) & 1);
            named_bar_sync(bar, GT);
            if (gtid == 0) {
                write_unusable(o, row_of(k), status);
                gs.cnt = 0;
                gs.first = INT_MAX;
                fence_proxy_async_smem();
                issue(k + kPcStages);
            }
            if (more && gs.abort) {  // the next row never landed
                aborted = true;
                k += kPcGroups;
                break;
            }
            continue;
        }
        // A single code that holds more than half of the mass: its p^l, near 1, would cost the sum of the lower bounds
        // (which decides Omega = 1.01 - S_lo when S_lo < 0.99) its last digits in float.
        const int dominant = nmax == 1 && e0f > 0.5f * zf;

        // ---- sweep 3: both bounds of every code from its own radius; the sums of d, p^l, d^2, d p^l, p^l^2
        {
            // two codes at a time in packed fp32 (the exponentials, reciprocals and clamps stay scalar)
            float2 pA = f2(0.f), pB = f2(0.f), pAA = f2(0.f), pAB = f2(0.f), pBB = f2(0.f);
            float dom_rho = 0.f;
            bool dom_here = false;  // this thread holds the dominant code
            auto sweep = [&](auto look_out) {
                constexpr bool DOM = decltype(look_out)::value;
                const float2 L2 = f2(kLog2e), nm2 = f2(-m2), zf2 = f2(zf), neg1 = f2(-1.0f);
#pragma unroll
                for (int j = 0; j < JV; ++j) {
                    const int vi = gtid + j * GT;
                    if (vi < nvec) {
                        float2 c[NPV], rho[NPV];
                        Vec<T>::pairs(stage_vec(stage, vi), c);
                        Vec<T>::pairs(stage_vec(rstage, vi), rho);
#pragma unroll
                        for (int q = 0; q < NPV; ++q) {
                            const float2 x = __ffma2_rn(c[q], L2, nm2);
                            float2 ev = make_float2(ex2_approx(x.x), ex2_approx(x.y));
                            if (DOM) {  // the dominant code is taken out here (its terms become 0) and put in below
                                if (ev.x == e0f) {
                                    dom_rho = rho[q].x;
                                    dom_here = true;
                                    ev.x = 0.f;
                                }
                                if (ev.y == e0f) {
                                    dom_rho = rho[q].y;
                                    dom_here = true;
                                    ev.y = 0.f;
                                }
                            }
                            const float2 beta = code_beta2<RAW>(rho[q], a.r_max, beta_max);
                            const float2 w = __ffma2_rn(ev, neg1, zf2);
                            const float2 den_l = __ffma2_rn(beta, w, zf2), den_u = __ffma2_rn(beta, ev, zf2);
                            const float2 pr = __fmul2_rn(den_l, den_u);
                            const float2 rd = make_float2(rcp_approx(pr.x), rcp_approx(pr.y));
                            const float2 pl = __fmul2_rn(ev, __fmul2_rn(rd, den_u));
                            const float2 kd = __ffma2_rn(beta, beta, __fadd2_rn(beta, beta));
                            const float2 d = __fmul2_rn(__fmul2_rn(kd, rd), __fmul2_rn(ev, w));
                            pA = __fadd2_rn(pA, d);
                            pB = __fadd2_rn(pB, pl);
                            pAA = __ffma2_rn(d, d, pAA);
                            pAB = __ffma2_rn(d, pl, pAB);
                            pBB = __ffma2_rn(pl, pl, pBB);
                        }
                    }
                }
            };
            // only the warp that holds a dominant code pays for looking out for it (the branch is uniform in a warp)
            if (dominant && __any_sync(0xffffffffu, has_max)) sweep(std::true_type());
            else sweep(std::false_type());
            float sA = pA.x + pA.y, sB = pB.x + pB.y, sAA = pAA.x + pAA.y, sAB = pAB.x + pAB.y, sBB = pBB.x + pBB.y;
            if (dom_here) {
                // With w = z - e taken from the other codes' sum, 1 - p^l = (1 + beta) w / (z + beta w) =: q^l keeps its
                // digits, so p^l - 1 = -q^l and p^l^2 - 1 = q^l^2 - 2 q^l are what the dominant code adds; the units are
                // put back when the totals are formed.
                const float beta = code_beta<RAW>(dom_rho, a.r_max, beta_max);
                float pl, d;
                code_bounds(e0f, z_others, zf, beta, pl, d);
                const float ql = (z_others + beta * z_others) * rcp_approx(fmaf(beta, z_others, zf));
                sA += d;
                sB -= ql;
                sAA = fmaf(d, d, sAA);
                sAB = fmaf(d, 1.0f - ql, sAB);
                sBB += fmaf(ql, ql, -2.0f * ql);
            }
            const float r0 = warp_sum_pair(sA, sB, lane), r1 = warp_sum_pair(sAA, sAB, lane), r2 = warp_sum_f(sBB);
            if (lane == 0) {
                pk.sums[0][gwarp] = r0;
                pk.sums[2][gwarp] = r1;
                pk.sums[4][gwarp] = r2;
            }
            if (lane == 16) {
                pk.sums[1][gwarp] = r0;
                pk.sums[3][gwarp] = r1;
            }
        }
        if (more) first_sweep(k + kPcGroups, (it + 1) & 1);  // sweep 1 of the group's next row
        named_bar_sync(bar, GT);
        const bool next_abort = more && gs.abort;  // set only by this group's threads, before the barrier: uniform
        // A look at the totals in float, only to see whether the moment form of the variance is safe for this row
        // (every thread forms the same values, so the branch below is uniform).
        bool low_cv;
        {
            const float A = group_sum_f(pk.sums[0], lane), B = group_sum_f(pk.sums[1], lane) + (float)dominant,
                        AA = group_sum_f(pk.sums[2], lane), AB = group_sum_f(pk.sums[3], lane),
                        BB = group_sum_f(pk.sums[4], lane) + (float)dominant;
            const float S_lo = B, S_up = A + B;
            float k_lo = 1.f, k_up = 1.f;
            if (S_lo > 0.f && a.lo_cap < S_lo) k_lo = a.lo_cap * rcp_approx(S_lo);
            if (S_up > 0.f && a.hi_cap > S_up) k_up = a.hi_cap * rcp_approx(S_up);
            const float g = k_up - k_lo;
            const float mu = (k_up * A + g * B) * inv_n;
            const float var = (k_up * k_up * AA + 2.f * k_up * g * AB + g * g * BB) * inv_n - mu * mu;
            low_cv = !(var >= 0.1f * mu * mu);  // nearly uniform widths: the moment form cancels
        }
        if (low_cv) {
            // ---- sweep 4 (rare): sum of (delta_i - mu)^2 with the scales known, from the totals in double
            const PcTotals tt = row_totals(pk, lane, m, nmax, dominant);
            const PcScales sc = row_scales(tt, a.lo_cap, a.hi_cap, nn);
            const float fku = (float)sc.k_up, fg = (float)sc.g, fmu = (float)sc.mu;
            float sd = 0.f;
#pragma unroll
            for (int j = 0; j < JV; ++j) {
                const int vi = gtid + j * GT;
                if (vi < nvec) {
                    float c[VEC], rho[VEC];
                    Elem<T>::load(reinterpret_cast<const T *>(stage + (size_t)vi * 16), c);
                    Elem<T>::load(reinterpret_cast<const T *>(rstage + (size_t)vi * 16), rho);
#pragma unroll
                    for (int q = 0; q < VEC; ++q) {
                        float pl, d;
                        const float ev = ex2_approx(fmaf(c[q], kLog2e, -m2));
                        code_bounds(ev, zf - ev, zf, code_beta<RAW>(rho[q], a.r_max, beta_max), pl, d);
                        const float x = fmaf(fku, d, fg * pl) - fmu;
                        sd = fmaf(x, x, sd);
                    }
                }
            }
            sd = warp_sum_f(sd);
            if (lane == 0) pk.dev[gwarp] = sd;
            named_bar_sync(bar, GT);
        }
        if (gtid == 0) {  // every thread of the group has read the stage for the last time: refill it; the row's scalars
            gs.cnt = 0;
            gs.first = INT_MAX;
            fence_proxy_async_smem();
            issue(k + kPcStages);
            pk.lr = row_of(k);
            pk.m = m;
            pk.first = first;
            pk.nmax = nmax;
            pk.dominant = dominant;
            pk.low_cv = low_cv;
        }
        if (++filled == GW) {
            finish_parked(filled);
            filled = 0;
        }
        if (next_abort) {  // the next row never landed
            aborted = true;
            k += kPcGroups;
            break;
        }
    }
    if (filled > 0) finish_parked(filled);

    if (aborted && gtid == 0) {
        // A copy never arrived: mark this row and the rest of this group's rows.
        for (int k2 = k; row_of(k2) < a.rows; k2 += kPcGroups) write_unusable(o, row_of(k2), CIAR_ROW_TIMEOUT);
    }
    __syncthreads();
    if ((sh.grp[0].abort | sh.grp[1].abort) && threadIdx.x == 0) {
        // Give the copies still in flight a last bounded chance to land before the CTA leaves (of the two waits on
        // a stage, the one for a phase already complete returns at once).
        for (int s = 0; s < kPcStages; ++s) {
            mbar_wait_bounded(&sh.full[s], 0u, kDrainCycles);
            mbar_wait_bounded(&sh.full[s], 1u, kDrainCycles);
        }
    }
}

template <typename T, bool RAW, bool MAPPED>
cudaError_t launch_pc(const QuantifyArgs &a, cudaStream_t stream)
{
    constexpr size_t smem_max = (size_t)kPcStages * 2 * kPcRowBytes + sizeof(PcShared);
    static bool configured[64] = {};
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!configured[dev]) {
        err = cudaFuncSetAttribute(quantify_percode_kernel<T, RAW, MAPPED>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_max);
        if (err != cudaSuccess) return err;
        configured[dev] = true;
    }
    const size_t row_bytes = (size_t)(a.n / Elem<T>::kVec) * 16;
    const size_t smem = (size_t)kPcStages * 2 * row_bytes + sizeof(PcShared);
    const int64_t cap = sm_count();
    const unsigned grid = (unsigned)(a.rows < cap ? a.rows : cap);
    quantify_percode_kernel<T, RAW, MAPPED><<<grid, kPcThreads, smem, stream>>>(a);
    count_launch();
    return cudaGetLastError();
}

}  // namespace

bool quantify_percode_eligible(const QuantifyArgs &a, int dtype)
{
    const int vec = dtype == CIAR_F32 ? 4 : 8;
    if (a.radius_mode != CIAR_RADIUS_PER_CODE) return false;
    if (a.rm.pos != nullptr) {  // decode row map: a CTA lists its rows, and the list is of fixed size
        const int64_t grid = a.rows < sm_count() ? a.rows : sm_count();
        if (grid > 0 && (a.rows + grid - 1) / grid > kPcListCap) return false;
    }
    if (a.out.dense_p || a.out.dense_lo || a.out.dense_up) return false;
    if (a.vb % vec != 0 || a.n % vec != 0) return false;
    if (a.r_max > 30.0f) return false;  // the product of the two denominators must stay in float range: beta <= e^30
    return a.n >= 2048 && (a.n / vec) * 16 <= kPcRowBytes;
}

cudaError_t launch_quantify_percode(const QuantifyArgs &a, int dtype, cudaStream_t stream)
{
    if (a.rows == 0) return cudaSuccess;
    const bool raw = a.radius_is_raw != 0, mapped = a.rm.pos != nullptr;
    if (dtype == CIAR_F32) {
        if (mapped) return raw ? launch_pc<float, true, true>(a, stream) : launch_pc<float, false, true>(a, stream);
        return raw ? launch_pc<float, true, false>(a, stream) : launch_pc<float, false, false>(a, stream);
    }
    if (mapped) return raw ? launch_pc<__nv_bfloat16, true, true>(a, stream) : launch_pc<__nv_bfloat16, false, true>(a, stream);
    return raw ? launch_pc<__nv_bfloat16, true, false>(a, stream) : launch_pc<__nv_bfloat16, false, false>(a, stream);
}

}  // namespace ciar
