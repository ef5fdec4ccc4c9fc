// Streaming quantifier for rows too wide to sit on chip (more than 16384 codes, scalar or per-row radius).
//
// One persistent CTA of 32 warps per SM walks rows blockIdx.x, blockIdx.x + gridDim.x, ...  A row passes
// twice through a ring of three shared-memory stages, 64 KB at a time ("chunks"), filled by bulk (TMA)
// copies that one thread issues three chunks ahead:
//   pass A  softmax statistics on line: every warp keeps a running maximum of the codes it has seen and,
//           per lane, the sums of exp and of exp * exponent relative to it (rescaled when the maximum
//           moves; codes equal to the maximum are counted, not summed).  The warps' results are joined
//           once per row, in double.
//   pass B  with the maximum and the sum of exponentials known: the interval sums of the on-chip kernel
//           (power sums about Z / n with the few codes above theta listed; or the direct formulas),
//           accumulated per chunk in float and across chunks in double; the arg-max.
// A finished row is parked in the same form as the on-chip kernel parks it and finished by the same warp
// routine.  With one CTA per SM the rows in flight (one per SM) stay in the L2 between their two passes, so
// each logit comes from HBM once; the copies of pass A ask the L2 to keep their lines, those of pass B to
// drop them.
#include <type_traits>

#include "online_stats.cuh"
#include "quantify_finish.cuh"

namespace ciar {

namespace {

constexpr int kWThreads = 1024;  // one CTA per SM: the rows in flight on the GPU then fit in the L2 between their passes
constexpr int kWWarps = kWThreads / 32;
constexpr int kGroups = 2;  // halves of the CTA, each with its own ring and barrier: a row's chunks go to them in turn
constexpr int kGThreads = kWThreads / kGroups;
constexpr int kWJ = 4;                       // vectors per thread and chunk
constexpr int kChunkVecs = kGThreads * kWJ;  // 2048 vectors
constexpr int kChunkBytes = kChunkVecs * 16;
constexpr int kRingBytes = kQStages * kChunkBytes;

struct WShared {
    unsigned long long full[kGroups][kQStages];
    // pass A, per warp: running maximum, sums relative to it, number of codes equal to it, first chunk holding it
    float wm[kWWarps];
    double wz[kWWarps], wt[kWWarps];
    int wcnt[kWWarps], wchunk[kWWarps];
    double ws[kWWarps][5];  // pass B, per warp: the route's sums
    // by row parity (a thread may start the next row while another still reads this row's): lowest index holding the
    // maximum, codes above theta so far, what an unusable row contains
    int argmin[2], nlist[2], bad_nan[2], bad_finite[2];
    int abort;
    float list[kListCap];  // series route: exponentials of the codes above theta beyond the parked row's own slots
    Parked park[kPark];
};
static_assert(sizeof(WShared) + kGroups * kRingBytes <= 232448, "the ring and the scratch must fit in one SM's shared memory");

// One step of a group's walk: the group's c-th chunk of pass `pass` (0 = A, 1 = B) of the CTA's k-th row.
struct Item {
    int k, pass, c;
};

template <typename T>
__global__ void __launch_bounds__(kWThreads, 1) quantify_wide_kernel(const __grid_constant__ QuantifyArgs a)
{
    typedef Vec<T> V;
    constexpr int VEC = Elem<T>::kVec;
    constexpr int NPV = V::kPairs;    // float2 pairs per 16-byte vector
    constexpr int NP = kWJ * NPV;     // pairs per thread and chunk
    extern __shared__ __align__(128) unsigned char smem[];
    WShared &sh = *reinterpret_cast<WShared *>(smem + (size_t)kGroups * kRingBytes);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int gid = tid / kGThreads, tg = tid % kGThreads;  // group, and thread within it
    unsigned char *ring = smem + (size_t)gid * kRingBytes;
    unsigned long long *full = sh.full[gid];
    const ciar_quantify_out &o = a.out;

    if (tid == 0) {
#pragma unroll
        for (int s = 0; s < kGroups * kQStages; ++s) mbar_init(&sh.full[0][0] + s, 1);
        sh.abort = 0;
        mbar_init_fence();
    }
    __syncthreads();

    const int nvec = a.n / VEC;
    const int nch_row = (nvec + kChunkVecs - 1) / kChunkVecs;
    const int nch = (nch_row - gid + kGroups - 1) / kGroups;  // this group's chunks of a row: gid, gid + 2, ...
    const int nk = (int)((a.rows - blockIdx.x + gridDim.x - 1) / gridDim.x);  // rows this CTA walks (the grid never exceeds the rows)
    auto row_of = [&](int k) -> int64_t { return blockIdx.x + (int64_t)k * gridDim.x; };
    // the next row at or after `from` that has something to quantify (-1: none left)
    auto next_active = [&](int from) -> int {
        for (int kk = from; kk < nk; ++kk) {
            int64_t pr;
            if (map_row(a.rm, row_of(kk), pr)) return kk;
        }
        return -1;
    };
    // thread 0: positions past the end of a sequence among rows [from, to) get their outputs
    auto retire_skipped = [&](int from, int to) {
        for (int kk = from; kk < (to < 0 ? nk : to); ++kk) {
            const int64_t lr = row_of(kk);
            if (o.flag) o.flag[lr] = 0;
            if (o.row_status) o.row_status[lr] = 0;
        }
    };
    auto advance = [&](Item &it) {
        if (it.k < 0) return;
        if (++it.c < nch) return;
        it.c = 0;
        if (it.pass == 0) {
            it.pass = 1;
            return;
        }
        it.pass = 0;
        it.k = next_active(it.k + 1);
    };
    // a group's first thread: asks for the chunk of item `it`, the g-th of the group's walk, into stage g mod 3
    auto issue = [&](const Item &it, int g) {
        if (it.k < 0) return;
        int64_t pr;
        map_row(a.rm, row_of(it.k), pr);
        const int v0 = (it.c * kGroups + gid) * kChunkVecs;
        const uint32_t bytes = (uint32_t)min(kChunkVecs, nvec - v0) * 16u;
        const int s = g % kQStages;
        mbar_arrive_expect_tx(&full[s], bytes);
        // pass A's lines are wanted once more, by pass B, which is their last use
        bulk_copy_g2s_hint(ring + (size_t)s * kChunkBytes,
                           reinterpret_cast<const T *>(a.logits) + a.vb + pr * a.row_stride + (int64_t)v0 * VEC, bytes, &full[s],
                           it.pass == 0 ? l2_policy_evict_last() : l2_policy_evict_first());
    };
    // Every warp finishes one parked row.  Only the row parked last can have a list longer than its slot
    // (such a row is finished at once); the slot's part then moves next to the rest in the shared buffer.
    auto finish_parked = [&](int count) {
        __syncthreads();
        if (warp < count) {
            Parked &p = sh.park[warp];
            const float *list = p.list;
            if (p.nlist > kParkList) {
                for (int i = lane; i < kParkList; i += 32) sh.list[i] = p.list[i];
                __syncwarp();
                list = sh.list;
            }
            finish_row(a, p, list, lane, kQWarps);
        }
        __syncthreads();
    };
    int k = next_active(0);  // the row being swept
    Item pit = { k, 0, 0 };  // the item to ask for next, three ahead of the sweeps
    if (tid == 0) retire_skipped(0, k);
#pragma unroll 1
    for (int i = 0; i < kQStages; ++i) {
        if (tg == 0) issue(pit, i);
        advance(pit);
    }

    int g = 0, filled = 0, rp = 0;  // items swept, rows parked, parity of the rows swept
    bool aborted = false;

    // One pass of this group over its chunks of the row being swept: waits for each chunk, lets `body` sweep it,
    // and after the group's barrier (all its threads have read the stage) asks for the chunk three further on.
    // `body` gets a compile-time flag saying that the chunk is a whole one: every thread then owns kWJ vectors of
    // it.  Once a copy has failed to arrive nothing is waited for any more; the CTA leaves at its next barrier.
    auto for_chunks = [&](auto &&body) {
#pragma unroll 1
        for (int cl = 0; cl < nch; ++cl) {
            const int s = g % kQStages;
            const unsigned char *stage = ring + (size_t)s * kChunkBytes;
            const int c = cl * kGroups + gid;
            const int v0 = c * kChunkVecs;
            if (!sh.abort && !mbar_wait_bounded(&full[s], (uint32_t)(g / kQStages) & 1u, kWaitCycles)) sh.abort = 1;
            if (nvec - v0 >= kChunkVecs) {
                body(std::true_type(), c, stage, v0, kWJ);
            } else {
                int nj = (nvec - v0 - tg + kGThreads - 1) / kGThreads;
                nj = nj < 0 ? 0 : nj;
                body(std::false_type(), c, stage, v0, nj);
            }
            __syncwarp();
            named_bar_sync(kBarRow + gid, kGThreads);
            if (tg == 0 && !sh.abort) {
                fence_proxy_async_smem();
                issue(pit, g + kQStages);
            }
            advance(pit);
            ++g;
        }
    };

    while (k >= 0) {
        Parked &pk = sh.park[filled];
        if (tid == 0) {
            sh.argmin[rp] = INT_MAX;
            sh.nlist[rp] = 0;
            sh.bad_nan[rp] = sh.bad_finite[rp] = 0;
        }
        // ---- pass A: every warp's running maximum, and per lane the sums of exp and exp * exponent relative to it
        {
            OnlineStats st;
            st.reset();
            for_chunks([&](auto whole, int c, const unsigned char *stage, int, int nj) {
                online_sweep<T, kGThreads, kWJ, decltype(whole)::value, true>(st, stage, tg, nj, c);
            });
            // the warp's share of the row's statistics
            const double zw = warp_sum_d(st.zd), tw = warp_sum_d(st.td);
            int cw = st.cnt;
#pragma unroll
            for (int ofs = 16; ofs > 0; ofs >>= 1) cw += __shfl_xor_sync(0xffffffffu, cw, ofs);
            if (lane == 0) {
                sh.wm[warp] = st.m_w;
                sh.wz[warp] = zw;
                sh.wt[warp] = tw;
                sh.wcnt[warp] = cw;
                sh.wchunk[warp] = st.chunk;
            }
        }
        __syncthreads();  // both groups are through pass A: the warps' shares are out
        if (sh.abort) {
            aborted = true;
            break;
        }
        // ---- the row's statistics from the warps' (lane w joins warp w's share, rescaled to the row maximum)
        float m, m2, zf, c0, th, th_log, r;
        int status = 0;
        bool classify, series, direct;
        {
            const int w = lane & (kWWarps - 1);
            const float mw = sh.wm[w];
            m = warp_redux_max(mw);
            m2 = m * kLog2e;
            const float e0 = ex2_approx(fmaf(m, kLog2e, -m2));  // the exponential every maximum gets
            double zc = 0.0, tc = 0.0;
            int nc = 0;
            if (mw > -INFINITY) {
                const double zw = sh.wz[w], tw = sh.wt[w];
                const int cw = sh.wcnt[w];
                if (mw == m) {
                    zc = zw;
                    tc = tw;
                    nc = cw;
                } else {
                    const float mw2 = mw * kLog2e;
                    const double dl = (double)mw2 - (double)m2;
                    const double f = exp2(dl);
                    const double tot = zw + (double)cw * (double)ex2_approx(fmaf(mw, kLog2e, -mw2));
                    zc = tot * f;
                    tc = f * (tw + dl * tot);
                }
            }
#pragma unroll
            for (int ofs = kWWarps / 2; ofs > 0; ofs >>= 1) {
                zc += __shfl_xor_sync(0xffffffffu, zc, ofs);
                tc += __shfl_xor_sync(0xffffffffu, tc, ofs);
                nc += __shfl_xor_sync(0xffffffffu, nc, ofs);
            }
            zf = (float)(zc + (double)nc * (double)e0);
            classify = !(m > -INFINITY) || !(zf > 0.f) || !(zf < INFINITY);
            if (classify) status = CIAR_ROW_NAN;  // refined by pass B
            const int64_t lr = row_of(k);
            int64_t pr;
            map_row(a.rm, lr, pr);
            const float rho = a.radius_mode == CIAR_RADIUS_PER_ROW ? reinterpret_cast<const float *>(a.radius)[pr] : a.r_scalar;
            if (!(rho == rho)) status |= CIAR_ROW_NAN;
            r = row_radius(rho, a.radius_is_raw, a.r_max);
            series = r <= 1.0f;
            direct = !status && !series;
            c0 = zf * rcp_approx((float)a.n);
            th = 0.00390625f * ex2_approx(-r * kLog2e) * zf;  // clamp level: theta = 2^-8 e^-r, in units of exp(c - m)
            th_log = __log2f(th) - 1e-3f;  // a slightly low stand-in for log2(th): the test on a maximum errs on the safe side
            // Park what is known already.  Each sum goes in as a float pair (high part in warp 0's place, the
            // remainder in warp 1's, zeros in the others), so that the finishing routine's double sum is the sum.
            if (tid < kQWarps * 8 && (tid & 3) == 0) {
                const int wrow = tid >> 3;
                const double tot = (tid & 4) ? tc : zc;
                const float hi = (float)tot;
                pk.wsum[wrow][tid & 7] = wrow == 0 ? hi : (wrow == 1 ? (float)(tot - (double)hi) : 0.f);
            }
            if (tid == 0) {
                pk.lr = lr;
                pk.pr = pr;
                pk.m = m;
                pk.e0 = e0;
                pk.c0 = c0;
                pk.th = th;
                pk.rho = rho;
                pk.r = r;
                pk.nmax = nc;
                pk.series = series;
                pk.par = 0;
            }
        }
        // ---- pass B: with the maximum and the sum of exponentials known
        if (classify) {
            // an unusable row: what it contains, exactly as the row-status bits are defined
            int has_nan = 0, has_finite = 0;
            for_chunks([&](auto, int, const unsigned char *stage, int, int nj) {
                for (int j = 0; j < nj; ++j) {
                    const T *v = reinterpret_cast<const T *>(stage + (size_t)(tg + j * kGThreads) * 16);
#pragma unroll
                    for (int q = 0; q < VEC; ++q) {
                        const float c = Elem<T>::widen(v[q]);
                        if (!(c == c) || c == INFINITY) has_nan = 1;
                        if (c == c && fabsf(c) != INFINITY) has_finite = 1;
                    }
                }
            });
            if (has_nan) sh.bad_nan[rp] = 1;
            if (has_finite) sh.bad_finite[rp] = 1;
        } else if (status) {
            for_chunks([&](auto, int, const unsigned char *, int, int) {});  // the chunks were asked for already
        } else {
            // the first chunk in which this warp met the row maximum holds its candidates for the arg-max
            const int amchunk = sh.wm[warp] == m ? sh.wchunk[warp] : -1;
            auto arg_max = [&](int c, const unsigned char *stage, int v0, int nj) {
                if (c != amchunk) return;
                int best = INT_MAX;
                for (int j = nj - 1; j >= 0; --j) {
                    const T *v = reinterpret_cast<const T *>(stage + (size_t)(tg + j * kGThreads) * 16);
#pragma unroll
                    for (int q = VEC - 1; q >= 0; --q)
                        if (Elem<T>::widen(v[q]) == m) best = (v0 + tg + j * kGThreads) * VEC + q;
                }
                if (best != INT_MAX) atomicMin(&sh.argmin[rp], best);
            };
            if (series) {
                double a2 = 0.0, a3 = 0.0, a4 = 0.0;  // power sums of (e - c0) over the row
                for_chunks([&](auto whole, int c, const unsigned char *stage, int v0, int nj) {
                    constexpr bool W = decltype(whole)::value;
                    arg_max(c, stage, v0, nj);
                    typename V::Max mx = V::max_init();
                    float2 e[NP];
                    {
                        const float2 L2 = f2(kLog2e), nm2 = f2(-m2);
#pragma unroll
                        for (int j = 0; j < kWJ; ++j) {
                            if (W || j < nj) {
                                const uint4 &vv = stage_vec(stage, tg + j * kGThreads);
                                mx = V::fold_max(mx, vv);
                                float2 cc[NPV];
                                V::pairs(vv, cc);
#pragma unroll
                                for (int q = 0; q < NPV; ++q) {
                                    const float2 d = __ffma2_rn(cc[q], L2, nm2);
                                    e[j * NPV + q] = make_float2(ex2_once(d.x), ex2_once(d.y));
                                }
                            } else {
#pragma unroll
                                for (int q = 0; q < NPV; ++q) e[j * NPV + q] = f2(0.f);
                            }
                        }
                    }
                    // Codes above th are listed and clamped to th.  Most warps hold none in a chunk (seen from the
                    // largest logit of the warp's part), and a vector holding none is skipped on one comparison.
                    const float wmc = warp_redux_max(V::max_value(mx));
                    if (__builtin_expect(fmaf(wmc, kLog2e, -m2) > th_log, 0)) {
#pragma unroll
                        for (int j = 0; j < kWJ; ++j) {
                            float2 gm = e[j * NPV];
#pragma unroll
                            for (int q = 1; q < NPV; ++q) gm = make_float2(fmaxf(gm.x, e[j * NPV + q].x), fmaxf(gm.y, e[j * NPV + q].y));
                            if (fmaxf(gm.x, gm.y) > th) {
#pragma unroll
                                for (int q = 0; q < 2 * NPV; ++q) {
                                    float &ev = (q & 1) ? e[j * NPV + q / 2].y : e[j * NPV + q / 2].x;
                                    if (ev > th) {
                                        const int slot = atomicAdd(&sh.nlist[rp], 1);
                                        if (slot < kParkList) pk.list[slot] = ev;
                                        else if (slot < kListCap) sh.list[slot] = ev;
                                        ev = th;
                                    }
                                }
                            }
                        }
                    }
                    // over the chunk in float, over the row in double
                    float2 T2 = f2(0.f), T3 = f2(0.f), T4 = f2(0.f);
                    const float2 nc0 = f2(-c0);
#pragma unroll
                    for (int i = 0; i < NP; ++i) {
                        if (W || i / NPV < nj) {
                            const float2 y = __fadd2_rn(e[i], nc0);
                            const float2 y2 = __fmul2_rn(y, y);
                            T2 = __fadd2_rn(T2, y2);
                            T3 = __ffma2_rn(y2, y, T3);
                            T4 = __ffma2_rn(y2, y2, T4);
                        }
                    }
                    a2 += (double)(T2.x + T2.y);
                    a3 += (double)(T3.x + T3.y);
                    a4 += (double)(T4.x + T4.y);
                });
                const double s2 = warp_sum_d(a2), s3 = warp_sum_d(a3), s4 = warp_sum_d(a4);
                if (lane == 0) {
                    sh.ws[warp][0] = s2;
                    sh.ws[warp][1] = s3;
                    sh.ws[warp][2] = s4;
                }
            } else {
                // both bounds of every code
                const DirectConst dc = make_direct_const(r, a.n);
                const float invz = 1.0f / zf;
                double acc[5] = { 0.0, 0.0, 0.0, 0.0, 0.0 };
                for_chunks([&](auto, int c, const unsigned char *stage, int v0, int nj) {
                    arg_max(c, stage, v0, nj);
                    float ps[5] = { 0.f, 0.f, 0.f, 0.f, 0.f };
#pragma unroll 1
                    for (int j = 0; j < nj; ++j) {
                        const T *v = reinterpret_cast<const T *>(stage + (size_t)(tg + j * kGThreads) * 16);
                        float cc[VEC];
                        Elem<T>::load(v, cc);
#pragma unroll
                        for (int q = 0; q < VEC; ++q) {
                            const float ev = ex2_approx(fmaf(cc[q], kLog2e, -m2));
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
#pragma unroll
                    for (int q = 0; q < 5; ++q) acc[q] += (double)ps[q];
                });
#pragma unroll
                for (int q = 0; q < 5; ++q) {
                    const double tot = warp_sum_d(acc[q]);
                    if (lane == 0) sh.ws[warp][q] = tot;
                }
            }
        }
        __syncthreads();  // both groups are through pass B: the warps' sums, the list and the arg-max are complete
        if (sh.abort) {
            aborted = true;
            break;
        }
        if (classify) {
            status = 0;
            if (sh.bad_nan[rp]) status |= CIAR_ROW_NAN;
            if (!sh.bad_finite[rp]) status |= CIAR_ROW_NO_FINITE;
            if (!status) status = CIAR_ROW_NAN;  // sums overflowed without any single bad logit
        }
        // ---- park the rest: the route's sums (series: powers 2, 3, 4; direct: pl, dd, pl^2, pl dd, dd^2)
        if (tid < kQWarps * 8 && (tid & 3) != 0) {
            const int wrow = tid >> 3, slot = tid & 7;
            const int q = slot == 1 ? 0 : slot == 5 ? 1 : slot == 2 ? 2 : slot == 6 ? 3 : slot == 3 ? 4 : -1;
            double tot = 0.0;
            if (!status && q >= 0 && (q < 3 || direct))
                for (int ww = 0; ww < kWWarps; ++ww) tot += sh.ws[ww][q];
            const float hi = (float)tot;
            pk.wsum[wrow][slot] = wrow == 0 ? hi : (wrow == 1 ? (float)(tot - (double)hi) : 0.f);
        }
        const int nlist = sh.nlist[rp];
        if (tid == 0) {
            pk.argmin = sh.argmin[rp];
            pk.nlist = nlist;
            pk.status = status;
        }
        rp ^= 1;
        if (++filled == kPark || nlist > kParkList) {  // a list longer than the row's own slots sits in the shared buffer: finish now
            finish_parked(filled);
            filled = 0;
        }
        const int kprev = k;
        k = next_active(k + 1);
        if (tid == 0) retire_skipped(kprev + 1, k);
    }
    if (filled > 0) finish_parked(filled);

    if (aborted && tg == 0) {
        // A copy never arrived.  Mark this row and the rest of this CTA's rows, then give the copies
        // still in flight a last bounded chance to land before the CTA leaves.
        if (tid == 0)
            for (int k2 = k; k2 < nk; ++k2) write_unusable(o, row_of(k2), CIAR_ROW_TIMEOUT);
        for (int i = 0; i < kQStages; ++i)
            mbar_wait_bounded(&full[(g + i) % kQStages], (uint32_t)((g + i) / kQStages) & 1u, kDrainCycles);
    }
}

cudaError_t launch_wide(const QuantifyArgs &a, int dtype, cudaStream_t stream)
{
    constexpr size_t smem = (size_t)kGroups * kRingBytes + sizeof(WShared);
    static bool configured[64] = {};
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!configured[dev]) {
        err = cudaFuncSetAttribute(quantify_wide_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (err == cudaSuccess)
            err = cudaFuncSetAttribute(quantify_wide_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (err != cudaSuccess) return err;
        configured[dev] = true;
    }
    const int64_t cap = (int64_t)sm_count();
    const unsigned grid = (unsigned)(a.rows < cap ? a.rows : cap);
    if (dtype == CIAR_F32) quantify_wide_kernel<float><<<grid, kWThreads, smem, stream>>>(a);
    else quantify_wide_kernel<__nv_bfloat16><<<grid, kWThreads, smem, stream>>>(a);
    count_launch();
    return cudaGetLastError();
}

}  // namespace

bool quantify_wide_eligible(const QuantifyArgs &a, int dtype)
{
    const int vec = dtype == CIAR_F32 ? 4 : 8;
    if (a.radius_mode == CIAR_RADIUS_PER_CODE) return false;
    if (a.out.dense_p || a.out.dense_lo || a.out.dense_up) return false;
    if (a.vb % vec != 0 || a.n % vec != 0) return false;
    return a.n > 16384 && a.n <= (1 << 28);
}

cudaError_t launch_quantify_wide(const QuantifyArgs &a, int dtype, cudaStream_t stream)
{
    if (a.rows == 0) return cudaSuccess;
    return launch_wide(a, dtype, stream);
}

}  // namespace ciar
