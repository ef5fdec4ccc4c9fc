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
#include "quantify_finish.cuh"

namespace ciar {

namespace {

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

// FULL: every thread owns exactly JV vectors (the row has 512 * JV of them).  MAPPED: the rows go through a
// position map (decode mode), so some of them hold nothing to quantify.
template <typename T, int NT, int JV, int MINB, bool FULL, bool MAPPED>
__global__ void __launch_bounds__(NT, MINB) quantify_stream_kernel(const __grid_constant__ QuantifyArgs a)
{
    constexpr int NW = NT / 32;  // warps; as many rows are parked before the CTA finishes them, one per warp
    typedef Vec<T> V;
    constexpr int VEC = Elem<T>::kVec;
    constexpr int NPV = V::kPairs;  // float2 pairs per 16-byte vector
    constexpr int NP = JV * NPV;    // pairs per thread
    constexpr int kStageBytes = NT * JV * 16;
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
        nj = (nvec - tid + NT - 1) / NT;
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
            finish_row(a, p, list, lane, NW);
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
        if constexpr (MAPPED) {
            for (int kk = from; kk < nk; ++kk) {
                int64_t pr;
                if (map_row(a.rm, row_of(kk), pr)) return kk;
            }
            return -1;
        } else {
            return from < nk ? from : -1;
        }
    };
    // Thread 0: the positions past the end of a sequence among rows [from, to) get their outputs, and each hands
    // its stage's turn to the row three further on.  Only called when the stages of those rows are free.
    auto retire_skipped = [&](int from, int to) {
        if constexpr (MAPPED) {
            for (int kk = from; kk < (to < 0 ? nk : to); ++kk) {
                const int64_t lr = row_of(kk);
                if (o.flag) o.flag[lr] = 0;
                if (o.row_status) o.row_status[lr] = 0;
                issue(kk + kQStages);
            }
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
            if (FULL || j < nj) mx = V::fold_max(mx, stage_vec(stage, tid + j * NT));
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
        named_bar_sync(kBarRow, NT);
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
        const float m = warp_redux_max(sh.wmax[par][lane & (NW - 1)]);
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
                    V::pairs(stage_vec(stage, tid + j * NT), c);
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
                const T *v = reinterpret_cast<const T *>(stage + (size_t)(tid + j * NT) * 16);
#pragma unroll
                for (int q = 0; q < VEC; ++q) {
                    const float d = fmaf(Elem<T>::widen(v[q]), kLog2e, -m2);
                    ts = fmaf(ex2_approx(d), fmaxf(d, kNegHuge), ts);
                }
            }
        }
        const float e0 = ex2_approx(fmaf(m, kLog2e, -m2));  // the exponential every maximum got
        if (sh.wmax[par][warp] == m) {
            // This warp owns a maximum.  A term near 1 would cost the small terms their low bits, so the sum of a
            // thread that holds one is formed again without the terms equal to e0 (they come back exactly, as a
            // count), by the whole warp, a code per lane; the lowest such code competes for the arg-max.
            typename V::Max mx = V::max_init();
#pragma unroll
            for (int j = 0; j < JV; ++j)
                if (FULL || j < nj) mx = V::fold_max(mx, stage_vec(stage, tid + j * NT));
            for (unsigned holders = __ballot_sync(0xffffffffu, V::max_value(mx) == m); holders != 0; holders &= holders - 1) {
                const int h = __ffs((int)holders) - 1;
                const int htid = (tid & ~31) + h;
                const int hn = (FULL ? JV : __shfl_sync(0xffffffffu, nj, h)) * VEC;  // the thread's codes
                float zz = 0.f;
                int cnt = 0, first = INT_MAX;
                for (int i = lane; i < hn; i += 32) {
                    const int vi = htid + (i / VEC) * NT;
                    const float c = Elem<T>::widen(reinterpret_cast<const T *>(stage + (size_t)vi * 16)[i % VEC]);
                    const float ev = ex2_approx(fmaf(c, kLog2e, -m2));
                    if (ev == e0) ++cnt; else zz += ev;
                    if (c == m) first = min(first, vi * VEC + i % VEC);
                }
                zz = warp_sum_f(zz);
                cnt = __reduce_add_sync(0xffffffffu, cnt);
                first = __reduce_min_sync(0xffffffffu, first);
                if (lane == h) zs = zz;
                if (lane == 0) {
                    if (cnt > 0) atomicAdd(&sh.nmax[it & 3], cnt);
                    if (first != INT_MAX) atomicMin(&sh.argmin[par], first);
                }
            }
        }
        {
            const float zt = warp_sum_pair(zs, ts, lane);  // lanes 0..15: z, lanes 16..31: t
            if ((lane & 15) == 0) pk.wsum[warp][lane >> 2] = zt;
        }
        __syncwarp();
        named_bar_sync(kBarRow, NT);
        if (sh.abort) {
            aborted = true;
            break;
        }
        float z = pk.wsum[lane & (NW - 1)][0];
#pragma unroll
        for (int ofs = NW / 2; ofs > 0; ofs >>= 1) z += __shfl_xor_sync(0xffffffffu, z, ofs);
        const int nmax = sh.nmax[it & 3];
        z = fmaf((float)nmax, e0, z);
        const float rho = pk.rho;

        int status = 0;
        if (!(m > -INFINITY) || !(z > 0.f) || !(z < INFINITY)) {
            // an unusable row (NaN / +inf logit, no finite logit): classify it from the landed bytes
            // exactly as the row-status bits are defined
            if (tid == 0) sh.bad_nan = sh.bad_finite = 0;
            named_bar_sync(kBarRow, NT);
            int has_nan = 0, has_finite = 0;
            for (int j = 0; j < nj; ++j) {
                const T *v = reinterpret_cast<const T *>(stage + (size_t)(tid + j * NT) * 16);
#pragma unroll
                for (int q = 0; q < VEC; ++q) {
                    const float c = Elem<T>::widen(v[q]);
                    if (!(c == c) || c == INFINITY) has_nan = 1;
                    if (c == c && fabsf(c) != INFINITY) has_finite = 1;
                }
            }
            if (has_nan) sh.bad_nan = 1;
            if (has_finite) sh.bad_finite = 1;
            named_bar_sync(kBarRow, NT);
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
                const T *v = reinterpret_cast<const T *>(stage + (size_t)(tid + j * NT) * 16);
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
            named_bar_sync(kBarRow, NT);
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
        if (++filled == NW || long_pending) {
            finish_parked(filled);
            filled = 0;
        }
        k = kn;
        ++it;
        if (MAPPED && k >= 0 && !ahead) {  // the next row's first sweep could not run ahead: it runs here, with a barrier of its own
            first_sweep(k, it);
            __syncwarp();
            named_bar_sync(kBarRow, NT);
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

template <typename T, int NT, int JV, int MINB, bool FULL, bool MAPPED>
cudaError_t launch_one(const QuantifyArgs &a, cudaStream_t stream)
{
    constexpr size_t smem = (size_t)kQStages * NT * JV * 16 + sizeof(QShared);
    static bool configured[64] = {};
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!configured[dev]) {
        err = cudaFuncSetAttribute(quantify_stream_kernel<T, NT, JV, MINB, FULL, MAPPED>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   (int)smem);
        if (err != cudaSuccess) return err;
        configured[dev] = true;
    }
    const int64_t cap = (int64_t)sm_count() * MINB;
    const unsigned grid = (unsigned)(a.rows < cap ? a.rows : cap);
    quantify_stream_kernel<T, NT, JV, MINB, FULL, MAPPED><<<grid, NT, smem, stream>>>(a);
    count_launch();
    return cudaGetLastError();
}

template <typename T, int NT, int JV, int MINB>
cudaError_t launch_jv(const QuantifyArgs &a, cudaStream_t stream)
{
    const int nvec = a.n / Elem<T>::kVec;
    const bool mapped = a.rm.pos != nullptr;
    if (nvec == NT * JV) return mapped ? launch_one<T, NT, JV, MINB, true, true>(a, stream) : launch_one<T, NT, JV, MINB, true, false>(a, stream);
    return mapped ? launch_one<T, NT, JV, MINB, false, true>(a, stream) : launch_one<T, NT, JV, MINB, false, false>(a, stream);
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
        if (a.n <= 4096) return launch_jv<float, 512, 2, 2>(a, stream);
        if (a.n <= 8192) return launch_jv<float, 512, 4, 2>(a, stream);
        return launch_jv<float, 512, 8, 1>(a, stream);
    }
    // Short rows go to CTAs of 256 threads, three per SM: a thread then still owns 16 or 32 codes of a row, over
    // which the per-row work (reductions, barrier, parking) is spread.
    if (a.n <= 4096) return launch_jv<__nv_bfloat16, 256, 2, 3>(a, stream);
    if (a.n <= 8192) return launch_jv<__nv_bfloat16, 256, 4, 3>(a, stream);
    return launch_jv<__nv_bfloat16, 512, 4, 2>(a, stream);
}

}  // namespace ciar
