// Discrete top-k quantifier: per row, the k most probable codes by a radix select over the logits' bit
// patterns (8-bit digits, per-warp histograms in shared memory, no sort), then the interval score of the
// quantifier over those k codes alone.
//
// One CTA of 256 threads walks rows blockIdx.x, blockIdx.x + gridDim.x, ...  A row that fits (up to 64 KB) is
// copied to shared memory once and every later sweep reads it there; wider rows are re-read through L1 / L2.
//   1. copy + maximum;
//   2. select: 2 (bf16) or 4 (fp32) digit passes, most significant first.  Each warp counts the digits of the
//      codes whose key still matches the prefix (lanes with equal digits are merged by match.any, so the
//      count is a plain read-modify-write of the merged lanes' leader); the CTA's totals are scanned from the
//      top bin down to the bin that holds the k-th largest key;
//   3. ties: codes equal to the k-th key are taken by lowest index.  Warps own contiguous stretches of the row,
//      count their ties, and the warp in which the quota runs out finds the index where it does;
//   4. softmax sums of the row and of the set (one exponential per code), entropy sum of the set;
//   5. interval sums over the set (bounds from p = e / Z_set), normalisation step and score in double;
//   6. optionally the set's code ids in ascending order (the warps' stretches compacted in order).
#include "ciar_internal.h"
#include "interval_math.cuh"

namespace ciar {

namespace {

constexpr int kTkStageBytes = 64 * 1024;

// Order-preserving 32-bit key of a logit: a larger float has a larger key; -0 and +0 share one key.
__device__ __forceinline__ uint32_t order_key(float x)
{
    uint32_t b = __float_as_uint(x);
    if (x == 0.f) b = 0u;
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

template <typename T>
struct KeyBits;
template <>
struct KeyBits<float> {
    static constexpr int kPasses = 4;
    static constexpr uint32_t kMask = 0xffffffffu;
};
template <>
struct KeyBits<__nv_bfloat16> {
    static constexpr int kPasses = 2;  // the widened value's low 16 bits carry nothing: they are masked off
    static constexpr uint32_t kMask = 0xffff0000u;
};

template <typename T>
__device__ __forceinline__ float key_value(uint32_t key)
{
    const uint32_t b = (key & 0x80000000u) ? (key ^ 0x80000000u) : (~key & KeyBits<T>::kMask);
    return __uint_as_float(b);
}

struct TkShared {
    uint32_t hist[kWarps][256];
    uint32_t total[256];
    float fs[kWarps];
    double ds[5 * kWarps];
    int wcount[kWarps];
    uint32_t prefix;     // key bits fixed so far
    int remaining;       // how many of the codes matching the prefix are still wanted
    int cutoff;          // slice-relative index below which codes equal to the k-th key are taken
    int ties;
};

// Is slice-relative code i with key `key` in the set?
__device__ __forceinline__ bool in_set(uint32_t key, int i, uint32_t kth, int cutoff)
{
    return key > kth || (key == kth && i < cutoff);
}

__device__ __forceinline__ void write_unusable_topk(const ciar_topk_out &o, int64_t row, int k, int status)
{
    const float nanv = __int_as_float(0x7fc00000);
    if (threadIdx.x == 0) {
        if (o.kth_logit) o.kth_logit[row] = nanv;
        if (o.n_above) o.n_above[row] = -1;
        if (o.mass) o.mass[row] = nanv;
        if (o.entropy) o.entropy[row] = nanv;
        if (o.S_lo) o.S_lo[row] = nanv;
        if (o.S_up) o.S_up[row] = nanv;
        if (o.omega) o.omega[row] = nanv;
        if (o.sigma) o.sigma[row] = nanv;
        if (o.score) o.score[row] = nanv;
        if (o.flag) o.flag[row] = 1;
        if (o.row_status) o.row_status[row] = (uint8_t)status;
    }
    if (o.indices)
        for (int j = threadIdx.x; j < k; j += kThreads) o.indices[row * (int64_t)k + j] = -1;
}

template <typename T>
__global__ void __launch_bounds__(kThreads) topk_kernel(TopkArgs a, int staged)
{
    constexpr int V = Elem<T>::kVec;
    constexpr int P = KeyBits<T>::kPasses;
    constexpr uint32_t KM = KeyBits<T>::kMask;
    extern __shared__ __align__(16) unsigned char tk_stage[];
    __shared__ TkShared sh;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int vec_begin = a.vb / V, vec_end = (a.vb + a.n + V - 1) / V, nvec = vec_end - vec_begin;
    const int vw = (nvec + kWarps - 1) / kWarps;  // vectors of a warp's contiguous stretch
    const int seg_b = vec_begin + warp * vw, seg_e = min(vec_end, seg_b + vw);
    const ciar_topk_out &o = a.out;

    for (int64_t row = blockIdx.x; row < a.rows; row += gridDim.x) {
        const T *grow = reinterpret_cast<const T *>(a.logits) + row * a.row_stride;
        __syncthreads();  // the previous row is no longer read
        if (staged) {
            const uint4 *src = reinterpret_cast<const uint4 *>(grow) + vec_begin;
            uint4 *dst = reinterpret_cast<uint4 *>(tk_stage);
            for (int vi = tid; vi < nvec; vi += kThreads) dst[vi] = src[vi];
            __syncthreads();
        }
        // vector vi of the row sits at stage vector vi - vec_begin
        const T *rowp = staged ? reinterpret_cast<const T *>(tk_stage) - (size_t)vec_begin * V : grow;
        const RowView<T> rv(rowp, a.vb, a.n);
        RowStats st;
        row_stats(rv, sh.fs, sh.ds, st);

        int status = 0;
        if (st.m == -INFINITY) status |= CIAR_ROW_NO_FINITE;
        else if (!(st.z_raw < INFINITY) || !(st.z_raw > 0.0)) status |= CIAR_ROW_NAN;
        double r_row = (double)a.r_scalar;
        if (a.radius_mode == CIAR_RADIUS_PER_ROW) r_row = (double)reinterpret_cast<const float *>(a.radius)[row];
        if (!(r_row == r_row)) status |= CIAR_ROW_NAN;
        if (status) {
            write_unusable_topk(o, row, a.k, status);
            continue;
        }

        // ---- 2. radix select of the k-th largest key
        if (tid == 0) {
            sh.prefix = 0u;
            sh.remaining = a.k;
        }
#pragma unroll 1
        for (int pass = 0; pass < P; ++pass) {
            const int shift = 24 - 8 * pass;
            const uint32_t fixed = pass == 0 ? 0u : (0xffffffffu << (shift + 8));
            for (int b = lane; b < 256; b += 32) sh.hist[warp][b] = 0u;
            __syncthreads();
            const uint32_t prefix = sh.prefix;
            for (int v0 = vec_begin + warp * 32; v0 < vec_end; v0 += kThreads) {
                const int vi = v0 + lane;
                float v[V];
                int i0 = 0;
                const bool have = vi < vec_end;
                if (have) i0 = rv.load(vi, v, -INFINITY);
#pragma unroll
                for (int k = 0; k < V; ++k) {
                    const int i = i0 + k;
                    const uint32_t key = have ? (order_key(v[k]) & KM) : 0u;
                    const bool hit = have && i >= 0 && i < a.n && (key & fixed) == prefix;
                    const unsigned act = __ballot_sync(0xffffffffu, hit);
                    if (act == 0u) continue;
                    if (hit) {
                        const uint32_t digit = (key >> shift) & 255u;
                        const unsigned peers = __match_any_sync(act, digit);
                        if (lane == __ffs((int)peers) - 1) sh.hist[warp][digit] += (uint32_t)__popc(peers);
                    }
                    __syncwarp();
                }
            }
            __syncthreads();
            {
                uint32_t t = 0;
#pragma unroll
                for (int w = 0; w < kWarps; ++w) t += sh.hist[w][tid];  // kThreads == 256 bins
                sh.total[tid] = t;
            }
            __syncthreads();
            if (warp == 0) {
                // lane L owns bins 255 - 8L .. 248 - 8L; scan from the top bin down
                const int top = 255 - 8 * lane;
                uint32_t s = 0;
#pragma unroll
                for (int j = 0; j < 8; ++j) s += sh.total[top - j];
                uint32_t incl = s;
#pragma unroll
                for (int d = 1; d < 32; d <<= 1) {
                    const uint32_t up = __shfl_up_sync(0xffffffffu, incl, d);
                    if (lane >= d) incl += up;
                }
                const uint32_t excl = incl - s, rem = (uint32_t)sh.remaining;
                if (excl < rem && rem <= incl) {
                    uint32_t c = excl;
                    for (int j = 0; j < 8; ++j) {
                        const uint32_t t = sh.total[top - j];
                        if (c + t >= rem) {
                            sh.prefix = prefix | ((uint32_t)(top - j) << shift);
                            sh.remaining = (int)(rem - c);
                            sh.ties = (int)t;
                            break;
                        }
                        c += t;
                    }
                }
            }
            __syncthreads();
        }
        const uint32_t kth = sh.prefix;
        const int need = sh.remaining, ties = sh.ties;  // of the `ties` codes equal to the k-th key, `need` are taken

        // ---- 3. where the quota of ties runs out (index order)
        if (ties == need) {
            if (tid == 0) sh.cutoff = a.n;
        } else {
            int cnt = 0;
            for (int v0 = seg_b; v0 < seg_e; v0 += 32) {
                const int vi = v0 + lane;
                if (vi < seg_e) {
                    float v[V];
                    const int i0 = rv.load(vi, v, -INFINITY);
#pragma unroll
                    for (int k = 0; k < V; ++k)
                        cnt += (i0 + k >= 0 && i0 + k < a.n && (order_key(v[k]) & KM) == kth) ? 1 : 0;
                }
            }
            cnt = __reduce_add_sync(0xffffffffu, cnt);
            if (lane == 0) sh.wcount[warp] = cnt;
            __syncthreads();
            int before = 0;
            for (int w = 0; w < warp; ++w) before += sh.wcount[w];
            const int mine = need - before;  // ties this warp's stretch still has to give
            if (mine > 0 && mine <= cnt) {
                int running = 0;
                for (int v0 = seg_b; v0 < seg_e; v0 += 32) {
                    const int vi = v0 + lane;
                    unsigned bits = 0u;
                    int i0 = 0;
                    if (vi < seg_e) {
                        float v[V];
                        i0 = rv.load(vi, v, -INFINITY);
#pragma unroll
                        for (int k = 0; k < V; ++k)
                            if (i0 + k >= 0 && i0 + k < a.n && (order_key(v[k]) & KM) == kth) bits |= 1u << k;
                    }
                    const int c = __popc(bits);
                    int incl = c;
#pragma unroll
                    for (int d = 1; d < 32; d <<= 1) {
                        const int up = __shfl_up_sync(0xffffffffu, incl, d);
                        if (lane >= d) incl += up;
                    }
                    const int tot = __shfl_sync(0xffffffffu, incl, 31);
                    if (running + tot >= mine) {
                        const int excl = running + incl - c;
                        if (excl < mine && mine <= excl + c) {
                            int cc = excl;
                            for (int k = 0; k < V; ++k)
                                if ((bits >> k) & 1u) {
                                    if (++cc == mine) sh.cutoff = i0 + k + 1;
                                }
                        }
                        break;
                    }
                    running += tot;
                }
            }
        }
        __syncthreads();
        const int cutoff = sh.cutoff;

        // ---- 4. softmax sums of the set (codes equal to the row maximum are counted, not summed)
        const float m = st.m, m2 = st.m2;
        double acc[5] = { 0.0, 0.0, 0.0, 0.0, 0.0 };
        for (int vi = vec_begin + tid; vi < vec_end; vi += kThreads) {
            float v[V];
            const int i0 = rv.load(vi, v, -INFINITY);
            float z = 0.f, t = 0.f;
            int cm = 0;
#pragma unroll
            for (int k = 0; k < V; ++k) {
                const int i = i0 + k;
                if (i < 0 || i >= a.n || !in_set(order_key(v[k]) & KM, i, kth, cutoff)) continue;
                if (v[k] == m) {
                    ++cm;
                } else {
                    const float d = fmaf(v[k], kLog2e, -m2);
                    const float e = ex2_approx(d);
                    z += e;
                    t = fmaf(e, fmaxf(d, kNegHuge), t);
                }
            }
            acc[0] += (double)z;
            acc[1] += (double)t;
            acc[2] += (double)cm;
        }
        block_sum<5>(acc, sh.ds);
        const double off = (double)m * (double)kLog2e - (double)m2;
        const double scale = exp2(off), unscale = exp2(-off);
        const double zk_others_raw = acc[0] + (acc[2] - 1.0) * scale;  // everything in the set but one maximum code
        const double zk_raw = zk_others_raw + scale;
        const double zk = zk_raw * unscale;
        const double tk = (acc[1] + acc[2] * scale * off) * unscale - off * zk;
        const double mass = zk_raw / st.z_raw;
        const double entropy = log(zk) - kLn2D * tk / zk;

        // ---- 5. interval sums over the set
        const RadiusConst krow = radius_const(clamp_radius(r_row, a.radius_is_raw, (double)a.r_max));
        const float invz = (float)(1.0 / zk_raw);
        const float pmaxf = (float)(scale / zk_raw), omp_max = (float)(zk_others_raw / zk_raw);
        double sums[5] = { 0, 0, 0, 0, 0 };
        for (int vi = vec_begin + tid; vi < vec_end; vi += kThreads) {
            float v[V];
            const int i0 = rv.load(vi, v, -INFINITY);
            float sA = 0.f, sB = 0.f, sAA = 0.f, sAB = 0.f, sBB = 0.f;
#pragma unroll
            for (int k = 0; k < V; ++k) {
                const int i = i0 + k;
                if (i < 0 || i >= a.n || !in_set(order_key(v[k]) & KM, i, kth, cutoff)) continue;
                float pl, d;
                if (v[k] == m) {
                    bounds_from_p_omp(pmaxf, omp_max, krow, pl, d);
                } else {
                    const float p = ex2_approx(fmaf(v[k], kLog2e, -m2)) * invz;
                    bounds_from_p_omp(p, 1.0f - p, krow, pl, d);
                }
                sA += d;
                sB += pl;
                sAA = fmaf(d, d, sAA);
                sAB = fmaf(d, pl, sAB);
                sBB = fmaf(pl, pl, sBB);
            }
            sums[0] += (double)sA; sums[1] += (double)sB; sums[2] += (double)sAA;
            sums[3] += (double)sAB; sums[4] += (double)sBB;
        }
        block_sum<5>(sums, sh.ds);
        const double nn = (double)a.k;
        const ScoreParts sp = score_parts(sums[0], sums[1], sums[2], sums[3], sums[4], nn, (double)a.lo_cap, (double)a.hi_cap);
        double var = sp.var;
        if (!(var >= 0.1 * sp.mu * sp.mu)) {
            // nearly equal widths: the moment form cancels; sum (delta - mu)^2 over the set directly
            const float fku = (float)sp.k_up, fg = (float)sp.g, fmu = (float)sp.mu;
            double dev[1] = { 0.0 };
            for (int vi = vec_begin + tid; vi < vec_end; vi += kThreads) {
                float v[V];
                const int i0 = rv.load(vi, v, -INFINITY);
                float s = 0.f;
#pragma unroll
                for (int k = 0; k < V; ++k) {
                    const int i = i0 + k;
                    if (i < 0 || i >= a.n || !in_set(order_key(v[k]) & KM, i, kth, cutoff)) continue;
                    float pl, d;
                    if (v[k] == m) {
                        bounds_from_p_omp(pmaxf, omp_max, krow, pl, d);
                    } else {
                        const float p = ex2_approx(fmaf(v[k], kLog2e, -m2)) * invz;
                        bounds_from_p_omp(p, 1.0f - p, krow, pl, d);
                    }
                    const float x = fmaf(fku, d, fg * pl) - fmu;
                    s = fmaf(x, x, s);
                }
                dev[0] += (double)s;
            }
            block_sum<1>(dev, sh.ds);
            var = dev[0] / nn;
        }
        const double sigma = sqrt(var > 0.0 ? var : 0.0);
        const double score = sp.omega * sigma;
        if (tid == 0) {
            if (o.kth_logit) o.kth_logit[row] = key_value<T>(kth);
            if (o.n_above) o.n_above[row] = a.k - need;
            if (o.mass) o.mass[row] = (float)mass;
            if (o.entropy) o.entropy[row] = (float)entropy;
            if (o.S_lo) o.S_lo[row] = (float)sp.S_lo;
            if (o.S_up) o.S_up[row] = (float)sp.S_up;
            if (o.omega) o.omega[row] = (float)sp.omega;
            if (o.sigma) o.sigma[row] = (float)sigma;
            if (o.score) o.score[row] = (float)score;
            if (o.flag) o.flag[row] = (uint8_t)(score > (double)a.tau);
            if (o.row_status) o.row_status[row] = 0;
        }

        // ---- 6. the set's code ids in ascending order
        if (o.indices) {
            int32_t *dst = o.indices + row * (int64_t)a.k;
            int cnt = 0;
            for (int v0 = seg_b; v0 < seg_e; v0 += 32) {
                const int vi = v0 + lane;
                if (vi < seg_e) {
                    float v[V];
                    const int i0 = rv.load(vi, v, -INFINITY);
#pragma unroll
                    for (int k = 0; k < V; ++k)
                        cnt += (i0 + k >= 0 && i0 + k < a.n && in_set(order_key(v[k]) & KM, i0 + k, kth, cutoff)) ? 1 : 0;
                }
            }
            cnt = __reduce_add_sync(0xffffffffu, cnt);
            __syncthreads();  // wcount may still be read by step 3
            if (lane == 0) sh.wcount[warp] = cnt;
            __syncthreads();
            int pos = 0;
            for (int w = 0; w < warp; ++w) pos += sh.wcount[w];
            for (int v0 = seg_b; v0 < seg_e && cnt > 0; v0 += 32) {
                const int vi = v0 + lane;
                unsigned bits = 0u;
                int i0 = 0;
                if (vi < seg_e) {
                    float v[V];
                    i0 = rv.load(vi, v, -INFINITY);
#pragma unroll
                    for (int k = 0; k < V; ++k)
                        if (i0 + k >= 0 && i0 + k < a.n && in_set(order_key(v[k]) & KM, i0 + k, kth, cutoff)) bits |= 1u << k;
                }
                const int c = __popc(bits);
                int incl = c;
#pragma unroll
                for (int d = 1; d < 32; d <<= 1) {
                    const int up = __shfl_up_sync(0xffffffffu, incl, d);
                    if (lane >= d) incl += up;
                }
                int w = pos + incl - c;
                for (int k = 0; k < V; ++k)
                    if ((bits >> k) & 1u) dst[w++] = i0 + k + a.vb;
                pos += __shfl_sync(0xffffffffu, incl, 31);
            }
        }
    }
}

template <typename T>
cudaError_t launch_topk_typed(const TopkArgs &a, cudaStream_t stream)
{
    constexpr int V = Elem<T>::kVec;
    const int nvec = (a.vb + a.n + V - 1) / V - a.vb / V;
    const int staged = (size_t)nvec * 16 <= (size_t)kTkStageBytes ? 1 : 0;
    const size_t smem = staged ? (size_t)nvec * 16 : 0;
    static bool attr_set = false;
    if (!attr_set) {
        const cudaError_t err = cudaFuncSetAttribute(topk_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTkStageBytes);
        if (err != cudaSuccess) return err;
        attr_set = true;
    }
    const int64_t cap = (int64_t)sm_count() * 3;
    const unsigned grid = (unsigned)(a.rows < cap ? a.rows : cap);
    topk_kernel<T><<<grid, kThreads, smem, stream>>>(a, staged);
    count_launch();
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_topk(const TopkArgs &a, int dtype, cudaStream_t stream)
{
    if (a.rows == 0) return cudaSuccess;
    if (dtype == CIAR_F32) return launch_topk_typed<float>(a, stream);
    return launch_topk_typed<__nv_bfloat16>(a, stream);
}

}  // namespace ciar
