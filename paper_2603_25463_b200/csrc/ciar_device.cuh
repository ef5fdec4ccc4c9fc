// Device-side helpers shared by the CIAR kernels: 128-bit row loads with exact widening of
// bf16 / fp32 logits to fp32, block-wide reductions, and the row addressing of the decode loop.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "ciar.h"

namespace ciar {

constexpr int kThreads = 256;  // threads per CTA of the row kernels
constexpr int kWarps = kThreads / 32;
constexpr float kLog2e = 1.4426950408889634f;
constexpr double kLog2eD = 1.4426950408889634074;
constexpr double kLn2D = 0.69314718055994530942;
constexpr float kNegHuge = -1.0e30f;  // exp2 argument floor: keeps 0 * (-inf) out of the sums

// Where the rows of a launch live.  Plain mode: logical row lr is physical row lr.  Decode mode
// (pos != nullptr): logical row lr = q * window + j is position pos[q] + j of request q, physical
// row q * seq_len + pos[q] + j; it does not exist when that position is past the sequence end.
struct RowMap {
    const int32_t *pos;
    int32_t seq_len;
    int32_t window;
};

__device__ __forceinline__ bool map_row(const RowMap &rm, int64_t lr, int64_t &phys)
{
    if (rm.pos == nullptr) {
        phys = lr;
        return true;
    }
    const int64_t q = lr / rm.window;
    const int32_t j = (int32_t)(lr - q * rm.window);
    const int32_t p = rm.pos[q] + j;
    phys = q * (int64_t)rm.seq_len + p;
    return p < rm.seq_len;
}

// Number of rows of the window that starts at logical row w * window (a window cut short by the
// sequence end in decode mode; 0 for a finished request).
__device__ __forceinline__ int32_t window_len(const RowMap &rm, int64_t w)
{
    if (rm.pos == nullptr) return rm.window;
    const int32_t left = rm.seq_len - rm.pos[w];
    return left < 0 ? 0 : (left < rm.window ? left : rm.window);
}

template <typename T>
struct Elem;
template <>
struct Elem<float> {
    static constexpr int kVec = 4;
    static __device__ __forceinline__ float widen(float x) { return x; }
    static __device__ __forceinline__ void load(const float *p, float (&v)[4])
    {
        const float4 t = *reinterpret_cast<const float4 *>(p);
        v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
    }
};
template <>
struct Elem<__nv_bfloat16> {
    static constexpr int kVec = 8;
    static __device__ __forceinline__ float widen(__nv_bfloat16 x) { return __bfloat162float(x); }
    static __device__ __forceinline__ void load(const __nv_bfloat16 *p, float (&v)[8])
    {
        const uint4 t = *reinterpret_cast<const uint4 *>(p);
        v[0] = __uint_as_float(t.x << 16); v[1] = __uint_as_float(t.x & 0xffff0000u);
        v[2] = __uint_as_float(t.y << 16); v[3] = __uint_as_float(t.y & 0xffff0000u);
        v[4] = __uint_as_float(t.z << 16); v[5] = __uint_as_float(t.z & 0xffff0000u);
        v[6] = __uint_as_float(t.w << 16); v[7] = __uint_as_float(t.w & 0xffff0000u);
    }
};

// The valid slice [vb, vb + n) of a row seen as 16-byte vectors.  Vector vi covers row elements
// vi*kVec .. vi*kVec + kVec - 1; the first and last vector may stick out of the slice, and those
// lanes are filled with `pad` without touching memory.
template <typename T>
struct RowView {
    const T *row;  // 16-byte aligned base of the row
    int32_t vb, n;
    int32_t vec_begin, vec_end;

    __device__ __forceinline__ RowView(const T *r, int32_t valid_begin, int32_t valid_count)
        : row(r), vb(valid_begin), n(valid_count)
    {
        constexpr int V = Elem<T>::kVec;
        vec_begin = vb / V;
        vec_end = (vb + n + V - 1) / V;
    }
    // loads vector vi; returns the slice-relative index of its lane 0 (may be negative)
    __device__ __forceinline__ int32_t load(int32_t vi, float (&v)[Elem<T>::kVec], float pad) const
    {
        constexpr int V = Elem<T>::kVec;
        const int32_t e0 = vi * V;
        if (e0 >= vb && e0 + V <= vb + n) {
            Elem<T>::load(row + e0, v);
        } else {
#pragma unroll
            for (int k = 0; k < V; ++k) {
                const int32_t idx = e0 + k;
                v[k] = (idx >= vb && idx < vb + n) ? Elem<T>::widen(row[idx]) : pad;
            }
        }
        return e0 - vb;
    }
};

__device__ __forceinline__ float ex2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ float rcp_approx(float x)
{
    float y;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ float warp_max(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Block-wide max; every thread gets the result.  `scratch` holds kWarps floats.
__device__ __forceinline__ float block_max(float v, float *scratch)
{
    v = warp_max(v);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    __syncthreads();
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    float r = scratch[0];
#pragma unroll
    for (int w = 1; w < kWarps; ++w) r = fmaxf(r, scratch[w]);
    return r;
}

// Block-wide sums of K doubles at once; every thread gets the results.  `scratch` holds
// K * kWarps doubles.  The order of the additions is fixed, so results are deterministic.
template <int K>
__device__ __forceinline__ void block_sum(double (&v)[K], double *scratch)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int k = 0; k < K; ++k) v[k] = warp_sum(v[k]);
    __syncthreads();
    if (lane == 0) {
#pragma unroll
        for (int k = 0; k < K; ++k) scratch[k * kWarps + warp] = v[k];
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < K; ++k) {
        double r = scratch[k * kWarps];
#pragma unroll
        for (int w = 1; w < kWarps; ++w) r += scratch[k * kWarps + w];
        v[k] = r;
    }
}

// Softmax statistics of one row held as (m, z): m = max, z = sum exp(c - m), computed by the
// whole CTA.  The exponent is formed as fma(c, log2e, -m2) with m2 = fl(m * log2e); the common
// offset m * log2e - m2 scales every term alike and is taken out of z again in double.
struct RowStats {
    float m;       // row maximum (-inf if no finite code)
    float m2;      // fl(m * log2e): subtracted inside the exponent
    double z_raw;  // sum of exp2(fma(c, log2e, -m2)) as computed
    double z;      // sum exp(c - m), offset corrected
    double t;      // sum exp(c - m) * (c - m) * log2e (<= 0), offset corrected; for the entropy
};

template <typename T>
__device__ __forceinline__ void row_stats(const RowView<T> &rv, float *fscratch, double *dscratch, RowStats &st)
{
    constexpr int V = Elem<T>::kVec;
    float m = -INFINITY;
    for (int32_t vi = rv.vec_begin + threadIdx.x; vi < rv.vec_end; vi += kThreads) {
        float v[V];
        rv.load(vi, v, -INFINITY);
#pragma unroll
        for (int k = 0; k < V; ++k) m = fmaxf(m, v[k]);
    }
    m = block_max(m, fscratch);
    st.m = m;
    const float m2 = m * kLog2e;
    st.m2 = m2;
    double acc[3] = { 0.0, 0.0, 0.0 };
    // fp32 partial sums over short runs, folded into double so that long rows lose nothing.  Codes equal to the
    // maximum are counted, not summed: their term 2^off is put in exactly below (an approximate exponential
    // of a term near 1 would leave its error, ~1e-7, in ln z of a row that is all but one-hot).
    int32_t vi = rv.vec_begin + threadIdx.x;
    while (vi < rv.vec_end) {
        float z = 0.f, t = 0.f;
        int cnt = 0;
#pragma unroll 4
        for (int it = 0; it < 8 && vi < rv.vec_end; ++it, vi += kThreads) {
            float v[V];
            rv.load(vi, v, -INFINITY);
#pragma unroll
            for (int k = 0; k < V; ++k) {
                const float d = fmaf(v[k], kLog2e, -m2);
                const float e = ex2_approx(d);  // NaN logits stay NaN here and poison z on purpose
                if (v[k] == m) {
                    ++cnt;
                } else {
                    z += e;
                    t = fmaf(e, fmaxf(d, kNegHuge), t);  // -inf logit: e = 0 and 0 * (-1e30) = 0
                }
            }
        }
        acc[0] += (double)z;
        acc[1] += (double)t;
        acc[2] += (double)cnt;
    }
    block_sum<3>(acc, dscratch);
    // exponent actually used: c*log2e_f - m2 = (c - m)*log2e_f + off, off = m*log2e_f - m2, so
    // z_raw = 2^off * z and t_raw = 2^off * (t + off * z); a maximum code's own terms are 2^off and 2^off * off
    // (a +inf maximum makes off NaN, which marks the row as before)
    const double off = (double)m * (double)kLog2e - (double)m2;
    const double scale = exp2(off);
    acc[0] += acc[2] * scale;
    acc[1] += acc[2] * scale * off;
    st.z_raw = acc[0];
    const double unscale = exp2(-off);
    st.z = acc[0] * unscale;
    st.t = acc[1] * unscale - off * st.z;
}

}  // namespace ciar
