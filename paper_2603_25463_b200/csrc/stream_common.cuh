// Building blocks of the streaming row kernels: bulk (TMA) global->shared copies completed on an
// mbarrier, bounded mbarrier waits, named CTA barriers, packed fp32x2 arithmetic and warp-wide
// reductions.  sm_100a only.
#pragma once

#include "ciar_device.cuh"

namespace ciar {

__device__ __forceinline__ uint32_t smem_addr(const void *p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ void mbar_init(unsigned long long *bar, uint32_t arrivals)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(arrivals) : "memory");
}

__device__ __forceinline__ void mbar_init_fence()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

// One arrival that also announces `bytes` of asynchronous copy traffic for the current phase.
__device__ __forceinline__ void mbar_arrive_expect_tx(unsigned long long *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(unsigned long long *bar, uint32_t parity)
{
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(smem_addr(bar)), "r"(parity)
        : "memory");
    return done != 0;
}

// Waits for the phase with the given parity to complete, giving up after about `max_cycles` SM
// clocks (a second is ~2e9).  Returns false when it gave up; the phase has then NOT been consumed.
__device__ __forceinline__ bool mbar_wait_bounded(unsigned long long *bar, uint32_t parity, long long max_cycles)
{
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    do {
        if (mbar_try_wait(bar, parity)) return true;
    } while (clock64() - t0 < max_cycles);
    return false;
}

// One plain arrival.
__device__ __forceinline__ void mbar_arrive(unsigned long long *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}

template <bool SLEEP>
__device__ __noinline__ bool wait_phase_slow(unsigned long long *bar, uint32_t parity, volatile int *abort_flag, long long limit)
{
    const long long t0 = clock64();
    for (;;) {
        if (mbar_try_wait(bar, parity)) return true;
        if (SLEEP) __nanosleep(40);
        if (*abort_flag) return false;
        if (clock64() - t0 > limit) {
            *abort_flag = 1;
            return false;
        }
    }
}

// Waits for the phase of the given parity; gives up (and tells everybody) after about `limit` clocks.
// SLEEP: the wait is for data that may take a while (a row in flight); the warp naps between polls.
template <bool SLEEP = true>
__device__ __forceinline__ bool wait_phase(unsigned long long *bar, uint32_t parity, int *abort_flag, long long limit)
{
    if (mbar_try_wait(bar, parity)) return true;
    return wait_phase_slow<SLEEP>(bar, parity, abort_flag, limit);
}

// Bulk copy of `bytes` (a multiple of 16; both addresses 16-byte aligned) from global to this
// CTA's shared memory; completion is signalled on `bar` as `bytes` of transaction count.
__device__ __forceinline__ void bulk_copy_g2s(void *dst_smem, const void *src_gmem, uint32_t bytes, unsigned long long *bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_addr(dst_smem)),
                 "l"(src_gmem), "r"(bytes), "r"(smem_addr(bar))
                 : "memory");
}

// L2 eviction policies for a bulk copy: keep the lines (they are read once more soon) / drop them first.
__device__ __forceinline__ unsigned long long l2_policy_evict_last()
{
    unsigned long long p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}

__device__ __forceinline__ unsigned long long l2_policy_evict_first()
{
    unsigned long long p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}

// bulk_copy_g2s with an L2 eviction policy for the lines it reads
__device__ __forceinline__ void bulk_copy_g2s_hint(void *dst_smem, const void *src_gmem, uint32_t bytes, unsigned long long *bar,
                                                   unsigned long long policy)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
                     smem_addr(dst_smem)),
                 "l"(src_gmem), "r"(bytes), "r"(smem_addr(bar)), "l"(policy)
                 : "memory");
}

// Orders earlier generic-proxy accesses of shared memory before later asynchronous-proxy ones.
__device__ __forceinline__ void fence_proxy_async_smem()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void named_bar_sync(int id, int threads)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

__device__ __forceinline__ void named_bar_arrive(int id, int threads)
{
    asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// Warp-wide float maximum in one instruction (ignores NaN operands).
__device__ __forceinline__ float warp_redux_max(float v)
{
    float r;
    asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(r) : "f"(v));
    return r;
}

__device__ __forceinline__ float warp_sum_f(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Sums two values over the warp with five shuffles: on return lanes 0..15 hold the sum of `a`,
// lanes 16..31 the sum of `b`.
__device__ __forceinline__ float warp_sum_pair(float a, float b, int lane)
{
    const bool upper = (lane & 16) != 0;
    const float send = upper ? a : b;
    float keep = upper ? b : a;
    keep += __shfl_xor_sync(0xffffffffu, send, 16);
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) keep += __shfl_xor_sync(0xffffffffu, keep, o);
    return keep;
}

// 2^x evaluated exactly once, where it is written: the compiler may neither drop nor repeat it, so the
// result is held rather than formed again from its operand later on.
__device__ __forceinline__ float ex2_once(float x)
{
    float y;
    asm volatile("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ float2 f2(float x, float y) { return make_float2(x, y); }
__device__ __forceinline__ float2 f2(float x) { return make_float2(x, x); }

// Two bf16 logits packed in one 32-bit word -> two floats (exact): element 0 is the low half.
__device__ __forceinline__ float2 unpack_bf16x2(uint32_t w)
{
    return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
}

// max of two packed bf16 pairs (NaN operands are ignored)
__device__ __forceinline__ uint32_t bf16x2_max(uint32_t a, uint32_t b)
{
    uint32_t r;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}

// A 16-byte vector of a landed row.  fold_max() folds it into a running maximum (bf16: two packed
// halves, NaN ignored), pairs() widens it to float2 pairs.
template <typename T>
struct Vec;

template <>
struct Vec<__nv_bfloat16> {
    static constexpr int kPairs = 4;
    typedef uint32_t Max;
    static __device__ __forceinline__ Max max_init() { return 0xFF80FF80u; }  // (-inf, -inf)
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
        c[0] = unpack_bf16x2(v.x);
        c[1] = unpack_bf16x2(v.y);
        c[2] = unpack_bf16x2(v.z);
        c[3] = unpack_bf16x2(v.w);
    }
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
};

__device__ __forceinline__ const uint4 &stage_vec(const unsigned char *stage, int vi)
{
    return *reinterpret_cast<const uint4 *>(stage + (size_t)vi * 16);
}

}  // namespace ciar
