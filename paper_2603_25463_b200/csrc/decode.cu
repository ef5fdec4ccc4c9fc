// Per-request bookkeeping of the decode loop: initialisation and the position advance that
// follows each verified window.
#include "ciar_internal.h"

namespace ciar {

namespace {

__global__ void decode_init_kernel(ciar_decode_state st, int32_t pos0)
{
    const int64_t total = (int64_t)st.requests * st.seq_len;
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (int64_t i = tid; i < total; i += (int64_t)gridDim.x * blockDim.x) st.tokens_out[i] = -1;
    if (tid < st.requests) st.pos[tid] = pos0;
    if (tid < 8) st.counters[tid] = 0;
}

__device__ __forceinline__ void bump(int64_t *c, int64_t v)
{
    if (v) atomicAdd(reinterpret_cast<unsigned long long *>(c), (unsigned long long)v);
}

// One thread per request: emit the kept draft tokens and the resampled token, advance pos.
__global__ void decode_update_kernel(DecodeUpdateArgs a)
{
    const int32_t q = blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= a.st.requests) return;
    const int32_t p0 = a.st.pos[q];
    const int32_t left = a.st.seq_len - p0;
    if (left <= 0) return;
    const int32_t wlen = left < a.window ? left : a.window;
    const int32_t f = a.first_flag[q];
    const int32_t acc = a.accepted_len[q];
    const int64_t row0 = (int64_t)q * a.st.seq_len + p0;
    for (int32_t j = 0; j < acc; ++j) a.st.tokens_out[row0 + j] = a.tokens[row0 + j];
    int32_t adv = acc;
    if (acc < wlen) {
        a.st.tokens_out[row0 + acc] = a.resampled_token[q];
        adv = acc + 1;
    }
    a.st.pos[q] = p0 + adv;
    int32_t flagged = 0;
    for (int32_t j = 0; j < wlen; ++j) flagged += a.flag[(int64_t)q * a.window + j] != 0;
    const int32_t sent = (a.mode == CIAR_VERIFY_PER_TOKEN) ? flagged : (wlen - f);
    bump(a.st.counters + 0, 1);
    bump(a.st.counters + 1, f < wlen);
    bump(a.st.counters + 2, sent);
    bump(a.st.counters + 3, flagged);
    bump(a.st.counters + 4, acc);
    bump(a.st.counters + 5, acc < wlen);
    bump(a.st.counters + 6, wlen);
    bump(a.st.counters + 7, p0 + adv >= a.st.seq_len);
}

}  // namespace

cudaError_t launch_decode_init(const ciar_decode_state &st, int32_t pos0, cudaStream_t stream)
{
    const int64_t total = (int64_t)st.requests * st.seq_len;
    int64_t blocks = (total + 255) / 256;
    const int64_t need = (st.requests + 255) / 256;
    if (blocks < need) blocks = need;
    if (blocks < 1) blocks = 1;
    if (blocks > 4096) blocks = 4096;
    if (need > 4096) blocks = need;
    decode_init_kernel<<<(unsigned)blocks, 256, 0, stream>>>(st, pos0);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_decode_update(const DecodeUpdateArgs &a, cudaStream_t stream)
{
    if (a.st.requests == 0) return cudaSuccess;
    decode_update_kernel<<<(a.st.requests + 127) / 128, 128, 0, stream>>>(a);
    count_launch();
    return cudaGetLastError();
}

}  // namespace ciar
