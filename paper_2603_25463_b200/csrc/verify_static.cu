// ciar_verify_static: the cloud-side verification for callers that have no way to hand over a
// workspace.  The scratch lives in a fixed array inside the library image instead.
#include <atomic>

#include "ciar_internal.h"

namespace {

// The scratch itself.  Every GPU that loads the library holds these bytes until the process exits.
static __device__ __align__(256) unsigned char g_verify_scratch[CIAR_STATIC_SCRATCH_BYTES];

// Device address of the scratch on the current device.  The array's name is only a handle in host
// code; the address a kernel can use comes from cudaGetSymbolAddress, asked once per device with
// that device current.
cudaError_t scratch_address(void **out)
{
    // (two host threads making the first call on a device at once both look the address up and store the same value)
    static std::atomic<void *> cached[64] = {};
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    void *p = cached[dev].load(std::memory_order_acquire);
    if (p == nullptr) {
        err = cudaGetSymbolAddress(&p, g_verify_scratch);
        if (err != cudaSuccess) return err;
        cached[dev].store(p, std::memory_order_release);
    }
    *out = p;
    return cudaSuccess;
}

}  // namespace

extern "C" ciar_status ciar_verify_static(const ciar_logits_desc *desc, const void *draft_logits, const void *target_logits,
                                          const int32_t *draft_tokens, const uint8_t *flag, const float *draft_row_max,
                                          const float *draft_sum_exp, const float *u_accept, const float *u_resample,
                                          const ciar_verify_params *params, const ciar_verify_out *out, void *stream)
{
    if (!desc || !params) return CIAR_ERR_INVALID_ARG;
    if (desc->rows < 0 || params->window < 1) return CIAR_ERR_INVALID_ARG;
    // more rows than the fixed scratch can serve: refuse before anything is launched
    if (ciar_workspace_bytes(desc->rows, params->window) > (size_t)CIAR_STATIC_SCRATCH_BYTES) return CIAR_ERR_WORKSPACE_TOO_SMALL;
    void *scratch = nullptr;
    if (scratch_address(&scratch) != cudaSuccess) return CIAR_ERR_CUDA;
    // ciar_verify zeroes the part of the scratch that must start at zero (the per-window arrival
    // counters) on the caller's stream before it launches; the rest is written before it is read.
    return ciar_verify(desc, draft_logits, target_logits, draft_tokens, flag, draft_row_max, draft_sum_exp, u_accept,
                       u_resample, params, out, scratch, (size_t)CIAR_STATIC_SCRATCH_BYTES, stream);
}
