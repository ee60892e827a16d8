// crisp_build_mask_static: mask projection for callers that cannot obtain device scratch memory.
//
// crisp_build_mask needs a small scratch workspace (the layer-wide maximum and one 64-bit score
// per coarse block) that its caller normally allocates.  Code that runs where allocation is
// off-limits has no way to provide it: a plug-in called inside a host framework that owns all
// device memory, a real-time or safety-certified loop that must not call the allocator after
// start-up, a callback running while another thread holds the allocator, or a process whose
// memory pool is already fully committed.  For those callers the scratch lives in the
// fixed-size device array below, which is part of the library image: every GPU that loads the
// library carries these CRISP_STATIC_SCRATCH_BYTES until the process exits, whether or not
// this entry point is ever used.
#include "crisp_internal.h"

namespace {

// The scratch itself.  In host code this name is only a handle for the runtime, not a device
// address; the address a kernel can use comes from cudaGetSymbolAddress (below).
static __device__ __align__(256) unsigned char g_static_scratch[CRISP_STATIC_SCRATCH_BYTES];

// Device address of g_static_scratch on the current device.  Asked for at every call: the lookup is cheap
// once the library's module is loaded on the device (the first call loads it), and an address kept
// across calls would go stale after cudaDeviceReset or in a second context on the same device.
crisp_status_t scratch_for_current_device(void **out) {
    void *p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return CRISP_CUDA_ERROR;
    *out = p;
    return CRISP_OK;
}

}  // namespace

extern "C" crisp_status_t crisp_build_mask_static(const float *d_saliency, int64_t ld_s,
                                                  const crisp_layer_desc_t *desc, void *d_mask_buf,
                                                  void *stream, crisp_mask_t *out) {
    if (out) *out = nullptr;
    size_t mask_bytes = 0, workspace_bytes = 0;
    crisp_status_t s = crisp_mask_sizes(desc, &mask_bytes, &workspace_bytes);
    if (s != CRISP_OK) return s;
    if (workspace_bytes > (size_t)CRISP_STATIC_SCRATCH_BYTES) return CRISP_BUFFER_TOO_SMALL;
    void *scratch = nullptr;
    s = scratch_for_current_device(&scratch);
    if (s != CRISP_OK) return s;
    // crisp_build_mask zeroes the whole workspace on `stream` before its first kernel, so what
    // an earlier call left in the shared array cannot leak into this one.
    return crisp_build_mask(d_saliency, ld_s, desc, d_mask_buf, scratch, stream, out);
}
