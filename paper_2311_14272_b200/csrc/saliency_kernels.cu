// Class-aware saliency score (Sec. III-C "Pruning Metric", Eq. 1): T_w = | (1/H) * sum_i g_i (.) W |, the
// first-order Taylor estimate with the gradient averaged over the H samples of the user's classes.
// The gradients come from the caller's training step, one tensor per sample or mini-batch:
//   crisp_saliency_accumulate  acc += g           (fp32 running sum, once per gradient tensor)
//   crisp_saliency_finish      S = |acc / H * W|   (fp32, the input of crisp_build_mask)
// Both are element-wise streams and HBM-bound: 16-byte accesses where the rows allow it, one grid-stride
// pass with a grid of a whole number of waves.
#include <cuda_bf16.h>

#include "crisp_internal.h"

namespace crisp {
namespace {

constexpr int kSalThreads = 256;

__device__ __forceinline__ float bf16_bits_to_float(uint32_t b) { return __uint_as_float(b << 16); }

// rows of k elements with leading dimensions in elements; kVec: every row start and k are multiples of 4
template <bool kBf16, bool kVec>
__global__ void __launch_bounds__(kSalThreads)
saliency_accumulate_kernel(const void *__restrict__ grad, int64_t ld_g, int rows, int k, float *__restrict__ acc,
                           int64_t ld_a, int first) {
    const int kq = kVec ? k / 4 : k;
    const int64_t total = (int64_t)rows * kq;
    for (int64_t i = (int64_t)blockIdx.x * kSalThreads + threadIdx.x; i < total; i += (int64_t)gridDim.x * kSalThreads) {
        const int r = (int)(i / kq), c = (int)(i - (int64_t)r * kq);
        if constexpr (kVec) {
            float4 g;
            if constexpr (kBf16) {
                const uint2 raw = *reinterpret_cast<const uint2 *>(reinterpret_cast<const uint16_t *>(grad) + r * ld_g + 4 * c);
                g = make_float4(bf16_bits_to_float(raw.x & 0xFFFFu), bf16_bits_to_float(raw.x >> 16),
                                bf16_bits_to_float(raw.y & 0xFFFFu), bf16_bits_to_float(raw.y >> 16));
            } else {
                g = *reinterpret_cast<const float4 *>(reinterpret_cast<const float *>(grad) + r * ld_g + 4 * c);
            }
            float4 *dst = reinterpret_cast<float4 *>(acc + r * ld_a + 4 * c);
            if (first) { *dst = g; continue; }
            float4 a = *dst;
            a.x += g.x; a.y += g.y; a.z += g.z; a.w += g.w;
            *dst = a;
        } else {
            const float g = kBf16 ? bf16_bits_to_float(reinterpret_cast<const uint16_t *>(grad)[r * ld_g + c])
                                  : reinterpret_cast<const float *>(grad)[r * ld_g + c];
            float *dst = acc + r * ld_a + c;
            *dst = first ? g : *dst + g;
        }
    }
}

// |s| as the mask projection reads it (NaN -> 0, Inf -> FLT_MAX), as ordered bits
__device__ __forceinline__ uint32_t canonical_key_bits(float v) {
    return __float_as_uint(fminf(fmaxf(v, 0.f), 3.402823466e+38f));
}

// max_key != nullptr: the layer-wide maximum of the canonical score is left there as well (one atomic per warp),
// which is the first thing the mask projection needs: it then does not have to stream S once more to find it.
template <bool kVec>
__global__ void __launch_bounds__(kSalThreads)
saliency_finish_kernel(const float *__restrict__ acc, int64_t ld_a, const uint16_t *__restrict__ w, int64_t ld_w,
                       int rows, int k, float inv_samples, float *__restrict__ s, int64_t ld_s,
                       uint32_t *__restrict__ max_key) {
    const int kq = kVec ? k / 4 : k;
    const int64_t total = (int64_t)rows * kq;
    uint32_t best = 0u;
    for (int64_t i = (int64_t)blockIdx.x * kSalThreads + threadIdx.x; i < total; i += (int64_t)gridDim.x * kSalThreads) {
        const int r = (int)(i / kq), c = (int)(i - (int64_t)r * kq);
        if constexpr (kVec) {
            const float4 a = *reinterpret_cast<const float4 *>(acc + r * ld_a + 4 * c);
            const uint2 raw = *reinterpret_cast<const uint2 *>(w + r * ld_w + 4 * c);
            float4 o;
            o.x = fabsf(a.x * inv_samples * bf16_bits_to_float(raw.x & 0xFFFFu));
            o.y = fabsf(a.y * inv_samples * bf16_bits_to_float(raw.x >> 16));
            o.z = fabsf(a.z * inv_samples * bf16_bits_to_float(raw.y & 0xFFFFu));
            o.w = fabsf(a.w * inv_samples * bf16_bits_to_float(raw.y >> 16));
            *reinterpret_cast<float4 *>(s + r * ld_s + 4 * c) = o;
            best = max(max(best, canonical_key_bits(o.x)), max(canonical_key_bits(o.y), max(canonical_key_bits(o.z), canonical_key_bits(o.w))));
        } else {
            const float v = fabsf(acc[r * ld_a + c] * inv_samples * bf16_bits_to_float(w[r * ld_w + c]));
            s[r * ld_s + c] = v;
            best = max(best, canonical_key_bits(v));
        }
    }
    if (max_key != nullptr) {
        best = __reduce_max_sync(0xFFFFFFFFu, best);
        if ((threadIdx.x & 31) == 0 && best) atomicMax(max_key, best);
    }
}

int wave_grid(int64_t work_items) {
    int dev = 0, sm_count = 0;                               // asked for at every call: the current device may change
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sm_count <= 0)
        sm_count = 148;
    const int64_t blocks = (work_items + kSalThreads - 1) / kSalThreads;
    const int64_t cap = (int64_t)sm_count * 8;               // 8 resident CTAs of 256 threads per SM
    return (int)(blocks < cap ? (blocks > 0 ? blocks : 1) : cap);
}

bool vec_ok(const void *p, int64_t ld, int elem_bytes, int k) {
    return k % 4 == 0 && (ld * elem_bytes) % (4 * elem_bytes) == 0 && reinterpret_cast<uintptr_t>(p) % (4 * elem_bytes) == 0;
}

}  // namespace
}  // namespace crisp

extern "C" {

CRISP_API crisp_status_t crisp_saliency_accumulate(const void *d_grad, int32_t grad_dtype, int64_t ld_g, int32_t rows,
                                                   int32_t k, float *d_acc, int64_t ld_acc, int32_t first, void *stream) {
    using namespace crisp;
    if (!d_grad || !d_acc || (grad_dtype != 0 && grad_dtype != 1) || (first != 0 && first != 1)) return CRISP_INVALID_ARG;
    if (rows <= 0 || k <= 0 || ld_g < k || ld_acc < k) return CRISP_BAD_SHAPE;
    const int gb = grad_dtype ? 4 : 2;
    if (reinterpret_cast<uintptr_t>(d_grad) % gb || reinterpret_cast<uintptr_t>(d_acc) % 4) return CRISP_INVALID_ARG;
    const bool vec = vec_ok(d_grad, ld_g, gb, k) && vec_ok(d_acc, ld_acc, 4, k);
    const int grid = wave_grid((int64_t)rows * (vec ? k / 4 : k));
    cudaStream_t st = (cudaStream_t)stream;
    if (grad_dtype == 0) {
        if (vec) saliency_accumulate_kernel<true, true><<<grid, kSalThreads, 0, st>>>(d_grad, ld_g, rows, k, d_acc, ld_acc, first);
        else saliency_accumulate_kernel<true, false><<<grid, kSalThreads, 0, st>>>(d_grad, ld_g, rows, k, d_acc, ld_acc, first);
    } else {
        if (vec) saliency_accumulate_kernel<false, true><<<grid, kSalThreads, 0, st>>>(d_grad, ld_g, rows, k, d_acc, ld_acc, first);
        else saliency_accumulate_kernel<false, false><<<grid, kSalThreads, 0, st>>>(d_grad, ld_g, rows, k, d_acc, ld_acc, first);
    }
    return cudaGetLastError() == cudaSuccess ? CRISP_OK : CRISP_CUDA_ERROR;
}

CRISP_API crisp_status_t crisp_saliency_finish(const float *d_acc, int64_t ld_acc, const uint16_t *d_w_bf16, int64_t ld_w,
                                               int32_t rows, int32_t k, int32_t samples, float *d_saliency, int64_t ld_s,
                                               void *stream) {
    return crisp_saliency_finish_max(d_acc, ld_acc, d_w_bf16, ld_w, rows, k, samples, d_saliency, ld_s, nullptr, stream);
}

CRISP_API crisp_status_t crisp_saliency_finish_max(const float *d_acc, int64_t ld_acc, const uint16_t *d_w_bf16,
                                                   int64_t ld_w, int32_t rows, int32_t k, int32_t samples,
                                                   float *d_saliency, int64_t ld_s, void *d_mask_workspace, void *stream) {
    using namespace crisp;
    if (d_mask_workspace && reinterpret_cast<uintptr_t>(d_mask_workspace) % kAlign) return CRISP_INVALID_ARG;
    if (!d_acc || !d_w_bf16 || !d_saliency || samples <= 0) return CRISP_INVALID_ARG;
    if (rows <= 0 || k <= 0 || ld_acc < k || ld_w < k || ld_s < k) return CRISP_BAD_SHAPE;
    if (reinterpret_cast<uintptr_t>(d_acc) % 4 || reinterpret_cast<uintptr_t>(d_w_bf16) % 2 ||
        reinterpret_cast<uintptr_t>(d_saliency) % 4)
        return CRISP_INVALID_ARG;
    const bool vec = vec_ok(d_acc, ld_acc, 4, k) && vec_ok(d_w_bf16, ld_w, 2, k) && vec_ok(d_saliency, ld_s, 4, k);
    const int grid = wave_grid((int64_t)rows * (vec ? k / 4 : k));
    const float inv = 1.0f / (float)samples;
    cudaStream_t st = (cudaStream_t)stream;
    uint32_t *max_key = reinterpret_cast<uint32_t *>(d_mask_workspace);
    if (max_key && cudaMemsetAsync(max_key, 0, kAlign, st) != cudaSuccess) return CRISP_CUDA_ERROR;
    if (vec) saliency_finish_kernel<true><<<grid, kSalThreads, 0, st>>>(d_acc, ld_acc, d_w_bf16, ld_w, rows, k, inv, d_saliency, ld_s, max_key);
    else saliency_finish_kernel<false><<<grid, kSalThreads, 0, st>>>(d_acc, ld_acc, d_w_bf16, ld_w, rows, k, inv, d_saliency, ld_s, max_key);
    return cudaGetLastError() == cudaSuccess ? CRISP_OK : CRISP_CUDA_ERROR;
}

}  // extern "C"
