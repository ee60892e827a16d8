// Direct SpMM on the canonical format (CUDA cores).  It follows the three steps of Sec. III-E
// literally: stage the activation rows of a kept block (step 1), pick for each stored weight
// the activation its offset names (step 2), multiply-accumulate in fp32 (step 3).  It accepts
// every shape and alignment and serves the layouts the tensor-core kernels cannot take.
#include <cuda_bf16.h>

#include "crisp_internal.h"

namespace crisp {

namespace {

constexpr int kTileN = 64;       // columns of Y per CTA
constexpr int kRowLanes = 4;     // thread rows; thread (ty, tx) owns rows ty, ty+4, ... of the tile

template <int BM, typename OutT>
__global__ void __launch_bounds__(kTileN * kRowLanes)
spmm_direct_kernel(Geometry g, const int32_t *__restrict__ blk_col,
                   const uint16_t *__restrict__ vals, const uint32_t *__restrict__ idx,
                   const uint16_t *__restrict__ x, int64_t ldx, int64_t ncols,
                   OutT *__restrict__ y, int64_t ldy, Epilogue epi) {
    extern __shared__ float xs[];                    // [bk][kTileN]
    const int tx = threadIdx.x % kTileN, ty = threadIdx.x / kTileN;
    const int rt = blockIdx.y;
    const int64_t c0 = (int64_t)blockIdx.x * kTileN;
    const int groups = g.groups();
    const int64_t vpb = g.vals_per_block();
    const uint32_t field = (1u << g.idx_bits) - 1u;
    constexpr int kAcc = BM / kRowLanes;
    float acc[kAcc];
#pragma unroll
    for (int i = 0; i < kAcc; ++i) acc[i] = 0.f;

    for (int slot = 0; slot < g.kkeep; ++slot) {
        const int blk = rt * g.kkeep + slot;
        const int jb = blk_col[blk];
        __syncthreads();
        for (int i = threadIdx.x; i < g.bk * kTileN; i += blockDim.x) {
            const int kr = i / kTileN, c = i - kr * kTileN;
            const int64_t krow = (int64_t)jb * g.bk + kr;
            float v = 0.f;
            if (krow < g.k && c0 + c < ncols)
                v = __uint_as_float((uint32_t)x[krow * ldx + c0 + c] << 16);
            xs[i] = v;
        }
        __syncthreads();
        const uint16_t *vb = vals + (int64_t)blk * vpb;
        const uint32_t *ib = idx + (int64_t)blk * (vpb * g.idx_bits / 32);
#pragma unroll
        for (int i = 0; i < kAcc; ++i) {
            const int r = ty + i * kRowLanes;
            int o = r * groups * g.n;
            float a = acc[i];
            for (int gi = 0; gi < groups; ++gi) {
                for (int v = 0; v < g.n; ++v, ++o) {
                    const int bit = o * g.idx_bits;
                    uint32_t t = __ldg(ib + (bit >> 5)) >> (bit & 31);
                    if ((bit & 31) + g.idx_bits > 32) t |= __ldg(ib + (bit >> 5) + 1) << (32 - (bit & 31));
                    t &= field;
                    const float wv = __uint_as_float((uint32_t)__ldg(vb + o) << 16);
                    a = fmaf(wv, xs[(gi * g.m + (int)t) * kTileN + tx], a);
                }
            }
            acc[i] = a;
        }
    }
    if (c0 + tx < ncols) {
#pragma unroll
        for (int i = 0; i < kAcc; ++i) {
            const int64_t row = (int64_t)rt * BM + ty + i * kRowLanes;
            if (row < g.rows) {
                float v = acc[i];
                if (epi.bias) v += epi.bias[row];
                if (epi.relu) v = fmaxf(v, 0.f);
                if constexpr (sizeof(OutT) == 2)
                    y[row * ldy + c0 + tx] = __bfloat16_as_ushort(__float2bfloat16_rn(v));
                else
                    y[row * ldy + c0 + tx] = v;
            }
        }
    }
}

template <typename OutT>
cudaError_t launch_typed(const Geometry &g, const int32_t *bc, const uint16_t *vals, const uint32_t *idx,
                         const uint16_t *x, int64_t ldx, int64_t ncols, OutT *y, int64_t ldy,
                         const Epilogue &epi, cudaStream_t st) {
    const int64_t gx = (ncols + kTileN - 1) / kTileN;
    const size_t smem = (size_t)g.bk * kTileN * sizeof(float);
    dim3 grid((unsigned)gx, (unsigned)g.nrt);
    const int threads = kTileN * kRowLanes;
    switch (g.bm) {
        case 32: spmm_direct_kernel<32, OutT><<<grid, threads, smem, st>>>(g, bc, vals, idx, x, ldx, ncols, y, ldy, epi); break;
        case 64: spmm_direct_kernel<64, OutT><<<grid, threads, smem, st>>>(g, bc, vals, idx, x, ldx, ncols, y, ldy, epi); break;
        case 128: spmm_direct_kernel<128, OutT><<<grid, threads, smem, st>>>(g, bc, vals, idx, x, ldx, ncols, y, ldy, epi); break;
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_spmm_direct(const Geometry &g, const int32_t *d_blk_col, const uint16_t *d_vals,
                               const uint32_t *d_idx, const uint16_t *d_x, int64_t ldx, int64_t ncols,
                               void *d_y, int64_t ldy, int y_dtype, const Epilogue &epi, cudaStream_t st) {
    if (y_dtype == 0)
        return launch_typed<uint16_t>(g, d_blk_col, d_vals, d_idx, d_x, ldx, ncols,
                                      reinterpret_cast<uint16_t *>(d_y), ldy, epi, st);
    return launch_typed<float>(g, d_blk_col, d_vals, d_idx, d_x, ldx, ncols,
                               reinterpret_cast<float *>(d_y), ldy, epi, st);
}

}  // namespace crisp
