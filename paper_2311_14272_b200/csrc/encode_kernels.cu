// Canonical compressed format of Sec. III-A: kept-block column list (Blocked-ELLPACK) plus,
// per kept value, its bf16 payload and a log2(M)-bit zero-based offset inside its M-vector.
#include "crisp_internal.h"

namespace crisp {

namespace {

// The M weights of one group as 16-bit patterns; one vector load when the layout allows it.
template <int M>
__device__ __forceinline__ void load_group(const uint16_t *__restrict__ w, int64_t ld, int rows, int k,
                                           int64_t row, int64_t col0, bool vec_ok, uint16_t v[M]) {
    if (row >= rows || col0 >= k) {
#pragma unroll
        for (int i = 0; i < M; ++i) v[i] = 0;
        return;
    }
    const uint16_t *p = w + row * ld + col0;
    if (vec_ok && col0 + M <= k) {
        if constexpr (M == 4) {
            const uint2 q = __ldg(reinterpret_cast<const uint2 *>(p));
            v[0] = (uint16_t)q.x; v[1] = (uint16_t)(q.x >> 16); v[2] = (uint16_t)q.y; v[3] = (uint16_t)(q.y >> 16);
        } else {
            const uint4 q = __ldg(reinterpret_cast<const uint4 *>(p));
            v[0] = (uint16_t)q.x; v[1] = (uint16_t)(q.x >> 16); v[2] = (uint16_t)q.y; v[3] = (uint16_t)(q.y >> 16);
            v[4] = (uint16_t)q.z; v[5] = (uint16_t)(q.z >> 16); v[6] = (uint16_t)q.w; v[7] = (uint16_t)(q.w >> 16);
        }
    } else {
#pragma unroll
        for (int i = 0; i < M; ++i) v[i] = (col0 + i < k) ? __ldg(p + i) : (uint16_t)0;
    }
}

// One CTA per kept block.  A thread takes whole groups of M elements (one vector load), so that the
// N values of a group land contiguously; values and offsets are staged in shared memory and written
// out with coalesced 16-byte stores.  Offsets go through a bit stream because a field may straddle
// two words (3-bit fields for M = 8).
template <int M>
__global__ void __launch_bounds__(256)
encode_block_kernel(const uint16_t *__restrict__ w, int64_t ld, Geometry g, bool vec_ok,
                    const int32_t *__restrict__ mask_blk_col, const uint32_t *__restrict__ nm_bits,
                    int32_t *__restrict__ blk_col, uint16_t *__restrict__ vals,
                    uint32_t *__restrict__ idx) {
    extern __shared__ uint32_t s_buf[];
    const int blk = blockIdx.x;                       // rt * kkeep + slot
    const int rt = blk / g.kkeep;
    const int jb = mask_blk_col[blk];
    const int groups = g.bk / M;
    const int vpb = g.bm * groups * g.n;
    const int idx_words = vpb * g.idx_bits / 32;
    const int val_words = (vpb + 1) / 2;
    uint32_t *s_idx = s_buf;                          // [idx_words]
    uint16_t *s_val = reinterpret_cast<uint16_t *>(s_buf + idx_words);   // [vpb]
    for (int i = threadIdx.x; i < idx_words; i += blockDim.x) s_idx[i] = 0u;
    if (threadIdx.x == 0) blk_col[blk] = jb;
    __syncthreads();

    for (int item = threadIdx.x; item < g.bm * groups; item += blockDim.x) {
        const int r = item / groups, gi = item - r * groups;
        const int64_t row = (int64_t)rt * g.bm + r;
        const int64_t col0 = (int64_t)jb * g.bk + (int64_t)gi * M;
        uint16_t v[M];
        load_group<M>(w, ld, g.rows, g.k, row, col0, vec_ok, v);
        uint32_t bits = (nm_bits[row * g.wpr + (col0 >> 5)] >> (col0 & 31)) & ((1u << M) - 1u);
        int o = item * g.n;
#pragma unroll
        for (int t = 0; t < M; ++t) {
            if ((bits >> t) & 1u) {
                s_val[o] = v[t];
                const int bit = o * g.idx_bits;
                const uint32_t lo = (uint32_t)t << (bit & 31);
                if (lo) atomicOr(&s_idx[bit >> 5], lo);
                if ((bit & 31) + g.idx_bits > 32) {
                    const uint32_t hi = (uint32_t)t >> (32 - (bit & 31));
                    if (hi) atomicOr(&s_idx[(bit >> 5) + 1], hi);
                }
                ++o;
            }
        }
    }
    __syncthreads();
    // vals_per_block is a multiple of 32 values = 64 bytes, the block's slice starts 64-byte aligned
    uint32_t *vout = reinterpret_cast<uint32_t *>(vals + (int64_t)blk * vpb);
    const uint32_t *s_val32 = reinterpret_cast<const uint32_t *>(s_val);
    for (int i = threadIdx.x; i < val_words; i += blockDim.x) vout[i] = s_val32[i];
    uint32_t *iout = idx + (int64_t)blk * idx_words;
    for (int i = threadIdx.x; i < idx_words; i += blockDim.x) iout[i] = s_idx[i];
}

__global__ void __launch_bounds__(256)
decode_block_kernel(Geometry g, const int32_t *__restrict__ blk_col,
                    const uint16_t *__restrict__ vals, const uint32_t *__restrict__ idx,
                    uint16_t *__restrict__ w, int64_t ld) {
    const int blk = blockIdx.x;
    const int rt = blk / g.kkeep;
    const int jb = blk_col[blk];
    const int groups = g.groups();
    const int64_t vpb = g.vals_per_block();
    const uint16_t *vin = vals + (int64_t)blk * vpb;
    const uint32_t *iin = idx + (int64_t)blk * (vpb * g.idx_bits / 32);
    const uint32_t field = (1u << g.idx_bits) - 1u;
    for (int o = threadIdx.x; o < (int)vpb; o += blockDim.x) {
        const int item = o / g.n;
        const int r = item / groups, gi = item - r * groups;
        const int bit = o * g.idx_bits;
        uint32_t t = iin[bit >> 5] >> (bit & 31);
        if ((bit & 31) + g.idx_bits > 32) t |= iin[(bit >> 5) + 1] << (32 - (bit & 31));
        t &= field;
        const int64_t row = (int64_t)rt * g.bm + r;
        const int64_t col = (int64_t)jb * g.bk + (int64_t)gi * g.m + t;
        if (row < g.rows && col < g.k) w[row * ld + col] = vin[o];
    }
}

}  // namespace

cudaError_t launch_encode_canonical(const uint16_t *d_w, int64_t ld, const Geometry &g,
                                    const int32_t *d_mask_blk_col, const uint32_t *d_nm_bits,
                                    int32_t *d_blk_col, uint16_t *d_vals, uint32_t *d_idx,
                                    cudaStream_t st) {
    const int nblocks = g.nrt * g.kkeep;
    if (nblocks == 0) return cudaSuccess;
    const size_t smem = (size_t)(g.vals_per_block() * g.idx_bits / 32) * sizeof(uint32_t) +
                        (size_t)(g.vals_per_block() + 2) * sizeof(uint16_t);
    // vector loads of a whole group need the group start aligned to its size in every row
    const size_t gbytes = (size_t)g.m * 2;
    const bool vec_ok = (reinterpret_cast<uintptr_t>(d_w) % gbytes == 0) && ((size_t)ld * 2 % gbytes == 0);
    if (g.m == 4)
        encode_block_kernel<4><<<nblocks, 256, smem, st>>>(d_w, ld, g, vec_ok, d_mask_blk_col, d_nm_bits,
                                                            d_blk_col, d_vals, d_idx);
    else
        encode_block_kernel<8><<<nblocks, 256, smem, st>>>(d_w, ld, g, vec_ok, d_mask_blk_col, d_nm_bits,
                                                            d_blk_col, d_vals, d_idx);
    return cudaGetLastError();
}

cudaError_t launch_decode(const Geometry &g, const int32_t *d_blk_col, const uint16_t *d_vals,
                          const uint32_t *d_idx, uint16_t *d_w, int64_t ld, cudaStream_t st) {
    cudaError_t e = cudaMemset2DAsync(d_w, (size_t)ld * 2, 0, (size_t)g.k * 2, (size_t)g.rows, st);
    if (e != cudaSuccess) return e;
    const int nblocks = g.nrt * g.kkeep;
    if (nblocks == 0) return cudaSuccess;
    decode_block_kernel<<<nblocks, 256, 0, st>>>(g, d_blk_col, d_vals, d_idx, d_w, ld);
    return cudaGetLastError();
}

}  // namespace crisp
