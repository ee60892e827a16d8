// Canonical compressed format of Sec. III-A: kept-block column list (Blocked-ELLPACK) plus,
// per kept value, its bf16 payload and a log2(M)-bit zero-based offset inside its M-vector.
#include "crisp_internal.h"

namespace crisp {

namespace {

// One CTA per kept block.  A thread takes whole groups of M elements, so that the N values of
// a group land contiguously; offsets go through a shared-memory bit stream because a field may
// straddle two words (3-bit fields for M = 8).
__global__ void __launch_bounds__(256)
encode_block_kernel(const uint16_t *__restrict__ w, int64_t ld, Geometry g,
                    const int32_t *__restrict__ mask_blk_col, const uint32_t *__restrict__ nm_bits,
                    int32_t *__restrict__ blk_col, uint16_t *__restrict__ vals,
                    uint32_t *__restrict__ idx) {
    extern __shared__ uint32_t s_idx[];
    const int blk = blockIdx.x;                       // rt * kkeep + slot
    const int rt = blk / g.kkeep;
    const int jb = mask_blk_col[blk];
    const int groups = g.groups();
    const int64_t vpb = g.vals_per_block();
    const int words = (int)(vpb * g.idx_bits / 32);
    for (int i = threadIdx.x; i < words; i += blockDim.x) s_idx[i] = 0u;
    if (threadIdx.x == 0) blk_col[blk] = jb;
    __syncthreads();

    uint16_t *vout = vals + (int64_t)blk * vpb;
    const uint32_t group_mask = (1u << g.m) - 1u;
    for (int item = threadIdx.x; item < g.bm * groups; item += blockDim.x) {
        const int r = item / groups, gi = item - r * groups;
        const int64_t row = (int64_t)rt * g.bm + r;
        const int64_t col0 = (int64_t)jb * g.bk + (int64_t)gi * g.m;
        uint32_t bits = (nm_bits[row * g.wpr + (col0 >> 5)] >> (col0 & 31)) & group_mask;
        int o = item * g.n;
        while (bits) {
            const int t = __ffs(bits) - 1;
            bits &= bits - 1;
            const int64_t col = col0 + t;
            vout[o] = (row < g.rows && col < g.k) ? w[row * ld + col] : (uint16_t)0;
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
    __syncthreads();
    uint32_t *iout = idx + (int64_t)blk * words;
    for (int i = threadIdx.x; i < words; i += blockDim.x) iout[i] = s_idx[i];
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
    const size_t smem = (size_t)(g.vals_per_block() * g.idx_bits / 32) * sizeof(uint32_t);
    encode_block_kernel<<<nblocks, 256, smem, st>>>(d_w, ld, g, d_mask_blk_col, d_nm_bits,
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
