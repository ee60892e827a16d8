// Canonical compressed format of Sec. III-A: kept-block column list (Blocked-ELLPACK) plus,
// per kept value, its bf16 payload and a log2(M)-bit zero-based offset inside its M-vector.
#include "crisp_internal.h"
#include "walks.cuh"

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
// TILE selects what else the CTA emits for 128-row blocks (one kept block = one tensor-core tile):
// 0 nothing, CRISP_PATH_DENSE the zero-expanded tile, CRISP_PATH_SPARSE the 2:4 compressed tile with
// its metadata (layouts: see the execution-image kernels of the tensor-core SpMM).
template <int M, int TILE>
__global__ void __launch_bounds__(256, 8)
encode_block_kernel(const uint16_t *__restrict__ w, int64_t ld, Geometry g, bool vec_ok,
                    const int32_t *__restrict__ mask_blk_col, const uint32_t *__restrict__ nm_bits,
                    int32_t *__restrict__ blk_col, uint16_t *__restrict__ vals,
                    uint32_t *__restrict__ idx, uint8_t *__restrict__ image, uint32_t a_bytes,
                    uint32_t entry_bytes, WalkArgs walks) {
    extern __shared__ uint32_t s_buf[];
    // The first walks.nctas CTAs build the walk lists of the tensor-core kernel instead of encoding a block:
    // that needs only the mask's block list, so it overlaps the encoding instead of following it.
    if ((int)blockIdx.x < walks.nctas) {
        __shared__ WalkShared s_walks;
        build_walks_body(g, walks, blockIdx.x, s_walks);
        return;
    }
    const int blk = (int)blockIdx.x - walks.nctas;   // rt * kkeep + slot
    const int rt = blk / g.kkeep;
    const int jb = mask_blk_col[blk];
    const int groups = g.bk / M;
    const int vpb = g.bm * groups * g.n;
    const int idx_words = vpb * g.idx_bits / 32;
    const int val_words = (vpb + 1) / 2;
    uint32_t *s_idx = s_buf;                          // [idx_words]
    uint16_t *s_val = reinterpret_cast<uint16_t *>(s_buf + idx_words);   // [vpb]
    uint8_t *tile = reinterpret_cast<uint8_t *>(s_buf + idx_words + (vpb + 7) / 8 * 4);   // [entry_bytes], 16-byte aligned
    for (int i = threadIdx.x; i < idx_words; i += blockDim.x) s_idx[i] = 0u;
    if constexpr (TILE != 0)
        for (uint32_t i = threadIdx.x; i < entry_bytes / 16; i += blockDim.x)
            reinterpret_cast<uint4 *>(tile)[i] = make_uint4(0, 0, 0, 0);
    if (threadIdx.x == 0) blk_col[blk] = jb;
    __syncthreads();

    // a thread takes eight consecutive elements of a row (one 16-byte load: two groups of 4 or one of 8)
    constexpr int kGroupsPerLoad = 8 / M;
    const int loads_per_row = g.bk / 8;
    for (int li = threadIdx.x; li < g.bm * loads_per_row; li += blockDim.x) {
      const int r = li / loads_per_row, c8 = li - r * loads_per_row;
      const int64_t row = (int64_t)rt * g.bm + r;
      const int64_t col8 = (int64_t)jb * g.bk + (int64_t)c8 * 8;
      uint16_t v8[8];
      load_group<8>(w, ld, g.rows, g.k, row, col8, vec_ok, v8);
      const uint32_t bits8 = (nm_bits[row * g.wpr + (col8 >> 5)] >> (col8 & 31)) & 0xFFu;
#pragma unroll
      for (int sub = 0; sub < kGroupsPerLoad; ++sub) {
        const int gi = c8 * kGroupsPerLoad + sub;
        const int item = r * groups + gi;
        const uint16_t *v = v8 + sub * M;
        const uint32_t bits = (bits8 >> (sub * M)) & ((1u << M) - 1u);
        if constexpr (TILE == CRISP_PATH_DENSE) {
#pragma unroll
            for (int t = 0; t < M; ++t)
                if ((bits >> t) & 1u) {
                    const int k = gi * M + t;
                    *reinterpret_cast<uint16_t *>(tile + (k >> 3) * 2048 + r * 16 + (k & 7) * 2) = v[t];
                }
        } else if constexpr (TILE == CRISP_PATH_SPARSE) {
            uint32_t *meta = reinterpret_cast<uint32_t *>(tile + a_bytes);
#pragma unroll
            for (int q = 0; q < M / 4; ++q) {                // aligned 4-groups: at most two kept values each
                const uint32_t qb = (bits >> (4 * q)) & 0xFu;
                int p0 = 0, p1 = 1;
                uint16_t v0 = 0, v1 = 0;
                if (qb) {
                    const int first = __ffs(qb) - 1;
                    const uint32_t rest = qb & (qb - 1);
                    if (rest) { p0 = first; v0 = v[4 * q + first]; p1 = __ffs(rest) - 1; v1 = v[4 * q + p1]; }
                    else if (first == 3) { p0 = 0; p1 = 3; v1 = v[4 * q + 3]; }
                    else { p0 = first; v0 = v[4 * q + first]; p1 = 3; }
                }
                const int k0 = gi * M + 4 * q, c0 = k0 >> 1;  // compressed column of the first slot (even)
                *reinterpret_cast<uint32_t *>(tile + (c0 >> 3) * 2048 + r * 16 + (c0 & 7) * 2) =
                    (uint32_t)v0 | ((uint32_t)v1 << 16);
                const int lrow = (r & 7) + 8 * ((k0 >> 4) & 1) + 16 * (r >> 4);
                atomicOr(&meta[lrow * 4 + (k0 >> 5)], ((uint32_t)p0 | ((uint32_t)p1 << 2)) << ((k0 & 15) + 16 * ((r >> 3) & 1)));
            }
        }
        // values in ascending position; the group's offsets are gathered in a register and merged into
        // the shared bit stream with one atomic (two if the field straddles a word)
        constexpr int kIdxBits = M == 4 ? 2 : 3;
        int o = item * g.n;
        const int bit0 = o * kIdxBits;
        uint32_t field = 0u;
        int cnt = 0;
#pragma unroll
        for (int t = 0; t < M; ++t) {
            if ((bits >> t) & 1u) {
                s_val[o + cnt] = v[t];
                field |= (uint32_t)t << (kIdxBits * cnt);
                ++cnt;
            }
        }
        if (field) {
            const int sh = bit0 & 31;
            atomicOr(&s_idx[bit0 >> 5], field << sh);
            if (sh + kIdxBits * cnt > 32) atomicOr(&s_idx[(bit0 >> 5) + 1], field >> (32 - sh));
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
    if constexpr (TILE != 0) {
        // with 128-row blocks the walk list of a CTA tile is its row tile's kept list: entry = blk
        uint4 *out = reinterpret_cast<uint4 *>(image + (int64_t)blk * entry_bytes);
        for (uint32_t i = threadIdx.x; i < entry_bytes / 16; i += blockDim.x) out[i] = reinterpret_cast<uint4 *>(tile)[i];
    }
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
                                    int tile_kind, uint8_t *d_image, uint32_t a_bytes, uint32_t entry_bytes,
                                    const WalkArgs *walks, cudaStream_t st) {
    const int nblocks = g.nrt * g.kkeep;
    if (nblocks == 0) return cudaSuccess;
    WalkArgs wa = {};
    if (walks) wa = *walks;
    const size_t vpb = (size_t)g.vals_per_block();
    size_t smem = (vpb * g.idx_bits / 32) * sizeof(uint32_t) + (vpb + 7) / 8 * 16 + 16;
    if (tile_kind != 0) smem += entry_bytes;
    // the 16-byte loads of eight elements need every row to start 16-byte aligned (block columns are multiples of 32)
    const size_t gbytes = 16;
    const bool vec_ok = (reinterpret_cast<uintptr_t>(d_w) % gbytes == 0) && ((size_t)ld * 2 % gbytes == 0);
#define CRISP_ENCODE_LAUNCH(MV, TV)                                                                          \
    do {                                                                                                     \
        auto kern = encode_block_kernel<MV, TV>;                                                             \
        if (smem > 48 * 1024) {                                                                              \
            cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); \
            if (e != cudaSuccess) return e;                                                                  \
        }                                                                                                    \
        kern<<<nblocks + wa.nctas, 256, smem, st>>>(d_w, ld, g, vec_ok, d_mask_blk_col, d_nm_bits, d_blk_col, \
                                                     d_vals, d_idx, d_image, a_bytes, entry_bytes, wa);      \
    } while (0)
    if (g.m == 4) {
        if (tile_kind == CRISP_PATH_SPARSE) CRISP_ENCODE_LAUNCH(4, CRISP_PATH_SPARSE);
        else if (tile_kind == CRISP_PATH_DENSE) CRISP_ENCODE_LAUNCH(4, CRISP_PATH_DENSE);
        else CRISP_ENCODE_LAUNCH(4, 0);
    } else {
        if (tile_kind == CRISP_PATH_SPARSE) CRISP_ENCODE_LAUNCH(8, CRISP_PATH_SPARSE);
        else if (tile_kind == CRISP_PATH_DENSE) CRISP_ENCODE_LAUNCH(8, CRISP_PATH_DENSE);
        else CRISP_ENCODE_LAUNCH(8, 0);
    }
#undef CRISP_ENCODE_LAUNCH
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
