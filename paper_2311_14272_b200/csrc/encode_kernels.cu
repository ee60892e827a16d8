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
    clear_header(walks);
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

// Fast path of encode_block_kernel for groups of 4 with one or two kept values (1:4, 2:4) and blocks 64 or 128
// elements deep, which is what the large layers use.  Everything a 4-group needs follows from its four mask
// bits, so it is looked up: a 16-entry table (built per CTA) gives, per nibble, the byte-permute selector that
// picks the two kept bf16 values out of the group's two registers, which of the two slots carry a value, the 2:4
// metadata nibble and the offset field.  Values, offsets, tile slots and metadata are then assembled in
// registers, combined across the lanes that share a 32-bit word with shuffles, and stored once: no shared-memory
// atomics, no zero-filling, a fraction of the instructions of the general kernel (which was bound by instruction
// issue).  Rows are visited so that rows r and r + 8 (whose metadata shares words) sit in the same warp.
// Output identical to encode_block_kernel's.  TILE: 0 or CRISP_PATH_SPARSE (128-row blocks).
template <int N, int TILE>
__global__ void __launch_bounds__(256, 8)
encode_block_m4_kernel(const uint16_t *__restrict__ w, int64_t ld, Geometry g, const int32_t *__restrict__ mask_blk_col,
                       const uint32_t *__restrict__ nm_bits, int32_t *__restrict__ blk_col, uint16_t *__restrict__ vals,
                       uint32_t *__restrict__ idx, uint8_t *__restrict__ image, uint32_t a_bytes, uint32_t entry_bytes,
                       WalkArgs walks) {
    extern __shared__ uint32_t s_buf[];
    __shared__ uint32_t s_lut[16], s_lut_mask[16];
    clear_header(walks);
    if ((int)blockIdx.x < walks.nctas) {
        __shared__ WalkShared s_walks;
        build_walks_body(g, walks, blockIdx.x, s_walks);
        return;
    }
    if (threadIdx.x < 16) {
        // nibble -> slots (a, b), their validity, metadata nibble, first kept position
        const uint32_t nib = threadIdx.x;
        int a = 0, b = 1, va = 0, vb = 0, first = 0;
        if (nib) {
            first = __ffs(nib) - 1;
            const uint32_t rest = nib & (nib - 1);
            if (rest) { a = first; va = 1; b = __ffs(rest) - 1; vb = 1; }
            else if (first == 3) { a = 0; b = 3; vb = 1; }
            else { a = first; va = 1; b = 3; }
        }
        const uint32_t sel = (uint32_t)(2 * a) | ((uint32_t)(2 * a + 1) << 4) | ((uint32_t)(2 * b) << 8) | ((uint32_t)(2 * b + 1) << 12);
        s_lut[nib] = sel | ((uint32_t)(a | (b << 2)) << 16) | ((uint32_t)first << 20);
        s_lut_mask[nib] = (va ? 0x0000FFFFu : 0u) | (vb ? 0xFFFF0000u : 0u);
    }
    const int blk = (int)blockIdx.x - walks.nctas;    // rt * kkeep + slot
    const int rt = blk / g.kkeep;
    const int jb = mask_blk_col[blk];
    const int groups = g.bk / 4;
    const int vpb = g.bm * groups * N;
    const int idx_words = vpb * 2 / 32;
    const int val_words = vpb / 2;
    uint32_t *s_idx = s_buf;                                                        // [idx_words]
    uint32_t *s_val32 = s_buf + idx_words;                                          // [vpb / 2]
    uint8_t *tile = reinterpret_cast<uint8_t *>(s_buf + idx_words + (vpb + 7) / 8 * 4);   // [entry_bytes], 16-byte aligned
    if (threadIdx.x == 0) blk_col[blk] = jb;
    if constexpr (TILE == CRISP_PATH_SPARSE)           // metadata words beyond block_k / 32 per row are never written
        for (uint32_t i = threadIdx.x; i < (entry_bytes - a_bytes) / 16; i += blockDim.x)
            reinterpret_cast<uint4 *>(tile + a_bytes)[i] = make_uint4(0, 0, 0, 0);
    __syncthreads();

    const int L = g.bk / 8;                            // 16-byte loads per row: 8 or 16
    const int lshift = L == 8 ? 3 : 4;
    for (int li = threadIdx.x; li < g.bm * L; li += blockDim.x) {
        const int q = li >> lshift, c8 = li & (L - 1);
        const int r = ((q & 1) << 3) | ((q >> 1) & 7) | (q & ~15);      // rows q, q ^ 1 of the walk are r, r ^ 8
        const int64_t row = (int64_t)rt * g.bm + r;
        const int64_t col8 = (int64_t)jb * g.bk + (int64_t)c8 * 8;
        uint32_t wv[4] = {0u, 0u, 0u, 0u};
        if (row < g.rows && col8 + 8 <= g.k) {
            const uint4 t = __ldg(reinterpret_cast<const uint4 *>(w + row * ld + col8));
            wv[0] = t.x; wv[1] = t.y; wv[2] = t.z; wv[3] = t.w;
        } else if (row < g.rows && col8 < g.k) {
            uint16_t v8[8];
            load_group<8>(w, ld, g.rows, g.k, row, col8, false, v8);
#pragma unroll
            for (int i = 0; i < 4; ++i) wv[i] = (uint32_t)v8[2 * i] | ((uint32_t)v8[2 * i + 1] << 16);
        }
        const uint32_t bits8 = (nm_bits[row * g.wpr + (col8 >> 5)] >> (col8 & 31)) & 0xFFu;
        const uint32_t e0 = s_lut[bits8 & 15u], e1 = s_lut[bits8 >> 4];
        const uint32_t p0 = __byte_perm(wv[0], wv[1], e0 & 0xFFFFu) & s_lut_mask[bits8 & 15u];
        const uint32_t p1 = __byte_perm(wv[2], wv[3], e1 & 0xFFFFu) & s_lut_mask[bits8 >> 4];
        const int item0 = r * groups + 2 * c8;                          // the thread's two groups: item0, item0 + 1
        if constexpr (TILE == CRISP_PATH_SPARSE) {
            // slot pairs of the two 4-groups: compressed columns 4 * c8 .. 4 * c8 + 3, one 8-byte store
            *reinterpret_cast<uint2 *>(tile + (c8 >> 1) * 2048 + r * 16 + (c8 & 1) * 8) = make_uint2(p0, p1);
            // metadata: this thread's two nibbles, the neighbour's (other half of the 16-element chunk) and those
            // of row r ^ 8 make one 32-bit word
            uint32_t mv = (((e0 >> 16) & 15u) | (((e1 >> 16) & 15u) << 4)) << (8 * (c8 & 1) + 16 * (q & 1));
            mv |= __shfl_xor_sync(0xFFFFFFFFu, mv, 1);
            mv |= __shfl_xor_sync(0xFFFFFFFFu, mv, L);
            if (((c8 | q) & 1) == 0) {
                const int lrow = (r & 7) + 8 * ((c8 >> 1) & 1) + 16 * (r >> 4);
                reinterpret_cast<uint32_t *>(tile + a_bytes)[lrow * 4 + (c8 >> 2)] = mv;
            }
        }
        if constexpr (N == 2) {
            // both values of a group are kept values in ascending position: the slot pair is the canonical pair
            *reinterpret_cast<uint2 *>(s_val32 + item0) = make_uint2(p0, p1);
            uint32_t f = (((e0 >> 16) & 15u) | (((e1 >> 16) & 15u) << 4)) << (8 * (c8 & 3));
            f |= __shfl_xor_sync(0xFFFFFFFFu, f, 1);
            f |= __shfl_xor_sync(0xFFFFFFFFu, f, 2);
            if ((c8 & 3) == 0) s_idx[(item0 >> 3)] = f;                  // 4 bits per group: 8 groups per word
        } else {
            // one kept value per group: it sits in slot 0, or in slot 1 when it is the group's last element
            const uint32_t v0 = (p0 & 0xFFFFu) | (p0 >> 16), v1 = (p1 & 0xFFFFu) | (p1 >> 16);
            s_val32[item0 >> 1] = v0 | (v1 << 16);
            uint32_t f = (((e0 >> 20) & 3u) | (((e1 >> 20) & 3u) << 2)) << (4 * (c8 & 7));
            f |= __shfl_xor_sync(0xFFFFFFFFu, f, 1);
            f |= __shfl_xor_sync(0xFFFFFFFFu, f, 2);
            f |= __shfl_xor_sync(0xFFFFFFFFu, f, 4);
            if ((c8 & 7) == 0) s_idx[(item0 >> 4)] = f;                  // 2 bits per group: 16 groups per word
        }
    }
    __syncthreads();
    uint32_t *vout = reinterpret_cast<uint32_t *>(vals + (int64_t)blk * vpb);
    for (int i = threadIdx.x; i < val_words; i += blockDim.x) vout[i] = s_val32[i];
    uint32_t *iout = idx + (int64_t)blk * idx_words;
    for (int i = threadIdx.x; i < idx_words; i += blockDim.x) iout[i] = s_idx[i];
    if constexpr (TILE != 0) {
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
    // groups of 4 with one or two kept values, 64- or 128-deep blocks, 16-byte aligned rows: the table-driven kernel
    const bool fast = g.m == 4 && g.n <= 2 && (g.bk == 64 || g.bk == 128) && vec_ok && tile_kind != CRISP_PATH_DENSE;
#define CRISP_ENCODE_FAST(NV, TV)                                                                            \
    do {                                                                                                     \
        auto kern = encode_block_m4_kernel<NV, TV>;                                                          \
        if (smem > 48 * 1024) {                                                                              \
            cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); \
            if (e != cudaSuccess) return e;                                                                  \
        }                                                                                                    \
        kern<<<nblocks + wa.nctas, 256, smem, st>>>(d_w, ld, g, d_mask_blk_col, d_nm_bits, d_blk_col, d_vals,  \
                                                    d_idx, d_image, a_bytes, entry_bytes, wa);               \
    } while (0)
    if (fast) {
        if (g.n == 2) { if (tile_kind == CRISP_PATH_SPARSE) CRISP_ENCODE_FAST(2, CRISP_PATH_SPARSE); else CRISP_ENCODE_FAST(2, 0); }
        else { if (tile_kind == CRISP_PATH_SPARSE) CRISP_ENCODE_FAST(1, CRISP_PATH_SPARSE); else CRISP_ENCODE_FAST(1, 0); }
    } else if (g.m == 4) {
        if (tile_kind == CRISP_PATH_SPARSE) CRISP_ENCODE_LAUNCH(4, CRISP_PATH_SPARSE);
        else if (tile_kind == CRISP_PATH_DENSE) CRISP_ENCODE_LAUNCH(4, CRISP_PATH_DENSE);
        else CRISP_ENCODE_LAUNCH(4, 0);
    } else {
        if (tile_kind == CRISP_PATH_SPARSE) CRISP_ENCODE_LAUNCH(8, CRISP_PATH_SPARSE);
        else if (tile_kind == CRISP_PATH_DENSE) CRISP_ENCODE_LAUNCH(8, CRISP_PATH_DENSE);
        else CRISP_ENCODE_LAUNCH(8, 0);
    }
#undef CRISP_ENCODE_LAUNCH
#undef CRISP_ENCODE_FAST
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
