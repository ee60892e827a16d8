// Mask projection kernels: saliency -> hybrid (block + N:M) mask.
//
// Algorithm 1 of the paper, restricted to one layer with the block keep count given:
//   K-M1a per group of M: keep the N largest (fine-grained N:M step), and the layer-wide maximum
//         of the canonical saliency (it sets the fixed-point scale): one pass over S from HBM
//   K-M1b block scores s_j = sum |T_w| as exact fixed-point integers: second pass over S, which
//         for layers up to the size of L2 is served from there
//   K-M2  per row of the block grid: keep the kkeep highest-scored blocks and clear the
//         bits of the pruned ones (blocks keep their positions)
// Coalesced 32-byte-per-lane accesses; K-M1a is bound by HBM bandwidth.
#include "crisp_internal.h"

namespace crisp {

namespace {

constexpr int kScoreFractionBits = 40;
constexpr int kM1Threads = 256;
constexpr int kM1ChunkK = 256;           // k-elements covered by one warp pass (32 lanes x 8)

// |s| as an order-preserving uint32 key: NaN -> 0, Inf -> FLT_MAX.
__device__ __forceinline__ uint32_t canonical_key(float s) {
    uint32_t u = __float_as_uint(s) & 0x7FFFFFFFu;
    if (u > 0x7F800000u) return 0u;
    if (u == 0x7F800000u) return 0x7F7FFFFFu;
    return u;
}

// Raw bits of eight consecutive saliency values; the caller guarantees row < rows, k0 + 8 <= k and
// 16-byte alignment.  Kept free of branches so that several of these can be in flight per lane.
__device__ __forceinline__ void load8_raw(const float *__restrict__ s, int64_t ld, int64_t row, int64_t k0,
                                          uint32_t key[8]) {
    const uint4 *p = reinterpret_cast<const uint4 *>(s + row * ld + k0);
    const uint4 a = __ldg(p), b = __ldg(p + 1);
    key[0] = a.x; key[1] = a.y; key[2] = a.z; key[3] = a.w;
    key[4] = b.x; key[5] = b.y; key[6] = b.z; key[7] = b.w;
}
// |s| with NaN -> 0 and Inf -> FLT_MAX in two instructions: max(|s|, 0) drops a NaN (the maximum of a NaN and a
// number is the number), min(., FLT_MAX) caps infinity; -0 becomes +0, denormals pass unchanged.
__device__ __forceinline__ uint32_t canonical_bits(uint32_t u) {
    return __float_as_uint(fminf(fmaxf(fabsf(__uint_as_float(u)), 0.f), 3.402823466e+38f));
}

// Eight consecutive saliency values of one row, zero beyond the matrix.
__device__ __forceinline__ void load8(const float *__restrict__ s, int64_t ld, int rows, int k,
                                      int64_t row, int64_t k0, bool vec_ok, uint32_t key[8]) {
    if (row >= rows || k0 >= k) {
#pragma unroll
        for (int i = 0; i < 8; ++i) key[i] = 0u;
        return;
    }
    const float *p = s + row * ld + k0;
    if (vec_ok && k0 + 8 <= k) {
        const float4 a = __ldg(reinterpret_cast<const float4 *>(p));
        const float4 b = __ldg(reinterpret_cast<const float4 *>(p) + 1);
        key[0] = canonical_key(a.x); key[1] = canonical_key(a.y);
        key[2] = canonical_key(a.z); key[3] = canonical_key(a.w);
        key[4] = canonical_key(b.x); key[5] = canonical_key(b.y);
        key[6] = canonical_key(b.z); key[7] = canonical_key(b.w);
    } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) key[i] = (k0 + i < k) ? canonical_key(__ldg(p + i)) : 0u;
    }
}

// Exponent of a positive finite float given by its bits (ilogb), denormals included.
__device__ __forceinline__ int key_exponent(uint32_t key) {
    const int e = (int)(key >> 23);
    return e ? e - 127 : (31 - __clz(key)) - 149;
}

// floor(value * 2^(40 - e_max)) for a non-negative finite float given by its bits, in integer
// arithmetic: the mantissa shifted by the exponent difference (exact, no rounding mode involved).
__device__ __forceinline__ unsigned long long fixed_point_score(uint32_t key, int e_max) {
    const int e = (int)(key >> 23);
    const uint32_t mant = e ? ((key & 0x7FFFFFu) | 0x800000u) : key;           // value = mant * 2^(max(e,1) - 150)
    const int sh = max(e, 1) - 150 + kScoreFractionBits - e_max;                 // <= 17 because value <= layer maximum
    const uint32_t down = mant >> min(max(-sh, 0), 31);                          // mant < 2^24: shifts >= 24 give 0
    const int up = max(sh, 0);                                                   // only one of the two shifts is non-zero
    return ((unsigned long long)__funnelshift_l(down, 0u, up) << 32) | (unsigned long long)(down << up);
}

// Bit i of the result is set iff element i is among the N largest of its group of M
// (ties to the lower index).  M is 4 or 8; the 8 keys hold two groups or one.
// For i < j, element i beats element j iff key[i] >= key[j].
template <int M>
__device__ __forceinline__ uint32_t top_n_bits(const uint32_t key[8], int n) {
    uint32_t bits = 0u;
#pragma unroll
    for (int g = 0; g < 8 / M; ++g) {
        int rank[M];
#pragma unroll
        for (int i = 0; i < M; ++i) rank[i] = 0;
#pragma unroll
        for (int i = 0; i < M; ++i)
#pragma unroll
            for (int j = i + 1; j < M; ++j) {
                const int i_wins = key[g * M + i] >= key[g * M + j];
                rank[j] += i_wins;
                rank[i] += 1 - i_wins;
            }
#pragma unroll
        for (int i = 0; i < M; ++i) bits |= (rank[i] < n ? 1u : 0u) << (g * M + i);
    }
    return bits;
}

// Groups of 4: the six pairwise outcomes index a 64-entry table of keep masks (built per CTA for
// the layer's n by keep_mask_of_outcomes), which replaces the rank arithmetic.
__device__ __forceinline__ uint32_t outcomes4(const uint32_t *k) {
    return (uint32_t)(k[0] >= k[1]) | ((uint32_t)(k[0] >= k[2]) << 1) | ((uint32_t)(k[0] >= k[3]) << 2) |
           ((uint32_t)(k[1] >= k[2]) << 3) | ((uint32_t)(k[1] >= k[3]) << 4) | ((uint32_t)(k[2] >= k[3]) << 5);
}
__device__ __forceinline__ uint32_t keep_mask_of_outcomes(uint32_t o, int n) {
    const int w01 = o & 1, w02 = (o >> 1) & 1, w03 = (o >> 2) & 1, w12 = (o >> 3) & 1, w13 = (o >> 4) & 1,
              w23 = (o >> 5) & 1;
    const int r0 = (1 - w01) + (1 - w02) + (1 - w03);
    const int r1 = w01 + (1 - w12) + (1 - w13);
    const int r2 = w02 + w12 + (1 - w23);
    const int r3 = w03 + w13 + w23;
    return (uint32_t)(r0 < n) | ((uint32_t)(r1 < n) << 1) | ((uint32_t)(r2 < n) << 2) | ((uint32_t)(r3 < n) << 3);
}

constexpr int kM1Rows = 32;              // rows per work item of K-M1a / K-M1b (divides every block height)
constexpr int kM1RowsPerWarp = kM1Rows / (kM1Threads / 32);

// One work item = 32 rows x 256 k-elements.  Warp w takes rows 4w..4w+3 (all loads issued first); lane l owns
// the 8 elements at k = chunk*256 + 8*l of each row, so a lane stays inside one block column.  Items are dealt
// out to a grid of resident CTAs (grid-stride), chunk fastest, so that a CTA streams along rows.
struct M1Item { int64_t row0; int chunk; };
__device__ __forceinline__ M1Item m1_item(int64_t it, int chunks) {
    M1Item x;
    const int64_t rg = it / chunks;
    x.chunk = (int)(it - rg * chunks);
    x.row0 = rg * kM1Rows;
    return x;
}

// The 8 canonical keys of the lane's elements of row `row` (zero beyond the matrix).
__device__ __forceinline__ void m1_load_rows(const float *__restrict__ s, int64_t ld, const Geometry &g, bool vec_ok,
                                             const M1Item &x, int warp, int64_t k0, uint32_t key[kM1RowsPerWarp][8]) {
    if (vec_ok && x.row0 + kM1Rows <= g.rows && (int64_t)(x.chunk + 1) * kM1ChunkK <= g.k) {   // interior item
#pragma unroll
        for (int i = 0; i < kM1RowsPerWarp; ++i) load8_raw(s, ld, x.row0 + warp * kM1RowsPerWarp + i, k0, key[i]);
#pragma unroll
        for (int i = 0; i < kM1RowsPerWarp; ++i)
#pragma unroll
            for (int j = 0; j < 8; ++j) key[i][j] = canonical_bits(key[i][j]);
    } else {
#pragma unroll
        for (int i = 0; i < kM1RowsPerWarp; ++i)
            load8(s, ld, g.rows, g.k, x.row0 + warp * kM1RowsPerWarp + i, k0, vec_ok, key[i]);
    }
}

// K-M1a: the fine-grained N:M step (which does not depend on the score scale) and the layer maximum (which fixes
// the scale) in ONE pass over S, the pass that comes from HBM: per group of M the N largest are marked, a lane
// stores its eight mask bits as one byte, and the largest key goes to max_key (one atomic per CTA).
// find_max = false when the caller already knows the maximum.
template <int M>
__global__ void __launch_bounds__(kM1Threads)
group_bits_kernel(const float *__restrict__ s, int64_t ld, Geometry g, bool vec_ok, int64_t items, int chunks,
                  bool find_max, uint32_t *__restrict__ max_key, uint32_t *__restrict__ nm_bits) {
    __shared__ uint8_t s_keep[64];
    __shared__ uint32_t s_best[kM1Threads / 32];
    if (M == 4 && threadIdx.x < 64) s_keep[threadIdx.x] = (uint8_t)keep_mask_of_outcomes(threadIdx.x, g.n);
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t best = 0u;
    for (int64_t it = blockIdx.x; it < items; it += gridDim.x) {
        const M1Item x = m1_item(it, chunks);
        const int64_t k0 = (int64_t)x.chunk * kM1ChunkK + lane * 8;
        uint32_t key[kM1RowsPerWarp][8];
        m1_load_rows(s, ld, g, vec_ok, x, warp, k0, key);
        const bool in_kp = k0 < g.kp();
#pragma unroll
        for (int i = 0; i < kM1RowsPerWarp; ++i) {
            const int64_t row = x.row0 + warp * kM1RowsPerWarp + i;
            uint32_t bits;
            if constexpr (M == 4)
                bits = (uint32_t)s_keep[outcomes4(key[i])] | ((uint32_t)s_keep[outcomes4(key[i] + 4)] << 4);
            else
                bits = top_n_bits<M>(key[i], g.n);
            // the lane's eight bits are byte (k0 / 8) mod 4 of their little-endian mask word: a warp stores 32
            // consecutive bytes of the row
            if (in_kp) reinterpret_cast<uint8_t *>(nm_bits + row * g.wpr)[k0 >> 3] = (uint8_t)bits;
#pragma unroll
            for (int j = 0; j < 8; ++j) best = max(best, key[i][j]);
        }
    }
    if (find_max) {
        best = __reduce_max_sync(0xFFFFFFFFu, best);
        if (lane == 0) s_best[warp] = best;
        __syncthreads();
        if (threadIdx.x == 0) {
#pragma unroll
            for (int w = 1; w < kM1Threads / 32; ++w) best = max(best, s_best[w]);
            if (best) atomicMax(max_key, best);
        }
    }
}

// Two fp32 values in one 64-bit register and the packed fp32 instructions of sm_100 on them (one instruction
// per pair; each half is rounded as the scalar instruction would round it).
__device__ __forceinline__ uint64_t f32x2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ float f32x2_sum(uint64_t v) {       // lo + hi
    float lo, hi;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
    return __fadd_rn(lo, hi);
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) { uint64_t r; asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b)); return r; }
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) { uint64_t r; asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b)); return r; }
__device__ __forceinline__ uint64_t sub2(uint64_t a, uint64_t b) { uint64_t r; asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b)); return r; }
__device__ __forceinline__ uint64_t add2_down(uint64_t a, uint64_t b) { uint64_t r; asm("add.rm.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b)); return r; }

// floor(v) of fp32 values 0 <= v < 2^41, two at a time, without a float-to-integer conversion per element (those
// run at a fraction of the fp32 rate and were what bound this kernel): v = r + d with r = v rounded DOWN to a
// multiple of 2^20 (add 1.5 * 2^43 rounding toward minus infinity: the sum lies in [2^43, 2^44), where fp32 steps
// by 2^20; subtracting the constant again is exact) and d = v - r exact, 0 <= d < 2^20; floor(d) by the same device
// with 1.5 * 2^23, where fp32 steps by 1.  r and floor(d) are then added up in fp32 over the eight elements of a
// row, which is exact (r / 2^20 <= 2^21 each, floor(d) < 2^20 each), and converted once.
__device__ __forceinline__ void floor_parts2(uint64_t v, uint64_t &r, uint64_t &fd) {
    const uint64_t big = f32x2(13194139533312.f, 13194139533312.f);            // 1.5 * 2^43
    const uint64_t mid = f32x2(12582912.f, 12582912.f);                        // 1.5 * 2^23
    r = sub2(add2_down(v, big), big);
    fd = sub2(add2_down(sub2(v, r), mid), mid);
}

// K-M1b: the block scores s_j = sum |T_w| as exact fixed-point integers, once the scale is known.  Second pass
// over S (for layers that fit, out of L2, where K-M1a left it).  Warps are independent (no shared memory, no
// barrier): a lane adds floor(|s| * 2^(40 - e_max)) of its counted elements (the N:M survivors, read back as the
// byte K-M1a stored, or all of them) over its warp's four rows, the four lanes of a 32-element word add up
// (a mask word never straddles a block: block_k is a multiple of 32), and one lane per word adds the partial
// score to the block's 64-bit total with an atomic (integer addition: any order gives the same sum).
__global__ void __launch_bounds__(kM1Threads)
block_score_kernel(const float *__restrict__ s, int64_t ld, Geometry g, bool vec_ok, int64_t items, int chunks,
                   const uint32_t *__restrict__ max_key, const uint32_t *__restrict__ nm_bits,
                   unsigned long long *__restrict__ score) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t mk = *max_key;
    if (!mk) return;                                         // an all-zero layer: every score stays 0
    const int e_max = key_exponent(mk);
    // floor(value * 2^(40 - e_max)): when that power of two is an fp32 number, the product is exact
    // (value <= layer maximum, so it stays below 2^41)
    const int scale_exp = kScoreFractionBits - e_max;
    const bool float_scale = scale_exp >= -126 && scale_exp <= 127;
    const float scale = float_scale ? __uint_as_float((uint32_t)(127 + scale_exp) << 23) : 0.f;
    for (int64_t it = blockIdx.x; it < items; it += gridDim.x) {
        const M1Item x = m1_item(it, chunks);
        const int64_t k0 = (int64_t)x.chunk * kM1ChunkK + lane * 8;
        const int rt = (int)(x.row0 / g.bm);
        uint32_t key[kM1RowsPerWarp][8];
        m1_load_rows(s, ld, g, vec_ok, x, warp, k0, key);
        const bool in_kp = k0 < g.kp();
        unsigned long long acc = 0ull;
        if (float_scale) {
#pragma unroll
            for (int i = 0; i < kM1RowsPerWarp; ++i) {
                const int64_t row = x.row0 + warp * kM1RowsPerWarp + i;
                uint32_t counted = 0xFFu;
                if (g.score_mode == 0) counted = in_kp ? reinterpret_cast<const uint8_t *>(nm_bits + row * g.wpr)[k0 >> 3] : 0u;
                // an element that is not counted is multiplied by zero instead of by the scale: its parts are zero
                uint64_t r_sum = f32x2(0.f, 0.f), d_sum = r_sum;             // exact: see floor_parts2
#pragma unroll
                for (int j = 0; j < 8; j += 2) {
                    const uint64_t sc = f32x2((counted >> j) & 1u ? scale : 0.f, (counted >> (j + 1)) & 1u ? scale : 0.f);
                    uint64_t r, fd;
                    floor_parts2(mul2(f32x2(__uint_as_float(key[i][j]), __uint_as_float(key[i][j + 1])), sc), r, fd);
                    r_sum = add2(r_sum, r);
                    d_sum = add2(d_sum, fd);
                }
                acc += ((unsigned long long)__float2uint_rn(f32x2_sum(r_sum) * 9.5367431640625e-07f) << 20) +
                       (unsigned long long)__float2uint_rn(f32x2_sum(d_sum));
            }
        } else {
#pragma unroll
            for (int i = 0; i < kM1RowsPerWarp; ++i) {
                const int64_t row = x.row0 + warp * kM1RowsPerWarp + i;
                uint32_t counted = 0xFFu;
                if (g.score_mode == 0) counted = in_kp ? reinterpret_cast<const uint8_t *>(nm_bits + row * g.wpr)[k0 >> 3] : 0u;
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    if ((counted >> j) & 1u) acc += fixed_point_score(key[i][j], e_max);
            }
        }
        acc += __shfl_xor_sync(0xFFFFFFFFu, acc, 1);
        acc += __shfl_xor_sync(0xFFFFFFFFu, acc, 2);
        // lanes that share a block column (block_k / 8 of them, 4, 8, 12 or 16): add up as far as the lane groups
        // of a power of two allow, then one atomic per group
        if (g.bk % 64 == 0) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, 4);
        if (g.bk % 128 == 0) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, 8);
        const int grp = g.bk % 128 == 0 ? 15 : (g.bk % 64 == 0 ? 7 : 3);
        if ((lane & grp) == 0 && in_kp && acc) {
            const int jb = (int)(k0 / g.bk);
            if (jb < g.nblk) atomicAdd(&score[(int64_t)rt * g.nblk + jb], acc);
        }
    }
}

// K-M2.  grid = (row tiles, block_rows / 32).  Every CTA ranks its row tile's block scores (cheap)
// and clears the mask words of pruned blocks in its own 32 rows; the CTA with blockIdx.y == 0 also
// emits the kept columns in ascending order.
__global__ void __launch_bounds__(256)
block_select_kernel(Geometry g, const unsigned long long *__restrict__ score,
                    int32_t *__restrict__ blk_col, uint32_t *__restrict__ nm_bits) {
    extern __shared__ unsigned long long sm[];
    unsigned long long *sc = sm;                                   // [nblk]
    int *kept = reinterpret_cast<int *>(sm + g.nblk);              // [nblk]
    __shared__ int s_warp_tot[8];
    __shared__ int s_base;
    const int rt = blockIdx.x;
    for (int j = threadIdx.x; j < g.nblk; j += blockDim.x) sc[j] = score[(int64_t)rt * g.nblk + j];
    if (threadIdx.x == 0) s_base = 0;
    __syncthreads();
    for (int j = threadIdx.x; j < g.nblk; j += blockDim.x) {
        const unsigned long long mine = sc[j];
        int rank = 0;
        for (int t = 0; t < g.nblk; ++t) {
            const unsigned long long o = sc[t];
            rank += (o > mine) || (o == mine && t < j);
        }
        kept[j] = rank < g.kkeep;
    }
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (blockIdx.y == 0) {
        // ascending compaction: block-wide exclusive scan over chunks of blockDim.x flags
        for (int j0 = 0; j0 < g.nblk; j0 += blockDim.x) {
            const int j = j0 + threadIdx.x;
            const int f = (j < g.nblk) ? kept[j] : 0;
            const uint32_t ballot = __ballot_sync(0xFFFFFFFFu, f);
            const int before = __popc(ballot & ((1u << lane) - 1u));
            if (lane == 0) s_warp_tot[warp] = __popc(ballot);
            __syncthreads();
            int warp_off = 0, tot = 0;
            for (int w = 0; w < (int)(blockDim.x >> 5); ++w) {
                if (w < warp) warp_off += s_warp_tot[w];
                tot += s_warp_tot[w];
            }
            if (f) blk_col[(int64_t)rt * g.kkeep + s_base + warp_off + before] = j;
            __syncthreads();
            if (threadIdx.x == 0) s_base += tot;
            __syncthreads();
        }
    }
    // final mask = group bits AND block kept: one warp per row, lanes stride over the row's words
    const int wpb = g.bk / 32;
    for (int r = warp; r < 32; r += 8) {
        uint32_t *row_words = nm_bits + ((int64_t)rt * g.bm + blockIdx.y * 32 + r) * g.wpr;
        for (int wc = lane; wc < g.wpr; wc += 32)
            if (!kept[wc / wpb]) row_words[wc] = 0u;
    }
}

}  // namespace

// workspace: [0] max key (uint32), padded to 256 B; then score[nrt * nblk] uint64.
size_t mask_workspace_bytes(const Geometry &g) {
    return kAlign + align_up((size_t)g.nrt * g.nblk * sizeof(unsigned long long));
}

cudaError_t launch_block_select(const Geometry &g, const void *d_workspace, int32_t *d_blk_col, uint32_t *d_nm_bits,
                                cudaStream_t st) {
    const unsigned long long *score =
        reinterpret_cast<const unsigned long long *>(reinterpret_cast<const uint8_t *>(d_workspace) + kAlign);
    const size_t smem = (size_t)g.nblk * (sizeof(unsigned long long) + sizeof(int));
    if (smem + 64 > 48 * 1024) {     // the longest rows (nblk near 4096) need the opt-in shared-memory size
        cudaError_t e = cudaFuncSetAttribute(block_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    block_select_kernel<<<dim3((unsigned)g.nrt, (unsigned)(g.bm / 32)), 256, smem, st>>>(g, score, d_blk_col, d_nm_bits);
    return cudaGetLastError();
}

cudaError_t launch_build_mask(const float *d_s, int64_t ld, const Geometry &g, int32_t *d_blk_col,
                              uint32_t *d_nm_bits, void *d_workspace, size_t workspace_bytes, bool max_known,
                              cudaStream_t st) {
    uint32_t *max_key = reinterpret_cast<uint32_t *>(d_workspace);
    unsigned long long *score =
        reinterpret_cast<unsigned long long *>(reinterpret_cast<uint8_t *>(d_workspace) + kAlign);
    // max_known: the first word already holds the layer's largest canonical |s| (written by the saliency kernel
    // that produced S), so only the scores are cleared and the pass over S that finds the maximum is skipped
    cudaError_t e = max_known ? cudaMemsetAsync(score, 0, workspace_bytes - kAlign, st)
                              : cudaMemsetAsync(d_workspace, 0, workspace_bytes, st);
    if (e != cudaSuccess) return e;
    const bool vec_ok = (ld % 4 == 0) && ((reinterpret_cast<uintptr_t>(d_s) & 15u) == 0);

    // work items of 32 rows x 256 k-elements, dealt out to at most eight resident CTAs per SM
    const int chunks = (int)((g.kp() + kM1ChunkK - 1) / kM1ChunkK);
    const int64_t items = (g.mp() / kM1Rows) * chunks;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
        sms = 148;
    // grids of resident CTAs: every CTA is on an SM from the start and takes its share of the items
    auto resident_grid = [&](const void *kern) {
        int per_sm = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kM1Threads, 0) != cudaSuccess || per_sm <= 0) per_sm = 4;
        const int64_t cap = (int64_t)sms * per_sm;
        return (int)(items < cap ? items : cap);
    };
    if (g.m == 4)
        group_bits_kernel<4><<<resident_grid((const void *)group_bits_kernel<4>), kM1Threads, 0, st>>>(
            d_s, ld, g, vec_ok, items, chunks, !max_known, max_key, d_nm_bits);
    else
        group_bits_kernel<8><<<resident_grid((const void *)group_bits_kernel<8>), kM1Threads, 0, st>>>(
            d_s, ld, g, vec_ok, items, chunks, !max_known, max_key, d_nm_bits);
    block_score_kernel<<<resident_grid((const void *)block_score_kernel), kM1Threads, 0, st>>>(
        d_s, ld, g, vec_ok, items, chunks, max_key, d_nm_bits, score);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    return launch_block_select(g, d_workspace, d_blk_col, d_nm_bits, st);
}

}  // namespace crisp
