// Tensor-core SpMM over kept blocks (sm_100a): TMA-staged, warp-specialised, tcgen05 MMA with
// TMEM accumulators.  Sec. III-E of the paper, mapped onto B200:
//   step 1 (load the activations of kept blocks): two producer threads walk the kept-block list of
//           a 128-row tile; per kept block one issues a tiled copy of the weight tile (from the
//           execution image), the other TMA tensor loads of the X rows [blk_col*Bk, +Bk) only;
//   step 2 (select activations by offset): either the 2:4 metadata drives tcgen05.mma.sp's operand
//           selection (sparse image), or the weight tile is stored zero-expanded so that the
//           selection is the identity (dense image);
//   step 3 (multiply-accumulate): tcgen05.mma, fp32 accumulators in tensor memory, epilogue warps
//           convert and TMA-store Y.
// A CTA is persistent over (128-row tile, column tile) pairs; all row tiles of a layer have the same
// number of kept blocks (uniform block pruning, Sec. III-A), so tiles are load-balanced by construction.
//
// The execution image is built by the kernels at the bottom of this file from the canonical format.
#include <cuda.h>
#include <cuda_bf16.h>

#include <atomic>
#include <new>

#include "crisp_internal.h"
#include "tc_common.cuh"
#include "walks.cuh"

namespace crisp {

using namespace tc;

namespace {

struct TcParams {
    const uint8_t *image;       // per walk entry: weight tile (+ metadata), entry_bytes each
    const int32_t *walk_col;    // [nst, wcap] block column of each walk entry
    const int32_t *walk_len;    // [nst]
    int32_t *status;
    void *y;                    // for edge chunks that TMA cannot clip exactly
    int64_t ldy;
    int nst, wcap, bk, n_col_tiles, num_tiles, rows;
    int64_t ncols;
    uint32_t a_bytes, entry_bytes, box_bytes, stage_bytes, num_stages;
    uint32_t group;             // kept blocks per pipeline stage (1, 2 or 4): [group weight tiles + metadata | group X tiles]
    uint32_t addends;           // sparse tiles (each a_bytes + metadata) per walk entry: 2 when a block with up to four
                                // values per aligned 4-group is multiplied as two 2:4-compliant addends
    uint32_t stg_bufs;          // staging tiles per epilogue warp (1, 2 or 4): stores in flight per warp
    uint32_t stg_tile_bytes;    // one staging tile: 16 or 32 rows of 128 bytes (= the row count of map_y's box)
    uint32_t stg_swz_mask;      // 16-byte chunk j of staging row r sits at j ^ (r & mask): 7 = 128-byte swizzle of
                                // map_y, 3 / 1 / 0 = 64-byte / 32-byte / none (convolution: span = inner box bytes)
    uint32_t walk_cache;        // walk lists are copied into shared memory at kernel start
    // Convolution as implicit GEMM: X is not a matrix in memory but an NHWC activation; a column tile is a
    // box of tw x th x tb output pixels and the X tile of a kept block (one filter tap, bk channels) is the
    // same box of the activation shifted by the tap, fetched by one 4-D TMA load (zero fill = zero padding).
    int conv;
    int cv_tw, cv_th, cv_tb;    // pixel box of a column tile (tw * th * tb = tile columns)
    int cv_tiles_x, cv_tiles_y; // column tiles per image row / per image column
    int cv_cpt;                 // k-blocks per filter tap = channels / bk
    int cv_kw, cv_pad;          // filter width, zero padding
    int cv_wo, cv_ho, cv_batch; // output width, height, images
    int cv_plain;               // Y rows are not TMA-addressable (wo * element size not a multiple of 16 bytes):
                                // the epilogue stores element by element
    int cv_tw_log2, cv_img_log2;   // log2(tw), log2(tw * th)
    int cv_nhwc;                // Y is [batch, ho, wo, ldy] (output channel fastest): the next convolution's activation
    // Thin layers (one CTA tile, at most 128 / stack rows; matrix mode): a tile covers `stack` column tiles, one per
    // group of 128 / stack accumulator lanes.  For group q the walk is run again with the image copy whose weights
    // sit in that group's rows (all other rows zero) against the X columns of column tile ct * stack + q.
    int stack;
    const float *bias;          // layer epilogue: Y = act(W*X + bias); nullptr = no bias
    int relu;
    unsigned long long wait_limit;   // cycles after which a wait gives up and the kernel reports CRISP_TIMEOUT
    int skip_fill;              // test hook (-1 = off): the producers leave out the loads of the skip_fill-th pipeline
                                // fill, so that the wait for it runs into wait_limit
    int a_map;                  // map_a views the image as rows of 256 bytes: weight tiles come in as tiled loads
    int x_map_3d;               // map_x views X as [ncols/64][k][64]: one load fetches all NT boxes
};

constexpr uint32_t kWideStageBytes = 2048;                      // epilogue staging tile: 16 rows x 128 bytes
// Epilogue warps: two per TMEM lane quarter, or four where short walks make the epilogue the longest role.
// Threads: warp 0 weight-tile producer, warp 1 MMA issuer, the epilogue warps, then one warp as the X producer.

// Where a tile's columns start: the first column (matrix mode) or the first output pixel (x, y, image) of
// the tile's box (convolution mode).
struct TileOrigin { int x, y, b; };

template <bool kConv>
__device__ __forceinline__ TileOrigin tile_origin(const TcParams &p, int ct, int tile_n) {
    TileOrigin o;
    if constexpr (!kConv) { o.x = ct * tile_n; o.y = 0; o.b = 0; return o; }
    const int per_image = p.cv_tiles_x * p.cv_tiles_y;
    const int bb = ct / per_image, r = ct - bb * per_image;
    const int by = r / p.cv_tiles_x;
    o.x = (r - by * p.cv_tiles_x) * p.cv_tw; o.y = by * p.cv_th; o.b = bb * p.cv_tb;
    return o;
}

// One epilogue chunk: 32 rows (one per lane) x 128 bytes.  Through the warp's 128B-swizzled staging
// tile and a TMA store, or, where TMA cannot clip exactly (it clips at 16-byte granularity), with
// guarded plain stores.
template <typename OutT, bool kConv>
__device__ __forceinline__ void store_chunk(const TcParams &p, const CUtensorMap *map_y, uint32_t stg, uint8_t *stg_gen,
                                            int lane, const uint32_t (&out)[32], const TileOrigin &org, int col0, int y0,
                                            uint32_t &slot) {
    constexpr int kOutCols = 128 / (int)sizeof(OutT);
    const int x0 = org.x + col0;             // matrix mode: first column of the chunk
    // convolution mode: the chunk is kOutCols / tw rows of tw pixels inside one image of the tile's box
    int cx = 0, cy = 0, cb = 0;
    bool inside = x0 < p.ncols;
    if constexpr (kConv) {
        const int per_image = p.cv_tw * p.cv_th;
        const int img = col0 / per_image;
        cx = org.x; cy = org.y + (col0 - img * per_image) / p.cv_tw; cb = org.b + img;
        inside = cx < p.cv_wo && cy < p.cv_ho && cb < p.cv_batch;
    }
    if constexpr (kConv) {
        if (p.cv_plain) {
            // Through the warp's staging tile, so that a store instruction covers consecutive pixels of one
            // row of W: lane r writes its row (swizzled 16-byte chunks), then for every row the lanes take the
            // chunk's pixels side by side.  Pixel c of the chunk is (image, y, x) in box order inside the tile,
            // clipped at the image borders.
            constexpr int kPer = kOutCols / 32;          // pixels per lane and row
            int64_t pix_off[kPer];
            uint32_t smem_off[kPer];
            bool pix_ok[kPer];
#pragma unroll
            for (int t = 0; t < kPer; ++t) {
                const int c = lane + 32 * t, col = col0 + c;
                const int img = col >> p.cv_img_log2, rem = col & ((1 << p.cv_img_log2) - 1);
                const int gy = org.y + (rem >> p.cv_tw_log2), gx = org.x + (rem & (p.cv_tw - 1)), gb = org.b + img;
                pix_ok[t] = gx < p.cv_wo && gy < p.cv_ho && gb < p.cv_batch;
                pix_off[t] = ((int64_t)gb * p.cv_ho + gy) * p.cv_wo + gx;
                smem_off[t] = (uint32_t)c * sizeof(OutT);
            }
            const int rpp = (int)(p.stg_tile_bytes / 128);      // rows per pass: 16 or 32
            for (int h = 0; h < 32 / rpp; ++h) {
                if (y0 + rpp * h >= p.rows) break;
                __syncwarp();
                if (lane / rpp == h) {
                    uint8_t *tile = stg_gen + (lane % rpp) * 128;
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        *reinterpret_cast<uint4 *>(tile + ((j ^ (lane & 7)) << 4)) =
                            make_uint4(out[4 * j], out[4 * j + 1], out[4 * j + 2], out[4 * j + 3]);
                }
                __syncwarp();
                for (int r = 0; r < rpp; ++r) {
                    const int row = y0 + rpp * h + r;
                    if (row >= p.rows) break;
                    OutT *yrow = reinterpret_cast<OutT *>(p.y) + (int64_t)row * p.ldy;
                    const uint8_t *trow = stg_gen + r * 128;
#pragma unroll
                    for (int t = 0; t < kPer; ++t) {
                        const uint32_t chunk = (smem_off[t] >> 4) ^ (uint32_t)((rpp * h + r) & 7);
                        const OutT v = *reinterpret_cast<const OutT *>(trow + (chunk << 4) + (smem_off[t] & 15u));
                        if (pix_ok[t]) yrow[pix_off[t]] = v;
                    }
                }
            }
            return;
        }
    }
    if (!kConv && x0 + kOutCols > p.ncols && (p.ncols * (int64_t)sizeof(OutT)) % 16 != 0) {
        const int row = y0 + lane;
        if (row < p.rows && x0 < p.ncols) {
            OutT *dst = reinterpret_cast<OutT *>(p.y) + (int64_t)row * p.ldy + x0;
            const int nvalid = (int)(p.ncols - x0);
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                if constexpr (sizeof(OutT) == 2) {
                    if (2 * i < nvalid) dst[2 * i] = (OutT)(out[i] & 0xFFFFu);
                    if (2 * i + 1 < nvalid) dst[2 * i + 1] = (OutT)(out[i] >> 16);
                } else {
                    if (i < nvalid) dst[i] = __uint_as_float(out[i]);
                }
            }
        }
        return;
    }
    // The warp cycles through stg_bufs staging tiles.  A 32-row tile takes the chunk in one pass and one
    // store; a 16-row tile (when shared memory is short) takes lanes 0..15, then lanes 16..31.
    const int passes = p.stg_tile_bytes == 4096 ? 1 : 2;
    for (int h = 0; h < passes; ++h) {
        if (y0 + 16 * h >= p.rows) break;
        if (lane == 0) {                         // the store that last used this tile has finished reading it
            if (p.stg_bufs == 4) bulk_wait_read<3>();
            else if (p.stg_bufs == 2) bulk_wait_read<1>();
            else bulk_wait_read<0>();
        }
        __syncwarp();
        const uint32_t tile_off = slot * p.stg_tile_bytes;
        if (passes == 1 || (lane >> 4) == h) {
            uint8_t *tile = stg_gen + tile_off + (passes == 1 ? lane : (lane & 15)) * 128;
#pragma unroll
            for (int j = 0; j < 8; ++j)          // map_y's swizzle: 16-byte chunk j of row r sits at j ^ (r & mask)
                *reinterpret_cast<uint4 *>(tile + ((j ^ (lane & (kConv ? p.stg_swz_mask : 7u))) << 4)) =
                    make_uint4(out[4 * j], out[4 * j + 1], out[4 * j + 2], out[4 * j + 3]);
        }
        fence_async_smem();
        __syncwarp();
        if (lane == 0) {
            if (inside) {
                if constexpr (kConv) tma_store_4d(map_y, stg + tile_off, cx, cy, cb, y0 + 16 * h);
                else tma_store_2d(map_y, stg + tile_off, x0, y0 + 16 * h);
            }
            bulk_commit();
        }
        slot = (slot + 1) & (p.stg_bufs - 1);
    }
}

// One epilogue chunk of a convolution whose output is NHWC: the lane holds one output channel (row y0 + lane) of
// kOutCols pixels, memory wants the 32 channels of a pixel side by side.  The chunk is transposed through the
// warp's staging tile, [pixel][32 channels] (64 or 128 bytes per pixel, 4096 bytes per chunk), and goes out
// as one 4-D bulk tensor store of {32 channels, tw, pixels / tw, 1} (it clips channels beyond `rows` and pixels
// outside the images), or, where the pixel pitch is not a multiple of 16 bytes, pixel by pixel with the 32
// lanes on consecutive channels.  `out` is packed as in store_chunk (bf16: pixels 2i, 2i+1 in word i).
template <typename OutT>
__device__ __forceinline__ void store_chunk_nhwc(const TcParams &p, const CUtensorMap *map_y, uint32_t stg, uint8_t *stg_gen,
                                                 int lane, const uint32_t (&out)[32], const TileOrigin &org, int col0, int y0) {
    constexpr int kOutCols = 128 / (int)sizeof(OutT);
    constexpr int kRowBytes = 32 * (int)sizeof(OutT);           // one pixel: 32 channels
    const int per_image = p.cv_tw * p.cv_th;
    const int img = col0 / per_image;
    const int cx = org.x, cy = org.y + (col0 - img * per_image) / p.cv_tw, cb = org.b + img;
    if (y0 >= p.rows) return;
    if (lane == 0 && !p.cv_plain) bulk_wait_read<0>();          // the previous store has finished reading the tile
    __syncwarp();
#pragma unroll
    for (int i = 0; i < 32; ++i) {
        if constexpr (sizeof(OutT) == 2) {
            *reinterpret_cast<uint16_t *>(stg_gen + (2 * i) * kRowBytes + lane * 2) = (uint16_t)(out[i] & 0xFFFFu);
            *reinterpret_cast<uint16_t *>(stg_gen + (2 * i + 1) * kRowBytes + lane * 2) = (uint16_t)(out[i] >> 16);
        } else {
            *reinterpret_cast<uint32_t *>(stg_gen + i * kRowBytes + lane * 4) = out[i];
        }
    }
    if (!p.cv_plain) {
        fence_async_smem();
        __syncwarp();
        if (lane == 0) {
            if (cx < p.cv_wo && cy < p.cv_ho && cb < p.cv_batch) tma_store_4d(map_y, stg, y0, cx, cy, cb);
            bulk_commit();
        }
        return;
    }
    __syncwarp();
    const bool row_ok = y0 + lane < p.rows;
    for (int c = 0; c < kOutCols; ++c) {
        const int col = col0 + c;
        const int im = col >> p.cv_img_log2, rem = col & ((1 << p.cv_img_log2) - 1);
        const int gy = org.y + (rem >> p.cv_tw_log2), gx = org.x + (rem & (p.cv_tw - 1)), gb = org.b + im;
        if (row_ok && gx < p.cv_wo && gy < p.cv_ho && gb < p.cv_batch)
            reinterpret_cast<OutT *>(p.y)[(((int64_t)gb * p.cv_ho + gy) * p.cv_wo + gx) * p.ldy + y0 + lane] =
                *reinterpret_cast<const OutT *>(stg_gen + c * kRowBytes + lane * (int)sizeof(OutT));
    }
    __syncwarp();
}

// The MMA issuer's loop, with the number of MMAs per kept block (NM) fixed at compile time: the loop is
// bound by this one thread's instruction latency, and a straight line of NM MMAs lets the compiler
// overlap the operand set-up of one MMA with the issue of the previous one.
// Descriptors of stage 0 are built once; a later stage or K step only moves the start-address field
// (16-byte units, low word), which cannot carry: shared memory is smaller than 2^18 bytes.  Per K step
// the weight tile advances by 4096 bytes, X by 32 rows (sparse image, 4096 bytes) or 16 rows (2048).
struct MmaRoleArgs {
    uint32_t ring, bar_full, bar_empty, bar_tfull, bar_tempty, tmem_base;
    const int32_t *walk_len;
    volatile int *abort_flag;
};
template <int kTileN, bool kSparse, int kAccStages, int NM, bool kConv>
__device__ __forceinline__ void mma_role(const TcParams &p, const MmaRoleArgs &a) {
    // matrix mode: X rows are columns-contiguous (MN-major operand, 64-column boxes box_bytes apart, a K
    // step is 32 or 16 rows); convolution mode: the activation tile is [pixel][bk channels] with the channels
    // contiguous (K-major operand, 128-byte rows in 1024-byte groups of 8, a K step is 64 or 32 bytes)
    constexpr uint32_t idesc = kConv ? (make_idesc(kTileN, kSparse) & ~(1u << 16)) : make_idesc(kTileN, kSparse);
    const uint64_t a_desc0 = make_smem_desc(a.ring, 2048, 128, kLayoutNone);
    const uint64_t b_desc0 = kConv ? make_smem_desc(a.ring + p.group * p.entry_bytes, 16, 1024, kLayoutSw128)
                                   : make_smem_desc(a.ring + p.group * p.entry_bytes, p.box_bytes, 1024, kLayoutSw128);
    constexpr uint32_t b_step = kConv ? (kSparse ? 4u : 2u) : (kSparse ? 256u : 128u);
    const uint64_t m_desc0 = make_smem_desc(a.ring + p.a_bytes, 128, 128, kLayoutNone);
    const uint32_t stage_step = p.stage_bytes >> 4, ring_span = p.num_stages * stage_step;
    const uint32_t a_step = p.entry_bytes >> 4, x_step = ((uint32_t)(kTileN / kBoxN) * p.box_bytes) >> 4;   // per block of a stage
    const int group = (int)p.group;
    uint32_t off = 0, full = a.bar_full, empty = a.bar_empty, ph = 0, acc = 0, acc_ph = 0, meta_buf = 0;
    if (group == 1) {
        // one kept block per stage: the plain loop (large tiles; every extra instruction here costs the headline cells)
        for (int t = blockIdx.x; t < p.num_tiles && !*a.abort_flag; t += gridDim.x) {
            const int len = min(a.walk_len[t % p.nst], p.wcap) * p.stack;
            if (!mbar_wait(a.bar_tempty + 8 * acc, acc_ph ^ 1u, a.abort_flag, p.wait_limit)) break;
            tc_fence_after();
            const uint32_t d_tmem = a.tmem_base + acc * kTileN;
            uint32_t accum = 0;
            bool ok = true;
            for (int e = 0; e < len; ++e) {
                if (!mbar_wait(full, ph, a.abort_flag, p.wait_limit)) { ok = false; break; }
                tc_fence_after();
                const uint64_t ad = a_desc0 + off, bd = b_desc0 + off;
                if constexpr (kSparse) {
                    const uint32_t meta_tmem = a.tmem_base + kAccStages * kTileN + 4 * meta_buf;
                    tmem_copy_128x128b(meta_tmem, m_desc0 + off);
#pragma unroll
                    for (int j = 0; j < NM; ++j)
                        mma_sparse(d_tmem, ad + j * 256, bd + j * b_step, idesc | (uint32_t)(j & 1), accum | (uint32_t)j,
                                   meta_tmem + (j & ~1));
                    meta_buf ^= 1u;
                    if (p.addends == 2) {               // second addend of the block: same X tile, same accumulator
                        const uint32_t sub = (p.a_bytes + kMetaBytes) >> 4;
                        const uint32_t meta2 = a.tmem_base + kAccStages * kTileN + 4 * meta_buf;
                        tmem_copy_128x128b(meta2, m_desc0 + off + sub);
#pragma unroll
                        for (int j = 0; j < NM; ++j)
                            mma_sparse(d_tmem, ad + sub + j * 256, bd + j * b_step, idesc | (uint32_t)(j & 1), 1u, meta2 + (j & ~1));
                        meta_buf ^= 1u;
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < NM; ++j) mma_dense(d_tmem, ad + j * 256, bd + j * b_step, idesc, accum | (uint32_t)j);
                }
                accum = 1u;
                mma_commit(empty);                      // stage reusable once these MMAs have read it
                off += stage_step; full += 8; empty += 8;
                if (off == ring_span) { off = 0; full = a.bar_full; empty = a.bar_empty; ph ^= 1u; }
            }
            if (!ok) break;
            mma_commit(a.bar_tfull + 8 * acc);          // accumulator complete
            if (++acc == kAccStages) { acc = 0; acc_ph ^= 1u; }
        }
        return;
    }
    for (int t = blockIdx.x; t < p.num_tiles && !*a.abort_flag; t += gridDim.x) {
        const int len = min(a.walk_len[t % p.nst], p.wcap);    // (the clamp keeps a list that was overwritten in bounds)
        if (!mbar_wait(a.bar_tempty + 8 * acc, acc_ph ^ 1u, a.abort_flag, p.wait_limit)) break;
        tc_fence_after();
        const uint32_t d_tmem = a.tmem_base + acc * kTileN;
        uint32_t accum = 0;
        bool ok = true;
        // a stacked tile walks its list once per lane group; a stage never spans two walks
        for (int q = 0; q < p.stack && ok; ++q) {
            for (int e = 0; e < len; e += group) {
                if (!mbar_wait(full, ph, a.abort_flag, p.wait_limit)) { ok = false; break; }
                tc_fence_after();
                const int cnt = min(group, len - e);
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    if (g >= cnt) break;
                    const uint64_t ad = a_desc0 + off + g * a_step, bd = b_desc0 + off + g * x_step;
                    if constexpr (kSparse) {
                        const uint32_t meta_tmem = a.tmem_base + kAccStages * kTileN + 4 * meta_buf;
                        tmem_copy_128x128b(meta_tmem, m_desc0 + off + g * a_step);
#pragma unroll
                        for (int j = 0; j < NM; ++j)
                            mma_sparse(d_tmem, ad + j * 256, bd + j * b_step, idesc | (uint32_t)(j & 1), accum | (uint32_t)j,
                                       meta_tmem + (j & ~1));
                        meta_buf ^= 1u;
                        if (p.addends == 2) {               // second addend of the block: same X tile, same accumulator
                            const uint32_t sub = (p.a_bytes + kMetaBytes) >> 4;
                            const uint32_t meta2 = a.tmem_base + kAccStages * kTileN + 4 * meta_buf;
                            tmem_copy_128x128b(meta2, m_desc0 + off + g * a_step + sub);
#pragma unroll
                            for (int j = 0; j < NM; ++j)
                                mma_sparse(d_tmem, ad + sub + j * 256, bd + j * b_step, idesc | (uint32_t)(j & 1), 1u, meta2 + (j & ~1));
                            meta_buf ^= 1u;
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < NM; ++j) mma_dense(d_tmem, ad + j * 256, bd + j * b_step, idesc, accum | (uint32_t)j);
                    }
                    accum = 1u;
                }
                mma_commit(empty);                      // stage reusable once these MMAs have read it
                off += stage_step; full += 8; empty += 8;
                if (off == ring_span) { off = 0; full = a.bar_full; empty = a.bar_empty; ph ^= 1u; }
            }
        }
        if (!ok) break;
        mma_commit(a.bar_tfull + 8 * acc);          // accumulator complete
        if (++acc == kAccStages) { acc = 0; acc_ph ^= 1u; }
    }
}

// ----------------------------------------------------------------------------------- kernel
//
// Shared memory (1024-byte aligned): num_stages x [weight tile | metadata (sparse) | NT boxes of X]
//                                    | 8 warps x stg_bufs staging tiles (16 or 32 rows) | barriers | TMEM base | abort flag
//                                    | walk lists (optional)
// Weight tile layout (no swizzle, K-major): [k/8][row][8 elements], i.e. 8x16-byte core matrices are
// contiguous, 128 bytes between 8-row groups, 2048 bytes between 16-byte K chunks.
// X box layout: TMA SWIZZLE_128B, 64 columns (128 bytes) x bk rows; MN-major operand with 1024 bytes
// between 8-row K groups and box_bytes between 64-column groups.
template <int NT, bool kSparse, int kAccStages, typename OutT, int kEpi, bool kConv>
__global__ void __launch_bounds__(96 + 32 * kEpi, 1)
spmm_tc_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_y,
               const __grid_constant__ CUtensorMap map_a, TcParams p) {
    constexpr int kTileN = NT * kBoxN;
    constexpr int kMetaCols = kSparse ? 8 : 0;                       // two 4-column metadata buffers
    constexpr int kTmemCols = (kAccStages * kTileN + kMetaCols) <= 256 ? 256 : 512;
    static_assert(kAccStages * kTileN + kMetaCols <= 512, "tensor memory is 512 columns");
    constexpr int kOutCols = 128 / (int)sizeof(OutT);                // columns of one 128-byte staging row

    extern __shared__ __align__(1024) uint8_t smem_raw[];     // the kernel has no static shared memory
    const uint32_t smem_base = smem_u32(smem_raw);
    uint8_t *smem_gen = smem_raw;
    if (smem_base & 1023u) {                 // swizzled operand tiles need it; checked, not assumed
        if (threadIdx.x == 0) atomicCAS(p.status, 0, (int)CRISP_CUDA_ERROR);
        return;
    }
    const uint32_t ring = smem_base;
    const uint32_t staging = ring + p.num_stages * p.stage_bytes;
    const uint32_t ctrl = staging + kEpi * p.stg_bufs * p.stg_tile_bytes;
    uint8_t *ctrl_gen = smem_gen + (ctrl - smem_base);
    // barriers: full[s], empty[s] (s < 8), tmem_full[2], tmem_empty[2]
    const uint32_t bar_full = ctrl, bar_empty = ctrl + 64, bar_tfull = ctrl + 128, bar_tempty = ctrl + 144;
    volatile uint32_t *tmem_base_slot = reinterpret_cast<volatile uint32_t *>(ctrl_gen + 160);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(ctrl_gen + 164);
    // Optional copy of the walk lists ([nst] lengths, then [nst][wcap] block columns): a tile with a short
    // walk would otherwise spend two dependent global loads per tile in the producer's serial loop.
    int32_t *s_walk = reinterpret_cast<int32_t *>(ctrl_gen + 256);

    // Set-up, ordered so that its round trips run side by side: warp 1 asks for tensor memory at once, every
    // thread asks for its first word of the walk lists before thread 0 builds the barriers, and the words are
    // stored to shared memory afterwards.
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (warp == 1) {
        tmem_alloc(smem_u32(const_cast<uint32_t *>(tmem_base_slot)), kTmemCols);
        tmem_relinquish();
    }
    const int walk_words = p.walk_cache ? p.nst * (p.wcap + 1) : 0;     // [nst] lengths, then [nst][wcap] columns
    int32_t walk_w0 = 0;
    if ((int)threadIdx.x < walk_words)
        walk_w0 = (int)threadIdx.x < p.nst ? p.walk_len[threadIdx.x] : p.walk_col[(int)threadIdx.x - p.nst];
    if (threadIdx.x == 0) {
        prefetch_tensormap(&map_a);
        prefetch_tensormap(&map_x);
        if (!(kConv && p.cv_plain)) prefetch_tensormap(&map_y);
        for (uint32_t s = 0; s < p.num_stages; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
        for (int a = 0; a < kAccStages; ++a) { mbar_init(bar_tfull + 8 * a, 1); mbar_init(bar_tempty + 8 * a, kEpi); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if ((int)threadIdx.x < walk_words) s_walk[threadIdx.x] = walk_w0;
    for (int i = threadIdx.x + blockDim.x; i < walk_words; i += blockDim.x)
        s_walk[i] = i < p.nst ? p.walk_len[i] : p.walk_col[i - p.nst];
    const int32_t *walk_len = p.walk_cache ? s_walk : p.walk_len;
    const int32_t *walk_col = p.walk_cache ? s_walk + p.nst : p.walk_col;
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_base_slot;
    const uint32_t x_blk_bytes = NT * p.box_bytes;           // X tile of one kept block
    const uint32_t tx_bytes = p.entry_bytes + x_blk_bytes;   // a stage of one block

    // Both single-thread roles below are bound by their own dependent-instruction latency (one warp per
    // scheduler, ~5 cycles per dependent instruction), so their per-block loops carry running addresses
    // (stage base, barrier, image row, descriptors) instead of recomputing them.
    if (warp == 0 || warp == 2 + kEpi) {
        // ------------------------------------------------ producers: step 1, kept blocks only
        // Issuing a tiled copy costs the issuing thread 90 to 170 cycles and every pass of its loop some 170 more
        // (measured with cycle stamps: wait 55, byte count 20, copy 155, loop 170), so one thread that brings
        // both operands fills a stage about every 450 cycles.  Two threads share the work by operand: warp 0
        // brings the weight tiles and posts the byte count of the whole stage (the only arrival the `full` barrier
        // expects), the warp after the epilogue warps walks the block columns and brings the X tiles.  Both wait
        // for the same `empty` phase, so neither writes a stage that is still being read; bytes of X that land
        // before the count is posted are carried by the barrier's transaction count until the arrival comes.
        if (lane == 0) {
            const uint32_t ring_end = ring + p.num_stages * p.stage_bytes;
            const uint32_t entry_rows = p.entry_bytes >> 8;      // image rows (256 bytes) per walk entry
            uint32_t dst = ring, full = bar_full, empty = bar_empty, ph = 0;
            int fill_no = 0;     // test hook: fill number p.skip_fill gets no copies, so its `full` barrier never
                                 // completes and the bounded wait of the MMA issuer ends the kernel with CRISP_TIMEOUT
            if (warp == 0) {
                if (p.group == 1) {       // one kept block per stage: the plain loop
                    for (int t = blockIdx.x; t < p.num_tiles && !*abort_flag; t += gridDim.x) {
                        const int st = t % p.nst;
                        const int len = min(walk_len[st], p.wcap);
                        const uint8_t *img = p.image + (int64_t)st * p.wcap * p.entry_bytes;
                        const int arow0 = (int)(((int64_t)st * p.wcap * p.entry_bytes) >> 8);
                        bool ok = true;
                        for (int q = 0; q < p.stack && ok; ++q) {             // image copy q (stack > 1 only with one CTA tile)
                            int arow = arow0 + q * p.wcap * (int)entry_rows;
                            const uint8_t *src = img + (int64_t)q * p.wcap * p.entry_bytes;
                            for (int e = 0; e < len; ++e) {
                                if (!mbar_wait(empty, ph ^ 1u, abort_flag, p.wait_limit)) { ok = false; break; }
                                mbar_expect_tx(full, tx_bytes);
                                if (fill_no++ != p.skip_fill) {
                                    // the weight tile comes in as a box of 256-byte image rows (tiled copies pipeline,
                                    // untiled bulk copies are served one at a time)
                                    if (p.a_map) tma_load_2d(dst, &map_a, 0, arow, full);
                                    else bulk_load(dst, src, p.entry_bytes, full);
                                }
                                arow += (int)entry_rows; src += p.entry_bytes;
                                dst += p.stage_bytes; full += 8; empty += 8;
                                if (dst == ring_end) { dst = ring; full = bar_full; empty = bar_empty; ph ^= 1u; }
                            }
                        }
                        if (!ok) break;
                    }
                } else {
                    for (int t = blockIdx.x; t < p.num_tiles && !*abort_flag; t += gridDim.x) {
                        const int st = t % p.nst;
                        const int len = min(walk_len[st], p.wcap);
                        const int arow0 = (int)(((int64_t)st * p.wcap * p.entry_bytes) >> 8);
                        bool ok = true;
                        for (int q = 0; q < p.stack && ok; ++q) {             // image copy q (stack > 1 only with one CTA tile)
                            int arow = arow0 + q * p.wcap * (int)entry_rows;
                            for (int e = 0; e < len; e += (int)p.group) {
                                if (!mbar_wait(empty, ph ^ 1u, abort_flag, p.wait_limit)) { ok = false; break; }
                                // A stage holds `group` consecutive walk entries.  Their weight tiles are one box of the
                                // image (a whole box also where the walk ends inside it: the rows beyond are the next
                                // entries of the image or, past its end, zero fill, and no MMA reads them); X comes per block.
                                const uint32_t cnt = (uint32_t)min((int)p.group, len - e);
                                mbar_expect_tx(full, p.group * p.entry_bytes + cnt * x_blk_bytes);
                                if (fill_no++ != p.skip_fill) tma_load_2d(dst, &map_a, 0, arow, full);   // (the weight map is tiled here)
                                arow += (int)(p.group * entry_rows);
                                dst += p.stage_bytes; full += 8; empty += 8;
                                if (dst == ring_end) { dst = ring; full = bar_full; empty = bar_empty; ph ^= 1u; }
                            }
                        }
                        if (!ok) break;
                    }
                }
            } else {
                if (p.group == 1) {       // one kept block per stage: the plain loop
                    constexpr int kAhead = 8;            // block columns held in registers ahead of their use
                    dst += p.entry_bytes;
                    for (int t = blockIdx.x; t < p.num_tiles && !*abort_flag; t += gridDim.x) {
                        const int st = t % p.nst, ct = t / p.nst;
                        const int len = min(walk_len[st], p.wcap);
                        const int32_t *cols = walk_col + (int64_t)st * p.wcap;
                        const TileOrigin org = tile_origin<kConv>(p, ct, kTileN);
                        // The block column of entry e is a load in this thread's serial loop; left where it is used
                        // it costs a round trip per stage.  Keep the next kAhead in registers.
                        bool ok = true;
                        for (int q = 0; q < p.stack && ok; ++q) {
                            const int xbox = (ct * p.stack + q) * NT;         // first 64-column box of this group's X columns
                            int col_q[kAhead];
#pragma unroll
                            for (int u = 0; u < kAhead; ++u) col_q[u] = u < len ? cols[u] : 0;
                            for (int e0 = 0; e0 < len && ok; e0 += kAhead) {
#pragma unroll
                                for (int u = 0; u < kAhead; ++u) {
                                    const int e = e0 + u;
                                    if (e >= len) break;
                                    const int jb = col_q[u];
                                    const int krow = jb * p.bk;
                                    if (e + kAhead < len) col_q[u] = cols[e + kAhead];
                                    if (!mbar_wait(empty, ph ^ 1u, abort_flag, p.wait_limit)) { ok = false; break; }
                                    if (fill_no++ != p.skip_fill) {
                                        if constexpr (kConv) {
                                            // block jb = filter tap (i, j), channels [c0, c0 + bk): the tile's pixel box
                                            // shifted by the tap; pixels outside the image read as zero (the padding)
                                            const int tap = jb / p.cv_cpt, c0 = (jb - tap * p.cv_cpt) * p.bk;
                                            const int ti = tap / p.cv_kw, tj = tap - ti * p.cv_kw;
                                            tma_load_4d(dst, &map_x, c0, org.x + tj - p.cv_pad, org.y + ti - p.cv_pad, org.b, full);
                                        } else if (p.x_map_3d) {
                                            tma_load_3d(dst, &map_x, 0, krow, xbox, full);       // the NT boxes of X as one copy
                                        } else {
#pragma unroll
                                            for (int b = 0; b < NT; ++b)
                                                tma_load_2d(dst + b * p.box_bytes, &map_x, (xbox + b) * kBoxN, krow, full);
                                        }
                                    }
                                    dst += p.stage_bytes; full += 8; empty += 8;
                                    if (dst == ring_end + p.entry_bytes) { dst = ring + p.entry_bytes; full = bar_full; empty = bar_empty; ph ^= 1u; }
                                }
                            }
                        }
                        if (!ok) break;
                    }
                } else {
                    constexpr int kAhead = 8;            // block columns held in registers ahead of their use
                    dst += p.group * p.entry_bytes;
                    const int gmask = (int)p.group - 1;
                    bool issue = true;
                    for (int t = blockIdx.x; t < p.num_tiles && !*abort_flag; t += gridDim.x) {
                        const int st = t % p.nst, ct = t / p.nst;
                        const int len = min(walk_len[st], p.wcap);
                        const int32_t *cols = walk_col + (int64_t)st * p.wcap;
                        const TileOrigin org = tile_origin<kConv>(p, ct, kTileN);
                        // The block column of entry e is a load in this thread's serial loop; left where it is used
                        // it costs a round trip per stage.  Keep the next kAhead in registers.
                        bool ok = true;
                        for (int q = 0; q < p.stack && ok; ++q) {
                            const int xbox = (ct * p.stack + q) * NT;         // first 64-column box of this group's X columns
                            int col_q[kAhead];
#pragma unroll
                            for (int u = 0; u < kAhead; ++u) col_q[u] = u < len ? cols[u] : 0;
                            for (int e0 = 0; e0 < len && ok; e0 += kAhead) {
#pragma unroll
                                for (int u = 0; u < kAhead; ++u) {
                                    const int e = e0 + u;
                                    if (e >= len) break;
                                    const int jb = col_q[u];
                                    const int krow = jb * p.bk;
                                    if (e + kAhead < len) col_q[u] = cols[e + kAhead];
                                    const int g = e & gmask;                  // position of the block in its stage
                                    if (g == 0) {
                                        if (!mbar_wait(empty, ph ^ 1u, abort_flag, p.wait_limit)) { ok = false; break; }
                                        issue = fill_no++ != p.skip_fill;
                                    }
                                    const uint32_t xdst = dst + (uint32_t)g * x_blk_bytes;
                                    if (issue) {
                                        if constexpr (kConv) {
                                            // block jb = filter tap (i, j), channels [c0, c0 + bk): the tile's pixel box
                                            // shifted by the tap; pixels outside the image read as zero (the padding)
                                            const int tap = jb / p.cv_cpt, c0 = (jb - tap * p.cv_cpt) * p.bk;
                                            const int ti = tap / p.cv_kw, tj = tap - ti * p.cv_kw;
                                            tma_load_4d(xdst, &map_x, c0, org.x + tj - p.cv_pad, org.y + ti - p.cv_pad, org.b, full);
                                        } else if (p.x_map_3d) {
                                            tma_load_3d(xdst, &map_x, 0, krow, xbox, full);      // the NT boxes of X as one copy
                                        } else {
#pragma unroll
                                            for (int b = 0; b < NT; ++b)
                                                tma_load_2d(xdst + b * p.box_bytes, &map_x, (xbox + b) * kBoxN, krow, full);
                                        }
                                    }
                                    if (g == gmask || e == len - 1) {         // last block of the stage
                                        dst += p.stage_bytes; full += 8; empty += 8;
                                        if (dst == ring_end + p.group * p.entry_bytes) {
                                            dst = ring + p.group * p.entry_bytes; full = bar_full; empty = bar_empty; ph ^= 1u;
                                        }
                                    }
                                }
                            }
                        }
                        if (!ok) break;
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer: steps 2 + 3
        if (lane == 0) {
            const MmaRoleArgs a{ring, bar_full, bar_empty, bar_tfull, bar_tempty, tmem_base, walk_len, abort_flag};
            const int nmma = kSparse ? p.bk / 32 : p.bk / 16;        // K = 32 (sparse) or K = 16 steps per block
            if constexpr (kSparse) {
                switch (nmma) {
                    case 1: mma_role<kTileN, true, kAccStages, 1, kConv>(p, a); break;
                    case 2: mma_role<kTileN, true, kAccStages, 2, kConv>(p, a); break;
                    case 3: mma_role<kTileN, true, kAccStages, 3, kConv>(p, a); break;
                    default: mma_role<kTileN, true, kAccStages, 4, kConv>(p, a); break;
                }
            } else {
                switch (nmma) {
                    case 2: mma_role<kTileN, false, kAccStages, 2, kConv>(p, a); break;
                    case 4: mma_role<kTileN, false, kAccStages, 4, kConv>(p, a); break;
                    case 6: mma_role<kTileN, false, kAccStages, 6, kConv>(p, a); break;
                    default: mma_role<kTileN, false, kAccStages, 8, kConv>(p, a); break;
                }
            }
        }
    } else if (warp < 2 + kEpi) {
        // ------------------------------------------------ epilogue: TMEM -> registers -> smem -> TMA store
        // Warp w may touch TMEM lanes 32*(w%4)..; the kEpi/4 warps that share a lane quarter split the
        // tile's columns among them when the shares are whole 64-column boxes: a warp first pulls its
        // whole share of the accumulator into registers and hands the accumulator back, so that the
        // next tile's MMAs overlap the conversion and the stores.
        constexpr int kParts = kEpi / 4;                                  // warps sharing a lane quarter
        constexpr bool kSplit = (kTileN / kParts) % 64 == 0;
        constexpr int kWarpCols = kSplit ? kTileN / kParts : kTileN;
        const int ew = warp - 2, q = warp & 3, half = ew >> 2;
        const uint32_t stg = staging + (uint32_t)ew * p.stg_bufs * p.stg_tile_bytes;
        uint8_t *stg_gen = smem_gen + (stg - smem_base);
        uint32_t acc = 0, acc_ph = 0, slot = 0;
        for (int t = blockIdx.x; t < p.num_tiles; t += gridDim.x) {
            const int st = t % p.nst, ct = t / p.nst;
            int go = 0;                                      // lane 0 waits, the warp follows it
            if (lane == 0) go = !*abort_flag && mbar_wait(bar_tfull + 8 * acc, acc_ph, abort_flag, p.wait_limit);
            go = __shfl_sync(0xFFFFFFFFu, go, 0);
            if (!go) break;
            tc_fence_after();
            const uint32_t t_addr = tmem_base + acc * kTileN + ((uint32_t)(32 * q) << 16);
            // lane quarter q holds rows 32q.. of the CTA tile; in a stacked tile it belongs to column-tile group
            // 32q / (128 / stack) and holds rows (32q) mod (128 / stack) of W
            // (stack is 1, 2 or 4: 32q / (128 / stack) = q * stack / 4)
            const int grp = (q * p.stack) >> 2;
            const int y0 = st * kTileM + 32 * q - grp * (kTileM >> (p.stack >> 1));
            TileOrigin org = tile_origin<kConv>(p, ct, kTileN);
            if constexpr (!kConv) org.x = (ct * p.stack + grp) * kTileN;
            // layer epilogue on the fp32 accumulator: this lane's row gets its bias, then the activation
            const bool fuse = p.bias != nullptr || p.relu != 0;
            const float bias_v = (p.bias != nullptr && y0 + lane < p.rows) ? p.bias[y0 + lane] : 0.f;
            const float floor_v = p.relu ? 0.f : -__int_as_float(0x7f800000);
            if (y0 >= p.rows) {
                // this lane quarter lies below the last row of W: nothing to drain
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_tempty + 8 * acc);
            } else if constexpr (kSplit) {
                uint32_t accr[kWarpCols];
#pragma unroll
                for (int i = 0; i < kWarpCols / 32; ++i)
                    tmem_ld32(t_addr + half * kWarpCols + 32 * i, *reinterpret_cast<uint32_t(*)[32]>(&accr[32 * i]));
                tmem_ld_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_tempty + 8 * acc);       // accumulator free for the next tile
                if (fuse) {
#pragma unroll
                    for (int i = 0; i < kWarpCols; ++i)
                        accr[i] = __float_as_uint(fmaxf(__uint_as_float(accr[i]) + bias_v, floor_v));
                }
#pragma unroll
                for (int c = 0; c < kWarpCols / kOutCols; ++c) {
                    uint32_t out[32];
                    if constexpr (sizeof(OutT) == 2) {
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            out[i] = pack_bf16(__uint_as_float(accr[c * 64 + 2 * i]), __uint_as_float(accr[c * 64 + 2 * i + 1]));
                    } else {
#pragma unroll
                        for (int i = 0; i < 32; ++i) out[i] = accr[c * 32 + i];
                    }
                    if (kConv && p.cv_nhwc) store_chunk_nhwc<OutT>(p, &map_y, stg, stg_gen, lane, out, org, half * kWarpCols + c * kOutCols, y0);
                    else store_chunk<OutT, kConv>(p, &map_y, stg, stg_gen, lane, out, org, half * kWarpCols + c * kOutCols, y0, slot);
                }
            } else {
                if (half == 0) {
#pragma unroll 1
                    for (int c = 0; c < kTileN / kOutCols; ++c) {
                        uint32_t out[32];
                        if constexpr (sizeof(OutT) == 2) {
                            uint32_t r0[32], r1[32];
                            tmem_ld32(t_addr + c * 64, r0);
                            tmem_ld32(t_addr + c * 64 + 32, r1);
                            tmem_ld_wait();
                            if (fuse) {
#pragma unroll
                                for (int i = 0; i < 32; ++i) {
                                    r0[i] = __float_as_uint(fmaxf(__uint_as_float(r0[i]) + bias_v, floor_v));
                                    r1[i] = __float_as_uint(fmaxf(__uint_as_float(r1[i]) + bias_v, floor_v));
                                }
                            }
#pragma unroll
                            for (int i = 0; i < 16; ++i) {
                                out[i] = pack_bf16(__uint_as_float(r0[2 * i]), __uint_as_float(r0[2 * i + 1]));
                                out[16 + i] = pack_bf16(__uint_as_float(r1[2 * i]), __uint_as_float(r1[2 * i + 1]));
                            }
                        } else {
                            tmem_ld32(t_addr + c * 32, out);
                            tmem_ld_wait();
                            if (fuse) {
#pragma unroll
                                for (int i = 0; i < 32; ++i) out[i] = __float_as_uint(fmaxf(__uint_as_float(out[i]) + bias_v, floor_v));
                            }
                        }
                        if (kConv && p.cv_nhwc) store_chunk_nhwc<OutT>(p, &map_y, stg, stg_gen, lane, out, org, c * kOutCols, y0);
                        else store_chunk<OutT, kConv>(p, &map_y, stg, stg_gen, lane, out, org, c * kOutCols, y0, slot);
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_tempty + 8 * acc);
            }
            if (++acc == kAccStages) { acc = 0; acc_ph ^= 1u; }
        }
        if (lane == 0) bulk_wait_read<0>();
    }

    // ------------------------------------------------ teardown (every wait above is bounded)
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        if (threadIdx.x == 0) atomicCAS(p.status, 0, (int)CRISP_TIMEOUT);
        // let copies that may still be in flight land before shared memory is released
        const unsigned long long t0 = clock64();
        while ((unsigned long long)(clock64() - t0) < 2000000ull) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// --------------------------------------------------------------------- execution image kernels

// Walk lists as a kernel of their own (the body, and what it builds, are described in walks.cuh).
__global__ void __launch_bounds__(256)
build_walks_kernel(Geometry g, WalkArgs a) {
    __shared__ WalkShared sh;
    build_walks_body(g, a, blockIdx.x, sh);
}

// One CTA per walk entry: assemble the entry's weight tile (and 2:4 metadata) in shared memory from
// the canonical values and offsets of the row tiles that keep this block column, zeros for row tiles
// that do not, then write it out with coalesced 16-byte stores.
// Dense image: element (row, k) of the tile at [k/8][row][k%8].
// Sparse image: per aligned 4-group two slots (ascending position, zero-padded); slot pair of group
// q stored at compressed columns 2q, 2q+1 in the same [c/8][row][c%8] layout.  Metadata (2048 bytes):
// 16-byte row L = row%8 + 8*((k/16)%2) + 16*(row/16), 32-bit word k/32, nibble of the 4-group at bit
// (k%16) + 16*((row/8)%2), value idx0 | idx1 << 2.
template <bool kSparse>
__global__ void __launch_bounds__(256)
build_image_kernel(Geometry g, const int32_t *__restrict__ blk_col, const uint16_t *__restrict__ vals,
                   const uint32_t *__restrict__ idx, int r, int nst, int wcap, int stack,
                   const int32_t *__restrict__ walk_col, const int32_t *__restrict__ walk_len, uint32_t a_bytes,
                   uint32_t entry_bytes, int addends, uint8_t *__restrict__ image) {
    extern __shared__ uint4 s_tile4[];
    uint8_t *tile = reinterpret_cast<uint8_t *>(s_tile4);
    __shared__ int s_blk[4];
    // image entries are ordered [copy][CTA tile][walk entry]; copy q of a stacked layer (one CTA tile of at most
    // 128 / stack rows) holds the same weights shifted down by q * 128 / stack rows
    const int per_copy = nst * wcap;
    const int copy = blockIdx.x / per_copy, in_copy = blockIdx.x - copy * per_copy;
    const int st = in_copy / wcap, e = in_copy - st * wcap;
    const int shift = copy * (kTileM / stack);
    if (e >= walk_len[st]) return;
    const int jb = walk_col[(int64_t)st * wcap + e];
    for (uint32_t i = threadIdx.x; i < entry_bytes / 16; i += blockDim.x) s_tile4[i] = make_uint4(0, 0, 0, 0);
    if (threadIdx.x < r) {
        // does row tile st*r + threadIdx.x keep block column jb, and in which slot?
        const int rt = st * r + threadIdx.x;
        int found = -1;
        if (rt < g.nrt) {
            const int32_t *bc = blk_col + (int64_t)rt * g.kkeep;
            int lo = 0, hi = g.kkeep - 1;
            while (lo <= hi) {
                const int mid = (lo + hi) >> 1;
                const int v = bc[mid];
                if (v == jb) { found = rt * g.kkeep + mid; break; }
                if (v < jb) lo = mid + 1; else hi = mid - 1;
            }
        }
        s_blk[threadIdx.x] = found;
    }
    __syncthreads();
    const int groups = g.groups();
    const int vpb = (int)g.vals_per_block();
    const int idx_words = vpb * g.idx_bits / 32;
    const uint32_t field = (1u << g.idx_bits) - 1u;
    // canonical values and offsets of one kept block, staged with coalesced 16-byte loads
    uint16_t *vb = reinterpret_cast<uint16_t *>(tile + entry_bytes);
    uint32_t *ib = reinterpret_cast<uint32_t *>(tile + entry_bytes + (size_t)vpb * 2);
    for (int sub = 0; sub < r; ++sub) {
        const int blk = s_blk[sub];
        if (blk < 0) continue;
        const int row0 = shift + sub * g.bm;
        __syncthreads();
        {
            const uint4 *vsrc = reinterpret_cast<const uint4 *>(vals + (int64_t)blk * vpb);      // vpb*2 is a multiple of 64
            for (int i = threadIdx.x; i < vpb / 8; i += blockDim.x) reinterpret_cast<uint4 *>(vb)[i] = __ldg(vsrc + i);
            const uint32_t *isrc = idx + (int64_t)blk * idx_words;
            for (int i = threadIdx.x; i < idx_words; i += blockDim.x) ib[i] = __ldg(isrc + i);
        }
        __syncthreads();
        if constexpr (!kSparse) {
            for (int o = threadIdx.x; o < vpb; o += blockDim.x) {
                const int item = o / g.n;
                const int lr = item / groups, gi = item - lr * groups;
                const int bit = o * g.idx_bits;
                uint32_t t = ib[bit >> 5] >> (bit & 31);
                if ((bit & 31) + g.idx_bits > 32) t |= ib[(bit >> 5) + 1] << (32 - (bit & 31));
                t &= field;
                const int k = gi * g.m + (int)t, row = row0 + lr;
                *reinterpret_cast<uint16_t *>(tile + (k >> 3) * 2048 + row * 16 + (k & 7) * 2) = vb[o];
            }
        } else {
            // one thread per (local row, 4-group): at most two kept values per addend.  With one addend the pattern
            // guarantees that; with two, the first two values (ascending position) go to the first addend and the
            // rest to the second, each a 2:4-compliant tile with its own metadata, sub bytes apart.
            const int quads = g.bk / 4;
            const uint32_t sub = a_bytes + kMetaBytes;
            for (int item = threadIdx.x; item < g.bm * quads; item += blockDim.x) {
                const int lr = item / quads, qd = item - lr * quads;
                const int row = row0 + lr;
                const int gi = (qd * 4) / g.m;
                uint16_t v4[4] = {0, 0, 0, 0};
                int pos4[4] = {0, 0, 0, 0}, cnt4 = 0;
                for (int vv = 0; vv < g.n; ++vv) {
                    const int o = (lr * groups + gi) * g.n + vv;
                    const int bit = o * g.idx_bits;
                    uint32_t t = ib[bit >> 5] >> (bit & 31);
                    if ((bit & 31) + g.idx_bits > 32) t |= ib[(bit >> 5) + 1] << (32 - (bit & 31));
                    t &= field;
                    const int k = gi * g.m + (int)t;
                    if ((k >> 2) == qd && cnt4 < 2 * addends) { v4[cnt4] = vb[o]; pos4[cnt4] = k & 3; ++cnt4; }
                }
                for (int a = 0; a < addends; ++a) {
                    uint16_t v[2] = {v4[2 * a], v4[2 * a + 1]};
                    int pos[2] = {pos4[2 * a], pos4[2 * a + 1]};
                    const int cnt = cnt4 - 2 * a < 0 ? 0 : (cnt4 - 2 * a > 2 ? 2 : cnt4 - 2 * a);
                    if (cnt == 0) { v[0] = v[1] = 0; pos[0] = 0; pos[1] = 1; }
                    else if (cnt == 1) {
                        v[1] = 0;
                        if (pos[0] == 3) { v[1] = v[0]; v[0] = 0; pos[1] = 3; pos[0] = 0; }
                        else pos[1] = 3;
                    }
                    uint8_t *ta = tile + a * sub;
                    uint32_t *meta = reinterpret_cast<uint32_t *>(ta + a_bytes);
                    const int c0 = 2 * qd;                   // even: both slots share one 16-byte chunk
                    *reinterpret_cast<uint32_t *>(ta + (c0 >> 3) * 2048 + row * 16 + (c0 & 7) * 2) =
                        (uint32_t)v[0] | ((uint32_t)v[1] << 16);
                    const uint32_t nib = (uint32_t)pos[0] | ((uint32_t)pos[1] << 2);
                    const int k0 = qd * 4;
                    const int lrow = (row & 7) + 8 * ((k0 >> 4) & 1) + 16 * (row >> 4);
                    atomicOr(&meta[lrow * 4 + (k0 >> 5)], nib << ((k0 & 15) + 16 * ((row >> 3) & 1)));
                }
            }
        }
    }
    if constexpr (kSparse) {
        // rows that carry no kept block here (row tiles that do not keep it, rows outside a stacked copy's
        // window) still need valid (distinct, ascending) index pairs
        for (int a = 0; a < addends; ++a) {
            uint32_t *meta = reinterpret_cast<uint32_t *>(tile + a * (a_bytes + kMetaBytes) + a_bytes);
            for (int item = threadIdx.x; item < kTileM * (g.bk / 4); item += blockDim.x) {
                const int row = item / (g.bk / 4), qd = item - row * (g.bk / 4);
                const int sub_rt = row >= shift ? (row - shift) / g.bm : r;
                if (sub_rt < r && s_blk[sub_rt] >= 0) continue;
                const int k0 = qd * 4;
                const int lrow = (row & 7) + 8 * ((k0 >> 4) & 1) + 16 * (row >> 4);
                atomicOr(&meta[lrow * 4 + (k0 >> 5)], 0x4u << ((k0 & 15) + 16 * ((row >> 3) & 1)));
            }
        }
    }
    __syncthreads();
    uint4 *out = reinterpret_cast<uint4 *>(image + (int64_t)blockIdx.x * entry_bytes);      // [copy][st][e]
    for (uint32_t i = threadIdx.x; i < entry_bytes / 16; i += blockDim.x) out[i] = s_tile4[i];
}

typedef void (*TcKernel)(const CUtensorMap, const CUtensorMap, const CUtensorMap, TcParams);

constexpr int kMaxDevices = 64;

// One instantiation of the kernel: its entry point, its block size, and the largest dynamic shared memory
// size opted into so far on each device (the attribute belongs to the function on one device).
struct TcVariant {
    TcKernel kern;
    int threads;
    std::atomic<size_t> *configured;     // [kMaxDevices]
};

template <int NT, bool kSparse, int kAccStages, typename OutT, int kEpi, bool kConv>
TcVariant make_variant() {
    static std::atomic<size_t> configured[kMaxDevices];
    return TcVariant{spmm_tc_kernel<NT, kSparse, kAccStages, OutT, kEpi, kConv>, 96 + 32 * kEpi, configured};
}

cudaError_t prepare_variant(const TcVariant &v, int device, size_t smem) {
    if (device < 0 || device >= kMaxDevices) return cudaErrorInvalidDevice;
    if (smem <= v.configured[device].load(std::memory_order_relaxed)) return cudaSuccess;
    cudaError_t e = cudaFuncSetAttribute(reinterpret_cast<const void *>(v.kern),
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e == cudaSuccess) v.configured[device].store(smem, std::memory_order_relaxed);
    return e;
}

// Multiprocessor count of a device, looked up once per device.
int sm_count_of(int device) {
    static std::atomic<int> cache[kMaxDevices];
    if (device < 0 || device >= kMaxDevices) return 148;
    int n = cache[device].load(std::memory_order_relaxed);
    if (n > 0) return n;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || n <= 0) n = 148;
    cache[device].store(n, std::memory_order_relaxed);
    return n;
}

}  // namespace

// ------------------------------------------------------------------------ tensor maps (host)

namespace tc {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

bool make_map_2d(CUtensorMap *map, CUtensorMapDataType dt, int elem_bytes, const void *base, uint64_t inner,
                 uint64_t outer, uint64_t ld_elems, uint32_t box_inner, uint32_t box_outer) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {inner, outer};
    cuuint64_t strides[1] = {ld_elems * (uint64_t)elem_bytes};
    cuuint32_t box[2] = {box_inner, box_outer};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, dt, 2, const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// X viewed as [ncols/64][k][64] (needs ncols % 64 == 0): box = 64 columns x bk rows x nt column groups,
// which lands in shared memory exactly like nt consecutive 2-D boxes.
bool make_map_x3d(CUtensorMap *map, const void *base, uint64_t ncols, uint64_t k, uint64_t ldx, uint32_t bk, uint32_t nt) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint64_t dims[3] = {(cuuint64_t)kBoxN, k, ncols / kBoxN};
    cuuint64_t strides[2] = {ldx * 2ull, (cuuint64_t)kBoxN * 2ull};
    cuuint32_t box[3] = {(cuuint32_t)kBoxN, bk, nt};
    cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The execution image as a matrix of 256-byte rows; one box = one walk entry (weight tile + metadata).
bool make_map_image(CUtensorMap *map, const void *image, uint64_t total_bytes, uint32_t entry_bytes) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn || entry_bytes % 256 != 0 || entry_bytes / 256 > 256 || total_bytes / 256 >= (1ull << 31)) return false;
    cuuint64_t dims[2] = {256, total_bytes / 256};
    cuuint64_t strides[1] = {256};
    cuuint32_t box[2] = {256, entry_bytes / 256};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(image), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// A 4-D tiled map (dims/box innermost first, strides of dimensions 1..3 in bytes).  The swizzle span is the
// inner box: 128, 64 or 32 bytes, none for 16.  (A store through a map whose span is wider than its inner
// box raised an illegal memory access on B200, although the map encodes.)
bool make_map_4d(CUtensorMap *map, CUtensorMapDataType dt, int elem_bytes, const void *base, const uint64_t (&dims)[4],
                 const uint64_t (&strides_bytes)[3], const uint32_t (&box)[4], bool swizzle) {
    EncodeTiledFn fn = encode_tiled_fn();
    const uint64_t inner = (uint64_t)box[0] * elem_bytes;
    if (!fn || (inner != 128 && inner != 64 && inner != 32 && inner != 16)) return false;
    const CUtensorMapSwizzle swz = !swizzle ? CU_TENSOR_MAP_SWIZZLE_NONE
                                 : inner == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : inner == 64 ? CU_TENSOR_MAP_SWIZZLE_64B
                                 : inner == 32 ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_NONE;
    cuuint64_t d[4] = {dims[0], dims[1], dims[2], dims[3]};
    cuuint64_t sb[3] = {strides_bytes[0], strides_bytes[1], strides_bytes[2]};
    cuuint32_t b[4] = {box[0], box[1], box[2], box[3]};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(map, dt, 4, const_cast<void *>(base), d, sb, b, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool tensor_maps_available() { return encode_tiled_fn() != nullptr; }

}  // namespace tc

// ------------------------------------------------------------------ interface to crisp_api.cu

bool tc_pattern_is_sparse(const Geometry &g) { return g.n <= 2; }   // <= 2 kept per aligned 4-group

TcImageLayout tc_image_layout(const Geometry &g, int kind) {
    const bool sparse = kind != CRISP_PATH_DENSE;
    TcImageLayout L;
    L.addends = kind == CRISP_PATH_SPARSE2 ? 2 : 1;
    L.r = kTileM / g.bm;
    L.nst = (g.nrt + L.r - 1) / L.r;
    const int64_t cap = (int64_t)L.r * g.kkeep;
    L.wcap = (int)(cap < g.nblk ? cap : g.nblk);
    // thin layers (a single CTA tile with at most 64 or 32 rows): 2 or 4 copies of every walk entry, shifted to
    // the other lane quarters, let one accumulator cover 2 or 4 column tiles (see launch_spmm_tc)
    L.stack = 1;
    if (L.nst == 1 && g.bm < kTileM) L.stack = g.rows <= 32 ? 4 : (g.rows <= 64 ? 2 : 1);
    L.a_bytes = (uint32_t)(kTileM * g.bk * 2) / (sparse ? 2 : 1);
    L.entry_bytes = (uint32_t)L.addends * (L.a_bytes + (sparse ? kMetaBytes : 0));
    L.walk_col_off = 0;
    L.walk_len_off = align_up((size_t)L.nst * L.wcap * sizeof(int32_t) + 4);
    L.image_off = L.walk_len_off + align_up((size_t)L.nst * sizeof(int32_t) + 4);
    L.total_bytes = L.image_off + align_up((size_t)L.stack * L.nst * L.wcap * L.entry_bytes + 16);
    return L;
}

WalkArgs tc_walk_args(const Geometry &g, int kind, const int32_t *d_blk_col, uint8_t *d_exec) {
    const TcImageLayout L = tc_image_layout(g, kind);
    WalkArgs a;
    a.blk_col = d_blk_col;
    a.r = L.r; a.nst = L.nst; a.wcap = L.wcap;
    a.nctas = g.nrt * g.kkeep == 0 ? 0 : L.nst;
    a.walk_col = reinterpret_cast<int32_t *>(d_exec + L.walk_col_off);
    a.walk_len = reinterpret_cast<int32_t *>(d_exec + L.walk_len_off);
    return a;
}

cudaError_t launch_build_image(const Geometry &g, int kind, const int32_t *d_blk_col, const uint16_t *d_vals,
                               const uint32_t *d_idx, uint8_t *d_exec, bool tiles_done, bool walks_done,
                               cudaStream_t st) {
    const bool sparse = kind != CRISP_PATH_DENSE;
    const TcImageLayout L = tc_image_layout(g, kind);
    if (g.nrt * g.kkeep == 0) return cudaSuccess;
    int32_t *walk_col = reinterpret_cast<int32_t *>(d_exec + L.walk_col_off);
    int32_t *walk_len = reinterpret_cast<int32_t *>(d_exec + L.walk_len_off);
    uint8_t *image = d_exec + L.image_off;
    if (!walks_done) build_walks_kernel<<<L.nst, 256, 0, st>>>(g, tc_walk_args(g, kind, d_blk_col, d_exec));
    if (tiles_done) return cudaGetLastError();       // the encode kernel already wrote the weight tiles
    const int grid = L.stack * L.nst * L.wcap;
    const size_t smem_img = (size_t)L.entry_bytes + (size_t)g.vals_per_block() * 2 + (size_t)(g.vals_per_block() * g.idx_bits / 32) * 4 + 16;
    if (smem_img > 48 * 1024) {      // large blocks with many kept values need the opt-in shared memory size
        cudaError_t e = sparse ? cudaFuncSetAttribute(build_image_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_img)
                               : cudaFuncSetAttribute(build_image_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_img);
        if (e != cudaSuccess) return e;
    }
    if (sparse)
        build_image_kernel<true><<<grid, 256, smem_img, st>>>(g, d_blk_col, d_vals, d_idx, L.r, L.nst, L.wcap, L.stack, walk_col,
                                                                    walk_len, L.a_bytes, L.entry_bytes, L.addends, image);
    else
        build_image_kernel<false><<<grid, 256, smem_img, st>>>(g, d_blk_col, d_vals, d_idx, L.r, L.nst, L.wcap, L.stack, walk_col,
                                                                     walk_len, L.a_bytes, L.entry_bytes, L.addends, image);
    return cudaGetLastError();
}

// Whether the tensor-core kernel can address these operands (TMA: 16-byte aligned base and pitch).
bool tc_operands_ok(const void *x, int64_t ldx, const void *y, int64_t ldy, int y_dtype, int64_t ncols) {
    const int ye = y_dtype ? 4 : 2;
    return (reinterpret_cast<uintptr_t>(x) % 16 == 0) && (reinterpret_cast<uintptr_t>(y) % 16 == 0) &&
           (ldx * 2) % 16 == 0 && (ldy * ye) % 16 == 0 && ncols < (1ll << 31) && encode_tiled_fn() != nullptr;
}

// Everything one launch needs, and the operands it was planned for.  Encoding three tensor maps costs a few
// microseconds of host time per call, which small layers notice; a product on the same buffers reuses the plan.
struct TcPlan {
    // key
    const void *x, *y, *bias;
    int64_t ldx, ldy, ncols;
    int y_dtype, relu, nt_override, group_override, device, skip_stage;
    unsigned long long wait_limit;
    bool has_conv;
    ConvGeom conv;
    // plan
    CUtensorMap mx, my, ma;
    TcParams p;
    TcVariant variant;
    int grid;
    size_t smem;
    crisp_launch_info_t info;
};

void tc_plan_destroy(TcPlan *plan) { delete plan; }

namespace {

bool same_conv(const ConvGeom &a, const ConvGeom &b) {
    return a.batch == b.batch && a.height == b.height && a.width == b.width && a.channels == b.channels &&
           a.kh == b.kh && a.kw == b.kw && a.pad == b.pad && a.nhwc_out == b.nhwc_out;
}

// Tile shape, shared-memory split, tensor maps and kernel variant for one product.
cudaError_t make_plan(const crisp_handle_s *h, int kind, const uint16_t *d_x, int64_t ldx, int64_t ncols, void *d_y,
                      int64_t ldy, int y_dtype, const ConvGeom *conv, int device, TcPlan *plan) {
    const Geometry &g = h->g;
    const uint8_t *d_exec = h->d_exec;
    const int nt_override = h->nt_override;
    const bool sparse = kind != CRISP_PATH_DENSE;
    const TcImageLayout L = tc_image_layout(g, kind);
    const int sm_count = sm_count_of(device);
    // column tile: 4 boxes (256 columns).  For the sparse image that leaves room for one accumulator
    // only (256 + 8 metadata columns), which still beats 3 boxes with two accumulators: the kernel is
    // bound by bytes into shared memory, and wider tiles amortise the weight tile over more columns.
    int nt = (nt_override >= 1 && nt_override <= 4) ? nt_override : 4;
    const int64_t boxes = (ncols + kBoxN - 1) / kBoxN;
    if (boxes < nt) nt = (int)boxes;
    // thin layers: a tile covers `stack` column tiles (one per group of accumulator lanes); not for the gather
    // (only where it pays: walks that stay short when repeated per group, and enough columns to keep every SM busy)
    int stack = conv ? 1 : L.stack;
    if (stack > 1 && (L.wcap * stack > 8 || (ncols + stack * nt * kBoxN - 1) / (stack * nt * kBoxN) < sm_count)) stack = 1;
    const int wlen = L.wcap * stack;                       // blocks per tile
    // small layers are latency-bound: narrower tiles (down to 2 boxes) until at least half of the SMs have one
    if (nt_override <= 0)
        while (nt > 2 && (int64_t)L.nst * ((ncols + stack * nt * kBoxN - 1) / (stack * nt * kBoxN)) < sm_count / 2) --nt;
    // Short walks: the epilogue and the accumulator hand-over are the longest chain.  One warp per 64-column
    // box and lane quarter; under the sparse image three boxes, so that two accumulators fit beside the
    // metadata columns and the next tile's MMAs do not wait for the drain.
    const bool short_walk = wlen <= 8 && nt_override <= 0;
    if (short_walk && wlen <= 2 && sparse && nt == 4 && !conv) nt = 3;
    TcParams p = {};
    if (conv) {
        // Pixel box of a column tile: tw * th * tb = 256 (or 128) output pixels, tw a power of two that divides
        // a 128-byte staging row, whole staging rows per image.  Among the shapes that fit, the one that
        // covers the fewest pixels outside the images wins (then the widest, then the tallest).
        if (nt == 3) nt = 4;
        if (nt < 2) nt = 2;
        const int f32c = y_dtype != 0 ? 32 : 64;
        int64_t best = -1;
        for (int tw = 32; tw >= 8; tw >>= 1)
            for (int th = 32; th >= 1; th >>= 1) {
                const int n_tile = nt * kBoxN;
                if (n_tile % (tw * th) != 0 || f32c % tw != 0 || (tw * th) % f32c != 0) continue;
                const int tb = n_tile / (tw * th);
                const int64_t covered = (int64_t)((conv->wo + tw - 1) / tw) * tw * ((conv->ho + th - 1) / th) * th *
                                        ((conv->batch + tb - 1) / tb) * tb;
                if (best < 0 || covered < best) { best = covered; p.cv_tw = tw; p.cv_th = th; p.cv_tb = tb; }
            }
        if (best < 0) return cudaErrorInvalidValue;
        p.conv = 1;
        p.cv_tiles_x = (conv->wo + p.cv_tw - 1) / p.cv_tw;
        p.cv_tiles_y = (conv->ho + p.cv_th - 1) / p.cv_th;
        p.cv_cpt = conv->channels / g.bk;
        p.cv_kw = conv->kw; p.cv_pad = conv->pad;
        p.cv_wo = conv->wo; p.cv_ho = conv->ho; p.cv_batch = conv->batch;
    }
    p.image = d_exec + L.image_off;
    p.walk_col = reinterpret_cast<const int32_t *>(d_exec + L.walk_col_off);
    p.walk_len = reinterpret_cast<const int32_t *>(d_exec + L.walk_len_off);
    p.status = h->d_status;
    p.bias = h->epilogue.bias; p.relu = h->epilogue.relu;
    p.wait_limit = h->wait_limit_cycles ? h->wait_limit_cycles : kWaitLimitCycles;
    p.skip_fill = h->debug_skip_stage;
    p.stack = stack;
    p.nst = L.nst; p.wcap = L.wcap; p.bk = g.bk; p.rows = g.rows; p.ncols = ncols; p.y = d_y; p.ldy = ldy;
    p.n_col_tiles = (int)((ncols + stack * nt * kBoxN - 1) / (stack * nt * kBoxN));
    if (conv) p.n_col_tiles = p.cv_tiles_x * p.cv_tiles_y * ((conv->batch + p.cv_tb - 1) / p.cv_tb);
    const int64_t tiles = (int64_t)p.n_col_tiles * L.nst;
    if (tiles > 0x7FFFFFFF) return cudaErrorInvalidValue;
    p.num_tiles = (int)tiles;
    p.a_bytes = L.a_bytes; p.entry_bytes = L.entry_bytes; p.addends = (uint32_t)L.addends;
    p.box_bytes = (uint32_t)(kBoxN * g.bk * 2);
    const uint32_t block_bytes = p.entry_bytes + nt * p.box_bytes;     // one kept block: weight tile (+ metadata) and X tile
    // Shared memory (the whole 227 KB; the base is 1024-aligned): the ring gets as many stages as fit next
    // to one staging tile per epilogue warp; what is left goes to the walk-list copy and to more staging
    // tiles.  Short walks are store-heavy and need no deep ring: they give stages up for staging tiles.
    const uint32_t avail = kSmemBudget + 1024;
    const uint32_t epi = short_walk && nt >= 3 ? 4u * (uint32_t)nt : 8u;
    const bool nhwc = conv && conv->nhwc_out;                // transposed chunks need whole 4096-byte staging tiles
    const uint32_t fixed = epi * (nhwc ? 2 * kWideStageBytes : kWideStageBytes) + 256;
    // Blocks per pipeline stage.  A stage costs each single-thread role (weight producer, X producer, MMA issuer)
    // a fixed 300 to 400 cycles of waits, barrier arrivals and loop overhead on top of its copies and MMAs, which
    // for short or narrow blocks is more than the tensor core needs for the block.  Where the ring still holds at
    // least three of them, a stage therefore takes two or four consecutive walk entries: one weight-tile copy, one
    // wait and one commit for all of them.  (Needs the tiled weight map; 256-column tiles of 64-deep blocks stay
    // at one block per stage, two would leave room for two stages only.)
    uint32_t group = 1;
    const bool bounded = h->group_override > 0;        // a caller's bound: the largest feasible size below it
    for (uint32_t g = 4; g >= 2; g >>= 1) {
        if (bounded ? (int)g > h->group_override : L.wcap < 16) continue;   // walks below 16 blocks gain nothing (measured)
        if ((g * p.entry_bytes) % 256 != 0 || (g * p.entry_bytes) / 256 > 256) continue;   // one box of the weight map
        if ((avail - fixed) / (g * block_bytes) >= 3) { group = g; break; }
    }
    p.group = group;
    p.stage_bytes = group * block_bytes;
    uint32_t stages = (avail - fixed) / p.stage_bytes;
    const uint32_t max_stages = block_bytes <= 24 * 1024 ? (wlen <= 8 ? 6u : 7u) : (wlen <= 8 ? 4u : 8u);
    if (stages > max_stages) stages = max_stages;
    if (stages < 2) return cudaErrorInvalidValue;
    p.num_stages = stages;
    uint32_t left = avail - fixed - stages * p.stage_bytes;
    const uint32_t cache_bytes = (uint32_t)align_up((size_t)L.nst * (L.wcap + 1) * sizeof(int32_t), 16);
    p.walk_cache = cache_bytes <= left ? 1u : 0u;
    if (p.walk_cache) left -= cache_bytes;
    // staging per warp beyond the one 16-row tile already counted: two 32-row tiles, two 16-row tiles, or none
    const uint32_t unit = epi * kWideStageBytes;
    if (nhwc) { p.stg_bufs = 1; p.stg_tile_bytes = 2 * kWideStageBytes; }
    else if (left >= 3 * unit) { p.stg_bufs = 2; p.stg_tile_bytes = 2 * kWideStageBytes; }
    else if (left >= unit) { p.stg_bufs = 2; p.stg_tile_bytes = kWideStageBytes; }
    else { p.stg_bufs = 1; p.stg_tile_bytes = kWideStageBytes; }
    plan->smem = (size_t)stages * p.stage_bytes + (size_t)epi * p.stg_bufs * p.stg_tile_bytes + 256 +
                 (p.walk_cache ? cache_bytes : 0);

    CUtensorMap &mx = plan->mx, &my = plan->my, &ma = plan->ma;
    p.a_map = make_map_image(&ma, p.image, (uint64_t)L.stack * L.nst * L.wcap * L.entry_bytes, group * L.entry_bytes);
    if (!p.a_map) {
        if (group > 1) return cudaErrorInvalidValue;         // excluded above: a box of `group` entries fits the map's limits
        ma = CUtensorMap{};
    }
    const bool f32 = y_dtype != 0;
    p.stg_swz_mask = 7;
    if (conv) {
        p.stg_swz_mask = (uint32_t)(p.cv_tw * (f32 ? 4 : 2)) / 16 - 1;      // 128 / 64 / 32 / 16-byte inner box of map_y
        p.cv_nhwc = conv->nhwc_out;
        p.cv_plain = (!p.cv_nhwc && ((int64_t)conv->wo * (f32 ? 4 : 2)) % 16 != 0) || (ldy * (f32 ? 4 : 2)) % 16 != 0 ||
                     reinterpret_cast<uintptr_t>(d_y) % 16 != 0;
        for (p.cv_tw_log2 = 0; (1 << p.cv_tw_log2) < p.cv_tw; ++p.cv_tw_log2) {}
        for (p.cv_img_log2 = 0; (1 << p.cv_img_log2) < p.cv_tw * p.cv_th; ++p.cv_img_log2) {}
        // activation [batch][height][width][channels] and Y [rows][batch][ho][wo] as 4-D tensors
        if (!p.a_map) return cudaErrorInvalidValue;
        p.x_map_3d = 0;
        const uint64_t c = (uint64_t)conv->channels, w = (uint64_t)conv->width, hh = (uint64_t)conv->height;
        const uint64_t xd[4] = {c, w, hh, (uint64_t)conv->batch}, xs[3] = {c * 2, w * c * 2, hh * w * c * 2};
        const uint32_t xb[4] = {(uint32_t)g.bk, (uint32_t)p.cv_tw, (uint32_t)p.cv_th, (uint32_t)p.cv_tb};
        if (!make_map_4d(&mx, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, d_x, xd, xs, xb)) return cudaErrorInvalidValue;
        const uint64_t es = f32 ? 4 : 2, wo = (uint64_t)conv->wo, ho = (uint64_t)conv->ho;
        const uint64_t yd[4] = {wo, ho, (uint64_t)conv->batch, (uint64_t)g.rows}, ys[3] = {wo * es, ho * wo * es, (uint64_t)ldy * es};
        const uint32_t yb[4] = {(uint32_t)p.cv_tw, (uint32_t)((f32 ? 32 : 64) / p.cv_tw), 1u, p.stg_tile_bytes / 128};
        if (p.cv_plain) my = CUtensorMap{};
        else if (p.cv_nhwc) {
            // Y [batch][ho][wo][ldy]: a chunk is {32 channels, tw, pixels / tw, 1}, laid out densely in the staging tile
            const uint64_t nd[4] = {(uint64_t)g.rows, wo, ho, (uint64_t)conv->batch};
            const uint64_t ns[3] = {(uint64_t)ldy * es, wo * (uint64_t)ldy * es, ho * wo * (uint64_t)ldy * es};
            const uint32_t nb[4] = {32u, (uint32_t)p.cv_tw, (uint32_t)((f32 ? 32 : 64) / p.cv_tw), 1u};
            if (!make_map_4d(&my, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (int)es, d_y, nd, ns, nb,
                             /*swizzle=*/false))
                return cudaErrorInvalidValue;
        } else if (!make_map_4d(&my, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (int)es, d_y, yd, ys, yb))
            return cudaErrorInvalidValue;
    } else {
        p.x_map_3d = (ncols % kBoxN == 0) &&
                     make_map_x3d(&mx, d_x, (uint64_t)ncols, (uint64_t)g.k, (uint64_t)ldx, (uint32_t)g.bk, (uint32_t)nt);
        if (!p.x_map_3d && !make_map_2d(&mx, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, d_x, (uint64_t)ncols, (uint64_t)g.k,
                                        (uint64_t)ldx, kBoxN, (uint32_t)g.bk))
            return cudaErrorInvalidValue;
        if (!make_map_2d(&my, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, f32 ? 4 : 2, d_y,
                         (uint64_t)ncols, (uint64_t)g.rows, (uint64_t)ldy, f32 ? 32 : 64, p.stg_tile_bytes / 128))
            return cudaErrorInvalidValue;
    }
    plan->grid = (int)(tiles < sm_count ? tiles : sm_count);
    plan->p = p;

    int acc = 2;
#define CRISP_TC_VARIANT_C(NTV, SP, ACC, EPI, CONV)                                                       \
    (acc = ACC, f32 ? make_variant<NTV, SP, ACC, float, EPI, CONV>() : make_variant<NTV, SP, ACC, uint16_t, EPI, CONV>())
#define CRISP_TC_VARIANT_E(NTV, SP, ACC, EPI) CRISP_TC_VARIANT_C(NTV, SP, ACC, EPI, false)
#define CRISP_TC_VARIANT(NTV, SP, ACC) CRISP_TC_VARIANT_E(NTV, SP, ACC, 8)
    if (conv) {                              // the gather uses 128- or 256-pixel tiles only
        if (sparse) {
            if (nt == 2) plan->variant = CRISP_TC_VARIANT_C(2, true, 2, 8, true);
            else plan->variant = epi == 16 ? CRISP_TC_VARIANT_C(4, true, 1, 16, true) : CRISP_TC_VARIANT_C(4, true, 1, 8, true);
        } else {
            if (nt == 2) plan->variant = CRISP_TC_VARIANT_C(2, false, 2, 8, true);
            else plan->variant = epi == 16 ? CRISP_TC_VARIANT_C(4, false, 2, 16, true) : CRISP_TC_VARIANT_C(4, false, 2, 8, true);
        }
    } else if (sparse) {
        switch (nt) {
            case 1: plan->variant = CRISP_TC_VARIANT(1, true, 2); break;
            case 2: plan->variant = CRISP_TC_VARIANT(2, true, 2); break;
            case 3: plan->variant = epi == 12 ? CRISP_TC_VARIANT_E(3, true, 2, 12) : CRISP_TC_VARIANT(3, true, 2); break;
            default: plan->variant = epi == 16 ? CRISP_TC_VARIANT_E(4, true, 1, 16) : CRISP_TC_VARIANT(4, true, 1); break;
        }
    } else {
        switch (nt) {
            case 1: plan->variant = CRISP_TC_VARIANT(1, false, 2); break;
            case 2: plan->variant = CRISP_TC_VARIANT(2, false, 2); break;
            case 3: plan->variant = CRISP_TC_VARIANT(3, false, 2); break;
            default: plan->variant = epi == 16 ? CRISP_TC_VARIANT_E(4, false, 2, 16) : CRISP_TC_VARIANT(4, false, 2); break;
        }
    }
#undef CRISP_TC_VARIANT
#undef CRISP_TC_VARIANT_E
#undef CRISP_TC_VARIANT_C
    crisp_launch_info_t &info = plan->info;
    info.path = kind;
    info.tile_cols = nt * kBoxN;
    info.accumulators = acc;
    info.stack = stack;
    info.epilogue_warps = plan->variant.threads / 32 - 3;
    info.stages = (int)stages;
    info.ctas = plan->grid;
    info.conv = conv ? 1 : 0;
    info.stage_blocks = (int)p.group;
    return prepare_variant(plan->variant, device, plan->smem);
}

}  // namespace

cudaError_t launch_spmm_tc(crisp_handle_s *h, int kind, const uint16_t *d_x, int64_t ldx, int64_t ncols,
                           void *d_y, int64_t ldy, int y_dtype, const ConvGeom *conv, cudaStream_t st) {
    int device = 0;
    cudaError_t e = cudaGetDevice(&device);
    if (e != cudaSuccess) return e;
    TcPlan *plan = h->plan;
    const bool hit = plan && plan->x == d_x && plan->y == d_y && plan->ldx == ldx && plan->ldy == ldy &&
                     plan->ncols == ncols && plan->y_dtype == y_dtype && plan->bias == h->epilogue.bias &&
                     plan->relu == h->epilogue.relu && plan->nt_override == h->nt_override &&
                     plan->group_override == h->group_override &&
                     plan->device == device && plan->skip_stage == h->debug_skip_stage &&
                     plan->wait_limit == h->wait_limit_cycles && plan->has_conv == (conv != nullptr) &&
                     (!conv || same_conv(plan->conv, *conv)) && plan->p.status == h->d_status &&
                     plan->info.path == kind;
    if (!hit) {
        if (!plan) {
            plan = new (std::nothrow) TcPlan;
            if (!plan) return cudaErrorMemoryAllocation;
            h->plan = plan;
        }
        plan->x = nullptr;                                  // not valid until the plan below is complete
        e = make_plan(h, kind, d_x, ldx, ncols, d_y, ldy, y_dtype, conv, device, plan);
        if (e != cudaSuccess) return e;
        plan->x = d_x; plan->y = d_y; plan->bias = h->epilogue.bias;
        plan->ldx = ldx; plan->ldy = ldy; plan->ncols = ncols;
        plan->y_dtype = y_dtype; plan->relu = h->epilogue.relu; plan->nt_override = h->nt_override;
        plan->group_override = h->group_override;
        plan->device = device; plan->skip_stage = h->debug_skip_stage; plan->wait_limit = h->wait_limit_cycles;
        plan->has_conv = conv != nullptr;
        if (conv) plan->conv = *conv;
    }
    plan->variant.kern<<<plan->grid, plan->variant.threads, plan->smem, st>>>(plan->mx, plan->my, plan->ma, plan->p);
    h->last = plan->info;
    return cudaGetLastError();
}

}  // namespace crisp
