// Internal declarations shared by the translation units of libcrisp.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "crisp.h"

namespace crisp {

// Layer epilogue applied to the fp32 accumulator before the store: Y = act(W*X + bias).
struct Epilogue {
    const float *bias;      // device, [rows] fp32, or nullptr
    int relu;               // max(., 0) after the bias
};

// Shape of one layer after padding to whole blocks.
struct Geometry {
    int rows, k, n, m, bm, bk;
    int score_mode;
    int nrt;        // row tiles
    int nblk;       // k-blocks per row tile
    int kkeep;      // kept k-blocks per row tile
    int wpr;        // uint32 words of bit mask per (padded) row = nblk * bk / 32
    int idx_bits;   // log2(m)
    __host__ __device__ int64_t mp() const { return (int64_t)nrt * bm; }
    __host__ __device__ int64_t kp() const { return (int64_t)nblk * bk; }
    __host__ __device__ int groups() const { return bk / m; }
    __host__ __device__ int64_t vals_per_block() const { return (int64_t)bm * groups() * n; }
    __host__ __device__ int64_t nnz() const { return (int64_t)nrt * kkeep * vals_per_block(); }
    __host__ __device__ int64_t idx_words() const { return (nnz() * idx_bits + 31) / 32; }
};

constexpr size_t kAlign = 256;
inline size_t align_up(size_t x, size_t a = kAlign) { return (x + a - 1) / a * a; }

}  // namespace crisp

struct crisp_mask_s {
    crisp::Geometry g;
    int32_t *d_blk_col;     // [nrt, kkeep]
    uint32_t *d_nm_bits;    // [mp, wpr]
    int image_kind;         // CRISP_PATH_* of the execution image crisp_encode will lay out: fixed when the
                            // mask is built, so that crisp_encode_sizes and crisp_encode always agree
};

namespace crisp {
// Launch plan of the tensor-core kernel for one set of operands (spmm_tc.cu); cached in the handle so that
// repeated products on the same buffers skip the tensor-map encoding.
struct TcPlan;
void tc_plan_destroy(TcPlan *plan);
}  // namespace crisp

struct crisp_handle_s {
    crisp::Geometry g;
    // canonical format
    int32_t *d_blk_col;
    uint16_t *d_vals;
    uint32_t *d_idx;
    // execution image
    int32_t *d_status;      // first word of the exec buffer
    uint8_t *d_exec;        // payload after the 256-byte header
    size_t exec_payload_bytes;
    int exec_kind;          // CRISP_PATH_* the image was laid out for (DIRECT = none)
    int forced_path;        // -1 = default
    crisp::Epilogue epilogue;
    int nt_override;        // tuning: 64-column boxes per CTA tile (0 = chosen by the library)
    int group_override;     // tuning: most kept blocks a pipeline stage may take (0 = chosen by the library)
    unsigned long long wait_limit_cycles;   // bound of every in-kernel wait (0 = default)
    int debug_skip_stage;   // test hook: the producer leaves out the loads of this pipeline fill (-1 = none)
    crisp::TcPlan *plan;    // cached launch plan of the last tensor-core product (or nullptr)
    crisp_launch_info_t last;               // what the last product on this handle launched
};

namespace crisp {

struct WalkArgs;

// mask_kernels.cu
cudaError_t launch_build_mask(const float *d_s, int64_t ld, const Geometry &g, int32_t *d_blk_col,
                              uint32_t *d_nm_bits, void *d_workspace, size_t workspace_bytes, bool max_known,
                              cudaStream_t st);
// per-row-tile selection alone, on the scores and group bits an earlier launch_build_mask left behind
cudaError_t launch_block_select(const Geometry &g, const void *d_workspace, int32_t *d_blk_col, uint32_t *d_nm_bits,
                                cudaStream_t st);
size_t mask_workspace_bytes(const Geometry &g);

// encode_kernels.cu
cudaError_t launch_encode_canonical(const uint16_t *d_w, int64_t ld, const Geometry &g,
                                    const int32_t *d_mask_blk_col, const uint32_t *d_nm_bits,
                                    int32_t *d_blk_col, uint16_t *d_vals, uint32_t *d_idx,
                                    int tile_kind, uint8_t *d_image, uint32_t a_bytes, uint32_t entry_bytes,
                                    const struct WalkArgs *walks, cudaStream_t st);
cudaError_t launch_decode(const Geometry &g, const int32_t *d_blk_col, const uint16_t *d_vals,
                          const uint32_t *d_idx, uint16_t *d_w, int64_t ld, cudaStream_t st);

// spmm_tc.cu: tensor-core path and its execution image
struct TcImageLayout {
    int r;                  // row tiles per 128-row CTA tile
    int nst;                // 128-row CTA tiles
    int wcap;               // capacity of one CTA tile's walk list (union of its row tiles' kept blocks)
    int stack;              // copies of the image, each shifted by 128 / stack rows (thin single-tile layers)
    uint32_t a_bytes;       // weight tile bytes per walk entry
    uint32_t entry_bytes;   // weight tile + metadata (two of each for the two-addend image)
    int addends;            // sparse tiles per walk entry: 1, or 2 for the two-addend image
    size_t walk_col_off, walk_len_off, image_off, total_bytes;   // offsets inside the exec payload
};
bool tc_pattern_is_sparse(const Geometry &g);
TcImageLayout tc_image_layout(const Geometry &g, int kind);      // kind: CRISP_PATH_DENSE / SPARSE / SPARSE2
// walk lists of the tensor-core kernel (walks.cuh): built by CTAs of the encode kernel (walks != nullptr in
// launch_encode_canonical, then walks_done below) or by a kernel of their own
struct WalkArgs tc_walk_args(const Geometry &g, int kind, const int32_t *d_mask_blk_col, uint8_t *d_exec);
cudaError_t launch_build_image(const Geometry &g, int kind, const int32_t *d_blk_col, const uint16_t *d_vals,
                               const uint32_t *d_idx, uint8_t *d_exec, bool tiles_done, bool walks_done,
                               cudaStream_t st);
bool tc_operands_ok(const void *x, int64_t ldx, const void *y, int64_t ldy, int y_dtype, int64_t ncols);
// Convolution geometry for the implicit-GEMM mode (stride 1): NHWC activation, ho x wo output pixels.
struct ConvGeom { int batch, height, width, channels, kh, kw, pad, ho, wo, nhwc_out; };
// conv == nullptr: d_x is the [k, ncols] matrix.  Otherwise d_x is the activation and ncols = batch*ho*wo.
// `h->plan` is reused when the operands, shape and epilogue are those of the previous call; `h->last` is filled in.
cudaError_t launch_spmm_tc(crisp_handle_s *h, int kind, const uint16_t *d_x, int64_t ldx, int64_t ncols,
                           void *d_y, int64_t ldy, int y_dtype, const ConvGeom *conv, cudaStream_t st);
// spmm_direct.cu
cudaError_t launch_spmm_direct(const Geometry &g, const int32_t *d_blk_col, const uint16_t *d_vals,
                               const uint32_t *d_idx, const uint16_t *d_x, int64_t ldx, int64_t ncols,
                               void *d_y, int64_t ldy, int y_dtype, const Epilogue &epi, cudaStream_t st);

}  // namespace crisp
