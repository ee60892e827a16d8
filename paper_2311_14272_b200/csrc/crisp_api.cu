// C ABI of libcrisp: argument checking, buffer carving and kernel dispatch.
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "crisp_internal.h"
#include "walks.cuh"

using crisp::align_up;
using crisp::Geometry;
using crisp::kAlign;

namespace {

constexpr int kMaxBlocksPerRowTile = 4096;   // block_select_kernel keeps a row tile's scores in shared memory
constexpr int kMaxRowTiles = 65535;          // grid.y

bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

crisp_status_t make_geometry(const crisp_layer_desc_t *d, Geometry *g) {
    if (!d) return CRISP_INVALID_ARG;
    if (d->rows <= 0 || d->k <= 0) return CRISP_BAD_SHAPE;
    if (d->m != 4 && d->m != 8) return CRISP_UNSUPPORTED;
    if (d->n < 1 || d->n > d->m) return CRISP_INVALID_ARG;
    if (d->block_rows != 32 && d->block_rows != 64 && d->block_rows != 128) return CRISP_UNSUPPORTED;
    if (d->block_k < 32 || d->block_k > 128 || d->block_k % 32 != 0) return CRISP_UNSUPPORTED;
    if (!(d->keep_ratio >= 0.0) || d->keep_ratio > 1.0) return CRISP_INVALID_ARG;
    if (d->score_mode != 0 && d->score_mode != 1) return CRISP_INVALID_ARG;
    g->rows = d->rows; g->k = d->k; g->n = d->n; g->m = d->m;
    g->bm = d->block_rows; g->bk = d->block_k; g->score_mode = d->score_mode;
    g->nrt = (d->rows + d->block_rows - 1) / d->block_rows;
    g->nblk = (d->k + d->block_k - 1) / d->block_k;
    if (g->nblk > kMaxBlocksPerRowTile || g->nrt > kMaxRowTiles) return CRISP_UNSUPPORTED;
    int kk = (int)std::floor(d->keep_ratio * (double)g->nblk + 0.5);
    g->kkeep = kk < 0 ? 0 : (kk > g->nblk ? g->nblk : kk);
    g->wpr = g->nblk * g->bk / 32;
    g->idx_bits = d->m == 4 ? 2 : 3;
    return CRISP_OK;
}

void fill_desc(const Geometry &g, double keep_ratio, crisp_layer_desc_t *d) {
    d->rows = g.rows; d->k = g.k; d->n = g.n; d->m = g.m;
    d->block_rows = g.bm; d->block_k = g.bk; d->keep_ratio = keep_ratio; d->score_mode = g.score_mode;
}

// Which execution image crisp_encode lays out.  Default: the 2:4 sparse-MMA image when every aligned
// 4-group keeps at most two values (n <= 2), the zero-expanded dense-tile image otherwise.  The
// environment variable CRISP_EXEC_IMAGE = dense | none overrides it (for measurements).  Evaluated once
// per mask, in crisp_build_mask, and carried by the mask from then on.
int image_kind(const Geometry &g) {
    const char *e = std::getenv("CRISP_EXEC_IMAGE");
    if (e && !std::strcmp(e, "none")) return CRISP_PATH_DIRECT;
    if (e && !std::strcmp(e, "dense")) return CRISP_PATH_DENSE;
    if (e && !std::strcmp(e, "sparse2") && !crisp::tc_pattern_is_sparse(g)) return CRISP_PATH_SPARSE2;
    return crisp::tc_pattern_is_sparse(g) ? CRISP_PATH_SPARSE : CRISP_PATH_DENSE;
}

size_t exec_payload_bytes(const Geometry &g, int kind) {
    if (kind == CRISP_PATH_DIRECT) return 0;
    return crisp::tc_image_layout(g, kind).total_bytes;
}

size_t blk_col_bytes(const Geometry &g) { return align_up((size_t)g.nrt * g.kkeep * sizeof(int32_t) + 4); }
size_t nm_bits_bytes(const Geometry &g) { return align_up((size_t)g.mp() * g.wpr * sizeof(uint32_t)); }
size_t vals_bytes(const Geometry &g) { return align_up((size_t)g.nnz() * sizeof(uint16_t) + 4); }
size_t idx_bytes(const Geometry &g) { return align_up((size_t)g.idx_words() * sizeof(uint32_t) + 4); }

}  // namespace

extern "C" {

const char *crisp_status_string(crisp_status_t s) {
    switch (s) {
        case CRISP_OK: return "ok";
        case CRISP_INVALID_ARG: return "invalid argument";
        case CRISP_UNSUPPORTED: return "unsupported pattern or size";
        case CRISP_BAD_SHAPE: return "bad shape";
        case CRISP_BUFFER_TOO_SMALL: return "buffer too small";
        case CRISP_CUDA_ERROR: return "CUDA error";
        case CRISP_TIMEOUT: return "bounded wait expired in a kernel";
    }
    return "unknown status";
}

crisp_status_t crisp_keep_count(const crisp_layer_desc_t *desc, int32_t *nblk, int32_t *kkeep) {
    Geometry g;
    crisp_status_t s = make_geometry(desc, &g);
    if (s != CRISP_OK) return s;
    if (nblk) *nblk = g.nblk;
    if (kkeep) *kkeep = g.kkeep;
    return CRISP_OK;
}

crisp_status_t crisp_mask_sizes(const crisp_layer_desc_t *desc, size_t *mask_bytes, size_t *workspace_bytes) {
    Geometry g;
    crisp_status_t s = make_geometry(desc, &g);
    if (s != CRISP_OK) return s;
    if (mask_bytes) *mask_bytes = blk_col_bytes(g) + nm_bits_bytes(g);
    if (workspace_bytes) *workspace_bytes = crisp::mask_workspace_bytes(g);
    return CRISP_OK;
}

crisp_status_t crisp_build_mask(const float *d_saliency, int64_t ld_s, const crisp_layer_desc_t *desc,
                                void *d_mask_buf, void *d_workspace, void *stream, crisp_mask_t *out) {
    return crisp_build_mask_ex(d_saliency, ld_s, desc, d_mask_buf, d_workspace, 0, stream, out);
}

crisp_status_t crisp_build_mask_ex(const float *d_saliency, int64_t ld_s, const crisp_layer_desc_t *desc,
                                   void *d_mask_buf, void *d_workspace, uint32_t flags, void *stream,
                                   crisp_mask_t *out) {
    if (!out) return CRISP_INVALID_ARG;
    if (flags & ~(uint32_t)CRISP_MASK_MAX_KNOWN) return CRISP_INVALID_ARG;
    *out = nullptr;
    Geometry g;
    crisp_status_t s = make_geometry(desc, &g);
    if (s != CRISP_OK) return s;
    if (!d_saliency || !d_mask_buf || !d_workspace) return CRISP_INVALID_ARG;
    if (!aligned(d_saliency, 4) || !aligned(d_mask_buf, kAlign) || !aligned(d_workspace, kAlign))
        return CRISP_INVALID_ARG;
    if (ld_s < g.k) return CRISP_BAD_SHAPE;
    crisp_mask_s *mk = new (std::nothrow) crisp_mask_s;
    if (!mk) return CRISP_CUDA_ERROR;
    mk->g = g;
    mk->d_blk_col = reinterpret_cast<int32_t *>(d_mask_buf);
    mk->d_nm_bits = reinterpret_cast<uint32_t *>(reinterpret_cast<uint8_t *>(d_mask_buf) + blk_col_bytes(g));
    mk->image_kind = image_kind(g);
    cudaError_t e = crisp::launch_build_mask(d_saliency, ld_s, g, mk->d_blk_col, mk->d_nm_bits, d_workspace,
                                             crisp::mask_workspace_bytes(g), (flags & CRISP_MASK_MAX_KNOWN) != 0,
                                             (cudaStream_t)stream);
    if (e != cudaSuccess) { delete mk; return CRISP_CUDA_ERROR; }
    *out = mk;
    return CRISP_OK;
}

crisp_status_t crisp_mask_reselect(crisp_mask_t mask, int32_t kkeep, const void *d_workspace, void *stream) {
    if (!mask || !d_workspace) return CRISP_INVALID_ARG;
    if (kkeep < 0 || kkeep > mask->g.kkeep) return CRISP_INVALID_ARG;     // the kept sets are nested: only downwards
    if (!aligned(d_workspace, kAlign)) return CRISP_INVALID_ARG;
    mask->g.kkeep = kkeep;
    cudaError_t e = crisp::launch_block_select(mask->g, d_workspace, mask->d_blk_col, mask->d_nm_bits, (cudaStream_t)stream);
    return e == cudaSuccess ? CRISP_OK : CRISP_CUDA_ERROR;
}

crisp_status_t crisp_prune_fraction(double kappa, int32_t n, int32_t m, double *prune_fraction) {
    if (!prune_fraction || n < 1 || m < n || !(kappa >= 0.0) || kappa > 1.0) return CRISP_INVALID_ARG;
    const double f = 1.0 - (1.0 - kappa) * (double)m / (double)n;
    *prune_fraction = f < 0.0 ? 0.0 : (f > 1.0 ? 1.0 : f);
    return CRISP_OK;
}

crisp_status_t crisp_keep_ratio_for_count(const crisp_layer_desc_t *desc, int32_t kkeep, double *keep_ratio) {
    Geometry g;
    crisp_status_t s = make_geometry(desc, &g);
    if (s != CRISP_OK) return s;
    if (!keep_ratio || kkeep < 0 || kkeep > g.nblk) return CRISP_INVALID_ARG;
    *keep_ratio = (double)kkeep / (double)g.nblk;     // floor(ratio * nblk + 0.5) gives kkeep back
    return CRISP_OK;
}

crisp_status_t crisp_mask_export(crisp_mask_t mask, int32_t *h_blk_col, uint32_t *h_nm_bits, void *stream) {
    if (!mask) return CRISP_INVALID_ARG;
    const Geometry &g = mask->g;
    cudaStream_t st = (cudaStream_t)stream;
    if (h_blk_col && g.nrt * g.kkeep > 0 &&
        cudaMemcpyAsync(h_blk_col, mask->d_blk_col, (size_t)g.nrt * g.kkeep * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return CRISP_CUDA_ERROR;
    if (h_nm_bits &&
        cudaMemcpyAsync(h_nm_bits, mask->d_nm_bits, (size_t)g.mp() * g.wpr * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return CRISP_CUDA_ERROR;
    return cudaStreamSynchronize(st) == cudaSuccess ? CRISP_OK : CRISP_CUDA_ERROR;
}

crisp_status_t crisp_mask_info(crisp_mask_t mask, crisp_layer_desc_t *desc, int32_t *nrt, int32_t *nblk, int32_t *kkeep) {
    if (!mask) return CRISP_INVALID_ARG;
    const Geometry &g = mask->g;
    if (desc) fill_desc(g, g.nblk ? (double)g.kkeep / g.nblk : 0.0, desc);
    if (nrt) *nrt = g.nrt;
    if (nblk) *nblk = g.nblk;
    if (kkeep) *kkeep = g.kkeep;
    return CRISP_OK;
}

crisp_status_t crisp_encode_sizes(crisp_mask_t mask, size_t *canonical_bytes, size_t *exec_bytes) {
    if (!mask) return CRISP_INVALID_ARG;
    const Geometry &g = mask->g;
    if (canonical_bytes) *canonical_bytes = blk_col_bytes(g) + vals_bytes(g) + idx_bytes(g);
    if (exec_bytes) *exec_bytes = kAlign + exec_payload_bytes(g, mask->image_kind);
    return CRISP_OK;
}

crisp_status_t crisp_encode(const uint16_t *d_w_bf16, int64_t ld_w, crisp_mask_t mask, void *d_canonical_buf,
                            void *d_exec_buf, void *stream, crisp_handle_t *out) {
    if (!out) return CRISP_INVALID_ARG;
    *out = nullptr;
    if (!mask || !d_w_bf16 || !d_canonical_buf || !d_exec_buf) return CRISP_INVALID_ARG;
    if (!aligned(d_w_bf16, 2) || !aligned(d_canonical_buf, kAlign) || !aligned(d_exec_buf, kAlign))
        return CRISP_INVALID_ARG;
    const Geometry &g = mask->g;
    if (ld_w < g.k) return CRISP_BAD_SHAPE;
    crisp_handle_s *h = new (std::nothrow) crisp_handle_s;
    if (!h) return CRISP_CUDA_ERROR;
    uint8_t *p = reinterpret_cast<uint8_t *>(d_canonical_buf);
    h->g = g;
    h->d_blk_col = reinterpret_cast<int32_t *>(p); p += blk_col_bytes(g);
    h->d_vals = reinterpret_cast<uint16_t *>(p); p += vals_bytes(g);
    h->d_idx = reinterpret_cast<uint32_t *>(p);
    h->d_status = reinterpret_cast<int32_t *>(d_exec_buf);
    h->d_exec = reinterpret_cast<uint8_t *>(d_exec_buf) + kAlign;
    h->exec_kind = mask->image_kind;
    h->exec_payload_bytes = exec_payload_bytes(g, h->exec_kind);
    h->forced_path = -1;
    h->epilogue = crisp::Epilogue{nullptr, 0};
    const char *nt_env = std::getenv("CRISP_TC_NT");          // 64-column boxes per CTA tile, tuning only; read once
    h->nt_override = nt_env ? std::atoi(nt_env) : 0;
    h->group_override = 0;
    h->wait_limit_cycles = 0;
    h->debug_skip_stage = -1;
    h->plan = nullptr;
    h->last = crisp_launch_info_t{-1, 0, 0, 1, 0, 0, 0, 0, 1};
    cudaStream_t st = (cudaStream_t)stream;
    // the status block is cleared by the encode kernel where one is launched with walk lists, else by a memset
    const bool clear_in_kernel = h->exec_kind != CRISP_PATH_DIRECT && (int64_t)g.nrt * g.kkeep > 0;
    cudaError_t e = clear_in_kernel ? cudaSuccess : cudaMemsetAsync(d_exec_buf, 0, kAlign, st);
    // 128-row blocks: one kept block is one tensor-core tile, so the encode kernel writes it directly
    const bool fuse_tiles = (h->exec_kind == CRISP_PATH_DENSE || h->exec_kind == CRISP_PATH_SPARSE) && g.bm == 128;
    crisp::TcImageLayout L = {};
    if (h->exec_kind != CRISP_PATH_DIRECT) L = crisp::tc_image_layout(g, h->exec_kind);
    // the walk lists of the tensor-core kernel depend on the mask only: CTAs of the encode kernel build them
    const bool tc = h->exec_kind != CRISP_PATH_DIRECT;
    crisp::WalkArgs walks = {};
    if (tc) walks = crisp::tc_walk_args(g, h->exec_kind, mask->d_blk_col, h->d_exec);
    walks.header = clear_in_kernel ? reinterpret_cast<uint32_t *>(d_exec_buf) : nullptr;
    if (e == cudaSuccess)
        e = crisp::launch_encode_canonical(d_w_bf16, ld_w, g, mask->d_blk_col, mask->d_nm_bits,
                                           h->d_blk_col, h->d_vals, h->d_idx, fuse_tiles ? h->exec_kind : 0,
                                           fuse_tiles ? h->d_exec + L.image_off : nullptr, L.a_bytes, L.entry_bytes,
                                           tc ? &walks : nullptr, st);
    if (e == cudaSuccess && tc)
        e = crisp::launch_build_image(g, h->exec_kind, h->d_blk_col, h->d_vals, h->d_idx,
                                      h->d_exec, fuse_tiles, /*walks_done=*/true, st);
    if (e != cudaSuccess) { delete h; return CRISP_CUDA_ERROR; }
    *out = h;
    return CRISP_OK;
}

crisp_status_t crisp_encoded_counts(crisp_handle_t h, int64_t *n_blk_col, int64_t *n_vals, int64_t *n_idx_words) {
    if (!h) return CRISP_INVALID_ARG;
    if (n_blk_col) *n_blk_col = (int64_t)h->g.nrt * h->g.kkeep;
    if (n_vals) *n_vals = h->g.nnz();
    if (n_idx_words) *n_idx_words = h->g.idx_words();
    return CRISP_OK;
}

crisp_status_t crisp_export(crisp_handle_t h, int32_t *h_blk_col, uint16_t *h_vals, uint32_t *h_idx, void *stream) {
    if (!h) return CRISP_INVALID_ARG;
    const Geometry &g = h->g;
    cudaStream_t st = (cudaStream_t)stream;
    if (g.nnz() > 0) {
        if (h_blk_col && cudaMemcpyAsync(h_blk_col, h->d_blk_col, (size_t)g.nrt * g.kkeep * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess)
            return CRISP_CUDA_ERROR;
        if (h_vals && cudaMemcpyAsync(h_vals, h->d_vals, (size_t)g.nnz() * 2, cudaMemcpyDeviceToHost, st) != cudaSuccess)
            return CRISP_CUDA_ERROR;
        if (h_idx && cudaMemcpyAsync(h_idx, h->d_idx, (size_t)g.idx_words() * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess)
            return CRISP_CUDA_ERROR;
    }
    return cudaStreamSynchronize(st) == cudaSuccess ? CRISP_OK : CRISP_CUDA_ERROR;
}

crisp_status_t crisp_decode(crisp_handle_t h, uint16_t *d_w_dense_bf16, int64_t ld, void *stream) {
    if (!h || !d_w_dense_bf16) return CRISP_INVALID_ARG;
    if (ld < h->g.k) return CRISP_BAD_SHAPE;
    cudaError_t e = crisp::launch_decode(h->g, h->d_blk_col, h->d_vals, h->d_idx, d_w_dense_bf16, ld, (cudaStream_t)stream);
    return e == cudaSuccess ? CRISP_OK : CRISP_CUDA_ERROR;
}

crisp_status_t crisp_set_epilogue(crisp_handle_t h, const float *d_bias_f32, int32_t relu) {
    if (!h || (relu != 0 && relu != 1)) return CRISP_INVALID_ARG;
    if (d_bias_f32 && !aligned(d_bias_f32, 4)) return CRISP_INVALID_ARG;
    h->epilogue = crisp::Epilogue{d_bias_f32, relu};
    return CRISP_OK;
}

crisp_status_t crisp_set_path(crisp_handle_t h, int32_t path) {
    if (!h) return CRISP_INVALID_ARG;
    if (path == -1 || path == CRISP_PATH_DIRECT) { h->forced_path = path; return CRISP_OK; }
    if (path != CRISP_PATH_DENSE && path != CRISP_PATH_SPARSE && path != CRISP_PATH_SPARSE2) return CRISP_INVALID_ARG;
    if (path != h->exec_kind) return CRISP_UNSUPPORTED;
    h->forced_path = path;
    return CRISP_OK;
}

crisp_status_t crisp_spmm(crisp_handle_t h, const uint16_t *d_x_bf16, int64_t ldx, int64_t ncols, void *d_y,
                          int64_t ldy, int32_t y_dtype, void *stream) {
    if (!h || !d_x_bf16 || !d_y) return CRISP_INVALID_ARG;
    if (y_dtype != 0 && y_dtype != 1) return CRISP_INVALID_ARG;
    if (ncols <= 0 || ldx < ncols || ldy < ncols) return CRISP_BAD_SHAPE;
    if (!aligned(d_x_bf16, 2) || !aligned(d_y, y_dtype ? 4 : 2)) return CRISP_INVALID_ARG;
    if ((ncols + 63) / 64 > 0x7FFFFFFFll) return CRISP_UNSUPPORTED;
    int path = h->forced_path >= 0 ? h->forced_path : h->exec_kind;
    if (h->g.kkeep == 0 || !crisp::tc_operands_ok(d_x_bf16, ldx, d_y, ldy, y_dtype, ncols)) path = CRISP_PATH_DIRECT;
    cudaError_t e;
    if (path == CRISP_PATH_DIRECT) {
        e = crisp::launch_spmm_direct(h->g, h->d_blk_col, h->d_vals, h->d_idx, d_x_bf16, ldx, ncols,
                                      d_y, ldy, y_dtype, h->epilogue, (cudaStream_t)stream);
        if (e == cudaSuccess) h->last = crisp_launch_info_t{CRISP_PATH_DIRECT, 0, 0, 1, 0, 0, 0, 0};
    } else {
        e = crisp::launch_spmm_tc(h, path, d_x_bf16, ldx, ncols, d_y, ldy, y_dtype, nullptr,
                                  (cudaStream_t)stream);
    }
    return e == cudaSuccess ? CRISP_OK : CRISP_CUDA_ERROR;
}

crisp_status_t crisp_spmm_conv(crisp_handle_t h, const uint16_t *d_act_nhwc, const crisp_conv_desc_t *cd, void *d_y,
                               int64_t ldy, int32_t y_dtype, void *stream) {
    if (!h || !d_act_nhwc || !cd || !d_y) return CRISP_INVALID_ARG;
    if (y_dtype != 0 && y_dtype != 1) return CRISP_INVALID_ARG;
    if (cd->batch <= 0 || cd->height <= 0 || cd->width <= 0 || cd->channels <= 0 || cd->kernel_h <= 0 ||
        cd->kernel_w <= 0 || cd->pad < 0)
        return CRISP_BAD_SHAPE;
    if (cd->y_layout != 0 && cd->y_layout != 1) return CRISP_INVALID_ARG;
    crisp::ConvGeom cg{cd->batch, cd->height, cd->width, cd->channels, cd->kernel_h, cd->kernel_w, cd->pad,
                       cd->height + 2 * cd->pad - cd->kernel_h + 1, cd->width + 2 * cd->pad - cd->kernel_w + 1,
                       cd->y_layout};
    if (cg.ho <= 0 || cg.wo <= 0) return CRISP_BAD_SHAPE;
    if ((int64_t)cd->kernel_h * cd->kernel_w * cd->channels != h->g.k) return CRISP_BAD_SHAPE;
    const int64_t ncols = (int64_t)cg.batch * cg.ho * cg.wo;
    if (ldy < (cg.nhwc_out ? (int64_t)h->g.rows : ncols)) return CRISP_BAD_SHAPE;
    const int es = y_dtype ? 4 : 2;
    // the gather needs whole k-blocks inside one filter tap, 128-byte channel slabs, and TMA-addressable tensors
    if (h->g.bk != 64 || cd->channels % h->g.bk != 0) return CRISP_UNSUPPORTED;
    if (!aligned(d_act_nhwc, 16)) return CRISP_UNSUPPORTED;
    if (!aligned(d_y, es)) return CRISP_INVALID_ARG;
    const int path = h->forced_path >= 0 ? h->forced_path : h->exec_kind;
    if (path == CRISP_PATH_DIRECT || h->g.kkeep == 0) return CRISP_UNSUPPORTED;
    cudaError_t e = crisp::launch_spmm_tc(h, path, d_act_nhwc, 0, ncols, d_y, ldy, y_dtype, &cg,
                                          (cudaStream_t)stream);
    if (e == cudaErrorInvalidValue) return CRISP_UNSUPPORTED;
    return e == cudaSuccess ? CRISP_OK : CRISP_CUDA_ERROR;
}

crisp_status_t crisp_last_launch(crisp_handle_t h, crisp_launch_info_t *out) {
    if (!h || !out) return CRISP_INVALID_ARG;
    *out = h->last;
    return CRISP_OK;
}

crisp_status_t crisp_set_stage_blocks(crisp_handle_t h, int32_t max_blocks) {
    if (!h || (max_blocks != 0 && max_blocks != 1 && max_blocks != 2 && max_blocks != 4)) return CRISP_INVALID_ARG;
    h->group_override = max_blocks;
    return CRISP_OK;
}

crisp_status_t crisp_set_tuning(crisp_handle_t h, int32_t tile_boxes, uint64_t wait_limit_cycles, int32_t skip_fill) {
    if (!h || tile_boxes < 0 || tile_boxes > 4 || skip_fill < -1) return CRISP_INVALID_ARG;
    h->nt_override = tile_boxes;
    h->wait_limit_cycles = wait_limit_cycles;
    h->debug_skip_stage = skip_fill;
    return CRISP_OK;
}

crisp_status_t crisp_reset_status(crisp_handle_t h, void *stream) {
    if (!h) return CRISP_INVALID_ARG;
    return cudaMemsetAsync(h->d_status, 0, sizeof(int32_t), (cudaStream_t)stream) == cudaSuccess ? CRISP_OK
                                                                                                 : CRISP_CUDA_ERROR;
}

crisp_status_t crisp_device_status(crisp_handle_t h, void *stream, int32_t *status_out) {
    if (!h || !status_out) return CRISP_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemcpyAsync(status_out, h->d_status, 4, cudaMemcpyDeviceToHost, st) != cudaSuccess) return CRISP_CUDA_ERROR;
    return cudaStreamSynchronize(st) == cudaSuccess ? CRISP_OK : CRISP_CUDA_ERROR;
}

crisp_status_t crisp_bytes_model(crisp_handle_t h, int64_t ncols, int32_t y_dtype, crisp_bytes_t *out) {
    if (!h || !out || ncols <= 0 || (y_dtype != 0 && y_dtype != 1)) return CRISP_INVALID_ARG;
    const Geometry &g = h->g;
    std::memset(out, 0, sizeof(*out));
    out->nnz = g.nnz();
    out->vals_bytes = 2 * g.nnz();
    out->idx_bytes = g.nnz() * g.idx_bits / 8;
    out->blk_col_bytes = 4ll * g.nrt * g.kkeep;
    out->y_bytes = (int64_t)g.rows * ncols * (y_dtype ? 4 : 2);
    out->useful_macs = g.nnz() * ncols;
    // rows of X that lie under at least one kept block: needs the block list on the host
    int64_t touched_rows = 0;
    if (g.nrt * g.kkeep > 0) {
        std::vector<int32_t> bc((size_t)g.nrt * g.kkeep);
        if (cudaMemcpy(bc.data(), h->d_blk_col, bc.size() * 4, cudaMemcpyDeviceToHost) != cudaSuccess)
            return CRISP_CUDA_ERROR;
        std::vector<char> seen((size_t)g.nblk, 0);
        for (int32_t j : bc) if (j >= 0 && j < g.nblk) seen[(size_t)j] = 1;
        for (int j = 0; j < g.nblk; ++j)
            if (seen[(size_t)j]) {
                const int64_t lo = (int64_t)j * g.bk, hi = lo + g.bk < g.k ? lo + g.bk : g.k;
                touched_rows += hi - lo;
            }
    }
    out->x_bytes = touched_rows * ncols * 2;
    const int64_t elems = (int64_t)g.nrt * g.kkeep * g.bm * g.bk;
    out->path = h->forced_path >= 0 ? h->forced_path : h->exec_kind;
    out->slot_macs = (out->path == CRISP_PATH_SPARSE ? elems / 2
                      : (out->path == CRISP_PATH_DENSE || out->path == CRISP_PATH_SPARSE2 ? elems : g.nnz())) * ncols;
    return CRISP_OK;
}

void crisp_mask_destroy(crisp_mask_t mask) { delete mask; }
void crisp_destroy(crisp_handle_t h) {
    if (h) crisp::tc_plan_destroy(h->plan);
    delete h;
}

}  // extern "C"
