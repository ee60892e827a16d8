/*
 * crisp.h - C ABI of libcrisp: CRISP hybrid structured sparsity on NVIDIA B200 (sm_100a).
 *
 * The library covers the inference-side hot path of the CRISP pruning framework
 * (Aggarwal, Binici, Mitra: "CRISP: Hybrid Structured Sparsity for Class-aware Model
 * Pruning"):
 *
 *   crisp_build_mask   saliency tensor -> hybrid mask: N of every M consecutive reduction
 *                      elements (Sec. III-A; Algorithm 1, fine-grained N:M step) inside an
 *                      equal number of kept coarse blocks per row of the block grid
 *                      (Sec. III-A "uniform block pruning"; Algorithm 1, block score, per-row
 *                      sort, select, prune).
 *   crisp_encode       dense weight + mask -> compressed format: Blocked-ELLPACK column index
 *                      per kept block and a log2(M)-bit offset per kept value (Sec. III-A),
 *                      plus an execution image laid out for the tensor cores.
 *   crisp_spmm         Y = W_hybrid * X, the three-step sparse product of Sec. III-E (load the
 *                      activations of kept blocks, select activations by offset, multiply-
 *                      accumulate), bf16 operands with fp32 accumulation.
 *
 * Conventions
 *   - W is [rows, k]: rows are output channels, k = kernel_h * kernel_w * in_channels is the
 *     reduction dimension and is contiguous.  N:M groups and coarse blocks run along k.
 *   - A "row tile" is block_rows consecutive rows of W (one row of the paper's block grid).
 *     nrt = ceil(rows / block_rows), nblk = ceil(k / block_k); shapes are zero-padded to
 *     whole blocks (padded saliency and weights count as 0).
 *   - X is [k, ncols] and Y is [rows, ncols], both row-major with ncols contiguous.
 *   - bf16 values are passed as uint16_t bit patterns.
 *   - Pointers named d_* are DEVICE memory owned by the caller; h_* are HOST memory owned by
 *     the caller.  The library never allocates or frees device memory in the calls below:
 *     the caller queries sizes, allocates, and keeps the buffers alive while the mask or
 *     handle that refers to them is in use.  Device buffers must be 256-byte aligned.
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).  All work is
 *     enqueued on it and is asynchronous, except the *_export calls and
 *     crisp_device_status, which synchronise the stream before returning.
 *   - Every call returns a crisp_status_t.  Argument errors are detected on the host before
 *     anything is launched.  No call throws, aborts or prints.
 */
#ifndef CRISP_H_
#define CRISP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define CRISP_API __attribute__((visibility("default")))
#else
#define CRISP_API
#endif

typedef enum {
    CRISP_OK = 0,
    CRISP_INVALID_ARG = 1,      /* null pointer, misaligned buffer, bad enum value            */
    CRISP_UNSUPPORTED = 2,      /* pattern or size outside what the kernels implement         */
    CRISP_BAD_SHAPE = 3,        /* non-positive extent, leading dimension too small           */
    CRISP_BUFFER_TOO_SMALL = 4,
    CRISP_CUDA_ERROR = 5,       /* a CUDA runtime/driver call or launch failed                */
    CRISP_TIMEOUT = 6           /* a bounded wait inside a kernel expired (device status)     */
} crisp_status_t;

/* One pruned layer.  Sec. III-A: N:M sparsity inside B x B blocks (generalised here to
 * block_rows x block_k). */
typedef struct {
    int32_t rows;        /* output channels, >= 1                                            */
    int32_t k;           /* reduction length, >= 1                                           */
    int32_t n;           /* kept elements per group, 1 <= n <= m                             */
    int32_t m;           /* group length along k: 4 or 8                                     */
    int32_t block_rows;  /* 32, 64 or 128                                                    */
    int32_t block_k;     /* 32, 64, 96 or 128 (a multiple of 32 and of m)                    */
    double  keep_ratio;  /* fraction of k-blocks kept in every row tile, in [0, 1]           */
    int32_t score_mode;  /* 0: block score sums the N:M survivors (Algorithm 1 prunes N:M
                            before it scores blocks); 1: sums every element of the block      */
} crisp_layer_desc_t;

typedef struct crisp_mask_s   *crisp_mask_t;    /* small host object, library-owned          */
typedef struct crisp_handle_s *crisp_handle_t;  /* small host object, library-owned          */

/* Roofline terms of one crisp_spmm call (bytes every algorithm must move, and multiply-
 * accumulate counts), see crisp_bytes_model. */
typedef struct {
    int64_t nnz;              /* stored weight values, padding included                      */
    int64_t vals_bytes;       /* 2 * nnz                                                     */
    int64_t idx_bytes;        /* nnz * log2(m) / 8                                           */
    int64_t blk_col_bytes;    /* 4 * nrt * kkeep                                             */
    int64_t x_bytes;          /* rows of X under at least one kept block, read once          */
    int64_t y_bytes;          /* rows * ncols * sizeof(Y element)                            */
    int64_t useful_macs;      /* nnz * ncols                                                 */
    int64_t slot_macs;        /* multiply-accumulate slots the chosen tensor-core path spends */
    int32_t path;             /* which SpMM kernel the handle runs, see CRISP_PATH_*         */
} crisp_bytes_t;

#define CRISP_PATH_DIRECT 0   /* CUDA-core kernel on the canonical format (any shape)        */
#define CRISP_PATH_DENSE  1   /* tcgen05 dense MMA over zero-expanded kept blocks            */
#define CRISP_PATH_SPARSE 2   /* tcgen05 sparse (2:4) MMA over compressed kept blocks        */
#define CRISP_PATH_SPARSE2 3  /* the same for patterns with up to four values per aligned 4-group
                                 (3:4, 4:8, ...): the block is split into two 2:4-compliant addends,
                                 both multiplied into one accumulator (opt-in, for measurements:
                                 the dense-tile image is the default for those patterns)        */

/* What the last crisp_spmm / crisp_spmm_conv on a handle really launched (crisp_last_launch).
 * `path` is the kernel family that ran, which differs from crisp_bytes_t.path when the operands
 * of that call could not be addressed by the tensor-core kernel (Sec. III-E is the same three
 * steps on every path). */
typedef struct {
    int32_t path;             /* CRISP_PATH_* of the kernel that was launched, -1 before any    */
    int32_t tile_cols;        /* columns of X / Y per CTA tile (0 on the direct path)           */
    int32_t accumulators;     /* tensor-memory accumulators per CTA                              */
    int32_t stack;            /* column tiles stacked in one accumulator (thin layers), else 1   */
    int32_t epilogue_warps;
    int32_t stages;           /* depth of the shared-memory ring                                 */
    int32_t ctas;             /* grid size                                                       */
    int32_t conv;             /* 1 if the activations were gathered from an NHWC tensor          */
    int32_t stage_blocks;     /* kept blocks per pipeline stage (1, 2 or 4)                      */
} crisp_launch_info_t;

/* kkeep = floor(keep_ratio * nblk + 0.5), clamped to [0, nblk], evaluated in double on the
 * host.  This is the "select by the current sparsity target" step of Algorithm 1 with the
 * per-layer ratio given by the caller.  Error: INVALID_ARG / BAD_SHAPE / UNSUPPORTED. */
CRISP_API crisp_status_t crisp_keep_count(const crisp_layer_desc_t *desc, int32_t *nblk, int32_t *kkeep);

/* Bytes of the mask buffer (kept-block list + bit mask) and of the scratch workspace that
 * crisp_build_mask needs for this layer. */
CRISP_API crisp_status_t crisp_mask_sizes(const crisp_layer_desc_t *desc, size_t *mask_bytes,
                                          size_t *workspace_bytes);

/*
 * Mask projection (Algorithm 1, N:M step, block score, per-row sort, select, prune).
 *   d_saliency  [rows, k] fp32, leading dimension ld_s >= k (elements).  Sign is ignored;
 *               NaN counts as 0, +-Inf as FLT_MAX.
 *   d_mask_buf  out, mask_bytes; holds blk_col[nrt, kkeep] (int32, ascending per row tile)
 *               and nm_bits[nrt*block_rows, nblk*block_k/32] (uint32, bit k%32 of word k/32).
 *   d_workspace scratch, workspace_bytes; afterwards it holds the layer's block scores (see
 *               crisp_mask_scores) until it is reused.
 *   out         receives a mask object that refers to d_mask_buf (not to d_saliency or
 *               d_workspace).  Free it with crisp_mask_destroy.
 * Steps: per group of m elements keep the n largest |s| (ties: lower k); block score =
 * exact fixed-point sum of floor(|s| * 2^(40 - e_max)), e_max = exponent of the largest |s|
 * in the layer; per row tile keep the kkeep highest scores (ties: lower column); final bit =
 * group bit AND block kept.  Blocks keep their positions (no column permutation).
 */
CRISP_API crisp_status_t crisp_build_mask(const float *d_saliency, int64_t ld_s,
                                          const crisp_layer_desc_t *desc,
                                          void *d_mask_buf, void *d_workspace, void *stream,
                                          crisp_mask_t *out);

/*
 * crisp_build_mask with options.  flags:
 *   CRISP_MASK_MAX_KNOWN  the first word of d_workspace already holds the bits of the layer's largest
 *                         canonical |s| (crisp_saliency_finish_max wrote it while it produced d_saliency):
 *                         the pass over the saliency that finds that maximum is skipped.  A wrong value gives
 *                         a wrong fixed-point scale, i.e. a different (still valid) block ranking.
 * flags = 0 is crisp_build_mask.
 */
#define CRISP_MASK_MAX_KNOWN 1u
CRISP_API crisp_status_t crisp_build_mask_ex(const float *d_saliency, int64_t ld_s,
                                             const crisp_layer_desc_t *desc, void *d_mask_buf,
                                             void *d_workspace, uint32_t flags, void *stream,
                                             crisp_mask_t *out);

/*
 * Keep fewer blocks of an existing mask without streaming the saliency again: the per-row-tile selection of
 * Algorithm 1 (sort per row, select, prune) re-run on the block scores and group bits that the mask's
 * crisp_build_mask left in d_workspace and d_mask_buf.  kkeep must not exceed the mask's current count
 * (the kept sets of one ranking are nested; INVALID_ARG otherwise).  Afterwards the mask is exactly what
 * crisp_build_mask would have produced with keep_ratio = kkeep / nblk.  Typical use: build once with
 * keep_ratio 1, let crisp_global_rank decide every layer's count, then reselect.
 */
CRISP_API crisp_status_t crisp_mask_reselect(crisp_mask_t mask, int32_t kkeep, const void *d_workspace,
                                             void *stream);

/* Algorithm 1's sparsity target kappa_p (fraction of ALL weights that are zero after step p) as the
 * fraction of coarse blocks to prune when n of every m elements survive inside kept blocks:
 * 1 - (1 - kappa) * m / n, clamped to [0, 1]. */
CRISP_API crisp_status_t crisp_prune_fraction(double kappa, int32_t n, int32_t m, double *prune_fraction);

/* The keep_ratio that makes crisp_keep_count return exactly kkeep for this layer. */
CRISP_API crisp_status_t crisp_keep_ratio_for_count(const crisp_layer_desc_t *desc, int32_t kkeep,
                                                    double *keep_ratio);

/*
 * Same result as crisp_build_mask, for callers that cannot hand over a scratch workspace
 * because they are not allowed to allocate device memory at the point of the call (a plug-in
 * inside a framework that owns all device memory, a loop that must stay allocation-free after
 * start-up, a process whose pool is fully committed).  The paper has no counterpart of this
 * call; it is a packaging variant of the mask projection.
 *
 * The scratch lives in a fixed array of CRISP_STATIC_SCRATCH_BYTES inside the library image;
 * every GPU that loads the library holds it until the process exits.  The call allocates and
 * frees no device memory and calls no allocating CUDA routine; the only allocation is the small
 * host object behind the returned crisp_mask_t (a few dozen bytes from the C++ heap, freed by
 * crisp_mask_destroy).  Inputs and outputs are still the caller's: d_saliency, d_mask_buf
 * (crisp_mask_sizes gives its size) and the returned mask.
 *
 * Limits and rules
 *   - The layer's workspace (256 bytes + 8 bytes per coarse block, i.e. per (row tile,
 *     k-block) pair) must fit: at most 32736 coarse blocks.  Larger layers are refused with
 *     CRISP_BUFFER_TOO_SMALL before anything is launched; use crisp_build_mask for them.
 *   - Every call looks up the array's device address with the current device current; the first
 *     call on a device also makes the runtime load the library's module there.  Make that first
 *     call during set-up, before any stream capture begins.  The address is never kept across
 *     calls, so cudaDeviceReset or a second context on the device cannot leave a stale one.
 *   - All calls on a device share the one array, and it keeps what the last call wrote.  Each
 *     call clears it on `stream` before use, so calls issued one after another on the same
 *     stream are safe; calls that may run concurrently on the GPU (different streams or host
 *     threads without ordering between them) race on it and give wrong masks.
 */
#define CRISP_STATIC_SCRATCH_BYTES (256 * 1024)
CRISP_API crisp_status_t crisp_build_mask_static(const float *d_saliency, int64_t ld_s,
                                                 const crisp_layer_desc_t *desc, void *d_mask_buf,
                                                 void *stream, crisp_mask_t *out);

/*
 * Class-aware saliency score (Sec. III-C "Pruning Metric", Eq. 1): the first-order Taylor estimate
 * T_w = | (1/H) * sum_i g_i (.) W | with the loss gradient g averaged over the H samples of the
 * user's classes.  The gradients are the caller's (one tensor per sample or mini-batch):
 *   crisp_saliency_accumulate   acc = g (first = 1) or acc += g (first = 0), fp32, in call order
 *   crisp_saliency_finish       S = | acc * (1 / samples) * W |, fp32: the input of crisp_build_mask
 * d_grad: [rows, k] bf16 (grad_dtype 0) or fp32 (1); d_acc, d_saliency: [rows, k] fp32; d_w_bf16:
 * [rows, k] bf16; leading dimensions in elements.  Arithmetic is fp32 in exactly this order (sum of
 * the samples in call order, times the rounded reciprocal of `samples`, times the weight), so the
 * result does not depend on the launch shape.  Nothing is allocated.
 */
CRISP_API crisp_status_t crisp_saliency_accumulate(const void *d_grad, int32_t grad_dtype, int64_t ld_g,
                                                   int32_t rows, int32_t k, float *d_acc, int64_t ld_acc,
                                                   int32_t first, void *stream);
CRISP_API crisp_status_t crisp_saliency_finish(const float *d_acc, int64_t ld_acc, const uint16_t *d_w_bf16,
                                               int64_t ld_w, int32_t rows, int32_t k, int32_t samples,
                                               float *d_saliency, int64_t ld_s, void *stream);
/* crisp_saliency_finish that also leaves the layer's largest score where crisp_build_mask_ex(...,
 * CRISP_MASK_MAX_KNOWN) expects it: d_mask_workspace is that layer's mask workspace (crisp_mask_sizes; its
 * first 256 bytes are cleared on `stream`, then the bits of max |S| - NaN read as 0, Inf as FLT_MAX - are
 * written to its first word).  NULL makes this crisp_saliency_finish.  Eq. 1 / Algorithm 1: the score and the
 * block scoring that follows it share one pass over the layer instead of two. */
CRISP_API crisp_status_t crisp_saliency_finish_max(const float *d_acc, int64_t ld_acc, const uint16_t *d_w_bf16,
                                                   int64_t ld_w, int32_t rows, int32_t k, int32_t samples,
                                                   float *d_saliency, int64_t ld_s, void *d_mask_workspace,
                                                   void *stream);

/*
 * Global rank selection across the layers of a network: Algorithm 1 of the paper between the
 * block scores and the pruning itself (Sec. III-C, "Pruning Algorithm": sort the block scores
 * inside every row of the block grid, add the o-th smallest score of every row into the
 * rank-column sum c_o, order all c_o of all layers increasingly, and prune from the front of
 * that order until the current sparsity target is met).  Pruning rank position o of a layer
 * removes one block from every row tile, so every row keeps the same number of blocks; the
 * result per layer is that number, kkeep, which crisp_build_mask then takes as
 * keep_ratio = kkeep / nblk.
 *
 * Inputs are the block scores crisp_build_mask leaves in its workspace.  After that call (with
 * any keep ratio) and until the workspace is reused, the workspace holds the bits of the
 * layer's largest |s| (uint32, byte 0; it fixes the unit of the scores, 2^(e_max - 40)) and the
 * [nrt, nblk] uint64 scores (byte 256); crisp_mask_scores returns the two addresses.
 *
 * Readings where the paper is silent:
 *   - rank sums of different layers are compared by their real values c * 2^(e_max - 40),
 *     exactly (128-bit integers); ties go to the lower layer index, then the lower o;
 *   - the target is a number of weights, floor(prune_fraction * total + 0.5) with total = sum
 *     over layers of nrt * nblk * block_elems; a rank position weighs nrt * block_elems;
 *     positions are pruned in order while the weight pruned so far is below the target.
 *     With Algorithm 1's overall sparsity kappa_p and N:M inside kept blocks,
 *     prune_fraction = 1 - (1 - kappa_p) * M / N;
 *   - the last min_keep rank positions of a layer are never pruned (0 lets a layer vanish).
 *
 * layers (host array) is read before the call returns.  d_workspace: crisp_global_rank_sizes
 * bytes, 256-byte aligned, scratch.  d_kkeep: device, int32 [n_layers], written on `stream`.
 * nblk <= 4096 per layer (CRISP_UNSUPPORTED beyond).  No device memory is allocated; the layer table is
 * staged through a small temporary host array, so the call is refused (CRISP_UNSUPPORTED) while
 * `stream` is being captured into a graph.
 */
typedef struct {
    const unsigned long long *d_scores;  /* device, [nrt, nblk] block scores                      */
    const uint32_t *d_max_key;           /* device, bits of the layer's largest |s|               */
    int32_t nrt, nblk;                   /* row tiles, k-blocks per row tile                      */
    int64_t block_elems;                 /* weights per block: block_rows * block_k               */
    int32_t min_keep;                    /* blocks per row tile that are never pruned             */
    int32_t reserved;                    /* 0                                                     */
} crisp_rank_layer_t;

CRISP_API crisp_status_t crisp_mask_scores(const crisp_layer_desc_t *desc, const void *d_workspace,
                                           const unsigned long long **d_scores, const uint32_t **d_max_key);
CRISP_API crisp_status_t crisp_global_rank_sizes(int32_t n_layers, const crisp_rank_layer_t *layers,
                                                 size_t *workspace_bytes);
CRISP_API crisp_status_t crisp_global_rank(int32_t n_layers, const crisp_rank_layer_t *layers,
                                           double prune_fraction, void *d_workspace, int32_t *d_kkeep,
                                           void *stream);

/* Copy the mask to host: h_blk_col [nrt*kkeep] int32, h_nm_bits [nrt*block_rows *
 * nblk*block_k/32] uint32.  Either may be NULL.  Synchronises `stream`. */
CRISP_API crisp_status_t crisp_mask_export(crisp_mask_t mask, int32_t *h_blk_col, uint32_t *h_nm_bits,
                                           void *stream);

/* Shape bookkeeping of a mask (any out pointer may be NULL). */
CRISP_API crisp_status_t crisp_mask_info(crisp_mask_t mask, crisp_layer_desc_t *desc, int32_t *nrt,
                                         int32_t *nblk, int32_t *kkeep);

/* Bytes of the canonical compressed format and of the execution image for this mask. */
CRISP_API crisp_status_t crisp_encode_sizes(crisp_mask_t mask, size_t *canonical_bytes,
                                            size_t *exec_bytes);

/*
 * Compress (Sec. III-A storage format; Algorithm 1 "f* = f (.) r").
 *   d_w_bf16        [rows, k] bf16, leading dimension ld_w >= k
 *   d_canonical_buf out: blk_col[nrt*kkeep] int32 | vals[nnz] bf16 | idx[ceil(nnz*b/32)] uint32
 *                   with b = log2(m).  Order of values: row tile, kept slot, local row,
 *                   group, value (ascending position); idx field o occupies bits
 *                   [o*b, o*b+b) of the uint32 stream, LSB first; offsets are zero-based
 *                   positions inside the m-vector (Sec. III-E example).  Values in the zero
 *                   padding are stored as 0.
 *   d_exec_buf      out: tensor-core-ready copy used by crisp_spmm (opaque) + status word.
 *   out             handle referring to both buffers (not to d_w_bf16 nor to the mask).
 */
CRISP_API crisp_status_t crisp_encode(const uint16_t *d_w_bf16, int64_t ld_w, crisp_mask_t mask,
                                      void *d_canonical_buf, void *d_exec_buf, void *stream,
                                      crisp_handle_t *out);

/* Element counts of the canonical arrays (for sizing the host buffers of crisp_export). */
CRISP_API crisp_status_t crisp_encoded_counts(crisp_handle_t h, int64_t *n_blk_col, int64_t *n_vals,
                                              int64_t *n_idx_words);

/* Copy the canonical format to host (any pointer may be NULL).  Synchronises `stream`. */
CRISP_API crisp_status_t crisp_export(crisp_handle_t h, int32_t *h_blk_col, uint16_t *h_vals,
                                      uint32_t *h_idx, void *stream);

/* Inverse of crisp_encode: scatter into a dense [rows, k] bf16 matrix (zeros elsewhere). */
CRISP_API crisp_status_t crisp_decode(crisp_handle_t h, uint16_t *d_w_dense_bf16, int64_t ld,
                                      void *stream);

/*
 * Y = W_hybrid * X (Sec. III-E, steps 1-3).
 *   d_x_bf16 [k, ncols] bf16, leading dimension ldx >= ncols
 *   d_y      [rows, ncols], leading dimension ldy >= ncols, bf16 (y_dtype 0, round to
 *            nearest even from the fp32 accumulator) or fp32 (y_dtype 1)
 * Rows of X under blocks that no row tile kept are never read.  A layer with kkeep = 0
 * yields Y = 0.  The tensor-core kernels need X and Y 16-byte aligned with ldx*2 and
 * ldy*sizeof(element) multiples of 16; other layouts run on the direct kernel.
 */
CRISP_API crisp_status_t crisp_spmm(crisp_handle_t h, const uint16_t *d_x_bf16, int64_t ldx,
                                    int64_t ncols, void *d_y, int64_t ldy, int32_t y_dtype, void *stream);

/*
 * The same product for a convolution layer without materialising X (Sec. III, Notation: the
 * K x K x R x S filter bank is the matrix W with one row per output channel; Sec. III-E step 1
 * loads "the input activations corresponding to the non-zero blocks").  The reduction index of W
 * is ordered (kernel row, kernel column, input channel), channel fastest, so a kept k-block of
 * block_k channels lies inside one filter tap, and its activations are a shifted window of the
 * input: they are fetched on the fly from the NHWC activation, the zero padding included.
 *
 *   Y[s, b, y, x] = sum_(i, j, r) W_hybrid[s, (i*kernel_w + j)*channels + r]
 *                                 * A[b, y + i - pad, x + j - pad, r]        (stride 1)
 *
 *   d_act_nhwc  [batch, height, width, channels] bf16, dense, 16-byte aligned
 *   d_y         y_layout 0: [rows, batch*ho*wo] bf16 (y_dtype 0) or fp32 (1), leading dimension ldy >=
 *               batch*ho*wo; y_layout 1: [batch, ho, wo, ldy] (NHWC, output channel fastest, ldy >= rows
 *               elements between pixels), which is the d_act_nhwc of the next convolution as it stands,
 *               so that layers chain without a transposition;
 *               ho = height + 2*pad - kernel_h + 1, wo likewise
 * The handle's k must equal kernel_h*kernel_w*channels (BAD_SHAPE otherwise).  Supported
 * (UNSUPPORTED otherwise; lower the convolution to a matrix and call crisp_spmm): block_k = 64,
 * channels a multiple of 64, a tensor-core execution image and at least one kept block.  Y is
 * written by bulk tensor stores when d_y is 16-byte aligned and wo*sizeof(Y element) and
 * ldy*sizeof(Y element) are multiples of 16 bytes (NHWC: when ldy*sizeof(Y element) is), element by
 * element otherwise (e.g. 28- or 14-pixel rows of bf16).  Same tolerance and status reporting as
 * crisp_spmm.
 */
typedef struct {
    int32_t batch, height, width, channels;   /* input activation, NHWC                         */
    int32_t kernel_h, kernel_w;               /* filter taps                                    */
    int32_t pad;                              /* zero padding on every side                     */
    int32_t y_layout;                         /* 0: Y [rows, batch*ho*wo]; 1: Y NHWC [batch, ho, wo, ldy] */
} crisp_conv_desc_t;

CRISP_API crisp_status_t crisp_spmm_conv(crisp_handle_t handle, const uint16_t *d_act_nhwc,
                                         const crisp_conv_desc_t *conv, void *d_y, int64_t ldy,
                                         int32_t y_dtype, void *stream);

/*
 * Layer epilogue for every later crisp_spmm / crisp_spmm_conv on this handle:
 *   Y = act(W_hybrid * X + bias),  act = max(., 0) when relu = 1, identity when 0,
 * applied to the fp32 accumulator before the store, so a bf16 Y is rounded once and can be the
 * next layer's X as it stands (pointwise layers: Y [rows, ncols] is the next X [k, ncols]).  The
 * paper prunes whole networks (Sec. IV: ResNet-50, VGG-16, MobileNetV2), whose layers end in a
 * bias (folded batch norm) and a ReLU; it gives no formula of its own for this step.
 *   d_bias_f32  device, [rows] fp32, read at every call (the caller keeps it alive), or NULL
 * (NULL, 0) restores the plain product.
 */
CRISP_API crisp_status_t crisp_set_epilogue(crisp_handle_t handle, const float *d_bias_f32, int32_t relu);

/* Restrict crisp_spmm of this handle to one kernel family (CRISP_PATH_*), or -1 for the
 * default choice.  UNSUPPORTED if the handle's execution image cannot serve that path. */
CRISP_API crisp_status_t crisp_set_path(crisp_handle_t h, int32_t path);

/* Kernel family and tile configuration of the last product launched through this handle. */
CRISP_API crisp_status_t crisp_last_launch(crisp_handle_t h, crisp_launch_info_t *out);

/* Tuning and failure-detection controls of the tensor-core kernels of this handle (all optional).
 *   tile_boxes        64-column boxes per CTA tile, 1..4; 0 = chosen by the library
 *   wait_limit_cycles every wait inside the kernel (on a pipeline stage, on an accumulator) gives
 *                     up after this many SM cycles, the kernel then lets its copies land, frees its
 *                     tensor memory, returns, and the device status reads CRISP_TIMEOUT; 0 = the
 *                     default of about two seconds
 *   skip_fill         test hook, -1 = off: every CTA leaves out the loads of its skip_fill-th
 *                     pipeline fill, so that the wait for them expires (use with a short limit)
 * The paper has no counterpart; Sec. III-E's pipeline has no failure model. */
CRISP_API crisp_status_t crisp_set_tuning(crisp_handle_t h, int32_t tile_boxes, uint64_t wait_limit_cycles,
                                          int32_t skip_fill);

/* Upper bound on the kept blocks that one pipeline stage of the tensor-core kernels takes (1, 2 or 4;
 * 0 = chosen by the library, the default).  A stage of several blocks shares one wait, one weight-tile copy
 * and one commit among them; results do not depend on it.  Takes effect at the next product.
 * The paper has no counterpart (Sec. III-E names no pipeline depth).  Error: INVALID_ARG. */
CRISP_API crisp_status_t crisp_set_stage_blocks(crisp_handle_t h, int32_t max_blocks);

/* Clear the device status word of the handle on `stream` (after a reported CRISP_TIMEOUT). */
CRISP_API crisp_status_t crisp_reset_status(crisp_handle_t h, void *stream);

/* Read the device status word of the handle (0 = no kernel reported a problem; otherwise a
 * crisp_status_t, e.g. CRISP_TIMEOUT when a bounded wait expired).  Synchronises `stream`. */
CRISP_API crisp_status_t crisp_device_status(crisp_handle_t h, void *stream, int32_t *status_out);

/* Algorithmic byte and multiply-accumulate counts of one crisp_spmm(ncols) call.  Reads the
 * kept-block list back with a blocking copy (not for use inside a timed region). */
CRISP_API crisp_status_t crisp_bytes_model(crisp_handle_t h, int64_t ncols, int32_t y_dtype,
                                           crisp_bytes_t *out);

CRISP_API void crisp_mask_destroy(crisp_mask_t mask);
CRISP_API void crisp_destroy(crisp_handle_t h);
CRISP_API const char *crisp_status_string(crisp_status_t s);

#ifdef __cplusplus
}
#endif
#endif /* CRISP_H_ */
