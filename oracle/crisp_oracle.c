/*
 * CPU oracle for the CRISP hybrid-sparsity path (test infrastructure only).
 *
 * Plain, slow, obviously-correct C.  It exists so that the CUDA library can be
 * checked against something written independently from the paper; it shares no
 * source, header, table or helper with the CUDA code and must never be called
 * from the product path.  Only the tests, the smoke check and the CPU-baseline
 * leg of the benchmark may load it.
 *
 * What it computes, in the paper's order:
 *   - Algorithm 1 "apply fine-grained N:M pruning": per group of M consecutive
 *     reduction elements keep the N of largest saliency            (Sec. III-A, III-C)
 *   - Algorithm 1 "s_j = sum_i |T_w^i|": per-block score             (Sec. III-C)
 *   - Algorithm 1 sort-per-row + select: the same number of blocks is kept in
 *     every row of the block grid; the lowest-scored are pruned      (Sec. III-C)
 *   - Algorithm 1 "f* = f (.) r": blocks keep their positions        (Sec. III-C)
 *   - Algorithm 1 rank-column sums c_o, their global order across layers and the
 *     selection by the sparsity target: how many blocks each layer keeps (Sec. III-C)
 *   - Sec. III-A storage: Blocked-ELLPACK column index per kept block and an
 *     offset in [0, M) per kept value (zero-based, Sec. III-E worked example)
 *   - Sec. III-E three-step sparse product, which equals the masked dense
 *     product; the oracle is that definition: decode, then an fp64 triple loop;
 *     for a convolution layer, the definition of the convolution (no lowering).
 *
 * Readings where the paper is silent:
 *   rows of W are output channels and groups/blocks run along the reduction
 *   dimension; ties go to the lower index; saliency enters as |s| with NaN -> 0
 *   and Inf -> FLT_MAX; the block score is an exact fixed-point integer sum so
 *   that it does not depend on summation order; shapes are zero-padded to whole
 *   blocks.
 *
 * All pointers are host memory.  bf16 values travel as uint16_t bit patterns.
 * Every function returns 0 on success and a negative value on a bad argument.
 */
#include <float.h>
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_SCORE_FRACTION_BITS 40

/* ------------------------------------------------------------------ helpers */

static double bf16_to_double(uint16_t b)
{
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* |s| with the non-finite cases made orderable. */
static float canonical_saliency(float s)
{
    if (isnan(s)) return 0.0f;
    s = fabsf(s);
    if (isinf(s)) return FLT_MAX;
    return s;
}

static int log2_exact(int m)
{
    int b = 0;
    while ((1 << b) < m) ++b;
    return ((1 << b) == m) ? b : -1;
}

static int get_bit(const uint32_t *bits, int64_t words_per_row, int64_t row, int64_t col)
{
    return (int)((bits[row * words_per_row + (col >> 5)] >> (col & 31)) & 1u);
}

static void set_bit(uint32_t *bits, int64_t words_per_row, int64_t row, int64_t col)
{
    bits[row * words_per_row + (col >> 5)] |= (1u << (col & 31));
}

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------- shape bookkeeping */

/* Blocks per row tile and how many of them survive: round-half-up of
 * keep_ratio * nblk, evaluated in IEEE double. */
int oracle_keep_count(int k, int block_k, double keep_ratio, int *nblk_out, int *kkeep_out)
{
    if (k <= 0 || block_k <= 0 || !(keep_ratio >= 0.0) || keep_ratio > 1.0) return -1;
    int nblk = (k + block_k - 1) / block_k;
    int kkeep = (int)floor(keep_ratio * (double)nblk + 0.5);
    if (kkeep < 0) kkeep = 0;
    if (kkeep > nblk) kkeep = nblk;
    *nblk_out = nblk;
    *kkeep_out = kkeep;
    return 0;
}

/* ------------------------------------------------------------- mask build */

/*
 * saliency : [rows, k] fp32, leading dimension ld
 * blk_col  : out, [nrt, kkeep] kept block columns per row tile, ascending
 * nm_bits  : out, [nrt*block_rows, ceil(nblk*block_k/32)] uint32, bit (k & 31) of
 *            word (k >> 5) of a row = 1 iff element (row, k) survives
 * score    : out, optional (may be NULL), [nrt, nblk] fixed-point block scores
 * score_mode 0: a block's score sums the saliency of its N:M survivors only
 *               (Algorithm 1 prunes N:M first, so pruned weights contribute 0)
 * score_mode 1: sums every element of the block
 */
int oracle_build_mask(const float *saliency, int64_t ld, int rows, int k,
                      int n, int m, int block_rows, int block_k, int kkeep, int score_mode,
                      int32_t *blk_col, uint32_t *nm_bits, uint64_t *score_out)
{
    if (!saliency || !nm_bits || rows <= 0 || k <= 0 || m <= 0 || n <= 0 || n > m) return -1;
    if (block_rows <= 0 || block_k <= 0 || block_k % m != 0 || ld < k) return -1;
    const int nrt = (rows + block_rows - 1) / block_rows;
    const int nblk = (k + block_k - 1) / block_k;
    if (kkeep < 0 || kkeep > nblk || (kkeep > 0 && !blk_col)) return -1;
    const int64_t mp = (int64_t)nrt * block_rows;
    const int64_t kp = (int64_t)nblk * block_k;
    const int64_t wpr = (kp + 31) / 32;

    /* step 1-2: padded, canonicalised saliency */
    float *sp = (float *)calloc((size_t)(mp * kp), sizeof(float));
    uint64_t *score = (uint64_t *)calloc((size_t)nrt * nblk, sizeof(uint64_t));
    uint32_t *group_bits = (uint32_t *)calloc((size_t)(mp * wpr), sizeof(uint32_t));
    if (!sp || !score || !group_bits) { free(sp); free(score); free(group_bits); return -2; }
    float smax = 0.0f;
    for (int r = 0; r < rows; ++r)
        for (int c = 0; c < k; ++c) {
            float v = canonical_saliency(saliency[(int64_t)r * ld + c]);
            sp[(int64_t)r * kp + c] = v;
            if (v > smax) smax = v;
        }

    /* step 3: N of M along k, largest saliency first, ties to the lower k */
    int *order = (int *)malloc(sizeof(int) * (size_t)m);
    for (int64_t r = 0; r < mp; ++r)
        for (int64_t g = 0; g < kp / m; ++g) {
            const float *v = sp + r * kp + g * m;
            for (int i = 0; i < m; ++i) order[i] = i;
            for (int i = 1; i < m; ++i) {              /* stable insertion sort, descending */
                int cur = order[i], j = i - 1;
                while (j >= 0 && v[order[j]] < v[cur]) { order[j + 1] = order[j]; --j; }
                order[j + 1] = cur;
            }
            for (int i = 0; i < n; ++i) set_bit(group_bits, wpr, r, g * m + order[i]);
        }
    free(order);

    /* step 4-5: fixed-point block scores  q(s) = floor(s * 2^(40 - e_max)) */
    if (smax > 0.0f) {
        const int e_max = ilogbf(smax);
        for (int64_t r = 0; r < mp; ++r)
            for (int64_t c = 0; c < kp; ++c) {
                if (score_mode == 0 && !get_bit(group_bits, wpr, r, c)) continue;
                double scaled = ldexp((double)sp[r * kp + c], ORACLE_SCORE_FRACTION_BITS - e_max);
                score[(r / block_rows) * nblk + (c / block_k)] += (uint64_t)floor(scaled);
            }
    }

    /* step 6-7: per row tile keep the kkeep best blocks (ties to the lower column) */
    memset(nm_bits, 0, (size_t)(mp * wpr) * sizeof(uint32_t));
    int *border = (int *)malloc(sizeof(int) * (size_t)nblk);
    char *kept = (char *)malloc((size_t)nblk);
    for (int rt = 0; rt < nrt; ++rt) {
        const uint64_t *sc = score + (int64_t)rt * nblk;
        for (int j = 0; j < nblk; ++j) border[j] = j;
        for (int i = 1; i < nblk; ++i) {
            int cur = border[i], j = i - 1;
            while (j >= 0 && sc[border[j]] < sc[cur]) { border[j + 1] = border[j]; --j; }
            border[j + 1] = cur;
        }
        memset(kept, 0, (size_t)nblk);
        for (int i = 0; i < kkeep; ++i) kept[border[i]] = 1;
        int slot = 0;
        for (int j = 0; j < nblk; ++j) {
            if (!kept[j]) continue;
            blk_col[(int64_t)rt * kkeep + slot++] = j;
            /* step 8: final mask = group bits AND block kept; positions unchanged */
            for (int64_t r = (int64_t)rt * block_rows; r < (int64_t)(rt + 1) * block_rows; ++r)
                for (int64_t c = (int64_t)j * block_k; c < (int64_t)(j + 1) * block_k; ++c)
                    if (get_bit(group_bits, wpr, r, c)) set_bit(nm_bits, wpr, r, c);
        }
    }
    if (score_out) memcpy(score_out, score, (size_t)nrt * nblk * sizeof(uint64_t));
    free(border); free(kept); free(sp); free(score); free(group_bits);
    return 0;
}

/* ------------------------------------------------------------ encode/decode */

/* Number of stored values and of uint32 words of offset metadata. */
int oracle_encoded_sizes(int rows, int block_rows, int block_k, int n, int m, int kkeep,
                         int64_t *nvals, int64_t *nidx_words)
{
    int b = log2_exact(m);
    if (b < 0 || rows <= 0) return -1;
    int64_t nrt = (rows + block_rows - 1) / block_rows;
    int64_t v = nrt * kkeep * block_rows * (block_k / m) * n;
    *nvals = v;
    *nidx_words = (v * b + 31) / 32;
    return 0;
}

/*
 * Canonical compressed format (Sec. III-A): for row tile rt, kept slot j, local
 * row r, group g, v-th survivor of the group in ascending position:
 *   vals[o] = W value, idx field o = its offset inside the M-vector (log2 M bits,
 *   packed LSB-first into a uint32 stream), o = (((rt*kkeep+j)*block_rows+r)*G+g)*n+v.
 * Elements in the zero padding are stored as 0x0000.
 */
int oracle_encode(const uint16_t *w, int64_t ld, int rows, int k,
                  int n, int m, int block_rows, int block_k, int kkeep,
                  const int32_t *blk_col, const uint32_t *nm_bits,
                  uint16_t *vals, uint32_t *idx)
{
    const int b = log2_exact(m);
    if (b < 0 || !w || !nm_bits || block_k % m != 0) return -1;
    const int nrt = (rows + block_rows - 1) / block_rows;
    const int nblk = (k + block_k - 1) / block_k;
    const int64_t wpr = ((int64_t)nblk * block_k + 31) / 32;
    const int groups = block_k / m;
    int64_t nvals, nwords;
    oracle_encoded_sizes(rows, block_rows, block_k, n, m, kkeep, &nvals, &nwords);
    memset(idx, 0, (size_t)nwords * sizeof(uint32_t));
    int64_t o = 0;
    for (int rt = 0; rt < nrt; ++rt)
        for (int j = 0; j < kkeep; ++j) {
            const int jb = blk_col[(int64_t)rt * kkeep + j];
            if (jb < 0 || jb >= nblk) return -3;
            for (int r = 0; r < block_rows; ++r) {
                const int64_t row = (int64_t)rt * block_rows + r;
                for (int g = 0; g < groups; ++g) {
                    int found = 0;
                    for (int t = 0; t < m; ++t) {
                        const int64_t col = (int64_t)jb * block_k + (int64_t)g * m + t;
                        if (!get_bit(nm_bits, wpr, row, col)) continue;
                        if (found == n) return -4;           /* more than N in a group */
                        vals[o] = (row < rows && col < k) ? w[row * ld + col] : (uint16_t)0;
                        const int64_t bit = o * b;
                        for (int q = 0; q < b; ++q)
                            if ((t >> q) & 1) idx[(bit + q) >> 5] |= 1u << ((bit + q) & 31);
                        ++o; ++found;
                    }
                    if (found != n) return -4;               /* fewer than N in a group */
                }
            }
        }
    return (o == nvals) ? 0 : -5;
}

/* Inverse scatter into a zeroed dense [rows, k] matrix of doubles (and/or bf16 bits). */
int oracle_decode(const int32_t *blk_col, const uint16_t *vals, const uint32_t *idx,
                  int rows, int k, int n, int m, int block_rows, int block_k, int kkeep,
                  double *w_dense, uint16_t *w_dense_bits)
{
    const int b = log2_exact(m);
    if (b < 0) return -1;
    const int nrt = (rows + block_rows - 1) / block_rows;
    const int groups = block_k / m;
    if (w_dense) memset(w_dense, 0, sizeof(double) * (size_t)rows * k);
    if (w_dense_bits) memset(w_dense_bits, 0, sizeof(uint16_t) * (size_t)rows * k);
    int64_t o = 0;
    for (int rt = 0; rt < nrt; ++rt)
        for (int j = 0; j < kkeep; ++j) {
            const int jb = blk_col[(int64_t)rt * kkeep + j];
            for (int r = 0; r < block_rows; ++r)
                for (int g = 0; g < groups; ++g)
                    for (int v = 0; v < n; ++v, ++o) {
                        const int64_t bit = o * b;
                        int t = 0;
                        for (int q = 0; q < b; ++q)
                            t |= (int)((idx[(bit + q) >> 5] >> ((bit + q) & 31)) & 1u) << q;
                        const int64_t row = (int64_t)rt * block_rows + r;
                        const int64_t col = (int64_t)jb * block_k + (int64_t)g * m + t;
                        if (row >= rows || col >= k) {
                            if (vals[o] != 0) return -6;     /* padding must hold zeros */
                            continue;
                        }
                        if (w_dense) w_dense[row * k + col] = bf16_to_double(vals[o]);
                        if (w_dense_bits) w_dense_bits[row * k + col] = vals[o];
                    }
        }
    return 0;
}

/* ------------------------------------------------------------------- product */

/*
 * The three hardware steps of Sec. III-E compute exactly the masked dense product
 *   Y[r, c] = sum_{t = 0}^{k-1} Wd[r, t] * X[t, c]
 * so the oracle is this definition in fp64, a literal triple loop (threads split
 * the rows of Y; each output is still one sequential sum over t).
 */
int oracle_spmm_fp64(const double *w_dense, int rows, int k,
                     const uint16_t *x, int64_t ldx, int64_t ncols, double *y)
{
    if (!w_dense || !x || !y || ldx < ncols) return -1;
#pragma omp parallel for schedule(dynamic, 1)
    for (int r = 0; r < rows; ++r)
        for (int64_t c = 0; c < ncols; ++c) {
            double acc = 0.0;
            for (int t = 0; t < k; ++t)
                acc += w_dense[(int64_t)r * k + t] * bf16_to_double(x[(int64_t)t * ldx + c]);
            y[(int64_t)r * ncols + c] = acc;
        }
    return 0;
}

/* Same definition for a chosen list of rows only: y is [nsel, ncols]. */
int oracle_spmm_fp64_rows(const double *w_dense, int rows, int k,
                          const uint16_t *x, int64_t ldx, int64_t ncols,
                          const int32_t *sel, int nsel, double *y)
{
    if (!w_dense || !x || !y || !sel || ldx < ncols) return -1;
    for (int i = 0; i < nsel; ++i) if (sel[i] < 0 || sel[i] >= rows) return -1;
#pragma omp parallel for schedule(dynamic, 1)
    for (int i = 0; i < nsel; ++i)
        for (int64_t c = 0; c < ncols; ++c) {
            double acc = 0.0;
            for (int t = 0; t < k; ++t)
                acc += w_dense[(int64_t)sel[i] * k + t] * bf16_to_double(x[(int64_t)t * ldx + c]);
            y[(int64_t)i * ncols + c] = acc;
        }
    return 0;
}

/*
 * Variant used only where the literal loop would take too long: for each row the
 * t loop is outermost and terms with Wd == 0 are skipped.  Every Y[r, c] is still
 * the sum over ascending t of the same products, so the result is identical up to
 * the sign of zero; the tests show equality on small shapes.
 */
int oracle_spmm_fp64_skipzero(const double *w_dense, int rows, int k,
                              const uint16_t *x, int64_t ldx, int64_t ncols, double *y)
{
    if (!w_dense || !x || !y || ldx < ncols) return -1;
#pragma omp parallel for schedule(dynamic, 1)
    for (int r = 0; r < rows; ++r) {
        double *yr = y + (int64_t)r * ncols;
        for (int64_t c = 0; c < ncols; ++c) yr[c] = 0.0;
        for (int t = 0; t < k; ++t) {
            const double wv = w_dense[(int64_t)r * k + t];
            if (wv == 0.0) continue;
            const uint16_t *xr = x + (int64_t)t * ldx;
            for (int64_t c = 0; c < ncols; ++c) yr[c] += wv * bf16_to_double(xr[c]);
        }
    }
    return 0;
}

/* --------------------------------------------- global rank selection (Algorithm 1) */

/*
 * Algorithm 1, the steps between the block scores and the pruning itself, over all
 * layers of a network (Sec. III-C, "Pruning Algorithm"):
 *   sort    : inside every row of a layer's block grid, order the block scores
 *             increasingly; S[rt][o] is the o-th smallest score of row tile rt;
 *   c_o     : add S[rt][o] over the row tiles rt, for every rank position o;
 *   C_o     : order all c_o of all layers increasingly ("globally across the network");
 *   select  : prune rank positions from the front of that order until the current
 *             sparsity target is met.
 * Pruning rank position o of a layer removes one block from every row tile, so every
 * row keeps the same number of blocks; since c_o cannot decrease with o, what a
 * layer loses is always its lowest rank positions, and the result per layer is one
 * number: kkeep = nblk - (pruned rank positions).
 *
 * Readings where the paper is silent:
 *   - A layer's scores are integers in units of 2^(scale_exp - 40) (the layer's own
 *     fixed-point scale); rank sums are compared across layers by their real values
 *     c * 2^scale_exp, exactly.  Ties go to the lower layer index, then the lower o.
 *   - The target is a number of weights: floor(prune_fraction * total + 0.5), total =
 *     sum over layers of nrt * nblk * block_elems (whole blocks).  A rank position
 *     weighs nrt * block_elems.  Positions are pruned in order while the weight
 *     pruned so far is still below the target (the shortest front that reaches it).
 *   - The last min_keep rank positions of a layer are never candidates.
 *
 * score[l] : [nrt[l]][nblk[l]] block scores of layer l
 * kkeep_out: [n_layers]
 */
typedef unsigned __int128 oracle_u128;

typedef struct {
    oracle_u128 c;
    int scale_exp, layer, o;
    uint64_t weight;
} oracle_rank_entry;

static int u128_bits(oracle_u128 v)
{
    int n = 0;
    while (v) { ++n; v >>= 1; }
    return n;
}

/* sign of a.c * 2^a.scale_exp - b.c * 2^b.scale_exp, then layer, then o */
static int rank_entry_cmp(const void *pa, const void *pb)
{
    const oracle_rank_entry *a = (const oracle_rank_entry *)pa, *b = (const oracle_rank_entry *)pb;
    int sign = 0;
    if (a->c == 0 || b->c == 0) {
        sign = (a->c != 0) - (b->c != 0);
    } else {
        const int top_a = u128_bits(a->c) + a->scale_exp, top_b = u128_bits(b->c) + b->scale_exp;
        if (top_a != top_b) {
            sign = top_a < top_b ? -1 : 1;
        } else {
            /* same leading bit position: bring both to the smaller exponent; the shifted one ends
             * with exactly as many bits as the other, so nothing is lost */
            oracle_u128 va = a->c, vb = b->c;
            if (a->scale_exp > b->scale_exp) va <<= (a->scale_exp - b->scale_exp);
            else vb <<= (b->scale_exp - a->scale_exp);
            sign = va < vb ? -1 : (va > vb ? 1 : 0);
        }
    }
    if (sign) return sign;
    if (a->layer != b->layer) return a->layer < b->layer ? -1 : 1;
    return a->o < b->o ? -1 : (a->o > b->o ? 1 : 0);
}

static int u64_cmp(const void *pa, const void *pb)
{
    const uint64_t a = *(const uint64_t *)pa, b = *(const uint64_t *)pb;
    return a < b ? -1 : (a > b ? 1 : 0);
}

int oracle_global_rank(int n_layers, const uint64_t *const *score, const int *nrt, const int *nblk,
                       const int *scale_exp, const int64_t *block_elems, const int *min_keep,
                       double prune_fraction, int32_t *kkeep_out)
{
    if (n_layers <= 0 || !score || !nrt || !nblk || !scale_exp || !block_elems || !min_keep || !kkeep_out) return -1;
    if (!(prune_fraction >= 0.0 && prune_fraction <= 1.0)) return -1;
    int64_t n_entries = 0;
    double total = 0.0;
    for (int l = 0; l < n_layers; ++l) {
        if (!score[l] || nrt[l] <= 0 || nblk[l] <= 0 || block_elems[l] <= 0 || min_keep[l] < 0) return -1;
        n_entries += nblk[l];
        total += (double)nrt[l] * (double)nblk[l] * (double)block_elems[l];
    }
    const uint64_t target = (uint64_t)floor(prune_fraction * total + 0.5);
    oracle_rank_entry *entry = (oracle_rank_entry *)malloc(sizeof(oracle_rank_entry) * (size_t)n_entries);
    if (!entry) return -2;
    int64_t n = 0;
    for (int l = 0; l < n_layers; ++l) {
        uint64_t *row = (uint64_t *)malloc(sizeof(uint64_t) * (size_t)nblk[l]);
        oracle_u128 *c = (oracle_u128 *)calloc((size_t)nblk[l], sizeof(oracle_u128));
        if (!row || !c) { free(row); free(c); free(entry); return -2; }
        for (int rt = 0; rt < nrt[l]; ++rt) {
            memcpy(row, score[l] + (int64_t)rt * nblk[l], sizeof(uint64_t) * (size_t)nblk[l]);
            qsort(row, (size_t)nblk[l], sizeof(uint64_t), u64_cmp);          /* sort per row, increasing */
            for (int o = 0; o < nblk[l]; ++o) c[o] += row[o];                /* c_o: sum down the column */
        }
        const int candidates = nblk[l] - min_keep[l];
        for (int o = 0; o < candidates; ++o) {
            entry[n].c = c[o]; entry[n].scale_exp = scale_exp[l]; entry[n].layer = l; entry[n].o = o;
            entry[n].weight = (uint64_t)nrt[l] * (uint64_t)block_elems[l];
            ++n;
        }
        kkeep_out[l] = nblk[l];
        free(row); free(c);
    }
    qsort(entry, (size_t)n, sizeof(oracle_rank_entry), rank_entry_cmp);      /* C_o: global order */
    uint64_t pruned = 0;
    for (int64_t i = 0; i < n && pruned < target; ++i) {                     /* select by the target */
        pruned += entry[i].weight;
        kkeep_out[entry[i].layer] -= 1;
    }
    free(entry);
    return 0;
}

/* ------------------------------------------------ convolution as implicit GEMM */

/*
 * The same product for a convolution layer (Sec. III, Notation: a K x K x R x S filter bank is the
 * matrix W with S rows, one per output channel, and K*K*R reduction elements; the paper runs the
 * hybrid pattern on that matrix).  The oracle is the definition of the convolution, with the
 * reduction index of W ordered (kernel row, kernel column, input channel), channel fastest:
 *
 *   Y[s, b, y, x] = sum over (i, j, r) of Wd[s, (i*kw + j)*R + r] * A[b, y + i - pad, x + j - pad, r]
 *
 * stride 1, zero padding `pad` on every side, A in NHWC order [batch, height, width, R] as bf16 bit
 * patterns, Y as [S, batch*ho*wo] with ho = height + 2*pad - kh + 1 (wo likewise), fp64 accumulation
 * in ascending (i, j, r) order.  w_dense is the decoded masked weight, [S, kh*kw*R] in fp64.
 */
int oracle_conv_fp64(const double *w_dense, int s_out, int kh, int kw, int r_in,
                     const uint16_t *act, int batch, int height, int width, int pad, double *y)
{
    if (!w_dense || !act || !y || s_out <= 0 || kh <= 0 || kw <= 0 || r_in <= 0) return -1;
    if (batch <= 0 || height <= 0 || width <= 0 || pad < 0) return -1;
    const int ho = height + 2 * pad - kh + 1, wo = width + 2 * pad - kw + 1;
    if (ho <= 0 || wo <= 0) return -1;
    const int64_t k = (int64_t)kh * kw * r_in, npix = (int64_t)batch * ho * wo;
#pragma omp parallel for schedule(dynamic, 1)
    for (int s = 0; s < s_out; ++s)
        for (int b = 0; b < batch; ++b)
            for (int oy = 0; oy < ho; ++oy)
                for (int ox = 0; ox < wo; ++ox) {
                    double acc = 0.0;
                    for (int i = 0; i < kh; ++i)
                        for (int j = 0; j < kw; ++j) {
                            const int iy = oy + i - pad, ix = ox + j - pad;
                            if (iy < 0 || iy >= height || ix < 0 || ix >= width) continue;   /* zero padding */
                            const uint16_t *a = act + (((int64_t)b * height + iy) * width + ix) * r_in;
                            const double *wr = w_dense + (int64_t)s * k + ((int64_t)i * kw + j) * r_in;
                            for (int r = 0; r < r_in; ++r) acc += wr[r] * bf16_to_double(a[r]);
                        }
                    y[(int64_t)s * npix + ((int64_t)b * ho + oy) * wo + ox] = acc;
                }
    return 0;
}

/* -------------------------------------------------------------- layer epilogue */

/*
 * The step that closes a layer of the networks the paper prunes (Sec. IV): per output channel a
 * bias, then optionally the rectifier.  In place on the fp64 product y [rows, ncols]:
 *   y[r, c] = max(y[r, c] + bias[r], 0)   (the max only when relu != 0; bias may be NULL)
 */
int oracle_bias_relu(double *y, int rows, int64_t ncols, const float *bias, int relu)
{
    if (!y || rows <= 0 || ncols <= 0) return -1;
    for (int r = 0; r < rows; ++r)
        for (int64_t c = 0; c < ncols; ++c) {
            double v = y[(int64_t)r * ncols + c] + (bias ? (double)bias[r] : 0.0);
            if (relu && v < 0.0) v = 0.0;
            y[(int64_t)r * ncols + c] = v;
        }
    return 0;
}

/* ---------------------------------------------------------------- saliency score */

/*
 * Class-aware saliency score, Sec. III-C "Pruning Metric", Eq. 1:
 *   T_w = | (1/H) * sum over the H samples of g_i  (.)  W |      (element-wise)
 * grads: H tensors [rows, k] laid out one after the other, as doubles (the values the caller's
 * gradients hold); w: bf16 bit patterns; out: fp64.
 */
int oracle_saliency(const double *grads, int samples, const uint16_t *w, int rows, int k, double *out)
{
    if (!grads || !w || !out || samples <= 0 || rows <= 0 || k <= 0) return -1;
    const int64_t n = (int64_t)rows * k;
    for (int64_t e = 0; e < n; ++e) {
        double sum = 0.0;
        for (int i = 0; i < samples; ++i) sum += grads[(int64_t)i * n + e];
        out[e] = fabs(sum / (double)samples * bf16_to_double(w[e]));
    }
    return 0;
}

/*
 * The same score in the precision and order in which a caller's fp32 accumulation produces it, for
 * comparisons where the score decides integers downstream (the mask): the H gradients are added in the
 * given order in fp32, the sum is multiplied by the fp32 reciprocal of H, then by the weight, each
 * product rounded to fp32; out = |.|.  (Eq. 1 fixes neither precision nor order; this is one evaluation of
 * it, within a few ulp of oracle_saliency.)  grads: H tensors [rows, k] as floats.
 */
int oracle_saliency_f32(const float *grads, int samples, const uint16_t *w, int rows, int k, float *out)
{
    if (!grads || !w || !out || samples <= 0 || rows <= 0 || k <= 0) return -1;
    const int64_t n = (int64_t)rows * k;
    const volatile float inv = 1.0f / (float)samples;
    for (int64_t e = 0; e < n; ++e) {
        volatile float sum = grads[e];
        for (int i = 1; i < samples; ++i) sum = sum + grads[(int64_t)i * n + e];
        volatile float t = sum * inv;              /* volatile: every step is rounded to fp32, nothing fused */
        t = t * (float)bf16_to_double(w[e]);
        out[e] = fabsf(t);
    }
    return 0;
}
