"""Pins of the CPU oracle against what the paper and plain mathematics fix.

None of these tests touches the CUDA library.  They are chosen so that a plausible
mistake in the oracle (a dropped term, a wrong sign or index, a transposed
operand, a one-based offset, a wrong tie rule) fails at least one of them.
"""
import itertools
import math
import os

import numpy as np
import pytest

import oracle
from paper_2311_14272_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------- small helpers

def rand_bf16(rng, shape, scale=1.0):
    return wl.f32_to_bf16_bits(rng.standard_normal(shape).astype(np.float32) * np.float32(scale))


def unpack_idx(idx_words, count, b):
    """Read `count` b-bit fields, LSB-first, from a uint32 stream (independent reader)."""
    bits = np.unpackbits(np.ascontiguousarray(idx_words).view(np.uint8), bitorder="little")
    out = np.zeros(count, dtype=np.int64)
    for q in range(b):
        out |= bits[q:count * b:b].astype(np.int64) << q
    return out


def numpy_group_mask(s, n, m):
    """Independent N:M selection: stable argsort of -|s| inside every group."""
    rows, k = s.shape
    g = np.abs(s).reshape(rows, k // m, m)
    order = np.argsort(-g, axis=2, kind="stable")
    mask = np.zeros_like(g, dtype=bool)
    np.put_along_axis(mask, order[:, :, :n], True, axis=2)
    return mask.reshape(rows, k)


def exact_q(v: float, e_max: int) -> int:
    """floor(v * 2^(40 - e_max)) in exact integer arithmetic."""
    mant, ex = math.frexp(float(v))            # v = mant * 2^ex, exactly
    num = int(mant * (1 << 53))                # exact: mant has <= 53 bits
    sh = ex - 53 + 40 - e_max
    return num << sh if sh >= 0 else num >> (-sh)


# ------------------------------------------------------------ P5: worked example

def _golden_rows():
    rows = []
    with open(os.path.join(GOLDEN, "offset_example.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            a, b, c = [p.split() for p in line.split("|")]
            rows.append((int(a[0]), int(a[1]), [float(v) for v in b], [int(v) for v in c]))
    return rows


@pytest.mark.parametrize("m,n,sal,offsets", _golden_rows())
def test_offset_convention_matches_paper_example(m, n, sal, offsets):
    """Section III-E: the second value of its M-vector has index 1 (zero-based)."""
    s = np.array([sal], dtype=np.float32)
    mask = oracle.build_mask(s, n, m, block_rows=1, block_k=m, keep_ratio=1.0)
    w = wl.f32_to_bf16_bits(np.array([sal], dtype=np.float32))
    vals, idx = oracle.encode(w, mask)
    got = unpack_idx(idx, n, int(math.log2(m)))
    assert list(got) == offsets
    assert list(wl.bf16_bits_to_f32(vals)) == [sal[o] for o in offsets]


# --------------------------------------------------------- keep-count rounding

@pytest.mark.parametrize("nblk,keep,expect", [
    (1, 0.5, 1), (5, 0.5, 3), (1, 0.4, 0), (3, 0.5, 2), (6, 0.5, 3), (10, 0.5, 5),
    (12, 0.5, 6), (18, 0.5, 9), (30, 0.5, 15), (64, 0.1, 6), (64, 0.25, 16),
    (36, 0.25, 9), (16, 0.5, 8), (7, 0.0, 0), (7, 1.0, 7),
])
def test_keep_count_rounds_half_up(nblk, keep, expect):
    got_nblk, kkeep = oracle.keep_count(nblk * 32, 32, keep)
    assert (got_nblk, kkeep) == (nblk, expect)
    # a ragged last block still counts as one block
    got_nblk, _ = oracle.keep_count(nblk * 32 - 5, 32, keep)
    assert got_nblk == nblk


# --------------------------------------------------- P1 / P2: invariants, counts

SHAPES = [
    # rows, k, n, m, bm, bk, keep
    (256, 1024, 2, 4, 32, 64, 0.5),      # config 1
    (128, 576, 1, 4, 64, 64, 0.25),
    (96, 144, 2, 8, 32, 32, 0.5),        # ragged k (144 = 4.5 blocks)
    (24, 27, 2, 4, 64, 64, 1.0),         # one padded block, ragged group at k = 27
    (70, 200, 3, 4, 32, 32, 0.4),
    (160, 256, 4, 8, 128, 64, 0.75),
    (64, 96, 8, 8, 32, 32, 0.67),        # n == m: block sparsity only
]


@pytest.mark.parametrize("rows,k,n,m,bm,bk,keep", SHAPES)
def test_mask_invariants_and_closed_forms(rows, k, n, m, bm, bk, keep):
    rng = np.random.default_rng(rows * 7 + k)
    s = rng.standard_normal((rows, k)).astype(np.float32)
    mk = oracle.build_mask(s, n, m, bm, bk, keep)
    nrt, nblk = mk.nrt, mk.nblk
    dense = mk.dense()
    assert dense.shape == (nrt * bm, nblk * bk)
    blocks = dense.reshape(nrt, bm, nblk, bk).transpose(0, 2, 1, 3)      # [rt, jb, r, c]
    kept = np.zeros((nrt, nblk), dtype=bool)
    for rt in range(nrt):
        cols = mk.blk_col[rt]
        assert len(cols) == mk.kkeep
        assert np.all(np.diff(cols) > 0)                                    # ascending, distinct
        assert np.all((cols >= 0) & (cols < nblk))
        kept[rt, cols] = True
    # Sec. III-A: exactly N per M inside kept blocks, nothing outside
    per_group = blocks.reshape(nrt, nblk, bm, bk // m, m).sum(axis=4)
    assert np.all(per_group[kept] == n)
    assert np.all(per_group[~kept] == 0)
    # every row of the block grid keeps the same number of blocks (Sec. III-A/III-C)
    assert np.all(kept.sum(axis=1) == mk.kkeep)
    # closed forms of Sec. III-A
    nnz = int(dense.sum())
    assert nnz == nrt * mk.kkeep * bm * bk * n // m
    kprime = mk.kkeep * bk
    sparsity = 1.0 - nnz / (nrt * bm * nblk * bk)
    assert sparsity == pytest.approx(1.0 - (kprime / (nblk * bk)) * (n / m), abs=1e-12)
    nvals, nwords = oracle.encoded_sizes(rows, bm, bk, n, m, mk.kkeep)
    assert nvals == nnz
    assert nwords == (nrt * bm * kprime * n // m * int(math.log2(m)) + 31) // 32
    # the N:M choice matches an independent numpy selection on the padded tensor
    sp = np.zeros((nrt * bm, nblk * bk), dtype=np.float32)
    sp[:rows, :k] = s
    want = numpy_group_mask(sp, n, m) & np.repeat(np.repeat(kept, bm, axis=0), bk, axis=1)
    assert np.array_equal(dense, want)


def test_block_scores_are_exact_fixed_point_sums():
    rng = np.random.default_rng(5)
    rows, k, n, m, bm, bk = 64, 128, 2, 4, 32, 32
    s = (rng.standard_normal((rows, k)) * np.exp(rng.uniform(-12, 3, (rows, k)))).astype(np.float32)
    for mode in (0, 1):
        mk = oracle.build_mask(s, n, m, bm, bk, 0.5, score_mode=mode)
        e_max = math.frexp(float(np.abs(s).max()))[1] - 1
        sel = numpy_group_mask(s, n, m) if mode == 0 else np.ones_like(s, dtype=bool)
        for rt in range(rows // bm):
            for jb in range(k // bk):
                blk = np.abs(s[rt * bm:(rt + 1) * bm, jb * bk:(jb + 1) * bk])
                bsel = sel[rt * bm:(rt + 1) * bm, jb * bk:(jb + 1) * bk]
                want = sum(exact_q(v, e_max) for v in blk[bsel])
                assert int(mk.score[rt, jb]) == want


def test_block_choice_is_topk_by_score_and_modes_differ():
    # block 0: one huge survivor per group, rest tiny;  block 1: uniformly medium
    s = np.zeros((2, 8), dtype=np.float32)
    s[:, 0:4] = [10.0, 9.0, 9.0, 9.0]     # survivors (1:4) sum 10, all-elements sum 37
    s[:, 4:8] = [12.0, 0.0, 0.0, 0.0]     # survivors sum 12,   all-elements sum 12
    m0 = oracle.build_mask(s, 1, 4, 2, 4, kkeep=1, score_mode=0)
    m1 = oracle.build_mask(s, 1, 4, 2, 4, kkeep=1, score_mode=1)
    assert list(m0.blk_col[0]) == [1]
    assert list(m1.blk_col[0]) == [0]


def test_non_finite_and_signed_saliency():
    s = np.array([[np.nan, -3.0, 2.0, -0.0, np.inf, 1e30, -np.inf, 5.0]], dtype=np.float32)
    mk = oracle.build_mask(s, 2, 4, 1, 4, 1.0)
    # group 0: |-3| and 2 win over NaN (-> 0) and -0;  group 1: the two infinities win
    assert list(mk.dense()[0].astype(int)) == [0, 1, 1, 0, 1, 0, 1, 0]


# ------------------------------------------------------------- tie-break rules

def test_ties_go_to_lower_index():
    s = np.ones((4, 16), dtype=np.float32)
    mk = oracle.build_mask(s, 2, 4, 2, 4, 0.5)
    assert mk.kkeep == 2
    assert np.array_equal(mk.blk_col, [[0, 1], [0, 1]])
    row = mk.dense()[0].astype(int)
    assert list(row) == [1, 1, 0, 0, 1, 1, 0, 0] + [0] * 8
    # partial tie inside a group: the larger wins, then the lower of the equal pair
    s2 = np.array([[1, 5, 1, 1]], dtype=np.float32)
    assert list(oracle.build_mask(s2, 2, 4, 1, 4, 1.0).dense()[0].astype(int)) == [1, 1, 0, 0]
    # tie between blocks with equal score: lower column kept, output ascending
    s3 = np.array([[1, 0, 0, 0, 2, 0, 0, 0, 1, 0, 0, 0]], dtype=np.float32)
    assert list(oracle.build_mask(s3, 1, 4, 1, 4, kkeep=2).blk_col[0]) == [0, 1]


# ------------------------------------------------------------- P3: brute force

def _all_hybrid_masks(nrt, nblk, bm, bk, n, m, kkeep):
    """Every mask with kkeep blocks per row tile and exactly N of M in kept blocks."""
    groups = bk // m
    group_choices = list(itertools.combinations(range(m), n))
    per_block = list(itertools.product(group_choices, repeat=bm * groups))
    tiles = []
    for blocks in itertools.combinations(range(nblk), kkeep):
        for fill in itertools.product(per_block, repeat=kkeep):
            tiles.append((blocks, fill))
    return tiles, groups


@pytest.mark.parametrize("n,kkeep", [(1, 1), (2, 1), (3, 1), (1, 2), (2, 2), (3, 2)])
def test_mask_is_the_unique_maximiser_of_retained_saliency(n, kkeep):
    """Enumerate every admissible hybrid mask of a tiny layer; the oracle's mask must
    retain the maximum total saliency, and be the only mask that does."""
    nrt, nblk, bm, bk, m = 2, 3, 1 if n == 2 and kkeep == 2 else 2, 4, 4
    rng = np.random.default_rng(100 * n + kkeep)
    vals = rng.choice(1 << 20, size=nrt * bm * nblk * bk, replace=False) + 1
    s = vals.reshape(nrt * bm, nblk * bk).astype(np.float32)        # integers: sums are exact
    if rng.random() < 0.5:
        s *= np.float32(-1.0)                                        # sign must not matter
    mk = oracle.build_mask(s, n, m, bm, bk, kkeep=kkeep)
    got = mk.dense()
    tiles, groups = _all_hybrid_masks(nrt, nblk, bm, bk, n, m, kkeep)
    a = np.abs(s).astype(np.int64)
    for rt in range(nrt):
        best, best_masks = -1, []
        for blocks, fill in tiles:
            mask = np.zeros((bm, nblk * bk), dtype=bool)
            for jb, groups_sel in zip(blocks, fill):
                for gi, sel in enumerate(groups_sel):
                    r, g = divmod(gi, groups)
                    for t in sel:
                        mask[r, jb * bk + g * m + t] = True
            tot = int(a[rt * bm:(rt + 1) * bm][mask].sum())
            if tot > best:
                best, best_masks = tot, [mask]
            elif tot == best:
                best_masks.append(mask)
        mine = got[rt * bm:(rt + 1) * bm]
        assert int(a[rt * bm:(rt + 1) * bm][mine].sum()) == best
        if len(best_masks) == 1:
            assert np.array_equal(mine, best_masks[0])


# ------------------------------------------------- P4: encode / decode round trip

@pytest.mark.parametrize("rows,k,n,m,bm,bk,keep", SHAPES)
def test_encode_decode_round_trip(rows, k, n, m, bm, bk, keep):
    rng = np.random.default_rng(rows + k)
    w = rand_bf16(rng, (rows, k), 0.05)
    w[w == 0x8000] = 0
    s = (np.abs(wl.bf16_bits_to_f32(w)) * rng.uniform(0.5, 1.5, (rows, k))).astype(np.float32)
    mk = oracle.build_mask(s, n, m, bm, bk, keep)
    vals, idx = oracle.encode(w, mk)
    wd, wb = oracle.decode(mk.blk_col, vals, idx, rows, k, n, m, bm, bk, mk.kkeep)
    want_bits = np.where(mk.dense()[:rows, :k], w, np.uint16(0))
    assert np.array_equal(wb, want_bits)                                   # == W (.) mask, bit for bit
    assert np.array_equal(wd, wl.bf16_bits_to_f32(want_bits).astype(np.float64))
    # encoding the decoded matrix under the same mask reproduces the encoding
    vals2, idx2 = oracle.encode(wb, mk)
    assert np.array_equal(vals, vals2) and np.array_equal(idx, idx2)
    # offsets, read by an independent bit reader, are ascending inside each group
    b = int(math.log2(m))
    offs = unpack_idx(idx, len(vals), b).reshape(-1, n)
    assert np.all(np.diff(offs, axis=1) > 0) if n > 1 else True
    assert offs.min() >= 0 and offs.max() < m
    # the stored order is (row tile, slot, local row, group, value)
    dense = mk.dense()
    o = 0
    for rt in range(min(mk.nrt, 2)):
        for j in range(mk.kkeep):
            jb = int(mk.blk_col[rt, j])
            for r in (0, bm - 1):
                base = ((rt * mk.kkeep + j) * bm + r) * (bk // m) * n
                row = rt * bm + r
                pos = np.flatnonzero(dense[row, jb * bk:(jb + 1) * bk])
                want_offs = pos % m
                assert list(unpack_idx(idx, len(vals), b)[base:base + len(pos)]) == list(want_offs)
                if row < rows:
                    cols = jb * bk + pos
                    exp = np.where(cols < k, w[row, np.minimum(cols, k - 1)], 0)
                    assert list(vals[base:base + len(pos)]) == list(exp)


def test_encode_rejects_a_mask_that_breaks_n_of_m():
    s = np.arange(1, 17, dtype=np.float32).reshape(2, 8)
    mk = oracle.build_mask(s, 2, 4, 2, 4, 1.0)
    mk.nm_bits[0, 0] |= 0xF
    with pytest.raises(ValueError):
        oracle.encode(np.ones((2, 8), dtype=np.uint16), mk)


# ------------------------------------------ P6 / P8: product against numpy, cases

def _setup(rows, k, ncols, n, m, bm, bk, keep, seed=0):
    rng = np.random.default_rng(seed)
    w = rand_bf16(rng, (rows, k), 0.05)
    s = (np.abs(wl.bf16_bits_to_f32(w)) * rng.uniform(0.5, 1.5, (rows, k))).astype(np.float32)
    x = rand_bf16(rng, (k, ncols))
    mk = oracle.build_mask(s, n, m, bm, bk, keep)
    vals, idx = oracle.encode(w, mk)
    wd, wb = oracle.decode(mk.blk_col, vals, idx, rows, k, n, m, bm, bk, mk.kkeep)
    return w, s, x, mk, wd, wb


def test_product_matches_numpy_fp64_gemm():
    w, s, x, mk, wd, _ = _setup(48, 96, 37, 2, 4, 16, 32, 0.67)
    y = oracle.spmm_fp64(wd, x)
    xd = wl.bf16_bits_to_f32(x).astype(np.float64)
    want = wd @ xd
    assert y.shape == (48, 37)
    assert np.allclose(y, want, rtol=1e-12, atol=1e-14)
    # non-square on purpose: a transposed operand or swapped stride cannot pass
    assert np.array_equal(oracle.spmm_fp64_skipzero(wd, x), y)
    sel = np.array([47, 0, 13], dtype=np.int32)
    assert np.array_equal(oracle.spmm_fp64_rows(wd, x, sel), y[sel])


def test_dense_special_case_n_equals_m_keep_all():
    """n == m and keep == 1 is a plain dense GEMM of W."""
    w, s, x, mk, wd, wb = _setup(32, 64, 20, 4, 4, 16, 32, 1.0, seed=3)
    assert np.array_equal(wb, w)
    want = wl.bf16_bits_to_f32(w).astype(np.float64) @ wl.bf16_bits_to_f32(x).astype(np.float64)
    assert np.allclose(oracle.spmm_fp64(wd, x), want, rtol=1e-12, atol=1e-14)


def test_keep_all_2of4_is_gemm_of_the_nm_masked_weight():
    w, s, x, mk, wd, wb = _setup(32, 64, 20, 2, 4, 16, 32, 1.0, seed=4)
    wm = np.where(numpy_group_mask(s, 2, 4), wl.bf16_bits_to_f32(w), 0).astype(np.float64)
    want = wm @ wl.bf16_bits_to_f32(x).astype(np.float64)
    assert np.allclose(oracle.spmm_fp64(wd, x), want, rtol=1e-12, atol=1e-14)


def test_no_kept_block_gives_zero_output():
    w, s, x, mk, wd, wb = _setup(16, 27, 9, 2, 4, 16, 64, 0.4, seed=5)   # nblk = 1 -> kkeep = 0
    assert mk.kkeep == 0 and mk.blk_col.shape == (1, 0)
    assert not mk.dense().any()
    assert np.count_nonzero(oracle.spmm_fp64(wd, x)) == 0


def test_identity_activation_returns_the_decoded_weight():
    w, s, x, mk, wd, wb = _setup(40, 64, 64, 1, 4, 8, 16, 0.5, seed=6)
    eye = wl.f32_to_bf16_bits(np.eye(64, dtype=np.float32))
    assert np.array_equal(oracle.spmm_fp64(wd, eye), wd)
    onehot = np.zeros((64, 3), dtype=np.float32)
    onehot[[5, 17, 63], [0, 1, 2]] = 1
    y = oracle.spmm_fp64(wd, wl.f32_to_bf16_bits(onehot))
    assert np.array_equal(y, wd[:, [5, 17, 63]])


# ------------------------------------------------------------ P7: invariances

def test_power_of_two_scaling_of_saliency_keeps_the_mask():
    rng = np.random.default_rng(8)
    s = rng.standard_normal((64, 256)).astype(np.float32)
    a = oracle.build_mask(s, 2, 8, 32, 32, 0.5)
    b = oracle.build_mask(s * np.float32(2.0 ** -9), 2, 8, 32, 32, 0.5)
    assert np.array_equal(a.blk_col, b.blk_col) and np.array_equal(a.nm_bits, b.nm_bits)
    assert np.array_equal(a.score, b.score)


def test_block_column_permutation_commutes():
    rng = np.random.default_rng(9)
    rows, k, ncols, n, m, bm, bk = 32, 128, 24, 2, 4, 16, 16
    w = rand_bf16(rng, (rows, k), 0.05)
    s = rng.uniform(0.1, 1.0, (rows, k)).astype(np.float32)
    x = rand_bf16(rng, (k, ncols))
    perm = rng.permutation(k // bk)
    colperm = (perm[:, None] * bk + np.arange(bk)[None, :]).reshape(-1)
    m1 = oracle.build_mask(s, n, m, bm, bk, 0.5)
    m2 = oracle.build_mask(s[:, colperm], n, m, bm, bk, 0.5)
    inv = np.argsort(perm)
    for rt in range(m1.nrt):
        assert sorted(inv[m1.blk_col[rt]]) == list(m2.blk_col[rt])

    def product(wbits, mk, xbits):
        v, i = oracle.encode(wbits, mk)
        wd, _ = oracle.decode(mk.blk_col, v, i, rows, k, n, m, bm, bk, mk.kkeep)
        return oracle.spmm_fp64(wd, xbits)

    y1 = product(w, m1, x)
    y2 = product(w[:, colperm], m2, x[colperm, :])
    assert np.allclose(y1, y2, rtol=1e-12, atol=1e-15)


def test_product_is_linear_in_x():
    w, s, x, mk, wd, _ = _setup(24, 64, 10, 2, 4, 8, 32, 0.5, seed=11)
    x2 = rand_bf16(np.random.default_rng(12), x.shape)
    xs = wl.f32_to_bf16_bits(np.zeros(x.shape, dtype=np.float32))
    ya, yb = oracle.spmm_fp64(wd, x), oracle.spmm_fp64(wd, x2)
    # exact sum of two bf16 operands is not a bf16 in general: feed the sum column-wise instead
    stacked = np.concatenate([x, x2], axis=1)
    ys = oracle.spmm_fp64(wd, stacked)
    assert np.array_equal(ys[:, :10], ya) and np.array_equal(ys[:, 10:], yb)
    assert np.count_nonzero(oracle.spmm_fp64(wd, xs)) == 0


# ----------------------------------------------------- workloads: shapes, seeds

def test_workload_tables_have_the_published_layer_shapes():
    cfg = wl.all_configs()
    assert [(l.rows, l.k, l.ncols) for l in cfg[1]] == [(256, 1024, 512)]
    assert [(l.rows, l.k, l.ncols) for l in cfg[2]] == [(256, 2304, 6272)]
    assert len(cfg[3]) == 13 and cfg[3][0].k == 27 and cfg[3][1].ncols == 16 * 224 * 224
    assert sum(l.rows * l.k * l.ncols for l in cfg[3]) == 16 * 15346630656 // 1
    assert len(cfg[4]) == 35
    assert {l.k for l in cfg[4]} == {16, 24, 32, 64, 96, 144, 160, 192, 320, 384, 576, 960}
    assert {l.ncols for l in cfg[4]} == {802816, 200704, 50176, 12544, 3136}
    assert len(cfg[5]) == 20
    assert all(0.1 <= l.keep_ratio <= 0.5 for l in cfg[3])


def test_generators_are_seeded_and_bf16_rounding_is_nearest_even():
    l = wl.config1()[0]
    w1, s1, x1 = wl.make_layer_inputs(l)
    w2, s2, x2 = wl.make_layer_inputs(l)
    assert np.array_equal(w1, w2) and np.array_equal(s1, s2) and np.array_equal(x1, x2)
    assert s1.dtype == np.float32 and w1.dtype == np.uint16 and x1.shape == (1024, 512)
    f = np.array([1.0, 1.00390625, 1.01171875, -2.5, 3.0e38], dtype=np.float32)
    # 1 + 2^-8 is a tie -> even (1.0); 1 + 3*2^-8 is a tie -> even (1 + 2^-6)
    assert list(wl.f32_to_bf16_bits(f)[:4]) == [0x3F80, 0x3F80, 0x3F82, 0xC020]
    assert np.array_equal(wl.bf16_bits_to_f32(wl.f32_to_bf16_bits(f[:1])), f[:1])
