"""CUDA path against the CPU oracle, through the C ABI, on the same seeded inputs.

Masks and encodings must match bit for bit; the product must satisfy
max |Y - Yref| <= 1e-2 * (1 + |Yref|) and ||Y - Yref||_F / ||Yref||_F <= 5e-3."""
import numpy as np
import pytest

import oracle
from paper_2311_14272_b200 import workloads as wl

from helpers import (assert_mask_and_encoding_equal, bf16_dev, check_tolerance, gpu_layer,
                     oracle_layer, to_dev, y_to_f64)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    from paper_2311_14272_b200 import binding as B
    B.load()
    assert torch.cuda.is_available()
    return B, torch


def rand_inputs(rows, k, ncols, seed, relu=False):
    rng = np.random.default_rng(seed)
    w = wl.f32_to_bf16_bits((rng.standard_normal((rows, k)) * 0.05).astype(np.float32))
    s = (np.abs(wl.bf16_bits_to_f32(w)) * rng.uniform(0.5, 1.5, (rows, k))).astype(np.float32)
    x = rng.standard_normal((k, ncols)).astype(np.float32)
    if relu:
        x = np.maximum(x, 0)
    return w, s, wl.f32_to_bf16_bits(x)


CASES = [
    # rows, k, ncols, n, m, bm, bk, keep   (several tiles and a ragged tail in every dimension)
    (256, 1024, 512, 2, 4, 32, 64, 0.5),
    (200, 576, 333, 1, 4, 64, 64, 0.25),
    (96, 144, 1000, 2, 8, 32, 32, 0.5),
    (24, 27, 130, 2, 4, 64, 64, 1.0),
    (70, 200, 77, 3, 4, 32, 32, 0.4),
    (300, 640, 520, 4, 8, 128, 64, 0.75),
    (260, 512, 264, 1, 8, 128, 64, 0.5),
    (64, 96, 50, 8, 8, 32, 32, 0.67),
    (130, 384, 96, 2, 4, 128, 128, 0.34),
    (64, 288, 40, 3, 8, 64, 96, 0.67),
    (384, 768, 576, 2, 4, 128, 64, 0.5),     # 3 CTA tiles, 2.25 column tiles
    (512, 512, 320, 1, 4, 64, 64, 0.25),
    (256, 256, 128, 2, 8, 32, 32, 0.5),
    # thin layers (one CTA tile of at most 32 / 64 rows) with few columns: too few tiles for the stacked
    # accumulator, so these run the ordinary tiles (the stacked path has its own cases below)
    (16, 32, 5000, 2, 8, 32, 32, 1.0),
    (24, 96, 3000, 2, 8, 32, 32, 0.67),
    (32, 192, 4100, 2, 4, 32, 64, 0.5),
    (64, 192, 2500, 2, 8, 32, 32, 0.5),      # two row tiles of 32 in the 64-row window
    (48, 256, 1111, 3, 4, 64, 64, 0.5),      # dense-tile image, 48 of 64 rows
]


# which execution image crisp_encode lays out: the default choice (2:4 sparse MMA when n <= 2, dense
# tiles otherwise), dense tiles forced, or none (CUDA-core kernel on the canonical format)
# "sparse2": patterns with more than two values per 4-group as two 2:4-compliant addends (others: the default image)
IMAGES = ["auto", "dense", "none", "sparse2"]


@pytest.fixture(params=IMAGES)
def image(request, monkeypatch):
    kind = request.param
    if kind == "auto":
        monkeypatch.delenv("CRISP_EXEC_IMAGE", raising=False)
    else:
        monkeypatch.setenv("CRISP_EXEC_IMAGE", kind)
    return kind


def expected_path(B, image, n, kkeep=1):
    if image == "none":
        return B.PATH_DIRECT
    if image == "dense":
        return B.PATH_DENSE
    if image == "sparse2" and n > 2:
        return B.PATH_SPARSE2
    return B.PATH_SPARSE if n <= 2 else B.PATH_DENSE


@pytest.mark.parametrize("rows,k,ncols,n,m,bm,bk,keep", CASES)
@pytest.mark.parametrize("y_dtype", [0, 1])
def test_layer_matches_oracle(env, image, rows, k, ncols, n, m, bm, bk, keep, y_dtype):
    B, torch = env
    w, s, x = rand_inputs(rows, k, ncols, seed=rows + k + ncols)
    mk, vals, idx, wd, wb = oracle_layer(w, s, n, m, bm, bk, keep)
    L = gpu_layer(B, torch, w, s, n, m, bm, bk, keep)
    assert_mask_and_encoding_equal(L, mk, vals, idx)
    dec = L.decode().view(torch.int16).cpu().numpy().view(np.uint16)
    assert np.array_equal(dec, wb)
    # ncols padded to a multiple of 8 in memory so that the tensor-core kernels can address X and Y
    ld = (ncols + 7) // 8 * 8
    xbuf = torch.zeros((k, ld), dtype=torch.bfloat16, device="cuda")
    xbuf[:, :ncols] = bf16_dev(x, torch)
    ybuf = torch.full((rows, ld), 5.0, dtype=torch.float32 if y_dtype else torch.bfloat16, device="cuda")
    assert L.bytes_model(ncols, y_dtype)["path"] == expected_path(B, image, n)
    L.spmm(xbuf[:, :ncols], y=ybuf[:, :ncols], y_dtype=y_dtype)
    torch.cuda.synchronize()
    assert L.device_status() == 0
    assert L.last_launch()["path"] == expected_path(B, image, n)          # the kernel family that really ran
    check_tolerance(y_to_f64(ybuf[:, :ncols], torch), oracle.spmm_fp64(wd, x))
    assert torch.all(ybuf[:, ncols:] == 5.0)                             # nothing written past ncols
    L.close()


def test_score_mode_all_elements(env):
    B, torch = env
    w, _, x = rand_inputs(128, 512, 64, seed=77)
    # odd block columns: one dominant element per group; even ones: four medium elements, so the
    # survivor sum and the all-element sum rank the blocks differently
    rng = np.random.default_rng(3)
    s = rng.uniform(0.9, 1.1, (128, 512)).astype(np.float32)
    odd = ((np.arange(512) // 64) % 2 == 1)
    s[:, odd & (np.arange(512) % 4 != 0)] *= np.float32(0.01)
    s[:, odd & (np.arange(512) % 4 == 0)] *= np.float32(1.5)
    mk, vals, idx, wd, wb = oracle_layer(w, s, 1, 4, 32, 64, 0.5, score_mode=1)
    mk0 = oracle.build_mask(s, 1, 4, 32, 64, 0.5, score_mode=0)
    assert not np.array_equal(mk.blk_col, mk0.blk_col)       # the two readings differ on this input
    L = gpu_layer(B, torch, w, s, 1, 4, 32, 64, 0.5, score_mode=1)
    assert_mask_and_encoding_equal(L, mk, vals, idx)
    L0 = gpu_layer(B, torch, w, s, 1, 4, 32, 64, 0.5, score_mode=0)
    v0, i0 = oracle.encode(w, mk0)
    assert_mask_and_encoding_equal(L0, mk0, v0, i0)


def test_padded_leading_dimensions_and_odd_alignment(env):
    B, torch = env
    w, s, x = rand_inputs(100, 250, 90, seed=5)
    mk, vals, idx, wd, wb = oracle_layer(w, s, 2, 4, 32, 64, 0.5)
    L = gpu_layer(B, torch, w, s, 2, 4, 32, 64, 0.5, ld_pad=3)       # ld = 253: scalar-load path
    assert_mask_and_encoding_equal(L, mk, vals, idx)
    xbuf = torch.zeros((250, 97), dtype=torch.bfloat16, device="cuda")
    xbuf[:, :90] = bf16_dev(x, torch)
    ybuf = torch.full((100, 101), 7.0, dtype=torch.bfloat16, device="cuda")
    L.spmm(xbuf[:, :90], y=ybuf[:, :90])
    # pitches of 97 and 101 elements are not multiples of 16 bytes: TMA cannot address them, and the call
    # must have fallen back to the CUDA-core kernel although the handle carries a tensor-core image
    assert L.bytes_model(90)["path"] == B.PATH_SPARSE and L.last_launch()["path"] == B.PATH_DIRECT
    check_tolerance(y_to_f64(ybuf[:, :90], torch), oracle.spmm_fp64(wd, x))
    assert torch.all(ybuf[:, 90:] == 7.0)                                # nothing written past ncols


def test_non_finite_negative_and_tied_saliency(env):
    B, torch = env
    rng = np.random.default_rng(11)
    rows, k = 64, 256
    w = wl.f32_to_bf16_bits(rng.standard_normal((rows, k)).astype(np.float32))
    s = rng.integers(0, 4, (rows, k)).astype(np.float32)               # many ties, many zeros
    s[rng.random((rows, k)) < 0.05] = np.nan
    s[rng.random((rows, k)) < 0.02] = np.inf
    s[rng.random((rows, k)) < 0.02] = -np.inf
    s *= np.where(rng.random((rows, k)) < 0.5, -1, 1).astype(np.float32)
    for (n, m) in [(2, 4), (3, 8)]:
        mk, vals, idx, wd, wb = oracle_layer(w, s, n, m, 32, 32, 0.5)
        L = gpu_layer(B, torch, w, s, n, m, 32, 32, 0.5)
        assert_mask_and_encoding_equal(L, mk, vals, idx)
    # all-zero saliency: every score ties at 0 -> first blocks, first n of every group
    z = np.zeros((rows, k), dtype=np.float32)
    mk, vals, idx, wd, wb = oracle_layer(w, z, 2, 4, 32, 32, 0.25)
    L = gpu_layer(B, torch, w, z, 2, 4, 32, 32, 0.25)
    assert_mask_and_encoding_equal(L, mk, vals, idx)
    # denormal-only saliency still ranks correctly
    d = (rng.integers(1, 1000, (rows, k)) * 1.4e-45).astype(np.float32)
    mk, vals, idx, wd, wb = oracle_layer(w, d, 1, 4, 32, 32, 0.5)
    L = gpu_layer(B, torch, w, d, 1, 4, 32, 32, 0.5)
    assert_mask_and_encoding_equal(L, mk, vals, idx)


def test_no_kept_block_writes_zeros(env):
    B, torch = env
    w, s, x = rand_inputs(64, 27, 50, seed=2)
    L = gpu_layer(B, torch, w, s, 2, 4, 64, 64, 0.4)
    assert L.kkeep == 0
    y = torch.full((64, 50), 3.0, dtype=torch.bfloat16, device="cuda")
    L.spmm(bf16_dev(x, torch), y=y)
    assert torch.count_nonzero(y).item() == 0
    assert L.export()[1].size == 0


@pytest.mark.parametrize("n,m,bm,bk,keep", [(2, 4, 32, 64, 0.5), (1, 8, 64, 32, 0.25), (4, 8, 128, 64, 1.0)])
def test_identity_activation_is_bit_exact(env, image, n, m, bm, bk, keep):
    """X = I: every output is a single product by 1, exact in fp32 and in bf16, so Y must equal
    the decoded weight bit for bit; this pins every index and offset path."""
    B, torch = env
    rows, k = 192, 256
    w, s, _ = rand_inputs(rows, k, 8, seed=n * 10 + m)
    mk, vals, idx, wd, wb = oracle_layer(w, s, n, m, bm, bk, keep)
    L = gpu_layer(B, torch, w, s, n, m, bm, bk, keep)
    eye = torch.eye(k, dtype=torch.bfloat16, device="cuda")
    y = L.spmm(eye)
    got = y.view(torch.int16).cpu().numpy().view(np.uint16)
    assert np.array_equal(got & 0x7FFF, wb & 0x7FFF)                      # (sign of zero aside)
    assert np.array_equal(wl.bf16_bits_to_f32(got), wl.bf16_bits_to_f32(wb))
    assert np.array_equal(y_to_f64(y, torch), oracle.spmm_fp64(wd, wl.f32_to_bf16_bits(np.eye(k, dtype=np.float32))))


def test_config1_full(env, image):
    B, torch = env
    l = wl.config1()[0]
    w, s, x = wl.make_layer_inputs(l)
    mk, vals, idx, wd, wb = oracle_layer(w, s, l.n, l.m, l.block_rows, l.block_k, l.keep_ratio)
    L = gpu_layer(B, torch, w, s, l.n, l.m, l.block_rows, l.block_k, l.keep_ratio)
    assert_mask_and_encoding_equal(L, mk, vals, idx)
    y = L.spmm(bf16_dev(x, torch))
    check_tolerance(y_to_f64(y, torch), oracle.spmm_fp64(wd, x))


def test_config2_full(env, image):
    B, torch = env
    l = wl.config2()[0]
    w, s, x = wl.make_layer_inputs(l)
    mk, vals, idx, wd, wb = oracle_layer(w, s, l.n, l.m, l.block_rows, l.block_k, l.keep_ratio)
    assert mk.kkeep == 9
    L = gpu_layer(B, torch, w, s, l.n, l.m, l.block_rows, l.block_k, l.keep_ratio)
    assert_mask_and_encoding_equal(L, mk, vals, idx)
    y = L.spmm(bf16_dev(x, torch))
    sel = np.array([0, 63, 64, 100, 255], dtype=np.int32)
    ref_rows = oracle.spmm_fp64_rows(wd, x, sel)                          # the literal definition
    full = oracle.spmm_fp64_skipzero(wd, x)                               # shown equal on small shapes
    assert np.array_equal(full[sel], ref_rows)
    check_tolerance(y_to_f64(y, torch), full)


# Thin layers with enough columns for the stacked accumulator: one accumulator covers `stack` column tiles,
# one per group of 128 / stack lanes, and the walk is repeated per group against that group's columns.
# ncols is chosen so that there are at least as many stacked tiles as SMs (148) plus a ragged tail.
STACKED = [
    # rows, k, n, m, bm, bk, keep, ncols, stack
    (16, 32, 2, 8, 32, 32, 1.0, 148 * 4 * 256 + 1000, 4),
    (32, 64, 2, 4, 32, 32, 1.0, 148 * 4 * 256 + 520, 4),       # two blocks, walked once per lane group
    (64, 32, 2, 8, 32, 32, 1.0, 148 * 2 * 256 + 328, 2),       # one-block walk: 192-column tiles, two accumulators
    (64, 64, 2, 8, 32, 32, 1.0, 148 * 2 * 256 + 776, 2),       # two row tiles of 32 in a 64-row window
    (48, 128, 1, 4, 64, 64, 0.5, 148 * 2 * 256 + 264, 2),      # 48 of 64 rows, one kept block of two
    (40, 64, 3, 4, 64, 64, 1.0, 148 * 2 * 256 + 128, 2),       # dense-tile image
]


@pytest.mark.parametrize("rows,k,n,m,bm,bk,keep,ncols,stack", STACKED)
@pytest.mark.parametrize("y_dtype", [0, 1])
@pytest.mark.parametrize("epilogue", [False, True])
def test_stacked_thin_layer_matches_oracle(env, rows, k, n, m, bm, bk, keep, ncols, stack, y_dtype, epilogue):
    B, torch = env
    w, s, x = rand_inputs(rows, k, ncols, seed=rows * 7 + k + stack)
    mk, vals, idx, wd, wb = oracle_layer(w, s, n, m, bm, bk, keep)
    L = gpu_layer(B, torch, w, s, n, m, bm, bk, keep)
    assert_mask_and_encoding_equal(L, mk, vals, idx)
    ref = oracle.spmm_fp64(wd, x)
    if epilogue:
        bias = np.random.default_rng(rows).standard_normal(rows).astype(np.float32)
        L.set_epilogue(to_dev(bias, torch), relu=True)
        ref = oracle.bias_relu(ref, bias, True)
    y = L.spmm(bf16_dev(x, torch), y_dtype=y_dtype)
    torch.cuda.synchronize()
    assert L.device_status() == 0
    info = L.last_launch()
    assert info["stack"] == stack, info                       # the stacked path is the one that ran
    assert info["path"] == (B.PATH_SPARSE if n <= 2 else B.PATH_DENSE)
    check_tolerance(y_to_f64(y, torch), ref)
    L.close()


def test_identity_activation_wide_single_accumulator_tile(env):
    """The launch configuration of the large layers (256-column tiles, sparse image, one accumulator) on
    X = [I I I ...]: column c of Y must be column c mod k of the decoded weight, bit for bit."""
    B, torch = env
    rows, k, n, m, bm, bk, keep = 256, 1024, 2, 4, 128, 64, 0.6     # walks of 10 blocks: the long-walk variant
    ncols = 19 * k                                            # enough tiles that the column tile is not narrowed
    w, s, _ = rand_inputs(rows, k, 8, seed=99)
    mk, vals, idx, wd, wb = oracle_layer(w, s, n, m, bm, bk, keep)
    L = gpu_layer(B, torch, w, s, n, m, bm, bk, keep)
    eye = torch.eye(k, dtype=torch.bfloat16, device="cuda").repeat(1, ncols // k)
    y = L.spmm(eye)
    torch.cuda.synchronize()
    info = L.last_launch()
    assert info["path"] == B.PATH_SPARSE and info["tile_cols"] == 256 and info["accumulators"] == 1, info
    got = wl.bf16_bits_to_f32(y.view(torch.int16).cpu().numpy().view(np.uint16))
    want = np.tile(wl.bf16_bits_to_f32(wb), (1, ncols // k))
    assert np.array_equal(got, want)
    assert L.device_status() == 0


def test_bounded_wait_reports_timeout_and_the_handle_stays_usable(env):
    """Failure detection: a pipeline fill whose copies never arrive must end the kernel through its bounded
    waits (status CRISP_TIMEOUT), and the next product on the same handle and stream must be correct."""
    B, torch = env
    rows, k, ncols, n, m, bm, bk, keep = 128, 256, 512, 2, 4, 128, 64, 0.5
    w, s, x = rand_inputs(rows, k, ncols, seed=4242)
    mk, vals, idx, wd, wb = oracle_layer(w, s, n, m, bm, bk, keep)
    L = gpu_layer(B, torch, w, s, n, m, bm, bk, keep)
    d_x = bf16_dev(x, torch)
    L.set_tuning(wait_limit_cycles=2_000_000, skip_fill=0)    # about a millisecond; every CTA's first fill
    L.spmm(d_x)
    torch.cuda.synchronize()
    assert L.device_status() == B.TIMEOUT
    L.set_tuning()                                            # defaults again
    L.reset_status()
    y = L.spmm(d_x)
    torch.cuda.synchronize()
    assert L.device_status() == 0
    check_tolerance(y_to_f64(y, torch), oracle.spmm_fp64(wd, x))


STAGE_CASES = [
    (256, 1024, 1000, 2, 4, 32, 64, 0.5),             # union walks of odd length, ragged last column tile
    (160, 960, 3136, 2, 8, 32, 32, 0.5),              # 32-deep blocks: up to four per stage
    (512, 2304, 1536, 1, 4, 64, 64, 0.25),            # two row tiles per CTA tile
    (128, 2048, 4096 + 64, 4, 8, 128, 64, 0.3),       # dense tiles, several tiles per CTA
    (128, 1024, 640, 3, 4, 128, 64, 0.45),            # 3:4, dense tiles
    (32, 64, 148 * 4 * 256 + 520, 2, 4, 32, 32, 1.0),  # stacked thin layer
]


@pytest.mark.parametrize("rows,k,ncols,n,m,bm,bk,keep", STAGE_CASES)
def test_blocks_per_stage_do_not_change_the_result(env, rows, k, ncols, n, m, bm, bk, keep):
    """A pipeline stage of 1, 2 or 4 kept blocks issues the same MMAs in the same order: the products are
    bit-identical, walks that end inside a stage included, and equal to the oracle's within the tolerance."""
    B, torch = env
    w, s, x = rand_inputs(rows, k, ncols, seed=rows + k + ncols)
    mk, vals, idx, wd, wb = oracle_layer(w, s, n, m, bm, bk, keep)
    L = gpu_layer(B, torch, w, s, n, m, bm, bk, keep)
    d_x = bf16_dev(x, torch)
    ys, used = {}, {}
    for g in (1, 2, 4, 0):
        L.set_stage_blocks(g)
        y = L.spmm(d_x)
        torch.cuda.synchronize()
        assert L.device_status() == 0
        info = L.last_launch()
        if info["path"] == B.PATH_DIRECT:
            pytest.skip("direct kernel: no pipeline stages")
        assert 1 <= info["stage_blocks"] <= (g or 4)
        ys[g], used[g] = y.clone(), info["stage_blocks"]
    assert used[1] == 1
    for g in (2, 4, 0):
        assert torch.equal(ys[1], ys[g]), (g, used)
    check_tolerance(y_to_f64(ys[1], torch), oracle.spmm_fp64(wd, x))
    L.close()


def test_longest_row_of_blocks(env):
    """4096 k-blocks per row tile: the per-row-tile selection holds a whole row of scores in shared memory
    (more than the default 48 KB at this length)."""
    B, torch = env
    rows, k = 32, 4096 * 32
    rng = np.random.default_rng(8)
    s = rng.uniform(0.1, 2.0, (rows, k)).astype(np.float32)
    w = wl.f32_to_bf16_bits(rng.standard_normal((rows, k)).astype(np.float32))
    mk, vals, idx, wd, wb = oracle_layer(w, s, 1, 4, 32, 32, 0.3)
    L = gpu_layer(B, torch, w, s, 1, 4, 32, 32, 0.3)
    assert_mask_and_encoding_equal(L, mk, vals, idx)
