"""Convolution as implicit GEMM (crisp_spmm_conv: the activations of kept blocks are gathered from the
NHWC input on the fly, Sec. III-E step 1) against the oracle's convolution by definition, through the C ABI.
Same bar as the matrix product: max |Y - Yref| <= 1e-2 (1 + |Yref|), relative Frobenius error <= 5e-3."""
import numpy as np
import pytest

import oracle
from paper_2311_14272_b200 import workloads as wl

from helpers import bf16_dev, check_tolerance, gpu_layer, oracle_layer, y_to_f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    from paper_2311_14272_b200 import binding as B
    B.load()
    assert torch.cuda.is_available()
    return B, torch


def conv_inputs(s_out, kh, kw, c, b, h, w, seed, relu=True):
    rng = np.random.default_rng(seed)
    k = kh * kw * c
    wt = wl.f32_to_bf16_bits((rng.standard_normal((s_out, k)) * np.sqrt(2.0 / k)).astype(np.float32))
    sal = (np.abs(wl.bf16_bits_to_f32(wt)) * rng.uniform(0.5, 1.5, (s_out, k))).astype(np.float32)
    a = rng.standard_normal((b, h, w, c)).astype(np.float32)
    if relu:
        a = np.maximum(a, 0)
    return wt, sal, wl.f32_to_bf16_bits(a)


CASES = [
    # s_out, kh, kw, pad, c, b, h, w, n, m, bm, keep      (bk = 64 always: a k-block is 64 channels of one tap)
    (96, 3, 3, 1, 64, 3, 12, 16, 2, 4, 32, 0.5),          # several pixel tiles, ragged rows of W
    (64, 3, 3, 1, 128, 2, 10, 24, 2, 4, 64, 0.5),         # two k-blocks per tap, width 24 (ragged tile in x)
    (200, 3, 3, 1, 64, 5, 9, 8, 1, 4, 128, 0.34),         # odd height and batch: ragged in y and across images
    (128, 1, 1, 0, 192, 2, 8, 16, 2, 8, 64, 0.67),        # pointwise
    (64, 5, 3, 1, 64, 2, 12, 16, 3, 4, 64, 0.6),          # dense-tile image (3:4), output shorter than input
    (160, 3, 3, 0, 64, 1, 18, 34, 4, 8, 32, 0.75),        # no padding: 16 x 32 outputs from 18 x 34
    (96, 3, 3, 1, 64, 3, 14, 14, 2, 4, 64, 0.5),          # 14-pixel rows: Y is stored element by element
    (128, 3, 3, 1, 128, 2, 28, 28, 1, 4, 64, 0.25),       # 28-pixel rows, two k-blocks per tap
    (64, 3, 3, 1, 64, 2, 9, 11, 3, 4, 32, 0.8),           # odd sizes in both directions, dense-tile image
]


@pytest.mark.parametrize("s_out,kh,kw,pad,c,b,h,w,n,m,bm,keep", CASES)
@pytest.mark.parametrize("y_dtype", [0, 1])
def test_conv_matches_oracle(env, s_out, kh, kw, pad, c, b, h, w, n, m, bm, keep, y_dtype):
    B, torch = env
    wt, sal, act = conv_inputs(s_out, kh, kw, c, b, h, w, seed=s_out + 7 * h + w)
    mk, vals, idx, wd, _wb = oracle_layer(wt, sal, n, m, bm, 64, keep)
    ref = oracle.conv_fp64(wd, kh, kw, act, pad)
    L = gpu_layer(B, torch, wt, sal, n, m, bm, 64, keep)
    ho, wo = h + 2 * pad - kh + 1, w + 2 * pad - kw + 1
    y = torch.full((s_out, b * ho * wo + 8), 7.0, dtype=torch.float32 if y_dtype else torch.bfloat16, device="cuda")
    L.spmm_conv(bf16_dev(act, torch), kh, kw, pad, y=y[:, : b * ho * wo], y_dtype=y_dtype)
    torch.cuda.synchronize()
    assert L.device_status() == 0
    check_tolerance(y_to_f64(y[:, : b * ho * wo], torch), ref)
    assert float(y[:, b * ho * wo:].float().min()) == 7.0 and float(y[:, b * ho * wo:].float().max()) == 7.0
    L.close()


def test_conv_blocks_per_stage_do_not_change_the_result(env):
    """The gather with 1, 2 or 4 filter-tap blocks per pipeline stage: bit-identical outputs."""
    B, torch = env
    s_out, kh, kw, pad, c, b, h, w = 128, 3, 3, 1, 64, 2, 20, 24
    wt, sal, act = conv_inputs(s_out, kh, kw, c, b, h, w, seed=77)
    L = gpu_layer(B, torch, wt, sal, 2, 4, 64, 64, 0.6)
    d_act = bf16_dev(act, torch)
    ys = {}
    for g in (1, 2, 4, 0):
        L.set_stage_blocks(g)
        y = L.spmm_conv(d_act, kh, kw, pad)
        torch.cuda.synchronize()
        assert L.device_status() == 0
        assert 1 <= L.last_launch()["stage_blocks"] <= (g or 4)
        ys[g] = y.clone()
    for g in (2, 4, 0):
        assert torch.equal(ys[1], ys[g]), g
    L.close()


def test_one_hot_taps_are_exact(env):
    """A weight with a single 1 per row picks shifted copies of the input: exact in bf16, border zeros included."""
    B, torch = env
    c, b, h, w = 64, 2, 8, 16
    rng = np.random.default_rng(3)
    act = wl.f32_to_bf16_bits(rng.standard_normal((b, h, w, c)).astype(np.float32))
    k = 9 * c
    wt = np.zeros((32, k), dtype=np.float32)
    picks = [(int(rng.integers(0, 9)), int(rng.integers(0, c))) for _ in range(32)]
    for r, (tap, ch) in enumerate(picks):
        wt[r, tap * c + ch] = 1.0
    wt = wl.f32_to_bf16_bits(wt)
    sal = np.abs(wl.bf16_bits_to_f32(wt)).astype(np.float32) + 1e-3
    L = gpu_layer(B, torch, wt, sal, 1, 4, 32, 64, 1.0)
    y = L.spmm_conv(bf16_dev(act, torch), 3, 3, 1)
    torch.cuda.synchronize()
    got = y.contiguous().view(torch.int16).cpu().numpy().view(np.uint16).reshape(32, b, h, w)
    padded = np.zeros((b, h + 2, w + 2, c), dtype=np.uint16)
    padded[:, 1:-1, 1:-1, :] = act
    for r, (tap, ch) in enumerate(picks):
        i, j = divmod(tap, 3)
        want = padded[:, i:i + h, j:j + w, ch]
        g, v = got[r].copy(), want.copy()
        g[g == 0x8000] = 0                      # the sign of a zero is not part of the result
        v[v == 0x8000] = 0
        assert np.array_equal(g, v)
    L.close()


def test_unsupported_shapes_are_refused(env):
    B, torch = env
    wt, sal, act = conv_inputs(64, 3, 3, 64, 1, 8, 14, seed=1)
    L = gpu_layer(B, torch, wt, sal, 2, 4, 64, 64, 0.5)
    with pytest.raises(B.CrispError):          # the handle's k is 9 * 64, not 9 * 32
        L.spmm_conv(bf16_dev(act[..., :32].copy(), torch), 3, 3, 1)
    wt2, sal2, act2 = conv_inputs(64, 3, 3, 32, 1, 8, 16, seed=2)
    L2 = gpu_layer(B, torch, wt2, sal2, 2, 4, 64, 32, 0.5)
    with pytest.raises(B.CrispError):          # 32-wide k-blocks
        L2.spmm_conv(bf16_dev(act2, torch), 3, 3, 1)
    L.close(); L2.close()


def test_vgg_layer_matches_lowered_product_and_sampled_oracle(env):
    """VGG-16 conv2_1 shape (128 x 576, 16 x 112 x 112 x 64): whole output against crisp_spmm on the lowered
    matrix (itself checked against the oracle at full size elsewhere), and two image strips against the
    oracle's convolution."""
    B, torch = env
    s_out, c, b, h, w = 128, 64, 16, 112, 112
    wt, sal, act = conv_inputs(s_out, 3, 3, c, b, h, w, seed=42)
    L = gpu_layer(B, torch, wt, sal, 2, 4, 64, 64, 0.4)
    a_d = bf16_dev(act, torch)
    y = L.spmm_conv(a_d, 3, 3, 1)
    # lowered matrix by torch (layout plumbing only): [9 * c, b * h * w], reduction ordered (i, j, channel)
    ap = torch.nn.functional.pad(a_d.float(), (0, 0, 1, 1, 1, 1))
    x = torch.stack([ap[:, i:i + h, j:j + w, :] for i in range(3) for j in range(3)], dim=0)      # [9, b, h, w, c]
    x = x.permute(0, 4, 1, 2, 3).reshape(9 * c, b * h * w).to(torch.bfloat16).contiguous()
    y2 = L.spmm(x)
    torch.cuda.synchronize()
    assert L.device_status() == 0
    d = (y.float() - y2.float()).abs()
    assert float(d.max()) <= 1e-2 * (1 + float(y2.float().abs().max()))
    assert float(d.norm() / y2.float().norm()) <= 5e-3
    _mk, _vals, _idx, wd, _wb = oracle_layer(wt, sal, 2, 4, 64, 64, 0.4)
    yv = y_to_f64(y, torch).reshape(s_out, b, h, w)
    for img, r0 in ((0, 0), (15, 100)):
        lo, hi = max(r0 - 1, 0), min(r0 + 12 + 1, h)
        strip = np.ascontiguousarray(act[img:img + 1, lo:hi])
        ref = oracle.conv_fp64(wd, 3, 3, strip, 1).reshape(s_out, hi - lo, w)
        inner = slice(1 if lo > 0 else 0, (hi - lo) - (1 if hi < h else 0))     # rows whose window lies inside the strip
        rows = np.arange(lo, hi)[inner]
        check_tolerance(yv[:, img, rows, :], ref[:, inner, :])
    L.close()


NHWC_CASES = [
    # s_out, kh, kw, pad, c, b, h, w, n, m, bm, keep
    (96, 3, 3, 1, 64, 3, 12, 16, 2, 4, 32, 0.5),          # ragged rows of W (96 of 128), several pixel tiles
    (200, 3, 3, 1, 64, 5, 9, 8, 1, 4, 128, 0.34),         # ragged in y, across images and in the channel blocks
    (64, 5, 3, 1, 64, 2, 12, 16, 3, 4, 64, 0.6),          # dense-tile image
    (128, 3, 3, 1, 128, 2, 28, 28, 1, 4, 64, 0.25),       # 28-pixel rows: fine in NHWC (the pixel pitch is what counts)
    (100, 3, 3, 1, 64, 2, 10, 12, 2, 4, 32, 0.5),         # 100 channels: pixel pitch of 200 bytes, stored pixel by pixel
]


@pytest.mark.parametrize("s_out,kh,kw,pad,c,b,h,w,n,m,bm,keep", NHWC_CASES)
@pytest.mark.parametrize("y_dtype", [0, 1])
def test_conv_with_nhwc_output_matches_oracle(env, s_out, kh, kw, pad, c, b, h, w, n, m, bm, keep, y_dtype):
    """Output channel fastest ([batch, ho, wo, rows]): the layout the next convolution reads."""
    B, torch = env
    wt, sal, act = conv_inputs(s_out, kh, kw, c, b, h, w, seed=s_out + 3 * h + w)
    mk, vals, idx, wd, _wb = oracle_layer(wt, sal, n, m, bm, 64, keep)
    ref = oracle.conv_fp64(wd, kh, kw, act, pad)                       # [s_out, b * ho * wo]
    L = gpu_layer(B, torch, wt, sal, n, m, bm, 64, keep)
    ho, wo = h + 2 * pad - kh + 1, w + 2 * pad - kw + 1
    y = torch.full((b, ho, wo, s_out), 7.0, dtype=torch.float32 if y_dtype else torch.bfloat16, device="cuda")
    guard = torch.full((64,), 7.0, dtype=y.dtype, device="cuda")        # allocated right after y
    L.spmm_conv(bf16_dev(act, torch), kh, kw, pad, y=y, y_dtype=y_dtype, nhwc_out=True)
    torch.cuda.synchronize()
    assert L.device_status() == 0
    got = y_to_f64(y.reshape(b * ho * wo, s_out), torch).T
    check_tolerance(got, ref)
    assert float(guard.float().min()) == 7.0 and float(guard.float().max()) == 7.0
    L.close()


def test_two_convolutions_chain_through_nhwc(env):
    """VGG-16 stand-in conv2_1 -> conv2_2 (64 -> 128 -> 128 channels, 3 x 3, bias + ReLU fused, bf16 hand-over): the
    first layer's NHWC output is the second layer's activation as it stands.  Each layer is checked against the
    oracle's convolution of what it actually read."""
    B, torch = env
    b, h, w = 2, 56, 56
    wt1, sal1, act = conv_inputs(128, 3, 3, 64, b, h, w, seed=21)
    wt2, sal2, _ = conv_inputs(128, 3, 3, 128, 1, 4, 4, seed=22)
    rng = np.random.default_rng(23)
    bias1 = rng.standard_normal(128).astype(np.float32) * 0.1
    bias2 = rng.standard_normal(128).astype(np.float32) * 0.1
    _m1, _v1, _i1, wd1, _ = oracle_layer(wt1, sal1, 2, 4, 64, 64, 0.4)
    _m2, _v2, _i2, wd2, _ = oracle_layer(wt2, sal2, 2, 4, 64, 64, 0.3)
    L1 = gpu_layer(B, torch, wt1, sal1, 2, 4, 64, 64, 0.4)
    L2 = gpu_layer(B, torch, wt2, sal2, 2, 4, 64, 64, 0.3)
    from helpers import to_dev
    L1.set_epilogue(to_dev(bias1, torch), relu=True)
    L2.set_epilogue(to_dev(bias2, torch), relu=True)
    y1 = L1.spmm_conv(bf16_dev(act, torch), 3, 3, 1, nhwc_out=True)            # [b, h, w, 128] bf16
    y2 = L2.spmm_conv(y1, 3, 3, 1, nhwc_out=True)
    torch.cuda.synchronize()
    assert L1.device_status() == 0 and L2.device_status() == 0
    ref1 = oracle.bias_relu(oracle.conv_fp64(wd1, 3, 3, act, 1), bias1, True)
    check_tolerance(y_to_f64(y1.reshape(b * h * w, 128), torch).T, ref1)
    y1_bits = y1.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)  # what the second layer read
    ref2 = oracle.bias_relu(oracle.conv_fp64(wd2, 3, 3, y1_bits, 1), bias2, True)
    check_tolerance(y_to_f64(y2.reshape(b * h * w, 128), torch).T, ref2)
    L1.close(); L2.close()
