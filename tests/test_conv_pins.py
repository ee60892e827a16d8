"""Pins for the oracle's convolution (the layer product of Sec. III with W viewed as an S x (K*K*R)
matrix): against an independently lowered im2col + matrix product, and on kernels whose result is
known without computing anything."""
import numpy as np
import pytest

import oracle
from paper_2311_14272_b200 import workloads as wl


def bf16(a):
    return wl.f32_to_bf16_bits(np.asarray(a, dtype=np.float32))


def im2col(act, kh, kw, pad):
    """[B,H,W,R] -> [kh*kw*R, B*Ho*Wo], reduction ordered (i, j, r), by numpy slicing of a padded copy."""
    b, h, w, r = act.shape
    ho, wo = h + 2 * pad - kh + 1, w + 2 * pad - kw + 1
    p = np.zeros((b, h + 2 * pad, w + 2 * pad, r), dtype=act.dtype)
    p[:, pad:pad + h, pad:pad + w, :] = act
    cols = np.empty((kh, kw, r, b, ho, wo), dtype=act.dtype)
    for i in range(kh):
        for j in range(kw):
            cols[i, j] = np.transpose(p[:, i:i + ho, j:j + wo, :], (3, 0, 1, 2))
    return cols.reshape(kh * kw * r, b * ho * wo)


@pytest.mark.parametrize("b,h,w,r,s,kh,kw,pad", [(2, 5, 7, 3, 4, 3, 3, 1), (1, 6, 4, 8, 5, 3, 3, 0),
                                                 (3, 4, 4, 2, 3, 1, 1, 0), (2, 5, 5, 4, 2, 5, 3, 2)])
def test_equals_im2col_product(b, h, w, r, s, kh, kw, pad):
    rng = np.random.default_rng(b * 100 + h)
    act = bf16(rng.standard_normal((b, h, w, r)))
    wd = rng.standard_normal((s, kh * kw * r))
    x = wl.bf16_bits_to_f32(im2col(act, kh, kw, pad)).astype(np.float64)
    got = oracle.conv_fp64(wd, kh, kw, act, pad)
    np.testing.assert_allclose(got, wd @ x, rtol=1e-12, atol=1e-12)
    if kh == kw == 1:
        # a 1x1 convolution is the plain product with the activation matrix
        np.testing.assert_allclose(got, oracle.spmm_fp64(wd, act.reshape(-1, r).T.copy()), rtol=0, atol=1e-12)


def test_one_hot_taps_shift_the_image():
    rng = np.random.default_rng(5)
    b, h, w, r = 2, 6, 5, 3
    act = bf16(rng.standard_normal((b, h, w, r)))
    a = wl.bf16_bits_to_f32(act).astype(np.float64)
    for (i, j, ch) in [(1, 1, 0), (0, 0, 2), (2, 1, 1), (1, 2, 0)]:
        wd = np.zeros((1, 9 * r))
        wd[0, (i * 3 + j) * r + ch] = 1.0
        got = oracle.conv_fp64(wd, 3, 3, act, 1).reshape(b, h, w)
        want = np.zeros((b, h, w))
        for y in range(h):
            for x in range(w):
                iy, ix = y + i - 1, x + j - 1
                if 0 <= iy < h and 0 <= ix < w:
                    want[:, y, x] = a[:, iy, ix, ch]
        assert np.array_equal(got, want)       # picks: exact, including the zero border


def test_all_ones_kernel_counts_the_window():
    act = bf16(np.ones((1, 4, 4, 2)))
    got = oracle.conv_fp64(np.ones((1, 18)), 3, 3, act, 1).reshape(4, 4)
    inside = np.array([[4, 6, 6, 4], [6, 9, 9, 6], [6, 9, 9, 6], [4, 6, 6, 4]]) * 2.0
    assert np.array_equal(got, inside)


def test_layer_epilogue_hand_values():
    # bias per row, then the rectifier: written out by hand
    y = np.array([[1.5, -2.0, 0.0], [-0.25, 4.0, -4.0]])
    b = np.array([0.5, -1.0], dtype=np.float32)
    assert np.array_equal(oracle.bias_relu(y), y)
    assert np.array_equal(oracle.bias_relu(y, b), [[2.0, -1.5, 0.5], [-1.25, 3.0, -5.0]])
    assert np.array_equal(oracle.bias_relu(y, b, relu=True), [[2.0, 0.0, 0.5], [0.0, 3.0, 0.0]])
    assert np.array_equal(oracle.bias_relu(y, None, relu=True), [[1.5, 0.0, 0.0], [0.0, 4.0, 0.0]])
    # against numpy on a random case
    rng = np.random.default_rng(0)
    y = rng.standard_normal((7, 13)); b = rng.standard_normal(7).astype(np.float32)
    np.testing.assert_array_equal(oracle.bias_relu(y, b, relu=True), np.maximum(y + b.astype(np.float64)[:, None], 0))


def test_saliency_score_hand_values_and_numpy():
    # Eq. 1 on values small enough to do by hand: mean gradient times weight, magnitude
    w = bf16(np.array([[2.0, -0.5, 4.0]]))
    g = np.array([[[1.0, 2.0, -1.0]], [[3.0, -2.0, -3.0]]])          # means 2, 0, -2
    assert np.array_equal(oracle.saliency(g, w), [[4.0, 0.0, 8.0]])
    rng = np.random.default_rng(4)
    g = rng.standard_normal((5, 6, 9))
    wb = bf16(rng.standard_normal((6, 9)))
    want = np.abs(g.mean(axis=0) * wl.bf16_bits_to_f32(wb).astype(np.float64))
    np.testing.assert_allclose(oracle.saliency(g, wb), want, rtol=1e-14, atol=0)
    # the three cases the paper lists keep their order: small*small < large*small ~ small*large < large*large
    w2 = bf16(np.array([[0.01, 1.0, 0.01, 1.0]]))
    g2 = np.array([[[0.01, 0.01, 1.0, 1.0]]])
    s = oracle.saliency(g2, w2)[0]
    assert s[0] < s[1] and s[0] < s[2] and s[1] < s[3] and s[2] < s[3]


def test_saliency_in_fp32_order_is_the_fp32_evaluation_and_close_to_fp64():
    """oracle.saliency_f32: sum of the samples in order in fp32, times fp32(1/H), times W, each step rounded to fp32
    (written out here with numpy's float32 scalars' arithmetic), and within a few ulp of the fp64 evaluation."""
    rng = np.random.default_rng(4)
    for h in (1, 3, 7):
        g = (rng.standard_normal((h, 9, 20)) * 1e-2).astype(np.float32)
        w = wl.f32_to_bf16_bits(rng.standard_normal((9, 20)).astype(np.float32))
        acc = g[0].copy()
        for i in range(1, h):
            acc = (acc + g[i]).astype(np.float32)
        inv = np.float32(1.0) / np.float32(h)
        want = np.abs(((acc * inv).astype(np.float32) * wl.bf16_bits_to_f32(w)).astype(np.float32))
        got = oracle.saliency_f32(g, w)
        assert got.dtype == np.float32 and np.array_equal(got, want)
        ref = oracle.saliency(g, w)
        assert np.all(np.abs(got - ref) <= 4 * 2.0 ** -24 * (h + 2) * np.abs(g).mean(axis=0) * np.abs(wl.bf16_bits_to_f32(w)) + 1e-45)
