"""Layer epilogue fused into the product (crisp_set_epilogue: Y = act(W X + bias) on the fp32 accumulator)
against the oracle, through the C ABI, for the tensor-core kernels, the CUDA-core kernel and the convolution;
and two pointwise layers chained through their bf16 output.  Same tolerance as the plain product."""
import numpy as np
import pytest

import oracle
from paper_2311_14272_b200 import workloads as wl

from helpers import bf16_dev, check_tolerance, gpu_layer, oracle_layer, to_dev, y_to_f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    from paper_2311_14272_b200 import binding as B
    B.load()
    assert torch.cuda.is_available()
    return B, torch


def rand_inputs(rows, k, ncols, seed):
    rng = np.random.default_rng(seed)
    w = wl.f32_to_bf16_bits((rng.standard_normal((rows, k)) * 0.05).astype(np.float32))
    s = (np.abs(wl.bf16_bits_to_f32(w)) * rng.uniform(0.5, 1.5, (rows, k))).astype(np.float32)
    x = wl.f32_to_bf16_bits(np.maximum(rng.standard_normal((k, ncols)), 0).astype(np.float32))
    bias = (rng.standard_normal(rows) * 0.3).astype(np.float32)
    return w, s, x, bias


CASES = [
    # rows, k, ncols, n, m, bm, bk, keep
    (256, 1024, 512, 2, 4, 32, 64, 0.5),
    (200, 576, 333, 1, 4, 64, 64, 0.25),      # ragged rows and columns
    (96, 144, 1000, 2, 8, 32, 32, 0.5),       # short walks: 12 or 16 epilogue warps
    (300, 640, 520, 3, 4, 128, 64, 0.75),     # dense-tile image
    (32, 32, 2048, 2, 8, 32, 32, 1.0),        # thin layers (too few columns for the stacked accumulator, which
    (64, 384, 1300, 2, 8, 32, 32, 0.5),       # test_gpu_parity.py covers with and without the epilogue)
]


@pytest.mark.parametrize("rows,k,ncols,n,m,bm,bk,keep", CASES)
@pytest.mark.parametrize("image", ["auto", "none"])
@pytest.mark.parametrize("y_dtype,use_bias,relu", [(0, True, True), (1, True, False), (0, False, True)])
def test_fused_epilogue_matches_oracle(env, monkeypatch, image, rows, k, ncols, n, m, bm, bk, keep, y_dtype, use_bias, relu):
    B, torch = env
    if image == "auto":
        monkeypatch.delenv("CRISP_EXEC_IMAGE", raising=False)
    else:
        monkeypatch.setenv("CRISP_EXEC_IMAGE", image)
    w, s, x, bias = rand_inputs(rows, k, ncols, seed=rows + k)
    _mk, _vals, _idx, wd, _wb = oracle_layer(w, s, n, m, bm, bk, keep)
    ref = oracle.bias_relu(oracle.spmm_fp64(wd, x), bias if use_bias else None, relu)
    L = gpu_layer(B, torch, w, s, n, m, bm, bk, keep)
    L.set_epilogue(to_dev(bias, torch) if use_bias else None, relu)
    y = L.spmm(bf16_dev(x, torch), y_dtype=y_dtype)
    torch.cuda.synchronize()
    assert L.device_status() == 0
    check_tolerance(y_to_f64(y, torch), ref)
    if relu:
        assert float(y.float().min()) >= 0.0
    # and back to the plain product
    L.set_epilogue(None, False)
    y = L.spmm(bf16_dev(x, torch), y_dtype=y_dtype)
    torch.cuda.synchronize()
    check_tolerance(y_to_f64(y, torch), oracle.spmm_fp64(wd, x))
    L.close()


def test_layer_without_kept_blocks_gives_the_bias(env):
    B, torch = env
    w, s, x, bias = rand_inputs(64, 27, 300, seed=9)
    L = gpu_layer(B, torch, w, s, 2, 4, 64, 64, 0.3)       # one padded block, keep 0.3 -> none kept
    assert L.kkeep == 0
    L.set_epilogue(to_dev(bias, torch), True)
    y = L.spmm(bf16_dev(x, torch), y_dtype=1)
    torch.cuda.synchronize()
    want = np.repeat(np.maximum(bias, 0)[:, None], 300, axis=1)
    assert np.array_equal(y.cpu().numpy(), want)
    L.close()


def test_convolution_with_epilogue(env):
    B, torch = env
    rng = np.random.default_rng(21)
    s_out, c, b, h, wd_ = 96, 64, 2, 12, 16
    k = 9 * c
    w = wl.f32_to_bf16_bits((rng.standard_normal((s_out, k)) * np.sqrt(2.0 / k)).astype(np.float32))
    s = (np.abs(wl.bf16_bits_to_f32(w)) * rng.uniform(0.5, 1.5, (s_out, k))).astype(np.float32)
    act = wl.f32_to_bf16_bits(np.maximum(rng.standard_normal((b, h, wd_, c)), 0).astype(np.float32))
    bias = (rng.standard_normal(s_out) * 0.5).astype(np.float32)
    _mk, _vals, _idx, wdense, _wb = oracle_layer(w, s, 2, 4, 32, 64, 0.5)
    ref = oracle.bias_relu(oracle.conv_fp64(wdense, 3, 3, act, 1), bias, True)
    L = gpu_layer(B, torch, w, s, 2, 4, 32, 64, 0.5)
    L.set_epilogue(to_dev(bias, torch), True)
    y = L.spmm_conv(bf16_dev(act, torch), 3, 3, 1)
    torch.cuda.synchronize()
    assert L.device_status() == 0
    check_tolerance(y_to_f64(y, torch), ref)
    L.close()


def test_two_pointwise_layers_chain_through_bf16(env):
    """MobileNetV2-style expand (ReLU) -> project: the first layer's bf16 Y is the second layer's X as it stands."""
    B, torch = env
    ncols = 1536
    w1, s1, x, b1 = rand_inputs(192, 32, ncols, seed=101)
    w2, s2, _x2, b2 = rand_inputs(32, 192, ncols, seed=102)
    L1 = gpu_layer(B, torch, w1, s1, 2, 8, 32, 32, 0.5)
    L2 = gpu_layer(B, torch, w2, s2, 2, 8, 32, 32, 0.5)
    L1.set_epilogue(to_dev(b1, torch), True)
    L2.set_epilogue(to_dev(b2, torch), False)
    y1 = L1.spmm(bf16_dev(x, torch))
    y2 = L2.spmm(y1, y_dtype=1)
    torch.cuda.synchronize()
    _m, _v, _i, wd1, _ = oracle_layer(w1, s1, 2, 8, 32, 32, 0.5)
    _m, _v, _i, wd2, _ = oracle_layer(w2, s2, 2, 8, 32, 32, 0.5)
    check_tolerance(y_to_f64(y1, torch), oracle.bias_relu(oracle.spmm_fp64(wd1, x), b1, True))
    y1_bits = y1.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)      # what layer 2 actually read
    check_tolerance(y_to_f64(y2, torch), oracle.bias_relu(oracle.spmm_fp64(wd2, y1_bits), b2, False))
    L1.close(); L2.close()
