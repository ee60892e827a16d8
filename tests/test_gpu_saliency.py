"""Class-aware saliency score (Sec. III-C, Eq. 1: T_w = |mean gradient (.) W|) on the GPU against the oracle,
through the C ABI.  Tolerance: the kernels add H fp32 values in call order and multiply twice, so
|S - S_ref| <= 4 * 2^-24 * (H + 2) * mean_i|g_i| * |w| (each of the H + 2 roundings moves the result by at most
2^-24 of the running magnitude; the factor 4 is slack).  The mask built from the GPU's scores must equal the
oracle's mask for the same scores bit for bit."""
import numpy as np
import pytest

import oracle
from paper_2311_14272_b200 import workloads as wl

from helpers import bf16_dev, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    from paper_2311_14272_b200 import binding as B
    B.load()
    assert torch.cuda.is_available()
    return B, torch


def gpu_saliency(B, torch, grads, grad_dtype, w_bits, pad=0):
    h, rows, k = grads.shape
    acc = torch.full((rows, k + pad), float("nan"), dtype=torch.float32, device="cuda")
    s = torch.full((rows, k + pad), -1.0, dtype=torch.float32, device="cuda")
    w_d = torch.zeros((rows, k + pad), dtype=torch.bfloat16, device="cuda")
    w_d[:, :k] = bf16_dev(w_bits, torch)
    for i in range(h):
        if grad_dtype == 0:
            g_d = torch.zeros((rows, k + pad), dtype=torch.bfloat16, device="cuda")
            g_d[:, :k] = bf16_dev(wl.f32_to_bf16_bits(grads[i].astype(np.float32)), torch)
        else:
            g_d = torch.zeros((rows, k + pad), dtype=torch.float32, device="cuda")
            g_d[:, :k] = to_dev(grads[i].astype(np.float32), torch)
        B.crisp_saliency_accumulate(g_d, grad_dtype, k + pad, rows, k, acc, k + pad, i == 0)
    B.crisp_saliency_finish(acc, k + pad, w_d, k + pad, rows, k, h, s, k + pad)
    torch.cuda.synchronize()
    assert pad == 0 or float(s[:, k:].min()) == -1.0          # nothing written beyond k
    return s[:, :k].contiguous()


@pytest.mark.parametrize("rows,k,h", [(64, 256, 1), (200, 576, 5), (33, 70, 8), (7, 27, 3), (512, 1024, 16)])
@pytest.mark.parametrize("grad_dtype", [0, 1])
@pytest.mark.parametrize("pad", [0, 3])
def test_saliency_matches_oracle(env, rows, k, h, grad_dtype, pad):
    B, torch = env
    rng = np.random.default_rng(rows * 7 + k + h)
    w_bits = wl.f32_to_bf16_bits((rng.standard_normal((rows, k)) * 0.05).astype(np.float32))
    grads = (rng.standard_normal((h, rows, k)) * 1e-2).astype(np.float32)
    if grad_dtype == 0:                                         # what the kernel reads: bf16-rounded gradients
        grads = wl.bf16_bits_to_f32(wl.f32_to_bf16_bits(grads))
    ref = oracle.saliency(grads, w_bits)
    got = gpu_saliency(B, torch, grads, grad_dtype, w_bits, pad).cpu().numpy().astype(np.float64)
    bound = 4 * 2.0 ** -24 * (h + 2) * np.abs(grads).astype(np.float64).mean(axis=0) * \
        np.abs(wl.bf16_bits_to_f32(w_bits).astype(np.float64)) + 1e-45
    assert np.all(np.abs(got - ref) <= bound), float((np.abs(got - ref) / bound).max())
    assert np.all(got >= 0)


def test_vector_and_scalar_paths_agree_bitwise(env):
    B, torch = env
    rng = np.random.default_rng(8)
    rows, k, h = 96, 640, 6
    w_bits = wl.f32_to_bf16_bits(rng.standard_normal((rows, k)).astype(np.float32))
    grads = rng.standard_normal((h, rows, k)).astype(np.float32)
    a = gpu_saliency(B, torch, grads, 1, w_bits, pad=0)        # 16-byte accesses
    b = gpu_saliency(B, torch, grads, 1, w_bits, pad=1)        # odd pitch: element accesses
    assert torch.equal(a, b)


def test_scores_feed_the_mask_projection(env):
    B, torch = env
    rng = np.random.default_rng(12)
    rows, k, h = 128, 512, 4
    w_bits = wl.f32_to_bf16_bits((rng.standard_normal((rows, k)) * 0.05).astype(np.float32))
    grads = (rng.standard_normal((h, rows, k)) * 1e-2).astype(np.float32)
    s = gpu_saliency(B, torch, grads, 1, w_bits)
    L = B.HybridLayer(rows, k, 2, 4, 32, 64, 0.5)
    L.build_mask(s)
    blk_col, nm_bits = L.export_mask()
    ref = oracle.build_mask(s.cpu().numpy(), 2, 4, 32, 64, keep_ratio=0.5)
    assert np.array_equal(blk_col, ref.blk_col) and np.array_equal(nm_bits, ref.nm_bits)
    L.close()


def test_argument_checks(env):
    B, torch = env
    g = torch.zeros((4, 8), dtype=torch.float32, device="cuda")
    with pytest.raises(B.CrispError):
        B.crisp_saliency_accumulate(g, 2, 8, 4, 8, g, 8, True)
    with pytest.raises(B.CrispError):
        B.crisp_saliency_accumulate(g, 1, 4, 4, 8, g, 8, True)
    with pytest.raises(B.CrispError):
        B.crisp_saliency_finish(g, 8, g, 8, 4, 8, 0, g, 8)
