"""Seeded synthetic inputs shaped like the paper's evaluated layers.

This module only *draws numbers and lists shapes*.  It holds none of the method's
arithmetic (no masking, no encoding, no products), so both the CPU oracle's tests
and the CUDA library's tests may feed from it without sharing any computation.

The paper (Section IV-A) evaluates ResNet-50, VGG-16 and MobileNetV2 pruned on
ImageNet / CIFAR-100.  Neither the datasets nor trained weights are used here:
only the layer *shapes* of those public architectures, with weights drawn from the
stated normal distributions and activations from N(0,1) (optionally rectified).

Conventions: a layer is the GEMM  Y[rows, ncols] = W[rows, k] @ X[k, ncols]  with
W holding output channels as rows and the reduction dimension k contiguous.
bf16 tensors are carried as numpy uint16 bit patterns.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import List

import numpy as np

BASE_SEED = 231114272


@dataclass(frozen=True)
class Layer:
    """One GEMM-shaped layer and its hybrid sparsity pattern."""
    config: int          # workload family 1..5
    index: int           # layer index inside the family (seed offset)
    name: str
    rows: int            # output channels (GEMM M)
    k: int               # reduction length (kernel_h * kernel_w * in_channels)
    ncols: int           # batch * output pixels (GEMM N)
    n: int               # N of N:M
    m: int               # M of N:M
    block_rows: int      # coarse block height (rows of W)
    block_k: int         # coarse block width (along k)
    keep_ratio: float    # fraction of k-blocks kept per row tile
    w_std: float         # standard deviation of the normal weights
    relu_x: bool         # activations are max(0, N(0,1)) instead of N(0,1)

    @property
    def seed(self) -> int:
        return BASE_SEED + 1000 * self.config + self.index


# --------------------------------------------------------------------------- bf16

def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16, returned as uint16 bit patterns."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    r = (u + 0x7FFF + lsb) >> 16
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << 16).view(np.float32)


# ---------------------------------------------------------------------- generators

def _normal_f32(rng: np.random.Generator, shape, chunk_rows: int = 256) -> np.ndarray:
    out = np.empty(shape, dtype=np.float32)
    flat = out.reshape(shape[0], -1)
    for r0 in range(0, shape[0], chunk_rows):
        r1 = min(shape[0], r0 + chunk_rows)
        flat[r0:r1] = rng.standard_normal((r1 - r0, flat.shape[1]), dtype=np.float32)
    return out


def make_weight(layer: Layer) -> np.ndarray:
    """W[rows, k] as bf16 bit patterns, ~N(0, w_std)."""
    rng = np.random.default_rng(layer.seed)
    w = _normal_f32(rng, (layer.rows, layer.k)) * np.float32(layer.w_std)
    return f32_to_bf16_bits(w)


def make_saliency(layer: Layer, w_bits: np.ndarray) -> np.ndarray:
    """S[rows, k] fp32 = |W| * U(0.5, 1.5): a stand-in for the class-aware score."""
    rng = np.random.default_rng(layer.seed + 13)
    u = rng.random((layer.rows, layer.k), dtype=np.float32) + np.float32(0.5)
    return (np.abs(bf16_bits_to_f32(w_bits)) * u).astype(np.float32)


def make_activation(layer: Layer, ncols: int | None = None) -> np.ndarray:
    """X[k, ncols] as bf16 bit patterns (N(0,1), rectified when layer.relu_x)."""
    nc = layer.ncols if ncols is None else ncols
    rng = np.random.default_rng(layer.seed + 7)
    x = _normal_f32(rng, (layer.k, nc))
    if layer.relu_x:
        np.maximum(x, np.float32(0), out=x)
    return f32_to_bf16_bits(x)


def make_layer_inputs(layer: Layer, ncols: int | None = None):
    w = make_weight(layer)
    s = make_saliency(layer, w)
    x = make_activation(layer, ncols)
    return w, s, x


# ------------------------------------------------------------------------- configs

def config1() -> List[Layer]:
    return [Layer(1, 0, "linear_256x1024", 256, 1024, 512, 2, 4, 32, 64, 0.5, 0.02, False)]


def config2() -> List[Layer]:
    k = 2304
    return [Layer(2, 0, "resnet50_layer3_conv3x3", 256, k, 32 * 14 * 14, 1, 4, 64, 64, 0.25,
                  float(np.sqrt(2.0 / k)), True)]


_VGG16 = [  # (out_channels, in_channels, output side) of the 13 3x3 convolutions
    (64, 3, 224), (64, 64, 224), (128, 64, 112), (128, 128, 112),
    (256, 128, 56), (256, 256, 56), (256, 256, 56),
    (512, 256, 28), (512, 512, 28), (512, 512, 28),
    (512, 512, 14), (512, 512, 14), (512, 512, 14),
]


def config3(batch: int = 16) -> List[Layer]:
    keep_rng = np.random.default_rng(BASE_SEED + 3000 + 29)
    keeps = keep_rng.uniform(0.1, 0.5, size=len(_VGG16))
    out = []
    for i, (co, ci, side) in enumerate(_VGG16):
        k = 9 * ci
        out.append(Layer(3, i, f"vgg16_conv{i}", co, k, batch * side * side, 2, 4, 64, 64,
                         float(keeps[i]), float(np.sqrt(2.0 / k)), True))
    return out


_MBV2 = [  # (expansion t, out channels c, repeats n, stride s) of the inverted-residual stages
    (1, 16, 1, 1), (6, 24, 2, 2), (6, 32, 3, 2), (6, 64, 4, 2),
    (6, 96, 3, 1), (6, 160, 3, 2), (6, 320, 1, 1),
]


def config4(batch: int = 64) -> List[Layer]:
    """All 1x1 (pointwise) convolutions: per block one expand and one project, plus
    the last 320->1280 convolution.  The first block (t = 1) is counted with a
    32->32 expand so that every block contributes two layers."""
    out: List[Layer] = []
    cin, side = 32, 112

    def add(name, co, ci, sd):
        out.append(Layer(4, len(out), name, co, ci, batch * sd * sd, 2, 8, 32, 32, 0.5,
                         float(np.sqrt(2.0 / ci)), True))

    b = 0
    for t, c, n, s in _MBV2:
        for r in range(n):
            stride = s if r == 0 else 1
            hidden = cin * t
            add(f"mbv2_b{b}_expand", hidden, cin, side)
            side = side // stride
            add(f"mbv2_b{b}_project", c, hidden, side)
            cin = c
            b += 1
    add("mbv2_last", 1280, cin, side)
    return out


SWEEP_NM = [(1, 4), (2, 4), (1, 8), (2, 8), (4, 8)]
SWEEP_KEEP = [1.0, 0.5, 0.25, 0.1]


def config5(rows: int = 4096, k: int = 4096, ncols: int = 8192) -> List[Layer]:
    out = []
    for (n, m) in SWEEP_NM:
        for keep in SWEEP_KEEP:
            # every cell prunes the same W / S / X: one seed for the whole sweep
            out.append(Layer(5, 0, f"sweep_{n}:{m}_keep{keep}", rows, k, ncols, n, m, 128, 64,
                             keep, 0.02, False))
    return out


def extra_sweep_cells(rows: int = 4096, k: int = 4096, ncols: int = 8192) -> List[Layer]:
    """3:4 on the sweep shape: the third pattern the paper's accelerator supports (Sec. III-D), which the
    five N:M ratios of the sweep do not contain.  Same W / S / X as the sweep."""
    return [Layer(5, 0, f"sweep_3:4_keep{keep}", rows, k, ncols, 3, 4, 128, 64, keep, 0.02, False)
            for keep in SWEEP_KEEP]


def sweep_cell(n: int, m: int, keep: float, **kw) -> Layer:
    for l in config5(**kw) + extra_sweep_cells(**kw):
        if (l.n, l.m) == (n, m) and abs(l.keep_ratio - keep) < 1e-12:
            return l
    raise KeyError((n, m, keep))


def all_configs():
    return {1: config1(), 2: config2(), 3: config3(), 4: config4(), 5: config5()}


def shrink(layer: Layer, rows=None, k=None, ncols=None) -> Layer:
    """Same pattern and distributions on a smaller shape (for parity cases the
    CPU oracle finishes in seconds)."""
    return replace(layer, rows=rows or layer.rows, k=k or layer.k, ncols=ncols or layer.ncols)
