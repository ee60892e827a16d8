"""Global rank selection (Algorithm 1: per-row sort of the block scores, rank-column sums c_o, global
order across layers, selection by the sparsity target; Sec. III-C) on the GPU against the CPU oracle,
through the C ABI.  All of it is integer work: kept-block counts, scores and masks must be identical."""
import numpy as np
import pytest

import oracle
from paper_2311_14272_b200 import workloads as wl

from helpers import to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    from paper_2311_14272_b200 import binding as B
    B.load()
    assert torch.cuda.is_available()
    return B, torch


def gpu_rank(B, torch, layers, frac):
    arr = B.make_rank_layers(layers)
    ws = torch.empty(B.crisp_global_rank_sizes(arr), dtype=torch.uint8, device="cuda")
    out = torch.full((len(layers),), -7, dtype=torch.int32, device="cuda")
    B.crisp_global_rank(arr, frac, ws, out)
    torch.cuda.synchronize()
    return out.cpu().numpy()


def float_bits(v):
    return int(np.array([v], dtype=np.float32).view(np.uint32)[0])


def synthetic(B, torch, scores, exps, elems, min_keep):
    """Device copies of hand-made score grids; the scale word carries 2^e as float bits."""
    keep_alive, layers = [], []
    for sc, e, be, mk in zip(scores, exps, elems, min_keep):
        d_sc = to_dev(np.ascontiguousarray(sc).view(np.int64), torch)
        d_mk = to_dev(np.array([float_bits(np.ldexp(1.0, e))], dtype=np.uint32).view(np.int32), torch)
        keep_alive += [d_sc, d_mk]
        layers.append((d_sc, d_mk, sc.shape[0], sc.shape[1], be, mk))
    return layers, keep_alive


@pytest.mark.parametrize("seed", range(12))
def test_synthetic_scores_match_oracle(env, seed):
    B, torch = env
    rng = np.random.default_rng(500 + seed)
    nl = int(rng.integers(1, 9))
    scores, exps, elems, mk = [], [], [], []
    for _ in range(nl):
        nrt = int(rng.integers(1, 40))
        nblk = int(rng.choice([1, 2, 3, 5, 17, 64, 100, 257]))
        hi = int(rng.choice([2, 7, 1 << 30, 1 << 55]))        # narrow ranges force ties within and across layers
        scores.append(rng.integers(0, hi, size=(nrt, nblk), dtype=np.uint64))
        exps.append(int(rng.integers(-20, 21)))
        elems.append(int(rng.choice([1024, 2048, 4096, 8192])))
        mk.append(int(rng.integers(0, min(nblk, 3) + 1)))
    layers, _keep = synthetic(B, torch, scores, exps, elems, mk)
    for frac in (0.0, 0.05, 0.3, 0.5, 0.75, 0.999, 1.0):
        want = oracle.global_rank(scores, exps, elems, frac, min_keep=mk)
        got = gpu_rank(B, torch, layers, frac)
        assert np.array_equal(got, want), (frac, got, want)


def test_rank_sums_beyond_64_bits_and_wide_scale_gaps(env):
    B, torch = env
    big = np.full((600, 3), (1 << 55) - 1, dtype=np.uint64)
    big[:, 1] -= 1
    big[:, 2] -= 5
    small = np.array([[3, 1, 2]], dtype=np.uint64)
    for exps in ([0, 70], [0, -3], [100, -100], [-100, 100], [0, 64]):
        layers, _keep = synthetic(B, torch, [big, small], exps, [64, 64], [0, 0])
        for frac in (0.0, 1 / 1803, 0.2, 0.34, 0.67, 0.9, 1.0):
            want = oracle.global_rank([big, small], exps, [64, 64], frac)
            assert np.array_equal(gpu_rank(B, torch, layers, frac), want), (exps, frac)


def test_degenerate_inputs(env):
    B, torch = env
    zeros = np.zeros((4, 6), dtype=np.uint64)
    one = np.array([[9]], dtype=np.uint64)
    rows = np.arange(12, dtype=np.uint64).reshape(2, 6)
    cases = [
        ([zeros], [0], [16], [0]),                   # an all-zero layer: ties everywhere
        ([one], [3], [4096], [0]),                   # a single block
        ([rows, zeros, one], [0, 0, 0], [32, 32, 32], [6, 0, 1]),   # no candidates in layers 0 and 2
        ([rows, rows], [5, 5], [32, 64], [0, 0]),    # equal values, different weights
        ([np.full((3, 4096), 5, dtype=np.uint64)], [0], [1024], [1]),   # the widest supported row
    ]
    for scores, exps, elems, mk in cases:
        layers, _keep = synthetic(B, torch, scores, exps, elems, mk)
        for frac in (0.0, 0.25, 0.5, 1.0):
            want = oracle.global_rank(scores, exps, elems, frac, min_keep=mk)
            assert np.array_equal(gpu_rank(B, torch, layers, frac), want), (elems, frac)


def test_argument_checks(env):
    B, torch = env
    sc = np.ones((2, 4), dtype=np.uint64)
    layers, _keep = synthetic(B, torch, [sc], [0], [16], [0])
    arr = B.make_rank_layers(layers)
    ws = torch.empty(B.crisp_global_rank_sizes(arr), dtype=torch.uint8, device="cuda")
    out = torch.zeros(1, dtype=torch.int32, device="cuda")
    for bad in (-0.1, 1.5, float("nan")):
        with pytest.raises(B.CrispError):
            B.crisp_global_rank(arr, bad, ws, out)
    with pytest.raises(B.CrispError):
        B.crisp_global_rank_sizes(B.make_rank_layers([(layers[0][0], layers[0][1], 2, 4097, 16, 0)]))
    with pytest.raises(B.CrispError):
        B.crisp_global_rank_sizes(B.make_rank_layers([(layers[0][0], layers[0][1], 2, 4, 16, 5)]))
    with pytest.raises(B.CrispError):
        B.crisp_global_rank(B.make_rank_layers([(0, layers[0][1], 2, 4, 16, 0)]), 0.5, ws, out)


def network(which):
    """(name, rows, k, n, m, bm, bk) of every layer, with the layers' own seeded saliency recipe."""
    cfg = {"vgg16": wl.config3, "mobilenetv2": wl.config4}[which]()
    return [l for l in cfg]


@pytest.mark.parametrize("which,fracs", [("vgg16", (0.5, 0.8)), ("mobilenetv2", (0.3, 0.6, 0.9))])
def test_network_selection_and_masks_match_oracle(env, which, fracs):
    """Scores come from crisp_build_mask's workspace; the selected counts go back into crisp_build_mask."""
    B, torch = env
    layers = network(which)
    gpu, sal, omask = [], [], []
    for l in layers:
        s = wl.make_saliency(l, wl.make_weight(l))
        L = B.HybridLayer(l.rows, l.k, l.n, l.m, l.block_rows, l.block_k, 1.0)
        L.build_mask(to_dev(s, torch))
        gpu.append(L)
        sal.append(s)
        omask.append(oracle.build_mask(s, l.n, l.m, l.block_rows, l.block_k, keep_ratio=1.0))
    torch.cuda.synchronize()
    # the scores the selection reads are the oracle's, bit for bit, and so is the scale
    for L, s, mk in zip(gpu, sal, omask):
        sc_ptr, mk_ptr = B.crisp_mask_scores(L.desc, L.workspace)
        off = sc_ptr - L.workspace.data_ptr()
        sc = L.workspace[off: off + 8 * L.nrt * L.nblk].view(torch.int64).cpu().numpy().view(np.uint64)
        assert np.array_equal(sc.reshape(L.nrt, L.nblk), mk.score)
        key = int(L.workspace[:4].view(torch.int32).cpu().numpy().view(np.uint32)[0])
        smax = float(np.array([key], dtype=np.uint32).view(np.float32)[0])
        assert (int(np.frexp(smax)[1]) - 1 if smax > 0 else 0) == oracle.score_scale_exp(s)
    exps = [oracle.score_scale_exp(s) for s in sal]
    elems = [l.block_rows * l.block_k for l in layers]
    for frac in fracs:
        for min_keep in (0, 1):
            want = oracle.global_rank([m.score for m in omask], exps, elems, frac, min_keep=[min_keep] * len(layers))
            got = gpu_rank(B, torch, [L.rank_layer(min_keep) for L in gpu], frac)
            assert np.array_equal(got, want), (frac, min_keep, got, want)
    # feed the last selection back: the masks are the oracle's masks for those counts
    for L, l, s, kk in zip(gpu, layers, sal, want):
        L.set_kkeep(int(kk))
        L.build_mask(to_dev(s, torch))
        ref = oracle.build_mask(s, l.n, l.m, l.block_rows, l.block_k, kkeep=int(kk))
        blk_col, nm_bits = L.export_mask()
        assert np.array_equal(blk_col, ref.blk_col)
        assert np.array_equal(nm_bits, ref.nm_bits)
        L.close()
