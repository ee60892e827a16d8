"""Full-size layers of the five workload families through the C ABI, in the launch configuration
bench.py times.

* Masks and encodings of EVERY layer of the VGG-16 and MobileNetV2 stand-ins and of all twenty sweep
  cells are compared with the oracle bit for bit (whole layer).
* The product of a selection of them is compared on at least 64 output rows (tile edges plus seeded
  ones; every column) that the oracle computes with its literal fp64 loop, and on the whole output
  against the property  Y = decode(W_hybrid) @ X  evaluated by a dense fp32 matmul (a library routine,
  used only as a second witness)."""
import numpy as np
import pytest

import oracle
from paper_2311_14272_b200 import workloads as wl

from helpers import ABS_TOL, FRO_TOL, assert_mask_and_encoding_equal, bf16_dev, check_tolerance, oracle_layer, y_to_f64

pytestmark = pytest.mark.gpu


def _layers():
    c3, c4, c5 = wl.config3(), wl.config4(), wl.config5()
    pick = [c3[0], c3[1], c3[5], c3[12],                 # VGG: K = 27 (one padded block), widest X, middle, last
            c4[0], c4[5], c4[32], c4[34],                # MobileNetV2: 32->32 @112^2, 144->24 (ragged), 960->320, 320->1280
            wl.sweep_cell(2, 4, 0.5), wl.sweep_cell(1, 8, 0.25), wl.sweep_cell(4, 8, 0.1), wl.sweep_cell(1, 4, 1.0)]
    return pick


@pytest.mark.parametrize("layer", _layers(), ids=lambda l: l.name)
def test_full_size_layer(layer):
    import torch
    from paper_2311_14272_b200 import binding as B
    B.load()
    w, s, x = wl.make_layer_inputs(layer)
    mk, vals, idx, wd, wb = oracle_layer(w, s, layer.n, layer.m, layer.block_rows, layer.block_k, layer.keep_ratio)
    L = B.HybridLayer(layer.rows, layer.k, layer.n, layer.m, layer.block_rows, layer.block_k, layer.keep_ratio)
    L.build_mask(torch.from_numpy(s).cuda()).encode(bf16_dev(w, torch))
    assert_mask_and_encoding_equal(L, mk, vals, idx)

    d_x = bf16_dev(x, torch)
    y = L.spmm(d_x)
    torch.cuda.synchronize()
    assert L.device_status() == 0
    if mk.kkeep > 0:                                        # the tensor-core kernel is the one that ran
        assert L.last_launch()["path"] == (B.PATH_SPARSE if layer.n <= 2 else B.PATH_DENSE)
    # sampled rows: first, last, tile edges and a few seeded ones, every column
    rng = np.random.default_rng(layer.seed)
    edges = [0, layer.rows - 1]
    for t in (layer.block_rows, 128):                      # first/last row of the first and last row tile / CTA tile
        edges += [t - 1, t, (layer.rows - 1) // t * t - 1, (layer.rows - 1) // t * t]
    sel = set(int(r) for r in edges if 0 <= r < layer.rows)
    want = min(layer.rows, 64)
    pool = rng.permutation(layer.rows)
    for r in pool:
        if len(sel) >= want:
            break
        sel.add(int(r))
    sel = np.array(sorted(sel), dtype=np.int32)
    assert len(sel) >= want
    ref = oracle.spmm_fp64_rows(wd, x, sel)
    got = y_to_f64(y[torch.from_numpy(sel.astype(np.int64)).cuda()], torch)
    check_tolerance(got, ref)
    # whole output against the dense product of the decoded weight
    dec = L.decode()
    assert np.array_equal(dec.view(torch.int16).cpu().numpy().view(np.uint16), wb)
    num = torch.zeros((), dtype=torch.float64, device="cuda")
    den = torch.zeros((), dtype=torch.float64, device="cuda")
    worst = torch.zeros((), dtype=torch.float32, device="cuda")
    step = max(1, (1 << 26) // max(1, layer.rows))          # column chunks keep the fp32 temporaries small
    dec32 = dec.float()
    for c0 in range(0, layer.ncols, step):
        yr = dec32 @ d_x[:, c0:c0 + step].float()
        diff = y[:, c0:c0 + step].float() - yr
        num += (diff.double() ** 2).sum()
        den += (yr.double() ** 2).sum()
        worst = torch.maximum(worst, (diff.abs() / (1 + yr.abs())).max())
    assert worst.item() <= ABS_TOL
    if den.item() > 0:
        assert (num / den).sqrt().item() <= FRO_TOL
    else:
        assert torch.count_nonzero(y).item() == 0
    L.close()


_SWEEP_INPUTS = {}


def _weight_and_saliency(layer):
    """W and S of a layer; the twenty sweep cells prune the same 4096 x 4096 pair."""
    if layer.name.startswith("sweep"):
        if not _SWEEP_INPUTS:
            w = wl.make_weight(layer)
            _SWEEP_INPUTS["ws"] = (w, wl.make_saliency(layer, w))
        return _SWEEP_INPUTS["ws"]
    w = wl.make_weight(layer)
    return w, wl.make_saliency(layer, w)


def _every_layer():
    return wl.config3() + wl.config4() + wl.config5()


@pytest.mark.parametrize("layer", _every_layer(), ids=lambda l: l.name)
def test_mask_and_encoding_of_every_layer(layer):
    import torch
    from paper_2311_14272_b200 import binding as B
    B.load()
    w, s = _weight_and_saliency(layer)
    mk, vals, idx, wd, wb = oracle_layer(w, s, layer.n, layer.m, layer.block_rows, layer.block_k, layer.keep_ratio)
    L = B.HybridLayer(layer.rows, layer.k, layer.n, layer.m, layer.block_rows, layer.block_k, layer.keep_ratio)
    L.build_mask(torch.from_numpy(s).cuda()).encode(bf16_dev(w, torch))
    assert_mask_and_encoding_equal(L, mk, vals, idx)
    assert np.array_equal(L.decode().view(torch.int16).cpu().numpy().view(np.uint16), wb)
    L.close()
