"""One pruning iteration of Algorithm 1 over a whole network (minus the fine-tuning), repeated for a schedule
of sparsity targets, on the GPU against the same sequence composed from the oracle's functions:

    saliency (Eq. 1)  ->  N:M step + block scores  ->  rank-column sums, global order, selection
    ->  per-row-tile selection with the selected count  ->  compressed format

The network is the MobileNetV2 stand-in (the 35 pointwise layers' weight shapes).  Every step's kept-block
counts, masks and encodings must equal the oracle's bit for bit.  Because the score goes on to decide the
mask, both sides evaluate Eq. 1 in the same precision and order (fp32, samples added in order).  Between
steps the weights are replaced by the pruned ones (decode of the previous step's encoding), as Algorithm 1
does before it fine-tunes."""
import numpy as np
import pytest

import oracle
from paper_2311_14272_b200 import workloads as wl

from helpers import bf16_dev, to_dev

pytestmark = pytest.mark.gpu

N, M, BM, BK = 2, 8, 32, 32
SAMPLES = 3
KAPPAS = [0.80, 0.86, 0.93]          # overall sparsity after each step; 2:8 alone gives 0.75


def oracle_step(weights, grads, kappa, min_keep):
    sal = [oracle.saliency_f32(g, w) for g, w in zip(grads, weights)]
    full = [oracle.build_mask(s, N, M, BM, BK, 1.0) for s in sal]
    exps = [oracle.score_scale_exp(s) for s in sal]
    prune_fraction = min(1.0, max(0.0, 1.0 - (1.0 - kappa) * M / N))
    kk = oracle.global_rank([f.score for f in full], exps, [BM * BK] * len(full), prune_fraction,
                            min_keep=[min_keep] * len(full))
    masks, encs = [], []
    for s, w, f, c in zip(sal, weights, full, kk):
        mk = oracle.build_mask(s, N, M, BM, BK, float(c) / f.nblk)
        assert mk.kkeep == c
        masks.append(mk)
        encs.append(oracle.encode(w, mk))
    return kk, masks, encs


def test_three_pruning_iterations_match_the_oracle():
    import torch
    from paper_2311_14272_b200 import binding as B
    B.load()
    shapes = [(l.rows, l.k) for l in wl.config4()]
    rng = np.random.default_rng(2311)
    w_host = [wl.f32_to_bf16_bits((rng.standard_normal(sh) * np.sqrt(2.0 / sh[1])).astype(np.float32)) for sh in shapes]
    net = B.PruningNetwork(shapes, N, M, BM, BK, min_keep=1)
    prev_kk = None
    for step, kappa in enumerate(KAPPAS):
        grads = [(rng.standard_normal((SAMPLES,) + sh) * 1e-2).astype(np.float32) for sh in shapes]
        d_w = [bf16_dev(w, torch) for w in w_host]
        d_g = [[to_dev(g[i], torch) for i in range(SAMPLES)] for g in grads]
        kk = net.step(d_w, d_g, kappa)
        torch.cuda.synchronize()
        want_kk, want_masks, want_encs = oracle_step(w_host, grads, kappa, 1)
        assert list(kk) == [int(c) for c in want_kk], (step, kk, want_kk)
        if prev_kk is not None:                      # the schedule tightens: no layer keeps more than before
            assert sum(kk) < sum(prev_kk)
        prev_kk = kk
        new_w = []
        for L, mk, (vals, idx), w in zip(net.layers, want_masks, want_encs, w_host):
            blk_col, nm_bits = L.export_mask()
            assert np.array_equal(blk_col, mk.blk_col) and np.array_equal(nm_bits, mk.nm_bits)
            bc, v, i = L.export()
            assert np.array_equal(bc, mk.blk_col) and np.array_equal(v, vals) and np.array_equal(i, idx)
            # the pruned weights go into the next iteration
            _wd, wb = oracle.decode(mk.blk_col, vals, idx, mk.rows, mk.k, N, M, BM, BK, mk.kkeep)
            assert np.array_equal(L.decode().view(torch.int16).cpu().numpy().view(np.uint16), wb)
            new_w.append(wb)
        w_host = new_w
    net.close()


@pytest.mark.parametrize("rows,k,n,m,bm,bk", [(256, 1024, 2, 4, 32, 64), (200, 576, 1, 8, 64, 64), (130, 384, 3, 4, 128, 128)])
def test_reselect_equals_a_fresh_mask(rows, k, n, m, bm, bk):
    """Built with keep ratio 1 and then narrowed twice: the same mask as built directly with the final count."""
    import torch
    from paper_2311_14272_b200 import binding as B
    B.load()
    rng = np.random.default_rng(rows + k)
    s = rng.uniform(0.0, 3.0, (rows, k)).astype(np.float32)
    L = B.HybridLayer(rows, k, n, m, bm, bk, 1.0)
    L.build_mask(to_dev(s, torch))
    for kkeep in (L.nblk - 1, max(1, L.nblk // 3), 0):
        L.reselect(kkeep)
        mk = oracle.build_mask(s, n, m, bm, bk, kkeep / L.nblk)
        assert mk.kkeep == kkeep
        blk_col, nm_bits = L.export_mask()
        assert np.array_equal(blk_col, mk.blk_col) and np.array_equal(nm_bits, mk.nm_bits)
    with pytest.raises(B.CrispError):
        B.crisp_mask_reselect(L.mask, 1, L.workspace)          # upwards: the cleared group bits are gone
    L.close()


def test_finish_max_feeds_the_mask_without_a_second_pass():
    """The maximum left by crisp_saliency_finish_max is the one crisp_build_mask finds itself: same scores, same mask."""
    import torch
    from paper_2311_14272_b200 import binding as B
    B.load()
    rows, k, h = 192, 640, 4
    rng = np.random.default_rng(5)
    w = wl.f32_to_bf16_bits((rng.standard_normal((rows, k)) * 0.05).astype(np.float32))
    grads = (rng.standard_normal((h, rows, k)) * 1e-2).astype(np.float32)
    grads[0, 3, 7] = np.inf                                     # canonical form: counts as FLT_MAX
    grads[1, 5, 9] = np.nan                                     # counts as 0
    L = B.HybridLayer(rows, k, 2, 4, 32, 64, 0.5)
    acc = torch.empty((rows, k), dtype=torch.float32, device="cuda")
    s = torch.empty((rows, k), dtype=torch.float32, device="cuda")
    d_w = bf16_dev(w, torch)
    for i in range(h):
        B.crisp_saliency_accumulate(to_dev(grads[i], torch), 1, k, rows, k, acc, k, i == 0)
    B.crisp_saliency_finish_max(acc, k, d_w, k, rows, k, h, s, k, L.workspace)
    L.build_mask_max_known(s)
    got = L.export_mask()
    scores = L.workspace[256:256 + 8 * L.nrt * L.nblk].view(torch.int64).cpu().numpy().copy()
    L.build_mask(s)                                             # finds the maximum itself
    ref = L.export_mask()
    assert np.array_equal(got[0], ref[0]) and np.array_equal(got[1], ref[1])
    assert np.array_equal(scores, L.workspace[256:256 + 8 * L.nrt * L.nblk].view(torch.int64).cpu().numpy())
    mk = oracle.build_mask(s.cpu().numpy(), 2, 4, 32, 64, 0.5)
    assert np.array_equal(got[0], mk.blk_col) and np.array_equal(got[1], mk.nm_bits)
    L.close()
