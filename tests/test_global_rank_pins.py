"""Pins for the oracle's global rank selection (Algorithm 1: per-row sort, rank-column sums c_o,
global order across layers, selection by the sparsity target; Sec. III-C).

The paper prints no worked numbers for these steps, so the oracle is pinned by a hand-worked case,
closed forms for special cases, and the properties that define the result: on tiny random networks
the selection is recomputed from the scores with Python's exact rationals and checked to be the
shortest front of the global order that reaches the target.
"""
from fractions import Fraction

import numpy as np
import pytest

import oracle


def _rank_columns(score):
    """c_o from the definition: sort every row increasingly, add down the columns (Python ints)."""
    rows = [sorted(int(v) for v in r) for r in np.asarray(score)]
    return [sum(r[o] for r in rows) for o in range(len(rows[0]))]


def _definition(scores, exps, elems, frac, min_keep):
    """Shortest front of the global increasing order (value, layer, o) whose weight reaches the target."""
    entries, total = [], 0
    for l, sc in enumerate(scores):
        nrt, nblk = sc.shape
        total += nrt * nblk * elems[l]
        c = _rank_columns(sc)
        for o in range(nblk - min_keep[l]):
            entries.append((Fraction(c[o]) * Fraction(2) ** exps[l], l, o, nrt * elems[l]))
    target = int(np.floor(frac * float(total) + 0.5))
    entries.sort()
    keep = [sc.shape[1] for sc in scores]
    pruned = 0
    for _, l, _, w in entries:
        if pruned >= target:
            break
        pruned += w
        keep[l] -= 1
    return keep, target, entries


def test_hand_worked_two_layers():
    # layer 0: rows [5,1,9],[2,8,3] -> sorted [1,5,9],[2,3,8] -> c = 3, 8, 17; a rank position weighs 2*4 = 8
    # layer 1: row [4,4] -> c = 4, 4; a rank position weighs 4.  total 32 weights, half = 16.
    # order: 3 (l0), 4 (l1,o0), 4 (l1,o1), 8, 17 -> 8 + 4 + 4 = 16 reached after three positions.
    sc = [np.array([[5, 1, 9], [2, 8, 3]], dtype=np.uint64), np.array([[4, 4]], dtype=np.uint64)]
    assert oracle.global_rank(sc, [0, 0], [4, 4], 0.5).tolist() == [2, 0]
    assert oracle.global_rank(sc, [0, 0], [4, 4], 0.0).tolist() == [3, 2]
    assert oracle.global_rank(sc, [0, 0], [4, 4], 1.0).tolist() == [0, 0]
    # one more weight than 8 needs the second position as well
    assert oracle.global_rank(sc, [0, 0], [4, 4], 9 / 32).tolist() == [2, 1]
    # protected last block of layer 1: its second position is no candidate, the front moves on to c = 8
    assert oracle.global_rank(sc, [0, 0], [4, 4], 0.5, min_keep=[0, 1]).tolist() == [1, 1]


def test_single_layer_closed_form():
    # one layer: positions are pruned lowest first, ceil(target / weight per position) of them
    rng = np.random.default_rng(7)
    for nrt, nblk, elems in ((1, 7, 16), (3, 9, 64), (4, 1, 8)):
        sc = rng.integers(0, 50, size=(nrt, nblk), dtype=np.uint64)
        for frac in (0.0, 0.1, 0.34, 0.5, 0.77, 1.0):
            target = int(np.floor(frac * nrt * nblk * elems + 0.5))
            expect = nblk - min(nblk, -(-target // (nrt * elems)))
            assert oracle.global_rank([sc], [0], [elems], frac).tolist() == [expect]


def test_identical_layers_alternate_lower_layer_first():
    sc = np.array([[1, 2, 3, 4]], dtype=np.uint64)
    # every position weighs 1 block of 4 weights; total 32; ties between the layers go to layer 0
    for k in range(9):
        got = oracle.global_rank([sc, sc], [0, 0], [4, 4], k / 8).tolist()
        assert got == [4 - (k + 1) // 2, 4 - k // 2]


def test_scale_exponent_orders_real_values():
    sc = np.array([[1, 2, 3]], dtype=np.uint64)
    # layer 0 in units of 1, layer 1 in units of 2: values 1,2,3 and 2,4,6
    # order: A0=1, A1=2 (tie with B0 -> lower layer), B0=2, A2=3, B1=4, B2=6
    expect = [[3, 3], [2, 3], [1, 3], [1, 2], [0, 2], [0, 1], [0, 0]]
    for k in range(7):
        assert oracle.global_rank([sc, sc], [0, 1], [1, 1], k / 6).tolist() == expect[k]
    # a huge scale gap: every position of the small-unit layer goes first
    assert oracle.global_rank([sc, sc], [100, -100], [1, 1], 0.5).tolist() == [3, 0]


def test_sums_beyond_64_bits():
    # 600 row tiles with scores near 2^55 give rank sums above 2^64
    big = np.full((600, 2), (1 << 55) - 1, dtype=np.uint64)
    big[:, 1] -= 1                                   # column 1 holds the smaller scores
    small = np.array([[3, 1]], dtype=np.uint64)
    # values: layer 0 -> 600*(2^55-2), 600*(2^55-1); layer 1 with exponent 70 -> 1*2^70, 3*2^70
    c0 = 600 * ((1 << 55) - 2)
    assert c0 > (1 << 64)
    order = sorted([(Fraction(c0), 0), (Fraction(c0 + 600), 0), (Fraction(1 << 70), 1), (Fraction(3 << 70), 1)])
    assert [l for _, l in order] == [0, 0, 1, 1]
    tot = 600 * 2 + 2
    assert oracle.global_rank([big, small], [0, 70], [1, 1], 600 / tot).tolist() == [1, 2]
    assert oracle.global_rank([big, small], [0, 70], [1, 1], 1201 / tot).tolist() == [0, 1]
    # and with the small layer scaled below the big one
    assert oracle.global_rank([big, small], [0, -3], [1, 1], 1 / tot).tolist() == [2, 1]


@pytest.mark.parametrize("seed", range(40))
def test_definition_on_tiny_networks(seed):
    rng = np.random.default_rng(1000 + seed)
    nl = int(rng.integers(1, 5))
    scores, exps, elems, mk = [], [], [], []
    for _ in range(nl):
        nrt, nblk = int(rng.integers(1, 4)), int(rng.integers(1, 6))
        hi = int(rng.choice([3, 10, 1 << 20]))       # small ranges force ties
        scores.append(rng.integers(0, hi, size=(nrt, nblk), dtype=np.uint64))
        exps.append(int(rng.integers(-3, 4)))
        elems.append(int(rng.choice([1, 4, 16])))
        mk.append(int(rng.integers(0, 2)) if nblk > 1 else 0)
    for frac in (0.0, 0.13, 0.4, 0.5, 0.81, 1.0):
        got = oracle.global_rank(scores, exps, elems, frac, min_keep=mk).tolist()
        keep, target, entries = _definition(scores, exps, elems, frac, mk)
        assert got == keep
        # properties that define the result, checked on the oracle's output itself
        pruned_w = sum((scores[l].shape[1] - got[l]) * scores[l].shape[0] * elems[l] for l in range(nl))
        cand_w = sum(w for _, _, _, w in entries)
        assert pruned_w >= min(target, cand_w)
        pruned = [(v, l, o, w) for v, l, o, w in entries if o < scores[l].shape[1] - got[l]]
        kept = [(v, l, o, w) for v, l, o, w in entries if o >= scores[l].shape[1] - got[l]]
        if pruned:
            assert pruned_w - max(pruned)[3] < target                  # the last one was needed
        if pruned and kept:
            assert max(pruned)[:3] < min(kept)[:3]                       # a front of the global order
        for l in range(nl):
            assert mk[l] <= got[l] <= scores[l].shape[1]


def test_monotone_in_target():
    rng = np.random.default_rng(3)
    scores = [rng.integers(0, 1000, size=(2, 6), dtype=np.uint64), rng.integers(0, 1000, size=(5, 4), dtype=np.uint64)]
    prev = None
    for frac in np.linspace(0, 1, 21):
        got = oracle.global_rank(scores, [0, 2], [16, 4], float(frac))
        if prev is not None:
            assert (got <= prev).all()
        prev = got


def test_feeds_the_mask_projection():
    # the kept-block count of a layer, turned into a keep ratio, gives that count back (Sec. III-C: the
    # selection decides how many blocks every row keeps; the mask projection then takes the best ones)
    rng = np.random.default_rng(11)
    s = [np.abs(rng.normal(size=(8, 32))).astype(np.float32) * sc for sc in (1.0, 0.01, 30.0)]
    masks = [oracle.build_mask(x, 2, 4, 4, 8, keep_ratio=1.0) for x in s]
    kk = oracle.global_rank([m.score for m in masks], [oracle.score_scale_exp(x) for x in s], [32] * 3, 0.5)
    # 3 layers x 2 row tiles x 4 blocks of 32 weights; every rank position weighs 64: half = 6 positions
    assert int(kk.sum()) == 6
    assert kk[1] <= kk[0] <= kk[2]               # the layer with the smallest saliency scale loses most
    for x, k in zip(s, kk):
        m = oracle.build_mask(x, 2, 4, 4, 8, keep_ratio=float(k) / 4)
        assert m.kkeep == int(k)
        assert (np.diff(m.blk_col, axis=1) > 0).all() if k > 1 else True
