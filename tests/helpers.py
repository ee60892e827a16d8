"""Shared plumbing of the GPU parity tests: run one layer through the C ABI and through the
oracle on the same seeded inputs."""
import numpy as np

import oracle
from paper_2311_14272_b200 import workloads as wl

ABS_TOL = 1e-2      # max |Y - Yref| <= ABS_TOL * (1 + |Yref|)
FRO_TOL = 5e-3      # ||Y - Yref||_F / ||Yref||_F


def to_dev(a, torch, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.view(dtype)
    return t.cuda()


def bf16_dev(bits, torch):
    return to_dev(bits.view(np.int16), torch).view(torch.bfloat16)


def y_to_f64(y, torch):
    if y.dtype == torch.bfloat16:
        bits = y.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
        return wl.bf16_bits_to_f32(bits).astype(np.float64)
    return y.cpu().numpy().astype(np.float64)


def check_tolerance(y, ref):
    err = np.abs(y - ref)
    assert np.all(err <= ABS_TOL * (1.0 + np.abs(ref))), f"max err {err.max()}"
    den = np.linalg.norm(ref)
    if den > 0:
        assert np.linalg.norm(y - ref) / den <= FRO_TOL
    else:
        assert np.count_nonzero(y) == 0


def oracle_layer(w, s, n, m, bm, bk, keep, score_mode=0):
    mk = oracle.build_mask(s, n, m, bm, bk, keep, score_mode=score_mode)
    vals, idx = oracle.encode(w, mk)
    wd, wb = oracle.decode(mk.blk_col, vals, idx, mk.rows, mk.k, n, m, bm, bk, mk.kkeep)
    return mk, vals, idx, wd, wb


def gpu_layer(B, torch, w, s, n, m, bm, bk, keep, score_mode=0, ld_pad=0):
    rows, k = w.shape
    L = B.HybridLayer(rows, k, n, m, bm, bk, keep, score_mode)
    if ld_pad:
        s_d = torch.full((rows, k + ld_pad), float("nan"), dtype=torch.float32, device="cuda")
        s_d[:, :k] = to_dev(s, torch)
        w_d = torch.full((rows, k + ld_pad), 1.0, dtype=torch.bfloat16, device="cuda")
        w_d[:, :k] = bf16_dev(w, torch)
        s_v, w_v = s_d[:, :k], w_d[:, :k]
    else:
        s_v, w_v = to_dev(s, torch), bf16_dev(w, torch)
    L.build_mask(s_v)
    L.encode(w_v)
    return L


def assert_mask_and_encoding_equal(L, mk, vals, idx):
    blk_col, nm_bits = L.export_mask()
    assert np.array_equal(blk_col, mk.blk_col)
    assert np.array_equal(nm_bits, mk.nm_bits)
    bc2, v2, i2 = L.export()
    assert np.array_equal(bc2, mk.blk_col)
    assert np.array_equal(v2, vals)
    assert np.array_equal(i2, idx)
