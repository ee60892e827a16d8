"""ctypes front end of the CPU oracle (``crisp_oracle.c``).

Test infrastructure only: the tests, the smoke check and the benchmark's
CPU-baseline leg load this; the CUDA library and its Python binding never do.
The wrapper only allocates numpy arrays and forwards pointers.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "crisp_oracle.c")
_LIB = os.path.join(_HERE, "libcrisp_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP for the row-parallel product)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp",
                               "-ffp-contract=off", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
    return _lib


def _p(a, t):
    return a.ctypes.data_as(C.POINTER(t)) if a is not None else None


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def keep_count(k: int, block_k: int, keep_ratio: float):
    nblk, kkeep = C.c_int(), C.c_int()
    rc = lib().oracle_keep_count(C.c_int(k), C.c_int(block_k), C.c_double(keep_ratio),
                                 C.byref(nblk), C.byref(kkeep))
    if rc:
        raise ValueError(f"oracle_keep_count rc={rc}")
    return nblk.value, kkeep.value


@dataclass
class Mask:
    rows: int
    k: int
    n: int
    m: int
    block_rows: int
    block_k: int
    kkeep: int
    blk_col: np.ndarray   # int32 [nrt, kkeep]
    nm_bits: np.ndarray   # uint32 [nrt*block_rows, ceil(nblk*block_k/32)]
    score: np.ndarray     # uint64 [nrt, nblk]

    @property
    def nrt(self):
        return (self.rows + self.block_rows - 1) // self.block_rows

    @property
    def nblk(self):
        return (self.k + self.block_k - 1) // self.block_k

    def dense(self) -> np.ndarray:
        """Boolean [nrt*block_rows, nblk*block_k] view of the bit mask."""
        bits = np.unpackbits(self.nm_bits.view(np.uint8), axis=1, bitorder="little")
        return bits[:, : self.nblk * self.block_k].astype(bool)


def build_mask(saliency: np.ndarray, n: int, m: int, block_rows: int, block_k: int,
               keep_ratio: float | None = None, score_mode: int = 0, kkeep: int | None = None) -> Mask:
    s = np.ascontiguousarray(saliency, dtype=np.float32)
    rows, k = s.shape
    nblk = (k + block_k - 1) // block_k
    if kkeep is None:
        nblk, kkeep = keep_count(k, block_k, keep_ratio)
    nrt = (rows + block_rows - 1) // block_rows
    wpr = (nblk * block_k + 31) // 32
    blk_col = np.zeros((nrt, kkeep), dtype=np.int32)
    nm_bits = np.zeros((nrt * block_rows, wpr), dtype=np.uint32)
    score = np.zeros((nrt, nblk), dtype=np.uint64)
    rc = lib().oracle_build_mask(_p(s, C.c_float), C.c_int64(s.strides[0] // 4), C.c_int(rows), C.c_int(k),
                                 C.c_int(n), C.c_int(m), C.c_int(block_rows), C.c_int(block_k),
                                 C.c_int(kkeep), C.c_int(score_mode),
                                 _p(blk_col, C.c_int32), _p(nm_bits, C.c_uint32), _p(score, C.c_uint64))
    if rc:
        raise ValueError(f"oracle_build_mask rc={rc}")
    return Mask(rows, k, n, m, block_rows, block_k, kkeep, blk_col, nm_bits, score)


def encoded_sizes(rows, block_rows, block_k, n, m, kkeep):
    nv, nw = C.c_int64(), C.c_int64()
    rc = lib().oracle_encoded_sizes(C.c_int(rows), C.c_int(block_rows), C.c_int(block_k), C.c_int(n),
                                    C.c_int(m), C.c_int(kkeep), C.byref(nv), C.byref(nw))
    if rc:
        raise ValueError(f"oracle_encoded_sizes rc={rc}")
    return nv.value, nw.value


def encode(w_bits: np.ndarray, mask: Mask):
    """-> (vals uint16 [nvals], idx uint32 [nwords]) in the canonical order."""
    w = np.ascontiguousarray(w_bits, dtype=np.uint16)
    nv, nw = encoded_sizes(mask.rows, mask.block_rows, mask.block_k, mask.n, mask.m, mask.kkeep)
    vals = np.zeros(nv, dtype=np.uint16)
    idx = np.zeros(nw, dtype=np.uint32)
    rc = lib().oracle_encode(_p(w, C.c_uint16), C.c_int64(w.strides[0] // 2), C.c_int(mask.rows), C.c_int(mask.k),
                             C.c_int(mask.n), C.c_int(mask.m), C.c_int(mask.block_rows), C.c_int(mask.block_k),
                             C.c_int(mask.kkeep), _p(np.ascontiguousarray(mask.blk_col), C.c_int32),
                             _p(np.ascontiguousarray(mask.nm_bits), C.c_uint32),
                             _p(vals, C.c_uint16), _p(idx, C.c_uint32))
    if rc:
        raise ValueError(f"oracle_encode rc={rc}")
    return vals, idx


def decode(blk_col, vals, idx, rows, k, n, m, block_rows, block_k, kkeep):
    """-> (dense fp64 [rows, k], dense bf16 bits [rows, k])."""
    wd = np.zeros((rows, k), dtype=np.float64)
    wb = np.zeros((rows, k), dtype=np.uint16)
    bc = np.ascontiguousarray(blk_col, dtype=np.int32)
    rc = lib().oracle_decode(_p(bc, C.c_int32), _p(np.ascontiguousarray(vals, dtype=np.uint16), C.c_uint16),
                             _p(np.ascontiguousarray(idx, dtype=np.uint32), C.c_uint32),
                             C.c_int(rows), C.c_int(k), C.c_int(n), C.c_int(m), C.c_int(block_rows),
                             C.c_int(block_k), C.c_int(kkeep), _p(wd, C.c_double), _p(wb, C.c_uint16))
    if rc:
        raise ValueError(f"oracle_decode rc={rc}")
    return wd, wb


def _spmm_call(fn, w_dense, x_bits):
    wd = np.ascontiguousarray(w_dense, dtype=np.float64)
    x = np.ascontiguousarray(x_bits, dtype=np.uint16)
    rows, k = wd.shape
    assert x.shape[0] == k
    y = np.empty((rows, x.shape[1]), dtype=np.float64)
    rc = fn(_p(wd, C.c_double), C.c_int(rows), C.c_int(k), _p(x, C.c_uint16),
            C.c_int64(x.shape[1]), C.c_int64(x.shape[1]), _p(y, C.c_double))
    if rc:
        raise ValueError(f"oracle spmm rc={rc}")
    return y


def spmm_fp64(w_dense, x_bits):
    """Y = Wd @ X by the literal fp64 triple loop."""
    return _spmm_call(lib().oracle_spmm_fp64, w_dense, x_bits)


def spmm_fp64_skipzero(w_dense, x_bits):
    return _spmm_call(lib().oracle_spmm_fp64_skipzero, w_dense, x_bits)


def spmm_fp64_rows(w_dense, x_bits, sel):
    wd = np.ascontiguousarray(w_dense, dtype=np.float64)
    x = np.ascontiguousarray(x_bits, dtype=np.uint16)
    sel = np.ascontiguousarray(sel, dtype=np.int32)
    rows, k = wd.shape
    y = np.empty((len(sel), x.shape[1]), dtype=np.float64)
    rc = lib().oracle_spmm_fp64_rows(_p(wd, C.c_double), C.c_int(rows), C.c_int(k), _p(x, C.c_uint16),
                                     C.c_int64(x.shape[1]), C.c_int64(x.shape[1]),
                                     _p(sel, C.c_int32), C.c_int(len(sel)), _p(y, C.c_double))
    if rc:
        raise ValueError(f"oracle_spmm_fp64_rows rc={rc}")
    return y


def score_scale_exp(saliency: np.ndarray) -> int:
    """Exponent e of a layer's largest canonical saliency (|s|, NaN -> 0, Inf -> FLT_MAX): one unit of
    the layer's block scores is worth 2^(e - 40).  0 for an all-zero layer."""
    s = np.abs(np.nan_to_num(np.asarray(saliency, dtype=np.float32), nan=0.0,
                             posinf=np.finfo(np.float32).max, neginf=np.finfo(np.float32).max))
    smax = float(s.max()) if s.size else 0.0
    return int(np.frexp(smax)[1]) - 1 if smax > 0 else 0      # smax = m * 2^e with m in [0.5, 1)


def global_rank(scores, scale_exps, block_elems, prune_fraction: float, min_keep=None) -> np.ndarray:
    """Algorithm 1, rank-column sums + global order + selection: kept blocks per row tile of every layer.

    scores[l]: uint64 [nrt_l, nblk_l]; scale_exps[l]: int; block_elems[l]: weights per block.
    """
    nl = len(scores)
    arrs = [np.ascontiguousarray(s, dtype=np.uint64) for s in scores]
    ptrs = (C.POINTER(C.c_uint64) * nl)(*[_p(a, C.c_uint64) for a in arrs])
    nrt = np.array([a.shape[0] for a in arrs], dtype=np.int32)
    nblk = np.array([a.shape[1] for a in arrs], dtype=np.int32)
    se = np.array(scale_exps, dtype=np.int32)
    be = np.array(block_elems, dtype=np.int64)
    mk = np.zeros(nl, dtype=np.int32) if min_keep is None else np.array(min_keep, dtype=np.int32)
    out = np.zeros(nl, dtype=np.int32)
    rc = lib().oracle_global_rank(C.c_int(nl), ptrs, _p(nrt, C.c_int), _p(nblk, C.c_int), _p(se, C.c_int),
                                  _p(be, C.c_int64), _p(mk, C.c_int), C.c_double(prune_fraction),
                                  _p(out, C.c_int32))
    if rc:
        raise ValueError(f"oracle_global_rank rc={rc}")
    return out


def conv_fp64(w_dense: np.ndarray, kh: int, kw: int, act_bits: np.ndarray, pad: int) -> np.ndarray:
    """Convolution by its definition (stride 1, zero padding): w_dense fp64 [S, kh*kw*R] with the reduction
    ordered (kernel row, kernel column, channel); act_bits bf16 patterns [B, H, W, R] -> fp64 [S, B*Ho*Wo]."""
    wd = np.ascontiguousarray(w_dense, dtype=np.float64)
    a = np.ascontiguousarray(act_bits, dtype=np.uint16)
    b, h, w, r = a.shape
    s = wd.shape[0]
    assert wd.shape[1] == kh * kw * r
    ho, wo = h + 2 * pad - kh + 1, w + 2 * pad - kw + 1
    y = np.zeros((s, b * ho * wo), dtype=np.float64)
    rc = lib().oracle_conv_fp64(_p(wd, C.c_double), C.c_int(s), C.c_int(kh), C.c_int(kw), C.c_int(r),
                                _p(a, C.c_uint16), C.c_int(b), C.c_int(h), C.c_int(w), C.c_int(pad),
                                _p(y, C.c_double))
    if rc:
        raise ValueError(f"oracle_conv_fp64 rc={rc}")
    return y


def bias_relu(y: np.ndarray, bias=None, relu: bool = False) -> np.ndarray:
    """Layer epilogue on an fp64 product [rows, ncols]: + bias[row] (fp32 values), then max(., 0) if relu."""
    out = np.ascontiguousarray(y, dtype=np.float64).copy()
    b = None if bias is None else np.ascontiguousarray(bias, dtype=np.float32)
    rc = lib().oracle_bias_relu(_p(out, C.c_double), C.c_int(out.shape[0]), C.c_int64(out.shape[1]),
                                _p(b, C.c_float), C.c_int(1 if relu else 0))
    if rc:
        raise ValueError(f"oracle_bias_relu rc={rc}")
    return out


def saliency(grads: np.ndarray, w_bits: np.ndarray) -> np.ndarray:
    """Eq. 1: |mean over samples of g  *  W|.  grads [H, rows, k] (any float), w_bits bf16 patterns -> fp64."""
    g = np.ascontiguousarray(grads, dtype=np.float64)
    w = np.ascontiguousarray(w_bits, dtype=np.uint16)
    h, rows, k = g.shape
    out = np.zeros((rows, k), dtype=np.float64)
    rc = lib().oracle_saliency(_p(g, C.c_double), C.c_int(h), _p(w, C.c_uint16), C.c_int(rows), C.c_int(k),
                               _p(out, C.c_double))
    if rc:
        raise ValueError(f"oracle_saliency rc={rc}")
    return out


def saliency_f32(grads: np.ndarray, w_bits: np.ndarray) -> np.ndarray:
    """Eq. 1 evaluated in fp32 in a fixed order (sum of the samples in order, times fp32(1/H), times W): the
    evaluation to use where the score goes on to decide a mask that is compared bit for bit."""
    g = np.ascontiguousarray(grads, dtype=np.float32)
    w = np.ascontiguousarray(w_bits, dtype=np.uint16)
    h, rows, k = g.shape
    out = np.zeros((rows, k), dtype=np.float32)
    rc = lib().oracle_saliency_f32(_p(g, C.c_float), C.c_int(h), _p(w, C.c_uint16), C.c_int(rows), C.c_int(k),
                                   _p(out, C.c_float))
    if rc:
        raise ValueError(f"oracle_saliency_f32 rc={rc}")
    return out
