"""ctypes binding of libcrisp's C ABI (see include/crisp.h).

Argument marshalling only: every step of the path runs in the CUDA kernels of
``libcrisp.so``.  PyTorch supplies device buffers and streams.  There is no CPU or
PyTorch fallback: if the shared library is missing, loading raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libcrisp.so")

OK, INVALID_ARG, UNSUPPORTED, BAD_SHAPE, BUFFER_TOO_SMALL, CUDA_ERROR, TIMEOUT = range(7)
PATH_DIRECT, PATH_DENSE, PATH_SPARSE, PATH_SPARSE2 = 0, 1, 2, 3
PATH_NAMES = {0: "direct", 1: "dense_tcgen05", 2: "sparse_tcgen05", 3: "sparse_tcgen05_two_addends"}


class LayerDesc(C.Structure):
    _fields_ = [("rows", C.c_int32), ("k", C.c_int32), ("n", C.c_int32), ("m", C.c_int32),
                ("block_rows", C.c_int32), ("block_k", C.c_int32), ("keep_ratio", C.c_double),
                ("score_mode", C.c_int32)]


class RankLayer(C.Structure):
    _fields_ = [("d_scores", C.c_void_p), ("d_max_key", C.c_void_p), ("nrt", C.c_int32), ("nblk", C.c_int32),
                ("block_elems", C.c_int64), ("min_keep", C.c_int32), ("reserved", C.c_int32)]


class ConvDesc(C.Structure):
    _fields_ = [("batch", C.c_int32), ("height", C.c_int32), ("width", C.c_int32), ("channels", C.c_int32),
                ("kernel_h", C.c_int32), ("kernel_w", C.c_int32), ("pad", C.c_int32), ("y_layout", C.c_int32)]


class LaunchInfo(C.Structure):
    _fields_ = [("path", C.c_int32), ("tile_cols", C.c_int32), ("accumulators", C.c_int32), ("stack", C.c_int32),
                ("epilogue_warps", C.c_int32), ("stages", C.c_int32), ("ctas", C.c_int32), ("conv", C.c_int32),
                ("stage_blocks", C.c_int32)]

    def as_dict(self):
        return {f: int(getattr(self, f)) for f, _ in self._fields_}


class BytesModel(C.Structure):
    _fields_ = [("nnz", C.c_int64), ("vals_bytes", C.c_int64), ("idx_bytes", C.c_int64),
                ("blk_col_bytes", C.c_int64), ("x_bytes", C.c_int64), ("y_bytes", C.c_int64),
                ("useful_macs", C.c_int64), ("slot_macs", C.c_int64), ("path", C.c_int32)]

    def as_dict(self):
        return {f: int(getattr(self, f)) for f, _ in self._fields_}


class CrispError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = crisp_status_string(code) if _lib is not None else str(code)
        super().__init__(f"{where}: {msg} (status {code})")


_lib = None


def load(path: Optional[str] = None):
    """Load libcrisp.so (built in-tree by ``paper_2311_14272_b200.build``)."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or LIB_PATH
    if not os.path.exists(p):
        raise FileNotFoundError(
            f"{p} not found: build it with `python -m paper_2311_14272_b200.build` "
            "(there is no fallback implementation)")
    lib = C.CDLL(p)
    vp, i32, i64, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t
    P = C.POINTER
    sig = {
        "crisp_keep_count": [P(LayerDesc), P(i32), P(i32)],
        "crisp_mask_sizes": [P(LayerDesc), P(sz), P(sz)],
        "crisp_build_mask": [vp, i64, P(LayerDesc), vp, vp, vp, P(vp)],
        "crisp_build_mask_static": [vp, i64, P(LayerDesc), vp, vp, P(vp)],
        "crisp_mask_export": [vp, vp, vp, vp],
        "crisp_mask_info": [vp, P(LayerDesc), P(i32), P(i32), P(i32)],
        "crisp_encode_sizes": [vp, P(sz), P(sz)],
        "crisp_encode": [vp, i64, vp, vp, vp, vp, P(vp)],
        "crisp_encoded_counts": [vp, P(i64), P(i64), P(i64)],
        "crisp_export": [vp, vp, vp, vp, vp],
        "crisp_decode": [vp, vp, i64, vp],
        "crisp_spmm": [vp, vp, i64, i64, vp, i64, i32, vp],
        "crisp_spmm_conv": [vp, vp, P(ConvDesc), vp, i64, i32, vp],
        "crisp_saliency_accumulate": [vp, i32, i64, i32, i32, vp, i64, i32, vp],
        "crisp_saliency_finish": [vp, i64, vp, i64, i32, i32, i32, vp, i64, vp],
        "crisp_saliency_finish_max": [vp, i64, vp, i64, i32, i32, i32, vp, i64, vp, vp],
        "crisp_build_mask_ex": [vp, i64, P(LayerDesc), vp, vp, C.c_uint32, vp, P(vp)],
        "crisp_mask_reselect": [vp, i32, vp, vp],
        "crisp_prune_fraction": [C.c_double, i32, i32, P(C.c_double)],
        "crisp_keep_ratio_for_count": [P(LayerDesc), i32, P(C.c_double)],
        "crisp_set_path": [vp, i32],
        "crisp_set_epilogue": [vp, vp, i32],
        "crisp_device_status": [vp, vp, P(i32)],
        "crisp_last_launch": [vp, P(LaunchInfo)],
        "crisp_set_tuning": [vp, i32, C.c_uint64, i32],
        "crisp_set_stage_blocks": [vp, i32],
        "crisp_reset_status": [vp, vp],
        "crisp_bytes_model": [vp, i64, i32, P(BytesModel)],
        "crisp_mask_scores": [P(LayerDesc), vp, P(vp), P(vp)],
        "crisp_global_rank_sizes": [i32, P(RankLayer), P(sz)],
        "crisp_global_rank": [i32, P(RankLayer), C.c_double, vp, vp, vp],
    }
    for name, args in sig.items():
        fn = getattr(lib, name)
        fn.argtypes = args
        fn.restype = C.c_int
    lib.crisp_mask_destroy.argtypes = [vp]
    lib.crisp_mask_destroy.restype = None
    lib.crisp_destroy.argtypes = [vp]
    lib.crisp_destroy.restype = None
    lib.crisp_status_string.argtypes = [C.c_int]
    lib.crisp_status_string.restype = C.c_char_p
    _lib = lib
    return lib


def crisp_status_string(code: int) -> str:
    return load().crisp_status_string(code).decode()


status_string = crisp_status_string


def _check(code: int, where: str):
    if code != OK:
        raise CrispError(code, where)


def _ptr(t) -> int:
    """Device (or host) address of a torch tensor / numpy array / int."""
    if t is None:
        return 0
    if isinstance(t, int):
        return t
    if hasattr(t, "data_ptr"):
        return t.data_ptr()
    return t.ctypes.data


def _stream(stream) -> int:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def make_desc(rows, k, n, m, block_rows, block_k, keep_ratio, score_mode=0) -> LayerDesc:
    return LayerDesc(rows, k, n, m, block_rows, block_k, float(keep_ratio), score_mode)


# ------------------------------------------------------------------ raw entry points

def crisp_keep_count(desc: LayerDesc):
    nblk, kkeep = C.c_int32(), C.c_int32()
    _check(load().crisp_keep_count(C.byref(desc), C.byref(nblk), C.byref(kkeep)), "crisp_keep_count")
    return nblk.value, kkeep.value


def crisp_mask_sizes(desc: LayerDesc):
    a, b = C.c_size_t(), C.c_size_t()
    _check(load().crisp_mask_sizes(C.byref(desc), C.byref(a), C.byref(b)), "crisp_mask_sizes")
    return a.value, b.value


def crisp_saliency_accumulate(d_grad, grad_dtype: int, ld_g: int, rows: int, k: int, d_acc, ld_acc: int, first: bool,
                              stream=None):
    _check(load().crisp_saliency_accumulate(_ptr(d_grad), grad_dtype, ld_g, rows, k, _ptr(d_acc), ld_acc,
                                            1 if first else 0, _stream(stream)), "crisp_saliency_accumulate")


def crisp_saliency_finish(d_acc, ld_acc: int, d_w, ld_w: int, rows: int, k: int, samples: int, d_saliency, ld_s: int,
                          stream=None):
    _check(load().crisp_saliency_finish(_ptr(d_acc), ld_acc, _ptr(d_w), ld_w, rows, k, samples, _ptr(d_saliency), ld_s,
                                        _stream(stream)), "crisp_saliency_finish")


def crisp_saliency_finish_max(d_acc, ld_acc: int, d_w, ld_w: int, rows: int, k: int, samples: int, d_saliency, ld_s: int,
                              d_mask_workspace, stream=None):
    _check(load().crisp_saliency_finish_max(_ptr(d_acc), ld_acc, _ptr(d_w), ld_w, rows, k, samples, _ptr(d_saliency),
                                            ld_s, _ptr(d_mask_workspace), _stream(stream)), "crisp_saliency_finish_max")


MASK_MAX_KNOWN = 1


def crisp_build_mask_ex(d_saliency, ld_s: int, desc: LayerDesc, d_mask_buf, d_workspace, flags: int, stream=None) -> int:
    out = C.c_void_p()
    _check(load().crisp_build_mask_ex(_ptr(d_saliency), ld_s, C.byref(desc), _ptr(d_mask_buf), _ptr(d_workspace),
                                      flags, _stream(stream), C.byref(out)), "crisp_build_mask_ex")
    return out.value


def crisp_mask_reselect(mask: int, kkeep: int, d_workspace, stream=None):
    _check(load().crisp_mask_reselect(mask, kkeep, _ptr(d_workspace), _stream(stream)), "crisp_mask_reselect")


def crisp_prune_fraction(kappa: float, n: int, m: int) -> float:
    out = C.c_double()
    _check(load().crisp_prune_fraction(float(kappa), n, m, C.byref(out)), "crisp_prune_fraction")
    return out.value


def crisp_keep_ratio_for_count(desc: LayerDesc, kkeep: int) -> float:
    out = C.c_double()
    _check(load().crisp_keep_ratio_for_count(C.byref(desc), kkeep, C.byref(out)), "crisp_keep_ratio_for_count")
    return out.value


def crisp_mask_scores(desc: LayerDesc, d_workspace):
    """-> (address of the [nrt, nblk] uint64 block scores, address of the max-key word) inside a workspace
    that crisp_build_mask has filled."""
    a, b = C.c_void_p(), C.c_void_p()
    _check(load().crisp_mask_scores(C.byref(desc), _ptr(d_workspace), C.byref(a), C.byref(b)), "crisp_mask_scores")
    return a.value, b.value


def make_rank_layers(layers):
    """layers: iterable of (d_scores, d_max_key, nrt, nblk, block_elems, min_keep) -> ctypes array."""
    layers = list(layers)
    arr = (RankLayer * len(layers))()
    for i, (sc, mk, nrt, nblk, be, keep) in enumerate(layers):
        arr[i] = RankLayer(_ptr(sc), _ptr(mk), nrt, nblk, be, keep, 0)
    return arr


def crisp_global_rank_sizes(rank_layers) -> int:
    out = C.c_size_t()
    _check(load().crisp_global_rank_sizes(len(rank_layers), rank_layers, C.byref(out)), "crisp_global_rank_sizes")
    return out.value


def crisp_global_rank(rank_layers, prune_fraction: float, d_workspace, d_kkeep, stream=None):
    _check(load().crisp_global_rank(len(rank_layers), rank_layers, float(prune_fraction), _ptr(d_workspace),
                                    _ptr(d_kkeep), _stream(stream)), "crisp_global_rank")


def crisp_build_mask(d_saliency, ld_s: int, desc: LayerDesc, d_mask_buf, d_workspace, stream=None) -> int:
    out = C.c_void_p()
    _check(load().crisp_build_mask(_ptr(d_saliency), ld_s, C.byref(desc), _ptr(d_mask_buf), _ptr(d_workspace),
                                   _stream(stream), C.byref(out)), "crisp_build_mask")
    return out.value


STATIC_SCRATCH_BYTES = 256 * 1024


def crisp_build_mask_static(d_saliency, ld_s: int, desc: LayerDesc, d_mask_buf, stream=None) -> int:
    """crisp_build_mask without a caller-provided workspace: the scratch is a fixed array inside
    the library, for callers that may not allocate device memory.  Layers whose workspace exceeds
    STATIC_SCRATCH_BYTES raise CrispError(BUFFER_TOO_SMALL).  Calls share that array, so they must
    not overlap on the GPU."""
    out = C.c_void_p()
    _check(load().crisp_build_mask_static(_ptr(d_saliency), ld_s, C.byref(desc), _ptr(d_mask_buf),
                                          _stream(stream), C.byref(out)), "crisp_build_mask_static")
    return out.value


def crisp_mask_info(mask: int):
    d, a, b, c = LayerDesc(), C.c_int32(), C.c_int32(), C.c_int32()
    _check(load().crisp_mask_info(mask, C.byref(d), C.byref(a), C.byref(b), C.byref(c)), "crisp_mask_info")
    return d, a.value, b.value, c.value


def crisp_mask_export(mask: int, h_blk_col, h_nm_bits, stream=None):
    _check(load().crisp_mask_export(mask, _ptr(h_blk_col), _ptr(h_nm_bits), _stream(stream)), "crisp_mask_export")


def crisp_encode_sizes(mask: int):
    a, b = C.c_size_t(), C.c_size_t()
    _check(load().crisp_encode_sizes(mask, C.byref(a), C.byref(b)), "crisp_encode_sizes")
    return a.value, b.value


def crisp_encode(d_w, ld_w: int, mask: int, d_canonical, d_exec, stream=None) -> int:
    out = C.c_void_p()
    _check(load().crisp_encode(_ptr(d_w), ld_w, mask, _ptr(d_canonical), _ptr(d_exec), _stream(stream),
                               C.byref(out)), "crisp_encode")
    return out.value


def crisp_encoded_counts(handle: int):
    a, b, c = C.c_int64(), C.c_int64(), C.c_int64()
    _check(load().crisp_encoded_counts(handle, C.byref(a), C.byref(b), C.byref(c)), "crisp_encoded_counts")
    return a.value, b.value, c.value


def crisp_export(handle: int, h_blk_col, h_vals, h_idx, stream=None):
    _check(load().crisp_export(handle, _ptr(h_blk_col), _ptr(h_vals), _ptr(h_idx), _stream(stream)), "crisp_export")


def crisp_decode(handle: int, d_w_dense, ld: int, stream=None):
    _check(load().crisp_decode(handle, _ptr(d_w_dense), ld, _stream(stream)), "crisp_decode")


def crisp_spmm(handle: int, d_x, ldx: int, ncols: int, d_y, ldy: int, y_dtype: int = 0, stream=None):
    _check(load().crisp_spmm(handle, _ptr(d_x), ldx, ncols, _ptr(d_y), ldy, y_dtype, _stream(stream)), "crisp_spmm")


def crisp_spmm_conv(handle: int, d_act_nhwc, conv: ConvDesc, d_y, ldy: int, y_dtype: int = 0, stream=None):
    _check(load().crisp_spmm_conv(handle, _ptr(d_act_nhwc), C.byref(conv), _ptr(d_y), ldy, y_dtype, _stream(stream)),
           "crisp_spmm_conv")


def crisp_set_epilogue(handle: int, d_bias_f32, relu: int):
    _check(load().crisp_set_epilogue(handle, _ptr(d_bias_f32), int(relu)), "crisp_set_epilogue")


def crisp_set_path(handle: int, path: int):
    _check(load().crisp_set_path(handle, path), "crisp_set_path")


def crisp_device_status(handle: int, stream=None) -> int:
    s = C.c_int32()
    _check(load().crisp_device_status(handle, _stream(stream), C.byref(s)), "crisp_device_status")
    return s.value


def crisp_last_launch(handle: int) -> dict:
    """Kernel family (`path`) and tile configuration of the last product launched through the handle."""
    info = LaunchInfo()
    _check(load().crisp_last_launch(handle, C.byref(info)), "crisp_last_launch")
    return info.as_dict()


def crisp_set_tuning(handle: int, tile_boxes: int = 0, wait_limit_cycles: int = 0, skip_fill: int = -1):
    _check(load().crisp_set_tuning(handle, tile_boxes, wait_limit_cycles, skip_fill), "crisp_set_tuning")


def crisp_set_stage_blocks(handle: int, max_blocks: int = 0):
    """Most kept blocks one pipeline stage may take (1, 2, 4; 0 = chosen by the library)."""
    _check(load().crisp_set_stage_blocks(handle, max_blocks), "crisp_set_stage_blocks")


def crisp_reset_status(handle: int, stream=None):
    _check(load().crisp_reset_status(handle, _stream(stream)), "crisp_reset_status")


def crisp_bytes_model(handle: int, ncols: int, y_dtype: int = 0) -> dict:
    b = BytesModel()
    _check(load().crisp_bytes_model(handle, ncols, y_dtype, C.byref(b)), "crisp_bytes_model")
    return b.as_dict()


def crisp_mask_destroy(mask: int):
    if mask:
        load().crisp_mask_destroy(mask)


def crisp_destroy(handle: int):
    if handle:
        load().crisp_destroy(handle)


# -------------------------------------------------- buffer-owning convenience wrapper

class HybridLayer:
    """Owns the device buffers of one pruned layer and forwards to the C ABI.

    ``build_mask`` -> ``encode`` -> ``spmm`` mirror crisp_build_mask / crisp_encode /
    crisp_spmm; tensors are torch CUDA tensors (bf16 tensors or their int16/uint16 views).
    """

    def __init__(self, rows, k, n, m, block_rows, block_k, keep_ratio, score_mode=0, device="cuda"):
        import torch
        self.torch = torch
        self.device = torch.device(device)
        self.desc = make_desc(rows, k, n, m, block_rows, block_k, keep_ratio, score_mode)
        self.nblk, self.kkeep = crisp_keep_count(self.desc)
        self.nrt = (rows + block_rows - 1) // block_rows
        mask_bytes, ws_bytes = crisp_mask_sizes(self.desc)
        self.mask_buf = torch.empty(mask_bytes, dtype=torch.uint8, device=self.device)
        self.workspace = torch.empty(ws_bytes, dtype=torch.uint8, device=self.device)
        self.mask = 0
        self.handle = 0
        self.canonical_buf = None
        self.exec_buf = None

    def build_mask(self, saliency, stream=None):
        assert saliency.is_cuda and saliency.dtype == self.torch.float32 and saliency.stride(1) == 1
        crisp_mask_destroy(self.mask)
        self.mask = crisp_build_mask(saliency, saliency.stride(0), self.desc, self.mask_buf, self.workspace, stream)
        return self

    def rank_layer(self, min_keep=0):
        """This layer's entry for crisp_global_rank (valid after build_mask, until the workspace is reused)."""
        sc, mk = crisp_mask_scores(self.desc, self.workspace)
        return (sc, mk, self.nrt, self.nblk, self.desc.block_rows * self.desc.block_k, min_keep)

    def set_kkeep(self, kkeep: int):
        """Keep ratio that makes the next build_mask keep exactly `kkeep` blocks per row tile."""
        self.desc.keep_ratio = crisp_keep_ratio_for_count(self.desc, kkeep)
        self.nblk, self.kkeep = crisp_keep_count(self.desc)
        assert self.kkeep == kkeep
        mask_bytes, ws_bytes = crisp_mask_sizes(self.desc)
        if self.mask_buf.numel() < mask_bytes:
            self.mask_buf = self.torch.empty(mask_bytes, dtype=self.torch.uint8, device=self.device)
        return self

    def build_mask_max_known(self, saliency, stream=None):
        """build_mask when the workspace already holds the layer maximum (crisp_saliency_finish_max wrote it)."""
        assert saliency.is_cuda and saliency.dtype == self.torch.float32 and saliency.stride(1) == 1
        crisp_mask_destroy(self.mask)
        self.mask = crisp_build_mask_ex(saliency, saliency.stride(0), self.desc, self.mask_buf, self.workspace,
                                        MASK_MAX_KNOWN, stream)
        return self

    def reselect(self, kkeep: int, stream=None):
        """Keep only the `kkeep` best blocks per row tile of the mask just built (no pass over the saliency)."""
        crisp_mask_reselect(self.mask, kkeep, self.workspace, stream)
        self.desc.keep_ratio = crisp_keep_ratio_for_count(self.desc, kkeep)
        self.kkeep = kkeep
        return self

    def export_mask(self, stream=None):
        import numpy as np
        wpr = self.nblk * self.desc.block_k // 32
        blk_col = np.zeros((self.nrt, self.kkeep), dtype=np.int32)
        nm_bits = np.zeros((self.nrt * self.desc.block_rows, wpr), dtype=np.uint32)
        crisp_mask_export(self.mask, blk_col, nm_bits, stream)
        return blk_col, nm_bits

    def encode(self, w, stream=None):
        assert w.is_cuda and w.element_size() == 2 and w.stride(1) == 1
        torch = self.torch
        cbytes, ebytes = crisp_encode_sizes(self.mask)
        if self.canonical_buf is None or self.canonical_buf.numel() < cbytes:
            self.canonical_buf = torch.empty(cbytes, dtype=torch.uint8, device=self.device)
        if self.exec_buf is None or self.exec_buf.numel() < ebytes:
            self.exec_buf = torch.empty(ebytes, dtype=torch.uint8, device=self.device)
        crisp_destroy(self.handle)
        self.handle = crisp_encode(w, w.stride(0), self.mask, self.canonical_buf, self.exec_buf, stream)
        return self

    def export(self, stream=None):
        import numpy as np
        nb, nv, nw = crisp_encoded_counts(self.handle)
        blk_col = np.zeros(nb, dtype=np.int32)
        vals = np.zeros(nv, dtype=np.uint16)
        idx = np.zeros(nw, dtype=np.uint32)
        crisp_export(self.handle, blk_col, vals, idx, stream)
        return blk_col.reshape(self.nrt, self.kkeep), vals, idx

    def decode(self, stream=None):
        torch = self.torch
        w = torch.empty((self.desc.rows, self.desc.k), dtype=torch.bfloat16, device=self.device)
        crisp_decode(self.handle, w, w.stride(0), stream)
        return w

    def spmm(self, x, y=None, y_dtype=0, stream=None):
        torch = self.torch
        assert x.is_cuda and x.element_size() == 2 and x.stride(1) == 1 and x.shape[0] == self.desc.k
        ncols = x.shape[1]
        if y is None:
            y = torch.empty((self.desc.rows, ncols), dtype=torch.float32 if y_dtype else torch.bfloat16,
                            device=self.device)
        crisp_spmm(self.handle, x, x.stride(0), ncols, y, y.stride(0), y_dtype, stream)
        return y

    def spmm_conv(self, act_nhwc, kernel_h, kernel_w, pad, y=None, y_dtype=0, stream=None, nhwc_out=False):
        """Convolution (stride 1) of an NHWC bf16 activation with this layer's weights, without an X matrix.
        nhwc_out: Y is [batch, ho, wo, rows] (the next convolution's activation) instead of [rows, batch*ho*wo]."""
        torch = self.torch
        assert act_nhwc.is_cuda and act_nhwc.element_size() == 2 and act_nhwc.is_contiguous() and act_nhwc.dim() == 4
        b, h, w, c = act_nhwc.shape
        ho, wo = h + 2 * pad - kernel_h + 1, w + 2 * pad - kernel_w + 1
        dt = torch.float32 if y_dtype else torch.bfloat16
        if y is None:
            y = torch.empty((b, ho, wo, self.desc.rows) if nhwc_out else (self.desc.rows, b * ho * wo), dtype=dt,
                            device=self.device)
        ldy = y.stride(2) if nhwc_out else y.stride(0)
        crisp_spmm_conv(self.handle, act_nhwc, ConvDesc(b, h, w, c, kernel_h, kernel_w, pad, 1 if nhwc_out else 0), y, ldy,
                        y_dtype, stream)
        return y

    def set_epilogue(self, bias=None, relu=False):
        """Y = act(W X + bias) for later products; `bias` is an fp32 CUDA tensor [rows] that this object keeps."""
        if bias is not None:
            assert bias.is_cuda and bias.dtype == self.torch.float32 and bias.numel() == self.desc.rows
        self._bias = bias
        crisp_set_epilogue(self.handle, bias, 1 if relu else 0)
        return self

    def set_path(self, path: int):
        crisp_set_path(self.handle, path)

    def device_status(self, stream=None) -> int:
        return crisp_device_status(self.handle, stream)

    def last_launch(self) -> dict:
        return crisp_last_launch(self.handle)

    def set_tuning(self, tile_boxes=0, wait_limit_cycles=0, skip_fill=-1):
        crisp_set_tuning(self.handle, tile_boxes, wait_limit_cycles, skip_fill)
        return self

    def set_stage_blocks(self, max_blocks=0):
        crisp_set_stage_blocks(self.handle, max_blocks)
        return self

    def reset_status(self, stream=None):
        crisp_reset_status(self.handle, stream)

    def bytes_model(self, ncols, y_dtype=0):
        return crisp_bytes_model(self.handle, ncols, y_dtype)

    def close(self):
        crisp_destroy(self.handle)
        crisp_mask_destroy(self.mask)
        self.handle = 0
        self.mask = 0

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class PruningNetwork:
    """One pruning iteration of Algorithm 1 over all layers of a network, without the fine-tuning that follows it:

        per layer   saliency of Eq. 1 from the caller's gradients   crisp_saliency_accumulate / _finish_max
        per layer   N:M step and block scores (keep ratio 1)        crisp_build_mask_ex(MAX_KNOWN)
        network     rank-column sums, global order, selection       crisp_global_rank
        per layer   keep the selected number of blocks              crisp_mask_reselect
        per layer   compress                                        crisp_encode

    This class only owns buffers and issues those calls in that order; every number is computed by the library.
    `shapes` is a list of (rows, k); the pattern (n:m, block shape) is shared by the layers.
    """

    def __init__(self, shapes, n, m, block_rows, block_k, min_keep=1, device="cuda"):
        import torch
        self.torch = torch
        self.device = torch.device(device)
        self.n, self.m = n, m
        self.min_keep = min_keep
        self.layers = [HybridLayer(r, k, n, m, block_rows, block_k, 1.0, device=device) for (r, k) in shapes]
        self.acc = [torch.empty((r, k), dtype=torch.float32, device=self.device) for (r, k) in shapes]
        self.sal = [torch.empty((r, k), dtype=torch.float32, device=self.device) for (r, k) in shapes]
        self.rank_arr = make_rank_layers([L.rank_layer(min_keep) for L in self.layers])
        self.rank_ws = torch.empty(crisp_global_rank_sizes(self.rank_arr), dtype=torch.uint8, device=self.device)
        self.d_kkeep = torch.zeros(len(shapes), dtype=torch.int32, device=self.device)

    def step(self, weights, grads, kappa, stream=None):
        """weights[l]: bf16 CUDA tensor [rows, k]; grads[l]: list of H gradient tensors (bf16 or fp32) of that shape;
        kappa: overall sparsity target of this iteration.  Returns the kept-block count of every layer; the layers'
        masks and handles (self.layers[l]) hold the result."""
        torch = self.torch
        for L, w, gs, acc, s in zip(self.layers, weights, grads, self.acc, self.sal):
            rows, k = L.desc.rows, L.desc.k
            for i, g in enumerate(gs):
                crisp_saliency_accumulate(g, 0 if g.dtype == torch.bfloat16 else 1, g.stride(0), rows, k, acc, k, i == 0,
                                          stream)
            crisp_saliency_finish_max(acc, k, w, w.stride(0), rows, k, len(gs), s, k, L.workspace, stream)
            L.desc.keep_ratio = 1.0
            L.nblk, L.kkeep = crisp_keep_count(L.desc)
            L.build_mask_max_known(s, stream)
        crisp_global_rank(self.rank_arr, crisp_prune_fraction(kappa, self.n, self.m), self.rank_ws, self.d_kkeep, stream)
        if stream is None:
            kk = self.d_kkeep.cpu().tolist()
        else:
            with torch.cuda.stream(stream):
                kk = self.d_kkeep.cpu().tolist()
        for L, w, c in zip(self.layers, weights, kk):
            L.reselect(c, stream)
            L.encode(w, stream)
        return kk

    def close(self):
        for L in self.layers:
            L.close()
