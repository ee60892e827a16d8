"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
header declares, and rejects bad arguments before touching the device."""
import ctypes as C
import os
import re

import pytest

from paper_2311_14272_b200 import binding as B
from paper_2311_14272_b200 import build as build_mod

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build_mod.build()
    return B.load()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "crisp.h")).read()
    return sorted(set(re.findall(r"CRISP_API[^;(]*?\b(crisp_\w+)\s*\(", text)))


def test_header_declares_the_three_named_calls():
    names = declared_symbols()
    for must in ("crisp_build_mask", "crisp_encode", "crisp_spmm"):
        assert must in names
    assert len(names) >= 15


def test_library_exports_every_declared_symbol(lib):
    for name in declared_symbols():
        assert hasattr(lib, name), name
    for name in declared_symbols():
        assert hasattr(B, name), f"binding lacks {name}"


def test_keep_count_and_sizes_on_host(lib):
    d = B.make_desc(256, 1024, 2, 4, 32, 64, 0.5)
    assert B.crisp_keep_count(d) == (16, 8)
    mask_bytes, ws_bytes = B.crisp_mask_sizes(d)
    assert mask_bytes >= 8 * 8 * 4 + 256 * 32 * 4 and mask_bytes % 256 == 0
    assert ws_bytes >= 8 * 16 * 8
    assert B.crisp_keep_count(B.make_desc(64, 27, 2, 4, 64, 64, 0.4)) == (1, 0)
    assert B.crisp_keep_count(B.make_desc(64, 160, 2, 8, 32, 32, 0.5)) == (5, 3)


@pytest.mark.parametrize("kw,code", [
    (dict(rows=0), B.BAD_SHAPE), (dict(k=-4), B.BAD_SHAPE), (dict(m=6), B.UNSUPPORTED),
    (dict(n=5), B.INVALID_ARG), (dict(n=0), B.INVALID_ARG), (dict(block_rows=48), B.UNSUPPORTED),
    (dict(block_k=16), B.UNSUPPORTED), (dict(block_k=160), B.UNSUPPORTED),
    (dict(keep_ratio=1.5), B.INVALID_ARG), (dict(keep_ratio=float("nan")), B.INVALID_ARG),
    (dict(score_mode=2), B.INVALID_ARG),
])
def test_bad_descriptors_are_rejected(lib, kw, code):
    base = dict(rows=64, k=128, n=2, m=4, block_rows=32, block_k=32, keep_ratio=0.5, score_mode=0)
    base.update(kw)
    with pytest.raises(B.CrispError) as ei:
        B.crisp_keep_count(B.make_desc(**base))
    assert ei.value.code == code


def test_null_and_misaligned_pointers_are_rejected_before_any_launch(lib):
    d = B.make_desc(64, 128, 2, 4, 32, 32, 0.5)
    out = C.c_void_p()
    assert lib.crisp_build_mask(None, 128, C.byref(d), 256, 256, None, C.byref(out)) == B.INVALID_ARG
    assert lib.crisp_build_mask(4096, 128, C.byref(d), 4096 + 8, 4096, None, C.byref(out)) == B.INVALID_ARG
    assert lib.crisp_build_mask(4096, 64, C.byref(d), 4096, 4096, None, C.byref(out)) == B.BAD_SHAPE
    assert out.value is None
    assert lib.crisp_encode(None, 128, None, None, None, None, C.byref(out)) == B.INVALID_ARG
    assert lib.crisp_spmm(None, None, 1, 1, None, 1, 0, None) == B.INVALID_ARG
    assert lib.crisp_device_status(None, None, None) == B.INVALID_ARG
    assert B.status_string(B.TIMEOUT) and B.status_string(0) == "ok"


def test_missing_library_fails_loudly(tmp_path):
    with pytest.raises(FileNotFoundError):
        B.load(str(tmp_path / "libcrisp.so"))


def test_block_count_limit_per_row_tile(lib):
    """Up to 4096 k-blocks per row tile are accepted (the longest row the selection kernels hold on chip),
    one more is refused on the host, before any launch."""
    ok = B.make_desc(32, 4096 * 32, 2, 4, 32, 32, 0.5)
    assert B.crisp_keep_count(ok) == (4096, 2048)
    B.crisp_mask_sizes(ok)
    with pytest.raises(B.CrispError) as ei:
        B.crisp_keep_count(B.make_desc(32, 4097 * 32, 2, 4, 32, 32, 0.5))
    assert ei.value.code == B.UNSUPPORTED


def test_handle_queries_reject_null(lib):
    info = B.LaunchInfo()
    assert lib.crisp_last_launch(None, C.byref(info)) == B.INVALID_ARG
    assert lib.crisp_set_tuning(None, 0, 0, -1) == B.INVALID_ARG
    assert lib.crisp_set_stage_blocks(None, 0) == B.INVALID_ARG
    assert lib.crisp_reset_status(None, None) == B.INVALID_ARG
