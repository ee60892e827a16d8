"""crisp_build_mask_static: the mask projection for callers that are not allowed to allocate
device memory when they call (plug-ins inside a framework that owns the GPU's memory, loops that
must stay allocation-free after start-up).  Its scratch is a fixed array inside the library, so
the test checks what a user relies on: the result is bit-identical to crisp_build_mask (and to the
CPU oracle's mask of the same saliency), a second call right after the first is not disturbed by what
the first left in the shared array, and a layer too large for the array is refused instead of
overrunning it."""
import ctypes as C

import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def _mask_via(B, torch, s_dev, desc, static):
    nblk, kkeep = B.crisp_keep_count(desc)
    nrt = (desc.rows + desc.block_rows - 1) // desc.block_rows
    mask_bytes, ws_bytes = B.crisp_mask_sizes(desc)
    mask_buf = torch.empty(mask_bytes, dtype=torch.uint8, device="cuda")
    if static:
        mask = B.crisp_build_mask_static(s_dev, s_dev.stride(0), desc, mask_buf)
    else:
        ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
        mask = B.crisp_build_mask(s_dev, s_dev.stride(0), desc, mask_buf, ws)
    blk_col = np.zeros((nrt, kkeep), dtype=np.int32)
    nm_bits = np.zeros((nrt * desc.block_rows, nblk * desc.block_k // 32), dtype=np.uint32)
    B.crisp_mask_export(mask, blk_col, nm_bits)
    B.crisp_mask_destroy(mask)
    return blk_col, nm_bits


def test_static_scratch_mask_matches_the_workspace_version_twice_in_a_row():
    import torch
    from paper_2311_14272_b200 import binding as B
    B.load()
    rng = np.random.default_rng(2311)
    # the second layer is smaller and has fewer blocks than the first: anything the first call
    # left behind in the shared scratch would corrupt its scores if it were not cleared
    layers = [(512, 1024, 2, 4, 64, 64, 0.5), (96, 200, 1, 8, 32, 32, 0.4)]
    for rows, k, n, m, bm, bk, keep in layers:
        s = (rng.standard_normal((rows, k)) * 3.0).astype(np.float32)
        s_dev = torch.from_numpy(s).cuda()
        desc = B.make_desc(rows, k, n, m, bm, bk, keep)
        want_cols, want_bits = _mask_via(B, torch, s_dev, desc, static=False)
        got_cols, got_bits = _mask_via(B, torch, s_dev, desc, static=True)
        assert np.array_equal(got_cols, want_cols)        # integer outputs: compared bit for bit,
        assert np.array_equal(got_bits, want_bits)        # the same bar as the other mask tests
        assert want_bits.any()
        import oracle
        mk = oracle.build_mask(s, n, m, bm, bk, keep)         # and both agree with the definition
        assert np.array_equal(got_cols, mk.blk_col) and np.array_equal(got_bits, mk.nm_bits)
    torch.cuda.synchronize()


def test_static_scratch_refuses_layers_beyond_its_size():
    import torch
    from paper_2311_14272_b200 import binding as B
    B.load()
    # 128 row tiles x 512 k-blocks = 65536 scores = 512 KiB of workspace > the 256 KiB array
    desc = B.make_desc(4096, 16384, 2, 4, 32, 32, 0.5)
    _, ws_bytes = B.crisp_mask_sizes(desc)
    assert ws_bytes > B.STATIC_SCRATCH_BYTES
    dummy = torch.zeros(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.CrispError) as ei:
        B.crisp_build_mask_static(dummy, 16384, desc, dummy)     # refused before any launch
    assert ei.value.code == B.BUFFER_TOO_SMALL
