"""The entry point that allocates nothing (waveal_bitmap_to_csr_noalloc), collected last.

Some users of this library cannot allocate device memory at the point where they call it:
a plug-in inside a serving engine receives tensors from a memory plan fixed up front, and a
cudaMalloc in the middle of a denoising loop would synchronise the whole device.  For them
the bitmap -> index-list conversion exists in a form whose scratch is a fixed array inside
the library.  The GPU test drives it through the C ABI with every buffer pre-allocated and
compares it with the ordinary entry point, bit for bit, on two calls in a row with different
masks (the shared scratch keeps the first call's contents when the second starts)."""
import ctypes

import numpy as np
import pytest

from paper_2609_34814_b200 import binding as wb
from paper_2609_34814_b200 import build as wbuild
from paper_2609_34814_b200 import inputs as I


def test_noalloc_rejects_oversized_problem_on_the_host():
    wbuild.build()
    lib = wb.load()
    limit = wb.noalloc_max_rows()
    assert limit == (1 << 20) // 4 - 1
    heads, rows = 64, limit // 64 + 1               # heads * rows just beyond the limit
    st = lib.waveal_bitmap_to_csr_noalloc(heads, rows, 8, 0x1000, 0x2000, None, 0, None)
    assert st == wb.ERR_UNSUPPORTED
    assert "built-in scratch" in wb.last_error() and "waveal_bitmap_to_csr" in wb.last_error()
    assert lib.waveal_bitmap_to_csr_noalloc(0, 4, 4, 0x1000, 0x2000, None, 0, None) == wb.ERR_INVALID_ARG


@pytest.mark.gpu
def test_noalloc_matches_the_workspace_entry_point_twice_in_a_row():
    import torch
    cases = [(I.scaled_config(I.CONFIGS["wan720p"], frames=6), [0, 1, 2, 3]),    # 169 blocks, 4 heads
             (I.scaled_config(I.CONFIGS["long720p"], frames=3), [5, 6])]          # 85 blocks, 2 heads: smaller, other data
    prepared = []
    for cfg, heads in cases:
        masks = [I.make_mask(cfg, h) for h in heads]
        bitmap = torch.from_numpy(np.stack([I.mask_to_bitmap(m) for m in masks]).view(np.int64)).cuda()
        ref_ptr, ref_idx = wb.bitmap_to_csr(bitmap, cfg.n_blocks)              # existing entry point
        # the caller of the no-allocation form owns and pre-sizes everything
        nnz = int(sum(m.sum() for m in masks))
        ptr = torch.full((len(heads) * cfg.n_blocks + 1,), -1, dtype=torch.int32, device="cuda")
        idx = torch.full((nnz,), -1, dtype=torch.int32, device="cuda")
        prepared.append((cfg, masks, bitmap, ref_ptr, ref_idx, ptr, idx))
    torch.cuda.synchronize()
    before = torch.cuda.memory_allocated()
    for cfg, masks, bitmap, ref_ptr, ref_idx, ptr, idx in prepared:             # two calls in a row
        wb.bitmap_to_csr_noalloc(bitmap, cfg.n_blocks, ptr, idx)
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated() == before                               # nothing came from torch either
    for cfg, masks, bitmap, ref_ptr, ref_idx, ptr, idx in prepared:
        assert torch.equal(ptr, ref_ptr) and torch.equal(idx, ref_idx)
        host_ptr, host_idx = I.masks_to_csr(masks)
        assert np.array_equal(ptr.cpu().numpy(), host_ptr) and np.array_equal(idx.cpu().numpy(), host_idx)


@pytest.mark.gpu
def test_noalloc_at_exactly_the_largest_accepted_size():
    """heads * n_q_blocks == waveal_noalloc_max_rows(): the scan then writes its last partial sum
    from the last int of the built-in array."""
    import torch
    heads, rows, cols = 3, 87381, 8
    assert heads * rows == wb.noalloc_max_rows()
    rng = np.random.default_rng(11)
    mask = rng.random((heads, rows, cols)) < 0.4
    words = np.zeros((heads, rows, 1), dtype=np.uint64)
    for j in range(cols):
        words[:, :, 0] |= mask[:, :, j].astype(np.uint64) << np.uint64(j)
    bitmap = torch.from_numpy(words.view(np.int64)).cuda()
    counts = mask.reshape(-1, cols).sum(axis=1)
    exp_ptr = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
    exp_idx = np.nonzero(mask.reshape(-1, cols))[1].astype(np.int32)
    ptr = torch.full((heads * rows + 1,), -1, dtype=torch.int32, device="cuda")
    idx = torch.full((int(exp_ptr[-1]),), -1, dtype=torch.int32, device="cuda")
    wb.bitmap_to_csr_noalloc(bitmap, cols, ptr, idx)
    torch.cuda.synchronize()
    assert np.array_equal(ptr.cpu().numpy(), exp_ptr) and np.array_equal(idx.cpu().numpy(), exp_idx)
