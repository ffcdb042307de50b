"""GPU parity of the planning kernels against the CPU oracle (through the C ABI)."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import waveal_oracle as wo
from paper_2609_34814_b200 import binding as wb
from paper_2609_34814_b200 import inputs as I
from gpu_util import Workload

pytestmark = pytest.mark.gpu


def _np(t):
    return t.cpu().numpy()


def _bitmap_dev(masks):
    bm = np.stack([I.mask_to_bitmap(m) for m in masks])
    return torch.from_numpy(bm.view(np.int64)).cuda()


def _check_plan(masks, heads, wave, iters, seed, mode, res, guard=None, ov_tol=0.02, ring_cut=False):
    """Integer outputs bit-exact; Stage 1 by equality or by overlap score; Stage 2 bit-exact
    given the GPU's own Stage-1 order."""
    exact = 0
    for li, h in enumerate(heads):
        mk = masks[li]
        ref = wo.plan_head(mk, wave, iters, seed, li, mode=mode, guard=guard, ring_cut=ring_cut)
        assert np.array_equal(_np(res.row_nnz[li]), ref["row_nnz"])
        assert np.array_equal(_np(res.col_count[li]), ref["col_count"])
        st = wo.guard_stats(mk, wave)
        assert _np(res.stats[li]).tolist()[:3] == [st["nnz"], st["ov_nat"], st["pair2"]]
        assert int(res.skip_flags[li]) == ref["flags"]
        order = _np(res.row_order[li]).astype(np.int64)
        order1 = _np(res.order1[li]).astype(np.int64)
        m_b = mk.shape[0]
        assert np.array_equal(np.sort(order), np.arange(m_b))          # P P^T = I
        assert np.array_equal(np.sort(order1), np.arange(m_b))
        if ref["flags"] & wo.FLAG_SKIPPED:
            assert np.array_equal(order, np.arange(m_b))
            continue
        # Stage 2 given the GPU's Stage-1 order: bit-exact
        if mode == wo.MODE_STAGE1_ONLY:
            assert np.array_equal(order, order1)
        else:
            assert np.array_equal(order, wo.stage2_order(order1, ref["row_nnz"], wave))
            for lo in range(0, m_b, wave):                              # within-wave descending counts
                n = ref["row_nnz"][order[lo:lo + wave]]
                assert (n[:-1] >= n[1:]).all()
        # Stage 1: identical permutation, else K/V-overlap score within 2 %
        if np.array_equal(order1, ref["order1"]):
            exact += 1
        else:
            a = wo.scores(mk, order, wave)["Ov"]
            b = wo.scores(mk, ref["row_order"], wave)["Ov"]
            assert abs(a / max(b, 1) - 1.0) <= ov_tol, (h, a, b)
        if mode != wo.MODE_STAGE2_ONLY:
            u = _np(res.embedding[li])
            assert abs(np.abs(u.sum(axis=0)).max()) < 1e-8              # retained directions orthogonal to 1
    return exact


CASES = [
    ("tiny", None, None, 16),
    ("wan480p", 8, 3, 37),        # 98 blocks (ragged), odd wave size
    ("wan480p", None, 4, 148),
    ("wan720p", None, 6, 148),
    ("ltxmixed", None, 3, 148),
    ("long720p", None, 2, 148),
]


@pytest.mark.parametrize("name,frames,heads,wave", CASES)
def test_plan_parity(name, frames, heads, wave):
    cfg = I.CONFIGS[name]
    if frames:
        cfg = I.scaled_config(cfg, frames=frames)
    hs = list(range(cfg.heads if heads is None else heads))
    masks = [I.make_mask(cfg, h) for h in hs]
    d = wb.plan_desc_default(heads=len(hs), n_q_blocks=cfg.n_blocks, n_kv_blocks=cfg.n_blocks, wave_size=wave,
                             mode=wb.FORCE_REORDER, seed=cfg.plan_seed)
    res = wb.plan_bitmap(d, _bitmap_dev(masks), debug=True)
    torch.cuda.synchronize()
    assert res.dev_status.tolist() == [0, 0, 0, 0]
    exact = _check_plan(masks, hs, wave, d.svd_iters, cfg.plan_seed, wo.MODE_FORCE_REORDER, res)
    assert exact >= 1          # fp64 on both sides: the permutation itself normally coincides


@pytest.mark.parametrize("mode", [wb.FORCE_REORDER, wb.STAGE1_ONLY])
def test_ring_cut_variant_matches_the_oracle(mode):
    """Stage-1 variant: ring opened at the largest angular gap.  Same checks as the plain plan, plus:
    the GPU's order1 is a rotation of the order1 it produces without the flag."""
    cfg = I.scaled_config(I.CONFIGS["long720p"], frames=12)
    hs = [0, 1, 2, 3]
    masks = [I.make_mask(cfg, h) for h in hs]
    bm = _bitmap_dev(masks)
    d = wb.plan_desc_default(heads=4, n_q_blocks=cfg.n_blocks, n_kv_blocks=cfg.n_blocks, wave_size=32, mode=mode,
                             seed=7, svd_iters=6)
    plain = wb.plan_bitmap(d, bm, debug=True)
    d.mode = mode | wb.RING_CUT_LARGEST_GAP
    res = wb.plan_bitmap(d, bm, debug=True)
    torch.cuda.synchronize()
    exact = _check_plan(masks, hs, 32, 6, 7, mode, res, ring_cut=True)
    assert exact >= 1
    m = cfg.n_blocks
    for li in range(4):
        a, b = _np(plain.order1[li]).tolist(), _np(res.order1[li]).tolist()
        assert any((a + a)[i:i + m] == b for i in range(m))
        ang = np.arctan2(_np(res.embedding[li])[:, 1], _np(res.embedding[li])[:, 0])
        assert b == wo.cut_ring_at_largest_gap(np.array(a), ang).tolist()


@pytest.mark.parametrize("mode", [wb.STAGE1_ONLY, wb.STAGE2_ONLY, wb.FORCE_NATURAL, wb.AUTO])
def test_plan_modes(mode):
    cfg = I.scaled_config(I.CONFIGS["long720p"], frames=12)
    hs = [0, 1, 2]
    masks = [I.make_mask(cfg, h) for h in hs]
    d = wb.plan_desc_default(heads=3, n_q_blocks=cfg.n_blocks, n_kv_blocks=cfg.n_blocks, wave_size=32, mode=mode,
                             seed=7, svd_iters=6)
    res = wb.plan_bitmap(d, _bitmap_dev(masks), debug=True)
    torch.cuda.synchronize()
    _check_plan(masks, hs, 32, 6, 7, mode, res)


def test_guard_decisions_per_head():
    # heads of different structure in one call: random, already-local, too sparse
    m = 96
    rnd = I.random_mask(m, m, 0.2, 5)
    loc = np.zeros((m, m), dtype=bool)
    for l in range(m // 8):
        loc[l * 8:(l + 1) * 8, (l * 8) % (m - 12):(l * 8) % (m - 12) + 12] = True
    sparse = np.eye(m, dtype=bool)
    sparse[0, :] = False
    sparse[0, 0] = True
    masks = [rnd, loc, sparse]
    guard = dict(wo.DEFAULT_GUARD, kv_bytes_per_head=2000, l2_bytes=3000, min_density_ppm=20000)
    d = wb.plan_desc_default(heads=3, n_q_blocks=m, n_kv_blocks=m, wave_size=8, mode=wb.AUTO, seed=3,
                             kv_bytes_per_head=2000, l2_bytes=3000, min_density_ppm=20000)
    res = wb.plan_bitmap(d, _bitmap_dev(masks), debug=True)
    torch.cuda.synchronize()
    flags = _np(res.skip_flags).tolist()
    assert flags[0] == 0
    assert flags[1] == wo.FLAG_ALREADY_LOCAL | wo.FLAG_SKIPPED
    assert flags[2] & wo.FLAG_TOO_SPARSE and flags[2] & wo.FLAG_SKIPPED
    _check_plan(masks, [0, 1, 2], 8, d.svd_iters, 3, wo.MODE_AUTO, res, guard=guard)
    # short-sequence case: the head's K+V fit the budget -> every head skipped
    d.kv_bytes_per_head, d.l2_bytes = 700, 3000
    res = wb.plan_bitmap(d, _bitmap_dev(masks), debug=True)
    torch.cuda.synchronize()
    assert all(f & wo.FLAG_SHORT_SEQ and f & wo.FLAG_SKIPPED for f in _np(res.skip_flags).tolist())
    assert np.array_equal(_np(res.row_order[0]), np.arange(m))


def test_plan_csr_entry_equals_bitmap_entry_and_bitmap_to_csr():
    cfg = I.scaled_config(I.CONFIGS["wan720p"], frames=5)
    w = Workload(cfg, heads=[0, 1, 2], need_tensors=False)
    d = wb.plan_desc_default(heads=3, n_q_blocks=cfg.n_blocks, n_kv_blocks=cfg.n_blocks, wave_size=20,
                             mode=wb.FORCE_REORDER, seed=11)
    a = wb.plan_bitmap(d, w.bitmap, debug=True)
    b = wb.plan_csr(d, w.ptr, w.idx, debug=True)
    torch.cuda.synchronize()
    for k in ("row_order", "row_nnz", "col_count", "order1", "stats", "skip_flags"):
        assert torch.equal(getattr(a, k), getattr(b, k)), k
    assert torch.equal(a.embedding, b.embedding)        # deterministic reductions: bit-identical
    ptr, idx = wb.bitmap_to_csr(w.bitmap, cfg.n_blocks)
    torch.cuda.synchronize()
    assert np.array_equal(_np(ptr), w.ptr_np) and np.array_equal(_np(idx), w.idx_np)
    # repeated call: bit-identical plan
    c = wb.plan_bitmap(d, w.bitmap, debug=True)
    torch.cuda.synchronize()
    assert torch.equal(a.row_order, c.row_order) and torch.equal(a.embedding, c.embedding)


def test_plan_out_of_range_index_is_reported_not_faulted():
    ptr = torch.tensor([0, 2, 3], dtype=torch.int32).cuda()
    idx = torch.tensor([0, 99, 1], dtype=torch.int32).cuda()
    d = wb.plan_desc_default(heads=1, n_q_blocks=2, n_kv_blocks=4, wave_size=2, mode=wb.FORCE_REORDER)
    res = wb.plan_csr(d, ptr, idx, debug=True)
    torch.cuda.synchronize()
    st = res.dev_status.tolist()
    assert st[0] == wb.ERR_BAD_MASK and st[3] == 99
    assert _np(res.row_nnz[0]).tolist() == [1, 1]       # the bad entry was skipped


@pytest.mark.parametrize("shape", [(1, 5), (7, 200), (130, 40), (64, 64)])
def test_plan_degenerate_and_rectangular(shape):
    m, n = shape
    masks = [np.ones((m, n), dtype=bool), I.random_mask(m, n, 0.3, 1), np.zeros((m, n), dtype=bool)]
    masks[2][:, 0] = True                                # identical rows
    wave = 9
    d = wb.plan_desc_default(heads=3, n_q_blocks=m, n_kv_blocks=n, wave_size=wave, mode=wb.FORCE_REORDER, seed=2)
    res = wb.plan_bitmap(d, _bitmap_dev(masks), debug=True)
    torch.cuda.synchronize()
    _check_plan(masks, [0, 1, 2], wave, d.svd_iters, 2, wo.MODE_FORCE_REORDER, res)
    # all-ones / identical rows: centred mask is zero -> natural order
    assert np.array_equal(_np(res.order1[0]), np.arange(m))
    assert np.array_equal(_np(res.order1[2]), np.arange(m))
    assert torch.isfinite(res.embedding).all()


def test_plan_large_block_count_uses_global_state():
    # 2*M_B + N_B beyond what shared memory holds: the iteration blocks live in the workspace
    m = 5000
    rng = np.random.default_rng(4)
    mk = np.zeros((m, m), dtype=bool)
    cols = rng.integers(0, m, size=(m, 6))
    mk[np.arange(m)[:, None], cols] = True
    mk[np.arange(m), np.arange(m)] = True
    d = wb.plan_desc_default(heads=1, n_q_blocks=m, n_kv_blocks=m, wave_size=148, mode=wb.FORCE_REORDER, seed=9,
                             svd_iters=5)
    res = wb.plan_bitmap(d, _bitmap_dev([mk]), debug=True)
    torch.cuda.synchronize()
    _check_plan([mk], [0], 148, 5, 9, wo.MODE_FORCE_REORDER, res)
