"""GPU parity of the block-sparse attention kernel against the CPU oracle (through the C ABI).

Tolerance (bf16 inputs, fp32 accumulation, bf16 output): max-abs 1e-2, mean-abs 1e-3."""
import dataclasses
import math

import numpy as np
import pytest
import torch

from oracle import waveal_oracle as wo
from paper_2609_34814_b200 import binding as wb
from paper_2609_34814_b200 import inputs as I
from gpu_util import Workload, run_attention, error_stats, assert_parity

pytestmark = pytest.mark.gpu
MAX_ABS, MEAN_ABS = 1e-2, 1e-3


def _oracle_head(w, li, scale=None):
    cfg = w.cfg
    Q, K, V = (w.head_f64(x, li) for x in "qkv")
    return wo.block_sparse_attention(Q, K, V, w.masks[li], cfg.block, cfg.block, cfg.seq, cfg.seq, scale)


def _small(name, frames, heads, **kw):
    cfg = I.CONFIGS[name]
    return dataclasses.replace(cfg, frames=frames, seq=frames * cfg.frame_tokens - kw.pop("cut", 0), heads=heads,
                               name=f"{name}_small", **kw)


SMALL = [
    ("tiny", I.CONFIGS["tiny"]),                              # 64x64 blocks, D=64, every row
    ("wan480p_r", _small("wan480p", 3, 2)),                   # 128x128, D=128, 4680 tokens: ragged last block (72)
    ("wan720p_r", _small("wan720p", 2, 2, cut=37)),           # 7163 tokens: ragged (123)
    ("ltx_r", _small("ltxmixed", 3, 2, cut=10)),              # 64x64 blocks, D=128, ragged, sink rows
    ("b128_d64", dataclasses.replace(_small("wan480p", 2, 2), head_dim=64)),
]


@pytest.mark.parametrize("name,cfg", SMALL, ids=[s[0] for s in SMALL])
def test_attention_full_parity_small(name, cfg):
    w = Workload(cfg)
    lse = torch.full((cfg.heads, cfg.seq), float("nan"), dtype=torch.float32, device="cuda")
    w.o.fill_(float("nan"))
    o, st = run_attention(w, lse=lse)
    assert st == [0, 0, 0, 0]
    for li in range(cfg.heads):
        ref, ref_lse = _oracle_head(w, li)
        g = o[li, :cfg.seq].float().cpu().numpy()
        mx, mean = error_stats(g, ref)
        assert mx <= MAX_ABS and mean <= MEAN_ABS, (name, li, mx, mean)
        assert np.abs(lse[li].cpu().numpy() - ref_lse).max() < 2e-3
        # padded query rows (beyond seq) are never written
        if cfg.seq_pad > cfg.seq:
            assert torch.isnan(o[li, cfg.seq:].float()).all()


def test_output_is_bitwise_invariant_under_row_order():
    # Section 4.1: reordering changes only the execution order; Table 3: outputs identical
    cfg = _small("wan720p", 4, 3)
    w = Workload(cfg)
    base, st = run_attention(w, out=torch.zeros_like(w.o))
    assert st[0] == 0
    d = wb.plan_desc_default(heads=3, n_q_blocks=cfg.n_blocks, n_kv_blocks=cfg.n_blocks, wave_size=16,
                             mode=wb.FORCE_REORDER, seed=5)
    plan = wb.plan_bitmap(d, w.bitmap)
    out1, st = run_attention(w, row_order=plan.row_order, out=torch.zeros_like(w.o))
    assert st[0] == 0 and torch.equal(base, out1)
    rng = np.random.default_rng(0)
    perm = np.stack([rng.permutation(cfg.n_blocks) for _ in range(3)]).astype(np.int32)
    out2, st = run_attention(w, row_order=torch.from_numpy(perm).cuda(), out=torch.zeros_like(w.o))
    assert st[0] == 0 and torch.equal(base, out2)
    out3, st = run_attention(w, row_order=plan.row_order, out=torch.zeros_like(w.o), interleaved=True)
    assert st[0] == 0 and torch.equal(base, out3)
    # run-to-run determinism
    out4, _ = run_attention(w, out=torch.zeros_like(w.o))
    assert torch.equal(base, out4)


def test_empty_rows_scale_and_strides():
    cfg = _small("wan480p", 2, 2)
    w = Workload(cfg)
    # empty list for some rows: O = 0, LSE = -inf
    masks = [m.copy() for m in w.masks]
    masks[0][3, :] = False
    masks[1][0, :] = False
    w.masks = masks
    ptr, idx = I.masks_to_csr(masks)
    w.ptr, w.idx = torch.from_numpy(ptr).cuda(), torch.from_numpy(idx).cuda()
    # strided layout: heads interleaved in one [tokens, heads, D] buffer
    buf = torch.empty((cfg.seq_pad, 2, 3, cfg.head_dim), dtype=torch.bfloat16, device="cuda")
    for t, src in enumerate((w.q, w.k, w.v)):
        buf[:, :, t].copy_(src.permute(1, 0, 2))
    w.q, w.k, w.v = (buf[:, :, t].permute(1, 0, 2) for t in range(3))
    o = torch.full((2, cfg.seq_pad, cfg.head_dim), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.empty((2, cfg.seq), dtype=torch.float32, device="cuda")
    scale = 0.05
    o, st = run_attention(w, out=o, lse=lse, scale=scale)
    assert st[0] == 0
    b = cfg.block
    assert (o[0, 3 * b:4 * b] == 0).all() and torch.isinf(lse[0, 3 * b:4 * b]).all()
    assert (o[1, :b] == 0).all() and (lse[1, :b] < 0).all()
    for li in range(2):
        ref, ref_lse = _oracle_head(w, li, scale)
        mx, mean = error_stats(o[li, :cfg.seq].float().cpu().numpy(), ref)
        assert mx <= MAX_ABS and mean <= MEAN_ABS
        fin = np.isfinite(ref_lse)
        assert np.abs(lse[li].cpu().numpy()[fin] - ref_lse[fin]).max() < 2e-3


def test_output_rows_at_16_byte_alignment_only():
    """O whose rows start at 16-byte but not 32-byte boundaries (the least the interface asks for):
    the kernel's narrower stores must write the same bits as the 32-byte ones."""
    cfg = _small("wan480p", 2, 2)
    w = Workload(cfg)
    base, st = run_attention(w)
    assert st[0] == 0
    n = 2 * cfg.seq_pad * cfg.head_dim
    buf = torch.full((n + 8,), float("nan"), dtype=torch.bfloat16, device="cuda")
    o = buf[8:].view(2, cfg.seq_pad, cfg.head_dim)
    assert o.data_ptr() % 32 == 16
    o, st = run_attention(w, out=o)
    assert st[0] == 0
    assert torch.equal(o[:, :cfg.seq], base[:, :cfg.seq])
    assert torch.isnan(buf[:8]).all()


def test_closed_forms_on_gpu():
    cfg = _small("wan480p", 2, 1)
    w = Workload(cfg)
    # constant V -> constant O
    w.v[:] = 0.75
    o, st = run_attention(w)
    assert st[0] == 0 and (o[0, :cfg.seq].float() - 0.75).abs().max().item() < 4e-3
    # Q = 0 -> O is the mean of the selected V rows (uniform weights), LSE = log(#keys)
    w.v.copy_(torch.stack([I.make_head_tensor(cfg, "v", 0)]).cuda())
    w.q.zero_()
    lse = torch.empty((1, cfg.seq), dtype=torch.float32, device="cuda")
    o, st = run_attention(w, lse=lse)
    V = w.head_f64("v", 0)
    b = cfg.block
    for i in (0, cfg.n_blocks // 2, cfg.n_blocks - 1):
        keys = np.concatenate([np.arange(j * b, min((j + 1) * b, cfg.seq)) for j in np.nonzero(w.masks[0][i])[0]])
        assert np.abs(o[0, i * b].float().cpu().numpy() - V[keys].mean(0)).max() < 4e-3
        assert abs(lse[0, i * b].item() - math.log(len(keys))) < 1e-3
    # large scores: the reference-max handling must not overflow
    w.q.copy_(torch.stack([I.make_head_tensor(cfg, "q", 0)]).cuda())
    o, st = run_attention(w, scale=4.0)
    ref, _ = _oracle_head(w, 0, 4.0)
    assert st[0] == 0 and np.isfinite(o[0, :cfg.seq].float().cpu().numpy()).all()
    assert_parity(o[0, :cfg.seq].float().cpu().numpy(), ref, "scale 4", one_hot=True)   # near one-hot softmax: |O| reaches 4


def _sample_tasks(nnz, rng, n_random=12):
    m_b = len(nnz)
    rows = {0, m_b - 1, int(np.argmin(nnz)), int(np.argmax(nnz))}
    rows.update(int(r) for r in rng.choice(m_b, size=min(n_random, m_b), replace=False))
    return sorted(rows)


FULL = ["wan480p", "wan720p", "ltxmixed", "long720p"]


@pytest.mark.parametrize("name", FULL)
def test_full_size_sampled_parity_and_invariance(name):
    """The four large workloads at full size, in the launch configuration the bench times: sampled
    (head, row) tasks against the oracle; the whole output bitwise natural vs planned order."""
    cfg = I.CONFIGS[name]
    w = Workload(cfg)
    W = wb.default_wave_size()
    d = wb.plan_desc_default(heads=cfg.heads, n_q_blocks=cfg.n_blocks, n_kv_blocks=cfg.n_blocks, wave_size=W,
                             mode=wb.FORCE_REORDER, seed=cfg.plan_seed)
    plan = wb.plan_bitmap(d, w.bitmap)
    nat, st = run_attention(w, out=torch.zeros_like(w.o))
    assert st == [0, 0, 0, 0]
    o, st = run_attention(w, row_order=plan.row_order)
    assert st == [0, 0, 0, 0]
    assert torch.equal(nat, o)
    order = plan.row_order.cpu().numpy()
    assert np.array_equal(np.sort(order, axis=1), np.tile(np.arange(cfg.n_blocks), (cfg.heads, 1)))
    rng = np.random.default_rng(cfg.tensor_seed)
    heads = sorted({0, cfg.heads - 1, *rng.choice(cfg.heads, size=2, replace=False).tolist()})
    b = cfg.block
    errs = []
    for h in heads:
        Q, K, V = (w.head_f64(x, h) for x in "qkv")
        nnz = wo.row_nnz(w.masks[h])
        for i in _sample_tasks(nnz, rng):
            lo, hi = i * b, min((i + 1) * b, cfg.seq)
            ref, _ = wo.attention_block_row(Q[lo:hi], K, V, np.nonzero(w.masks[h][i])[0], b, cfg.seq,
                                            1 / math.sqrt(cfg.head_dim))
            errs.append(error_stats(o[h, lo:hi].float().cpu().numpy(), ref))
    assert max(e[0] for e in errs) <= MAX_ABS and max(e[1] for e in errs) <= MEAN_ABS


def test_reference_growth_and_short_rows():
    """Scores that keep growing along a row force the rescale of O on both softmax teams and
    the merge of their sums; rows of one, two and three KV blocks exercise the hand-over of
    the running reference at the start of a task."""
    cfg = _small("wan480p", 3, 1)
    w = Workload(cfg)
    b, nb = cfg.block, cfg.n_blocks
    # keys of block j scaled by 1 + 0.35 j: the row max rises by far more than 2^8 overall
    k = w.k[0].float()
    for j in range(nb):
        k[j * b:(j + 1) * b] *= 1.0 + 0.35 * j
    w.k[0].copy_(k.to(torch.bfloat16))
    K64 = I.bf16_to_f64(w.k[0].cpu())
    Q64, V64 = w.head_f64("q", 0), w.head_f64("v", 0)
    # rows 0..2 get exactly 1, 2, 3 blocks; the others keep the generated lists
    mask = w.masks[0].copy()
    for r, cols in ((0, [0]), (1, [1, nb - 1]), (2, [0, 5, nb - 1])):
        mask[r, :] = False
        mask[r, cols] = True
    w.masks[0] = mask
    ptr_np, idx_np = I.masks_to_csr([mask])
    w.ptr, w.idx = torch.from_numpy(ptr_np).cuda(), torch.from_numpy(idx_np).cuda()
    lse = torch.empty((1, cfg.seq), dtype=torch.float32, device="cuda")
    o, st = run_attention(w, lse=lse, scale=1.0)
    assert st == [0, 0, 0, 0]
    ref, ref_lse = wo.block_sparse_attention(Q64, K64, V64, mask, b, b, cfg.seq, cfg.seq, 1.0)
    g = o[0, :cfg.seq].float().cpu().numpy()
    assert np.isfinite(g).all()
    assert_parity(g, ref, "growing scores", one_hot=True)                 # near one-hot rows: |O| reaches 4
    assert np.abs(lse[0].cpu().numpy() - ref_lse).max() < 5e-3 * max(1.0, np.abs(ref_lse).max() / 10)


def test_second_launch_recomputes_tasks_whose_reference_was_too_low():
    """Keys that are far larger in one late KV block push the exponents of the fixed-reference
    pass over its limit: those tasks must be listed, computed again with the max of every
    block, and agree with the oracle; harmless inputs list nothing."""
    cfg = _small("wan480p", 3, 1)
    w = Workload(cfg)
    b, nb = cfg.block, cfg.n_blocks
    d = wb.attn_desc(w.q, w.k, w.v, w.o, cfg.seq, cfg.seq, b)
    ws = torch.zeros((wb.bsattn_workspace_bytes(d),), dtype=torch.uint8, device="cuda")
    st = torch.zeros(4, dtype=torch.int32, device="cuda")
    wb.bsattn_fwd(d, w.q, w.k, w.v, w.o, w.ptr, w.idx, workspace=ws, dev_status=st)
    torch.cuda.synchronize()
    assert st.tolist() == [0, 0, 0, 0] and ws.view(torch.int32)[2].item() == 0
    # block 20 of K scaled by 40: scores there exceed everything before them by far more than 2^100
    jb = 20
    k = w.k[0].float()
    k[jb * b:(jb + 1) * b] *= 40.0
    w.k[0].copy_(k.to(torch.bfloat16))
    hit = [i for i in range(nb) if w.masks[0][i, jb] and np.nonzero(w.masks[0][i])[0].tolist().index(jb) >= 2]
    assert len(hit) >= 3
    o = torch.full_like(w.o, float("nan"))
    ws.zero_()
    wb.bsattn_fwd(d, w.q, w.k, w.v, o, w.ptr, w.idx, workspace=ws, dev_status=st)
    torch.cuda.synchronize()
    assert st.tolist() == [0, 0, 0, 0]
    n_redo = ws.view(torch.int32)[2].item()
    listed = sorted(ws.view(torch.int32)[8:8 + 2 * n_redo].view(-1, 2)[:, 1].tolist())
    assert n_redo >= 1 and set(listed) <= set(hit), (n_redo, listed, hit)
    K64 = I.bf16_to_f64(w.k[0].cpu())
    ref, _ = wo.block_sparse_attention(w.head_f64("q", 0), K64, w.head_f64("v", 0), w.masks[0], b, b, cfg.seq, cfg.seq)
    g = o[0, :cfg.seq].float().cpu().numpy()
    assert np.isfinite(g).all()
    assert_parity(g, ref, "two launches", one_hot=True)
    # the single-launch variant that takes the max of every block gives the same rows for the listed tasks
    o2 = torch.zeros_like(w.o)
    d2 = wb.attn_desc(w.q, w.k, w.v, o2, cfg.seq, cfg.seq, b, flags=wb.ATTN_ONLINE_MAX_ONLY)
    wb.bsattn_fwd(d2, w.q, w.k, w.v, o2, w.ptr, w.idx, workspace=ws, dev_status=st)
    torch.cuda.synchronize()
    assert wb.last_launch_count() == 2               # ticket table + one attention launch
    for i in listed:
        assert torch.equal(o[0, i * b:min((i + 1) * b, cfg.seq)], o2[0, i * b:min((i + 1) * b, cfg.seq)])
    assert_parity(o2[0, :cfg.seq].float().cpu().numpy(), ref, "max of every block", one_hot=True)


def test_isolated_huge_key_in_a_polynomial_slot_is_recomputed():
    """One key far above everything else, in a late KV block and at a column whose exponential is
    taken from the polynomial: the fixed-reference launch must notice (its polynomial saturates
    instead of wrapping around), list the task, and the second launch must match the oracle."""
    cfg = _small("wan480p", 3, 1)
    w = Workload(cfg)
    b, nb = cfg.block, cfg.n_blocks
    jb = 20
    for col in (0, 2, 3, 70):             # 2, 3 and 70 = 64 + 6 are polynomial slots of a 64-column chunk, 0 is not
        w2 = Workload(cfg)
        k = w2.k[0].float()
        k[jb * b + col] *= 300.0          # scores of about +-300 nats on this key
        w2.k[0].copy_(k.to(torch.bfloat16))
        d = wb.attn_desc(w2.q, w2.k, w2.v, w2.o, cfg.seq, cfg.seq, b)
        ws = torch.zeros((wb.bsattn_workspace_bytes(d),), dtype=torch.uint8, device="cuda")
        st = torch.zeros(4, dtype=torch.int32, device="cuda")
        o = torch.full_like(w2.o, float("nan"))
        wb.bsattn_fwd(d, w2.q, w2.k, w2.v, o, w2.ptr, w2.idx, workspace=ws, dev_status=st)
        torch.cuda.synchronize()
        assert st.tolist() == [0, 0, 0, 0]
        hit = [i for i in range(nb) if w2.masks[0][i, jb] and np.nonzero(w2.masks[0][i])[0].tolist().index(jb) >= 2]
        n_redo = ws.view(torch.int32)[2].item()
        listed = sorted(ws.view(torch.int32)[8:8 + 2 * n_redo].view(-1, 2)[:, 1].tolist())
        assert len(hit) >= 3 and listed == hit, (col, listed, hit)
        K64 = I.bf16_to_f64(w2.k[0].cpu())
        ref, _ = wo.block_sparse_attention(w2.head_f64("q", 0), K64, w2.head_f64("v", 0), w2.masks[0], b, b,
                                           cfg.seq, cfg.seq)
        g = o[0, :cfg.seq].float().cpu().numpy()
        assert np.isfinite(g).all()
        assert_parity(g, ref, f"huge key at column {col}", one_hot=True)


MASKS = ["dense", "random20"]


@pytest.mark.parametrize("kind", MASKS)
def test_dense_and_unstructured_masks_match_the_oracle(kind):
    """The two mask variants the bench offers beside the structured recipe: all pairs (Section 2.2:
    dense attention computes every pair) and 20 % uniform columns per row (the Random row of the
    paper's Table 1), on a small 128x128-block case with a ragged tail."""
    cfg = _small("wan480p", 2, 2, cut=19)
    w = Workload(cfg)
    nb = cfg.n_blocks
    if kind == "dense":
        masks = [np.ones((nb, nb), dtype=bool) for _ in range(cfg.heads)]
    else:
        masks = [I.random_mask(nb, nb, 0.20, 77 + h) for h in range(cfg.heads)]
        assert all(abs(m.mean() - 0.20) < 0.03 for m in masks)
    w.masks = masks
    ptr, idx = I.masks_to_csr(masks)
    w.ptr, w.idx = torch.from_numpy(ptr).cuda(), torch.from_numpy(idx).cuda()
    lse = torch.empty((cfg.heads, cfg.seq), dtype=torch.float32, device="cuda")
    o, st = run_attention(w, lse=lse)
    assert st == [0, 0, 0, 0]
    for li in range(cfg.heads):
        ref, ref_lse = _oracle_head(w, li)
        assert_parity(o[li, :cfg.seq].float().cpu().numpy(), ref, kind)
        assert np.abs(lse[li].cpu().numpy() - ref_lse).max() < 2e-3
    if kind == "dense":
        # all-ones mask == textbook softmax(scale Q K^T) V
        Q, K, V = (w.head_f64(x, 0)[:cfg.seq] for x in "qkv")
        s = (Q @ K.T) / math.sqrt(cfg.head_dim)
        p = np.exp(s - s.max(axis=1, keepdims=True))
        assert_parity(o[0, :cfg.seq].float().cpu().numpy(), (p / p.sum(axis=1, keepdims=True)) @ V, "textbook")


def test_bounded_wait_runs_out_and_the_kernel_leaves_cleanly():
    """Failure handling without a fault: with the self-test flag the loader never requests one K
    tile, the waits behind it give up after ~2 ms, and the call must report a TIMEOUT with
    every thread block gone through the common exit; the next ordinary call on the same
    workspace and status words must be correct."""
    import time
    cfg = _small("wan480p", 3, 2)
    w = Workload(cfg)
    b = cfg.block
    d = wb.attn_desc(w.q, w.k, w.v, w.o, cfg.seq, cfg.seq, b, flags=wb.ATTN_SELFTEST_LOST_TILE)
    ws = torch.zeros((wb.bsattn_workspace_bytes(d),), dtype=torch.uint8, device="cuda")
    st = torch.zeros(4, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    wb.bsattn_fwd(d, w.q, w.k, w.v, w.o, w.ptr, w.idx, workspace=ws, dev_status=st)
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    code, site, cta, thread = st.tolist()
    # whichever wait behind the lost tile ran out first: the Q K^T issuer (12), a loader's ring
    # slot (3: K, 4: V), the P V issuer (14) or a softmax warp (21)
    assert code == wb.ERR_TIMEOUT and site in (3, 4, 12, 14, 21), st.tolist()
    assert 0 <= cta < 148 and 0 <= thread < 640
    assert ws.view(torch.int32)[1].item() == 1            # abort flag seen by the other thread blocks
    assert dt < 1.0, dt                                   # milliseconds, not the 2 s production limit
    # same workspace, same status words (zeroed by the caller), ordinary call
    st.zero_()
    d = wb.attn_desc(w.q, w.k, w.v, w.o, cfg.seq, cfg.seq, b)
    w.o.fill_(float("nan"))
    wb.bsattn_fwd(d, w.q, w.k, w.v, w.o, w.ptr, w.idx, workspace=ws, dev_status=st)
    torch.cuda.synchronize()
    assert st.tolist() == [0, 0, 0, 0]
    for li in range(cfg.heads):
        ref, _ = _oracle_head(w, li)
        assert_parity(w.o[li, :cfg.seq].float().cpu().numpy(), ref, "after the self-test")
    # tensor memory was released by the aborted launch: many more launches still find it
    for _ in range(8):
        wb.bsattn_fwd(d, w.q, w.k, w.v, w.o, w.ptr, w.idx, workspace=ws, dev_status=st)
    torch.cuda.synchronize()
    assert st.tolist() == [0, 0, 0, 0]


def test_malformed_lists_are_reported_not_followed():
    cfg = _small("wan480p", 2, 1)
    w = Workload(cfg)
    b, nb = cfg.block, cfg.n_blocks
    good, _ = run_attention(w, out=torch.zeros_like(w.o))
    # entry of row_order out of range
    order = torch.arange(nb, dtype=torch.int32, device="cuda").view(1, nb).clone()
    order[0, 5] = nb + 3
    o, st = run_attention(w, row_order=order, out=torch.zeros_like(w.o))
    assert st == [wb.ERR_BAD_MASK, 31, 0, nb + 3]
    # decreasing row pointers: the task gets an empty list, the others are untouched
    ptr = w.ptr.clone()
    keep = w.ptr
    ptr[4] = ptr[3] - 1
    w.ptr = ptr
    o, st = run_attention(w, out=torch.full_like(w.o, float("nan")))
    assert st[0] == wb.ERR_BAD_MASK and st[1] == 32 and st[2] == 0
    assert (o[0, 3 * b:4 * b] == 0).all()
    assert torch.equal(o[0, 5 * b:cfg.seq], good[0, 5 * b:cfg.seq])
    w.ptr = keep
    # an index beyond the number of KV blocks: last of a list (site 33) and inside a list (site 30)
    idx = w.idx.clone()
    keep_idx = w.idx
    lo, hi = int(w.ptr_np[2]), int(w.ptr_np[3])
    idx[hi - 1] = nb + 7
    w.idx = idx
    o, st = run_attention(w, out=torch.zeros_like(w.o))
    assert st == [wb.ERR_BAD_MASK, 33, 0, nb + 7]
    idx = keep_idx.clone()
    idx[lo] = -4
    w.idx = idx
    o, st = run_attention(w, out=torch.zeros_like(w.o))
    assert st == [wb.ERR_BAD_MASK, 30, 0, -4]
    w.idx = keep_idx
    o, st = run_attention(w, out=torch.zeros_like(w.o))
    assert st == [0, 0, 0, 0] and torch.equal(o, good)


def test_identical_rows_share_a_tile_with_identical_bits():
    """64-row query blocks with the very same KV list at positions 2i, 2i+1 of the order run as one
    128-row tile: same bits as unshared, same as any other order, and equal to the oracle."""
    cfg = _small("ltxmixed", 4, 2, cut=10)          # 64x64 blocks, ragged tail, sink rows (full lists)
    w = Workload(cfg)
    nb = cfg.n_blocks
    # make sure identical lists exist beyond the sink rows: copy a few rows' lists
    masks = [m.copy() for m in w.masks]
    for m in masks:
        m[11] = m[10]
        m[nb - 1] = m[nb - 2]
        m[21, :] = False
        m[21, [3, 7]] = True                         # one tile, two blocks
        m[20] = m[21]
        m[31, :] = False
        m[31, [5]] = True                            # half a tile
        m[30] = m[31]
    w.masks = masks
    ptr, idx = I.masks_to_csr(masks)
    w.ptr, w.idx = torch.from_numpy(ptr).cuda(), torch.from_numpy(idx).cuda()
    b = cfg.block

    def run(order, flags=0):
        o = torch.full_like(w.o, float("nan"))
        lse = torch.full((cfg.heads, cfg.seq), float("nan"), dtype=torch.float32, device="cuda")
        d = wb.attn_desc(w.q, w.k, w.v, o, cfg.seq, cfg.seq, b, flags=flags)
        ws = torch.zeros((wb.bsattn_workspace_bytes(d),), dtype=torch.uint8, device="cuda")
        st = torch.zeros(4, dtype=torch.int32, device="cuda")
        wb.bsattn_fwd(d, w.q, w.k, w.v, o, w.ptr, w.idx, row_order=order, lse=lse, workspace=ws, dev_status=st)
        torch.cuda.synchronize()
        assert st.tolist() == [0, 0, 0, 0]
        return o, lse, int(ws.view(torch.int32)[6].item())

    # Stage 2 (descending count inside a wave) puts the full rows side by side
    d = wb.plan_desc_default(heads=cfg.heads, n_q_blocks=nb, n_kv_blocks=nb, wave_size=16, mode=wb.STAGE2_ONLY, seed=1)
    plan = wb.plan_bitmap(d, w.bitmap if False else torch.from_numpy(
        np.stack([I.mask_to_bitmap(m) for m in masks]).view(np.int64)).cuda())
    shared, lse_s, pairs = run(plan.row_order)
    alone, lse_a, none = run(plan.row_order, flags=wb.ATTN_NO_ROW_PAIRING)
    natural, lse_n, pairs_nat = run(None)
    assert none == 0 and pairs >= 4 and pairs_nat >= 4          # (10,11), (20,21), (30,31), the last two rows
    # rows that select every block pair up wherever they stand, also in natural order
    full_pairs = sum(int((m.sum(axis=1) == nb).sum()) // 2 for m in masks)
    assert full_pairs >= 2 and pairs_nat >= full_pairs and pairs >= full_pairs
    assert torch.equal(shared[:, :cfg.seq], alone[:, :cfg.seq]) and torch.equal(lse_s, lse_a)
    assert torch.equal(shared[:, :cfg.seq], natural[:, :cfg.seq]) and torch.equal(lse_s, lse_n)
    assert torch.isnan(shared[:, cfg.seq:].float()).all()        # rows beyond the sequence stay untouched
    for li in range(cfg.heads):
        ref, ref_lse = _oracle_head(w, li)
        assert_parity(shared[li, :cfg.seq].float().cpu().numpy(), ref, "shared tiles")
        assert np.abs(lse_s[li].cpu().numpy() - ref_lse).max() < 2e-3
    # a key far above the rest in a late block: tasks that share a tile are handed to the second
    # launch as two single blocks, and the result still equals the unshared one and the oracle
    k = w.k[0].float()
    k[9 * b + 2] *= 300.0
    w.k[0].copy_(k.to(torch.bfloat16))
    shared, lse_s, pairs = run(plan.row_order)
    alone, lse_a, _ = run(plan.row_order, flags=wb.ATTN_NO_ROW_PAIRING)
    assert pairs >= 4 and torch.equal(shared[:, :cfg.seq], alone[:, :cfg.seq])
    K64 = I.bf16_to_f64(w.k[0].cpu())
    ref, _ = wo.block_sparse_attention(w.head_f64("q", 0), K64, w.head_f64("v", 0), masks[0], b, b, cfg.seq, cfg.seq)
    assert_parity(shared[0, :cfg.seq].float().cpu().numpy(), ref, "shared tiles, second launch", one_hot=True)


@pytest.mark.parametrize("block,d", [(128, 128), (64, 128), (64, 64)])
def test_different_query_and_key_lengths_and_the_single_launch_variant(block, d):
    """M_B != N_B (the paper's problem statement allows it), both lengths ragged; the default two-launch
    call and the variant that takes the max of every tile must both match the oracle."""
    seq_q, seq_kv = 5 * block - 9, 11 * block - 37
    mq, nk = 5, 11
    rng = np.random.default_rng(block + d)
    H = 2
    g = torch.Generator().manual_seed(block * 7 + d)
    q = torch.randn((H, mq * block, d), generator=g).to(torch.bfloat16)
    k = torch.randn((H, nk * block, d), generator=g).to(torch.bfloat16)
    v = torch.randn((H, nk * block, d), generator=g).to(torch.bfloat16)
    masks = []
    for h in range(H):
        m = rng.random((mq, nk)) < 0.4
        m[:, nk - 1] |= rng.random(mq) < 0.7          # the ragged last KV block is in most lists
        m[np.arange(mq), np.arange(mq)] = True
        m[1] = True                                    # a row that selects everything
        m[3] = True                                    # and a second one: they share a tile on 64-row blocks
        if h == 1:
            m[:] = True                                # all five rows full: two pairs and one block on its own
        masks.append(m)
    ptr_np, idx_np = I.masks_to_csr(masks)
    ptr, idx = torch.from_numpy(ptr_np).cuda(), torch.from_numpy(idx_np).cuda()
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    for flags in (0, wb.ATTN_ONLINE_MAX_ONLY):
        o = torch.full_like(qd, float("nan"))
        lse = torch.full((H, seq_q), float("nan"), dtype=torch.float32, device="cuda")
        desc = wb.attn_desc(qd, kd, vd, o, seq_q, seq_kv, block, flags=flags)
        st = torch.zeros(4, dtype=torch.int32, device="cuda")
        wb.bsattn_fwd(desc, qd, kd, vd, o, ptr, idx, lse=lse, dev_status=st)
        torch.cuda.synchronize()
        assert st.tolist() == [0, 0, 0, 0]
        for h in range(H):
            Q64, K64, V64 = (I.bf16_to_f64(t[h]) for t in (q, k, v))
            ref, ref_lse = wo.block_sparse_attention(Q64, K64, V64, masks[h], block, block, seq_q, seq_kv)
            assert_parity(o[h, :seq_q].float().cpu().numpy(), ref, f"{block}x{d} flags {flags}")
            assert np.abs(lse[h].cpu().numpy() - ref_lse).max() < 2e-3
            assert torch.isnan(o[h, seq_q:].float()).all()
