"""GPU parity of the paper's drop-in reorder operators (Section 5), and equivalence of the
paper's deployment (gather Q and mask rows -> backend in natural order -> scatter O) with the
index-list path of waveal_bsattn_fwd."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import waveal_oracle as wo
from paper_2609_34814_b200 import binding as wb
from paper_2609_34814_b200 import inputs as I
from gpu_util import Workload, run_attention

pytestmark = pytest.mark.gpu


def test_gather_scatter_bit_exact():
    H, nb, b, D = 3, 11, 64, 128
    rng = np.random.default_rng(1)
    x = torch.from_numpy(rng.integers(-2**15, 2**15, size=(H, nb * b, D), dtype=np.int16)).cuda().view(torch.bfloat16)
    order = np.stack([rng.permutation(nb) for _ in range(H)]).astype(np.int32)
    od = torch.from_numpy(order).cuda()
    g = torch.zeros_like(x)
    wb.gather_rows(x, g, od, b)
    s = torch.zeros_like(x)
    wb.scatter_rows(g, s, od, b)
    torch.cuda.synchronize()
    xs = x.view(torch.int16).cpu().numpy()
    for h in range(H):
        assert np.array_equal(g[h].view(torch.int16).cpu().numpy(), wo.gather_blocks(xs[h], order[h], b))
    assert torch.equal(s.view(torch.int16), x.view(torch.int16))
    # strided source (heads interleaved) and mask rows as 1-row blocks of words
    buf = torch.zeros((nb * b, H, D), dtype=torch.bfloat16, device="cuda")
    buf.copy_(x.permute(1, 0, 2))
    g2 = torch.zeros_like(x)
    wb.gather_rows(buf.permute(1, 0, 2), g2, od, b)
    torch.cuda.synchronize()
    assert torch.equal(g2.view(torch.int16), g.view(torch.int16))
    words = torch.from_numpy(rng.integers(0, 2**62, size=(H, nb, 2), dtype=np.int64)).cuda()
    gw = torch.zeros_like(words)
    wb.gather_rows(words, gw, od, 1)
    torch.cuda.synchronize()
    for h in range(H):
        assert np.array_equal(gw[h].cpu().numpy(), words[h].cpu().numpy()[order[h]])


def test_paper_deployment_equals_index_list_path():
    cfg = dataclasses.replace(I.CONFIGS["wan480p"], frames=4, seq=4 * 1560 - 48, heads=2, name="dep")   # 48 blocks, padded seq
    # operate on the padded length so that whole blocks move
    cfg = dataclasses.replace(cfg, seq=cfg.seq_pad)
    w = Workload(cfg)
    d = wb.plan_desc_default(heads=2, n_q_blocks=cfg.n_blocks, n_kv_blocks=cfg.n_blocks, wave_size=12,
                             mode=wb.FORCE_REORDER, seed=3)
    plan = wb.plan_bitmap(d, w.bitmap)
    direct, st = run_attention(w, row_order=plan.row_order, out=torch.zeros_like(w.o))
    assert st[0] == 0
    # the paper's way: gather Q blocks and mask rows, run in natural order, scatter O back
    qg = torch.zeros_like(w.q)
    wb.gather_rows(w.q, qg, plan.row_order, cfg.block)
    words = w.bitmap.shape[2]
    pad = (-words) % 2                                            # rows of 16-byte multiples
    bm = torch.zeros((2, cfg.n_blocks, words + pad), dtype=torch.int64, device="cuda")
    bm[:, :, :words] = w.bitmap
    bmg = torch.zeros_like(bm)
    wb.gather_rows(bm, bmg, plan.row_order, 1)
    ptr, idx = wb.bitmap_to_csr(bmg[:, :, :words].contiguous(), cfg.n_blocks)
    og = torch.zeros_like(w.o)
    st = torch.zeros(4, dtype=torch.int32, device="cuda")
    wb.bsattn_fwd(wb.attn_desc(qg, w.k, w.v, og, cfg.seq, cfg.seq, cfg.block), qg, w.k, w.v, og, ptr, idx, dev_status=st)
    back = torch.zeros_like(w.o)
    wb.scatter_rows(og, back, plan.row_order, cfg.block)
    torch.cuda.synchronize()
    assert st.tolist()[0] == 0
    assert torch.equal(back, direct)                               # same bits: only the execution order differs
