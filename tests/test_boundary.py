"""Host-only checks of the C-ABI boundary: the library loads, exports every symbol the
header declares, struct layouts agree, and host-detectable errors return a status before
any CUDA work (so these run without a GPU)."""
import ctypes
import os
import re

import pytest

from paper_2609_34814_b200 import binding as wb
from paper_2609_34814_b200 import build as wbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    wbuild.build()
    return wb.load()


def test_exports_match_header(lib):
    header = open(os.path.join(ROOT, "include", "waveal.h")).read()
    declared = set(re.findall(r"\b(waveal_[a-z0-9_]+)\s*\(", header))
    assert declared == set(wb.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_struct_layouts():
    assert ctypes.sizeof(wb.PlanDesc) == 80
    assert ctypes.sizeof(wb.PlanOut) == 64
    assert ctypes.sizeof(wb.AttnDesc) == 96
    assert wb.PlanDesc.seed.offset == 24 and wb.PlanDesc.min_nnz.offset == 72
    assert wb.AttnDesc.q_stride.offset == 24 and wb.AttnDesc.order_heads_interleaved.offset == 88


def test_defaults_and_workspace_query(lib):
    d = wb.plan_desc_default()
    assert (d.svd_iters, d.mode, d.l2_fit_num, d.l2_fit_den, d.min_density_ppm, d.local_num, d.local_den) == \
        (5, wb.AUTO, 9, 16, 10000, 1, 2)
    with pytest.raises(wb.WavealError) as e:
        wb.plan_workspace_bytes(d)                       # heads etc. still 0
    assert e.value.status == wb.ERR_INVALID_ARG and "positive" in str(e.value)
    d.heads, d.n_q_blocks, d.n_kv_blocks = 2, 100, 130
    n = wb.plan_workspace_bytes(d)
    assert n >= 2 * 100 * 3 * 8 + 2 * 130 * 2 * 8
    d.n_q_blocks = 1 << 20
    with pytest.raises(wb.WavealError) as e:
        wb.plan_workspace_bytes(d)
    assert e.value.status == wb.ERR_UNSUPPORTED
    d.n_q_blocks, d.mode = 100, 9
    with pytest.raises(wb.WavealError):
        wb.plan_workspace_bytes(d)


def test_plan_host_errors_before_any_launch(lib):
    d = wb.plan_desc_default(heads=1, n_q_blocks=4, n_kv_blocks=4)
    out = wb.PlanOut()
    assert lib.waveal_plan_bitmap(ctypes.byref(d), None, None, 0, ctypes.byref(out), None) == wb.ERR_INVALID_ARG
    assert lib.waveal_plan_bitmap(ctypes.byref(d), 0x1000, 0x2000, 1 << 20, ctypes.byref(out), None) == wb.ERR_INVALID_ARG
    assert "row_order" in wb.last_error()
    out.row_order = 0x3000
    assert lib.waveal_plan_bitmap(ctypes.byref(d), 0x1000, 0x2000, 16, ctypes.byref(out), None) == wb.ERR_WORKSPACE
    assert lib.waveal_plan_bitmap(ctypes.byref(d), 0x1000, 0x2010, 1 << 20, ctypes.byref(out), None) == wb.ERR_INVALID_ARG
    assert lib.waveal_plan_csr(ctypes.byref(d), None, None, 0x2000, 1 << 20, ctypes.byref(out), None) == wb.ERR_INVALID_ARG
    assert lib.waveal_bitmap_to_csr(0, 4, 4, 0x1000, 0x2000, None, 0, 0x3000, 64, None) == wb.ERR_INVALID_ARG
    assert lib.waveal_bitmap_to_csr(1, 4, 4, 0x1000, 0x2000, None, 0, 0x3000, 4, None) == wb.ERR_WORKSPACE


def test_attention_host_errors_before_any_launch(lib):
    d = wb.AttnDesc()
    d.heads, d.seq_q, d.seq_kv, d.head_dim, d.block_q, d.block_kv = 2, 256, 256, 128, 128, 128
    for s in (d.q_stride, d.k_stride, d.v_stride, d.o_stride):
        s[0], s[1] = 256 * 128, 128
    n = ctypes.c_size_t()
    assert lib.waveal_bsattn_workspace_bytes(ctypes.byref(d), ctypes.byref(n)) == wb.OK
    assert n.value == 256                                # counters + 8 + 32 bytes per (head, query block), in units of 256
    d.heads, d.seq_q = 40, 75600
    assert lib.waveal_bsattn_workspace_bytes(ctypes.byref(d), ctypes.byref(n)) == wb.OK
    tasks = 40 * 591
    assert n.value == ((32 + 8 * tasks + 31) // 32 * 32 + 32 * tasks + 255) // 256 * 256
    d.heads, d.seq_q = 2, 256
    call = lambda q=0x1000, ws=0x9000, wsb=256, scale=0.0: lib.waveal_bsattn_fwd(
        ctypes.byref(d), q, 0x2000, 0x3000, 0x4000, None, 0x5000, 0x6000, None, ctypes.c_float(scale), ws, wsb,
        None, None)
    assert call(q=None) == wb.ERR_INVALID_ARG
    assert call(q=0x1004) == wb.ERR_INVALID_ARG and "aligned" in wb.last_error()
    assert call(ws=None) == wb.ERR_WORKSPACE
    assert call(wsb=8) == wb.ERR_WORKSPACE
    assert call(scale=float("nan")) == wb.ERR_INVALID_ARG
    d.head_dim = 96
    assert call() == wb.ERR_UNSUPPORTED
    d.head_dim, d.block_q = 128, 64
    assert call() == wb.ERR_UNSUPPORTED                  # block_q != block_kv
    d.block_q = 128
    d.q_stride[1] = 100
    assert call() == wb.ERR_INVALID_ARG
    assert wb.status_string(wb.ERR_TIMEOUT) == "device-side wait timed out"


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(wb, "_lib", None)
    monkeypatch.setattr(wb, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        wb.load()
