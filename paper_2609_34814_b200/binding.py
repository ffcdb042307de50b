"""ctypes binding of libwaveal.so: the same names as include/waveal.h, argument marshalling only.

Every step of the hot path runs inside the library's CUDA kernels; this module converts
torch tensors to pointers, allocates the workspaces the C ABI asks the caller to own, and
raises on a non-zero status.  It fails loudly when the library is missing: there is no CPU
fallback.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(PKG, "libwaveal.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_BAD_MASK, ERR_CUDA, ERR_TIMEOUT = range(7)
AUTO, FORCE_REORDER, FORCE_NATURAL, STAGE1_ONLY, STAGE2_ONLY = range(5)
FLAG_SKIPPED, FLAG_SHORT_SEQ, FLAG_TOO_SPARSE, FLAG_ALREADY_LOCAL = 1, 2, 4, 8

EXPORTS = ["waveal_plan_desc_default", "waveal_plan_workspace_bytes", "waveal_plan_bitmap", "waveal_plan_csr",
           "waveal_bitmap_to_csr", "waveal_bitmap_to_csr_noalloc", "waveal_noalloc_max_rows",
           "waveal_gather_rows", "waveal_scatter_rows", "waveal_bsattn_workspace_bytes", "waveal_bsattn_fwd",
           "waveal_default_wave_size", "waveal_last_launch_count", "waveal_status_string", "waveal_last_error"]


class PlanDesc(ctypes.Structure):
    _fields_ = [("heads", ctypes.c_int32), ("n_q_blocks", ctypes.c_int32), ("n_kv_blocks", ctypes.c_int32),
                ("wave_size", ctypes.c_int32), ("svd_iters", ctypes.c_int32), ("mode", ctypes.c_int32),
                ("seed", ctypes.c_uint64), ("kv_bytes_per_head", ctypes.c_int64), ("l2_bytes", ctypes.c_int64),
                ("l2_fit_num", ctypes.c_int32), ("l2_fit_den", ctypes.c_int32), ("min_density_ppm", ctypes.c_int32),
                ("local_num", ctypes.c_int32), ("local_den", ctypes.c_int32), ("min_nnz", ctypes.c_int64)]


class PlanOut(ctypes.Structure):
    _fields_ = [("row_order", ctypes.c_void_p), ("row_nnz", ctypes.c_void_p), ("skip_flags", ctypes.c_void_p),
                ("col_count", ctypes.c_void_p), ("order1", ctypes.c_void_p), ("embedding", ctypes.c_void_p),
                ("stats", ctypes.c_void_p), ("dev_status", ctypes.c_void_p)]


class AttnDesc(ctypes.Structure):
    _fields_ = [("heads", ctypes.c_int32), ("seq_q", ctypes.c_int32), ("seq_kv", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("block_q", ctypes.c_int32), ("block_kv", ctypes.c_int32),
                ("q_stride", ctypes.c_int64 * 2), ("k_stride", ctypes.c_int64 * 2), ("v_stride", ctypes.c_int64 * 2),
                ("o_stride", ctypes.c_int64 * 2), ("order_heads_interleaved", ctypes.c_int32),
                ("flags", ctypes.c_int32)]


class WavealError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"waveal status {status}: {message}")
        self.status = status


_lib = None


def load() -> ctypes.CDLL:
    """Loads the C-ABI library; raises if it was not built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2609_34814_b200.build` "
                               "(the library has no CPU fallback)")
        lib = ctypes.CDLL(LIB_PATH)
        P, I32, I64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
        lib.waveal_plan_desc_default.argtypes = [ctypes.POINTER(PlanDesc)]
        lib.waveal_plan_desc_default.restype = None
        lib.waveal_plan_workspace_bytes.argtypes = [ctypes.POINTER(PlanDesc), ctypes.POINTER(ctypes.c_size_t)]
        lib.waveal_plan_bitmap.argtypes = [ctypes.POINTER(PlanDesc), P, P, ctypes.c_size_t, ctypes.POINTER(PlanOut), P]
        lib.waveal_plan_csr.argtypes = [ctypes.POINTER(PlanDesc), P, P, P, ctypes.c_size_t, ctypes.POINTER(PlanOut), P]
        lib.waveal_bitmap_to_csr.argtypes = [I32, I32, I32, P, P, P, I64, P, ctypes.c_size_t, P]
        lib.waveal_bitmap_to_csr_noalloc.argtypes = [I32, I32, I32, P, P, P, I64, P]
        lib.waveal_bitmap_to_csr_noalloc.restype = ctypes.c_int
        lib.waveal_noalloc_max_rows.restype = ctypes.c_size_t
        for name in ("waveal_gather_rows", "waveal_scatter_rows"):
            getattr(lib, name).argtypes = [I32, I32, I32, I32, P, ctypes.POINTER(I64), P, ctypes.POINTER(I64), P, P]
            getattr(lib, name).restype = ctypes.c_int
        lib.waveal_bsattn_workspace_bytes.argtypes = [ctypes.POINTER(AttnDesc), ctypes.POINTER(ctypes.c_size_t)]
        lib.waveal_bsattn_fwd.argtypes = [ctypes.POINTER(AttnDesc), P, P, P, P, P, P, P, P, ctypes.c_float, P,
                                          ctypes.c_size_t, P, P]
        for name in ["waveal_plan_workspace_bytes", "waveal_plan_bitmap", "waveal_plan_csr", "waveal_bitmap_to_csr",
                     "waveal_gather_rows", "waveal_scatter_rows", "waveal_bsattn_workspace_bytes", "waveal_bsattn_fwd", "waveal_default_wave_size",
                     "waveal_last_launch_count"]:
            getattr(lib, name).restype = ctypes.c_int
        lib.waveal_status_string.argtypes = [ctypes.c_int]
        lib.waveal_status_string.restype = ctypes.c_char_p
        lib.waveal_last_error.restype = ctypes.c_char_p
        _lib = lib
    return _lib


def last_error() -> str:
    return load().waveal_last_error().decode()


def status_string(s: int) -> str:
    return load().waveal_status_string(s).decode()


def _check(status: int):
    if status != OK:
        raise WavealError(status, last_error() or status_string(status))


def _ptr(t) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        stream = torch.cuda.current_stream()
    return stream.cuda_stream or None


def default_wave_size() -> int:
    return int(load().waveal_default_wave_size())


def last_launch_count() -> int:
    return int(load().waveal_last_launch_count())


def plan_desc_default(**kw) -> PlanDesc:
    d = PlanDesc()
    load().waveal_plan_desc_default(ctypes.byref(d))
    for k, v in kw.items():
        setattr(d, k, v)
    return d


def plan_workspace_bytes(desc: PlanDesc) -> int:
    n = ctypes.c_size_t(0)
    _check(load().waveal_plan_workspace_bytes(ctypes.byref(desc), ctypes.byref(n)))
    return int(n.value)


class PlanResult:
    """Device tensors a plan call filled (torch tensors; the caller may pass its own)."""

    def __init__(self, **kw):
        self.__dict__.update(kw)


def _plan_outputs(desc: PlanDesc, device, debug: bool):
    import torch
    H, M, N = desc.heads, desc.n_q_blocks, desc.n_kv_blocks
    res = PlanResult(
        row_order=torch.empty((H, M), dtype=torch.int32, device=device),
        row_nnz=torch.empty((H, M), dtype=torch.int32, device=device),
        skip_flags=torch.empty((H,), dtype=torch.uint8, device=device),
        dev_status=torch.zeros((4,), dtype=torch.int32, device=device),
        col_count=None, order1=None, embedding=None, stats=None)
    if debug:
        res.col_count = torch.empty((H, N), dtype=torch.int32, device=device)
        res.order1 = torch.empty((H, M), dtype=torch.int32, device=device)
        res.embedding = torch.empty((H, M, 2), dtype=torch.float64, device=device)
        res.stats = torch.empty((H, 4), dtype=torch.int64, device=device)
    out = PlanOut(_ptr(res.row_order), _ptr(res.row_nnz), _ptr(res.skip_flags), _ptr(res.col_count),
                  _ptr(res.order1), _ptr(res.embedding), _ptr(res.stats), _ptr(res.dev_status))
    return res, out


def plan_bitmap(desc: PlanDesc, mask_bits, workspace=None, debug: bool = False, stream=None) -> PlanResult:
    """waveal_plan_bitmap.  mask_bits: cuda tensor of 64-bit words [heads, M_B, ceil(N_B/64)]."""
    import torch
    lib = load()
    if workspace is None:
        workspace = torch.empty((plan_workspace_bytes(desc) + 256,), dtype=torch.uint8, device=mask_bits.device)
    res, out = _plan_outputs(desc, mask_bits.device, debug)
    res.workspace = workspace
    _check(lib.waveal_plan_bitmap(ctypes.byref(desc), _ptr(mask_bits), _ptr(workspace), workspace.numel(),
                                  ctypes.byref(out), _stream(stream)))
    return res


def plan_csr(desc: PlanDesc, kv_row_ptr, kv_block_indices, workspace=None, debug: bool = False, stream=None) -> PlanResult:
    """waveal_plan_csr."""
    import torch
    lib = load()
    if workspace is None:
        workspace = torch.empty((plan_workspace_bytes(desc) + 256,), dtype=torch.uint8, device=kv_row_ptr.device)
    res, out = _plan_outputs(desc, kv_row_ptr.device, debug)
    res.workspace = workspace
    _check(lib.waveal_plan_csr(ctypes.byref(desc), _ptr(kv_row_ptr), _ptr(kv_block_indices), _ptr(workspace),
                               workspace.numel(), ctypes.byref(out), _stream(stream)))
    return res


def bitmap_to_csr(mask_bits, n_kv_blocks: int, capacity: Optional[int] = None, stream=None):
    """waveal_bitmap_to_csr.  Returns (kv_row_ptr, kv_block_indices) device tensors; when
    `capacity` is None the row pointers are computed first and their last entry read back
    (one synchronisation) to size the index array."""
    import torch
    lib = load()
    H, M, _ = mask_bits.shape
    dev = mask_bits.device
    ptr = torch.empty((H * M + 1,), dtype=torch.int32, device=dev)
    ws = torch.empty(((H * M + 1) * 4,), dtype=torch.uint8, device=dev)
    if capacity is None:
        _check(lib.waveal_bitmap_to_csr(H, M, n_kv_blocks, _ptr(mask_bits), _ptr(ptr), None, 0, _ptr(ws), ws.numel(),
                                        _stream(stream)))
        capacity = int(ptr[-1].item())
    idx = torch.empty((max(capacity, 1),), dtype=torch.int32, device=dev)
    _check(lib.waveal_bitmap_to_csr(H, M, n_kv_blocks, _ptr(mask_bits), _ptr(ptr), _ptr(idx), capacity, _ptr(ws),
                                    ws.numel(), _stream(stream)))
    return ptr, idx[:capacity]


def noalloc_max_rows() -> int:
    return int(load().waveal_noalloc_max_rows())


def bitmap_to_csr_noalloc(mask_bits, n_kv_blocks: int, kv_row_ptr, kv_block_indices, stream=None):
    """waveal_bitmap_to_csr_noalloc: for callers that cannot allocate device memory (an engine
    plug-in handed pre-planned tensors).  Every buffer is the caller's: `kv_row_ptr` int32
    [heads*M_B + 1] and `kv_block_indices` int32 [capacity] (or None for row pointers only)
    are filled on the stream; the call itself allocates nothing, here or in the library, and
    refuses problems with more than noalloc_max_rows() query-block rows."""
    H, M, _ = mask_bits.shape
    cap = 0 if kv_block_indices is None else kv_block_indices.numel()
    _check(load().waveal_bitmap_to_csr_noalloc(H, M, n_kv_blocks, _ptr(mask_bits), _ptr(kv_row_ptr),
                                               _ptr(kv_block_indices), cap, _stream(stream)))


def _move_rows(fn_name: str, src, dst, row_order, block: int, stream=None):
    """src, dst: [heads, n_blocks*block, row elements] tensors (last dim contiguous)."""
    H, rows, _ = src.shape
    assert src.stride(2) == 1 and dst.stride(2) == 1 and dst.shape == src.shape
    es = src.element_size()
    ss = (ctypes.c_int64 * 2)(src.stride(0) * es, src.stride(1) * es)
    ds = (ctypes.c_int64 * 2)(dst.stride(0) * es, dst.stride(1) * es)
    _check(getattr(load(), fn_name)(H, rows // block, block, src.shape[2] * es, _ptr(src), ss, _ptr(dst), ds,
                                    _ptr(row_order), _stream(stream)))


def gather_rows(src, dst, row_order, block: int, stream=None):
    """waveal_gather_rows: dst block p <- src block row_order[h][p]."""
    _move_rows("waveal_gather_rows", src, dst, row_order, block, stream)


def scatter_rows(src, dst, row_order, block: int, stream=None):
    """waveal_scatter_rows: dst block row_order[h][p] <- src block p."""
    _move_rows("waveal_scatter_rows", src, dst, row_order, block, stream)


RING_CUT_LARGEST_GAP = 16
ATTN_ONLINE_MAX_ONLY = 1
ATTN_SELFTEST_LOST_TILE = 256
ATTN_NO_ROW_PAIRING = 2


def attn_desc(q, k, v, o, seq_q: int, seq_kv: int, block: int, interleaved: bool = False, flags: int = 0) -> AttnDesc:
    """Descriptor for [heads, tokens, head_dim] tensors (head_dim contiguous)."""
    d = AttnDesc()
    d.heads, d.seq_q, d.seq_kv, d.head_dim = q.shape[0], seq_q, seq_kv, q.shape[2]
    d.block_q = d.block_kv = block
    for name, t in (("q_stride", q), ("k_stride", k), ("v_stride", v), ("o_stride", o)):
        assert t.stride(2) == 1, "head_dim must be contiguous"
        getattr(d, name)[0], getattr(d, name)[1] = t.stride(0), t.stride(1)
    d.order_heads_interleaved = 1 if interleaved else 0
    d.flags = flags
    return d


def bsattn_workspace_bytes(desc: AttnDesc) -> int:
    n = ctypes.c_size_t(0)
    _check(load().waveal_bsattn_workspace_bytes(ctypes.byref(desc), ctypes.byref(n)))
    return int(n.value)


def bsattn_fwd(desc: AttnDesc, q, k, v, o, kv_row_ptr, kv_block_indices, row_order=None, lse=None,
               scale: float = 0.0, workspace=None, dev_status=None, stream=None):
    """waveal_bsattn_fwd.  All tensors are cuda tensors owned by the caller; returns nothing
    (o, lse and dev_status are written on the stream)."""
    import torch
    lib = load()
    if workspace is None:
        workspace = torch.empty((bsattn_workspace_bytes(desc),), dtype=torch.uint8, device=q.device)
    _check(lib.waveal_bsattn_fwd(ctypes.byref(desc), _ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), _ptr(kv_row_ptr),
                                 _ptr(kv_block_indices), _ptr(row_order), ctypes.c_float(scale), _ptr(workspace),
                                 workspace.numel(), _ptr(dev_status), _stream(stream)))
    return workspace
