"""ctypes loader for oracle_attn.c (the C twin of the attention oracle).  TEST
INFRASTRUCTURE ONLY.  build() compiles the C file with gcc next to its source."""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "oracle_attn.c")
_LIB = os.path.join(_HERE, "liboracle_attn.so")
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", _SRC, "-o", _LIB, "-lm"])
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_attn_threads.restype = ctypes.c_int
        _lib.oracle_attn_tasks.restype = None
    return _lib


def threads() -> int:
    return int(_load().oracle_attn_threads())


def attn_tasks(q_bits: np.ndarray, k_bits: np.ndarray, v_bits: np.ndarray, block_q: int, block_kv: int,
               seq_q: int, seq_kv: int, scale: float, task_q_block: Sequence[int],
               kv_lists: Sequence[Sequence[int]]) -> Tuple[np.ndarray, np.ndarray]:
    """q_bits/k_bits/v_bits: uint16 [tokens, D] bf16 bit patterns of one head.  Returns
    O [n_tasks, block_q, D] and LSE [n_tasks, block_q] in float64 (tokens >= seq_q: NaN)."""
    lib = _load()
    d = q_bits.shape[1]
    n = len(task_q_block)
    tq = np.asarray(task_q_block, dtype=np.int32)
    ptr = np.zeros(n + 1, dtype=np.int32)
    ptr[1:] = np.cumsum([len(l) for l in kv_lists])
    idx = np.concatenate([np.asarray(l, dtype=np.int32) for l in kv_lists]) if n and ptr[-1] else np.zeros(0, np.int32)
    out = np.full((n, block_q, d), np.nan)
    lse = np.full((n, block_q), np.nan)
    q_bits, k_bits, v_bits = (np.ascontiguousarray(a, dtype=np.uint16) for a in (q_bits, k_bits, v_bits))
    P = ctypes.c_void_p
    lib.oracle_attn_tasks(P(q_bits.ctypes.data), P(k_bits.ctypes.data), P(v_bits.ctypes.data),
                          ctypes.c_int(d), ctypes.c_int(block_q), ctypes.c_int(block_kv),
                          ctypes.c_int(seq_q), ctypes.c_int(seq_kv), ctypes.c_double(scale),
                          ctypes.c_int(n), P(tq.ctypes.data), P(ptr.ctypes.data), P(idx.ctypes.data),
                          P(out.ctypes.data), P(lse.ctypes.data))
    return out, lse
