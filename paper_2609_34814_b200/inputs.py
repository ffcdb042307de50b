"""Seeded synthetic inputs: block masks and Q/K/V tensors shaped like the paper's workloads.

This module is the only code shared by the CUDA path's tests/bench and the CPU oracle.
It holds no arithmetic of the method itself (no popcounts, no embedding, no sorting of
rows, no attention): it only draws masks and tensors and converts a boolean mask to the
two storage formats the library accepts (a little-endian bitmap and per-row index lists).

The paper measures on Q/K/V captured from video diffusion transformers under four dynamic
sparse-attention methods (Section 6.1); none of that data is available, so the generators
below stand in for it.  They reproduce what the text states about those masks: a strong
diagonal, content-dependent scattered blocks (Section 6.6, mask visualisation), correlated
rows (Section 4.3) and widely varying per-row block counts (Section 3.3, root cause 2).

Generator ("videomask"), per head h with numpy Generator default_rng([mask_seed, h]):
  * the sequence is F frames of L_f tokens cut into blocks of b tokens; block i has centre
    token t_i, frame f_i = t_i // L_f and in-frame offset p_i = t_i % L_f;
  * structured candidates by priority: the diagonal block; the +-1..+-w_s neighbours whose
    centre lies in the same frame; for each frame offset +-1..+-F_band the block holding the
    same in-frame offset in that frame;
  * extras: the head owns G pools of ceil(kappa*rho*N_B) random columns, row i belongs to
    pool floor(G*p_i/L_f) (so similar rows sit one frame apart in natural order) and draws
    extras without replacement, from its pool with probability q, else uniformly;
  * the row's block count is n_i = clamp(round(rho_h*N_B*exp(sigma*z - sigma^2/2)), n_min,
    N_B), z ~ N(0,1); candidates are taken in priority order, then extras, until n_i;
  * optional "sink" rows (probability sink_frac) select every block.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional, Sequence, Tuple

import numpy as np


@dataclasses.dataclass(frozen=True)
class Config:
    name: str
    heads: int
    head_dim: int
    seq: int                 # true sequence length S
    block: int               # block_q == block_kv
    frames: int
    frame_tokens: int        # L_f
    rho: Tuple[float, float]  # per-head density drawn uniformly from [lo, hi]
    sigma: float = 0.6
    w_s: Tuple[int, int] = (3, 3)        # spatial half-window for (even, odd) heads
    f_band: Tuple[int, int] = (3, 3)     # temporal band for (even, odd) heads
    pools: int = 12
    pool_q: float = 0.8
    kappa: float = 1.5
    n_min: int = 4
    sink_frac: float = 0.0
    kind: str = "video"      # "video" or "tiny"
    tensor_seed: int = 0
    mask_seed: int = 0
    plan_seed: int = 0

    @property
    def n_blocks(self) -> int:
        return (self.seq + self.block - 1) // self.block

    @property
    def seq_pad(self) -> int:
        return self.n_blocks * self.block


CONFIGS = {
    # tiny correctness case: 4 frames x 1024 tokens, 64x64 blocks, D=64
    "tiny": Config("tiny", heads=2, head_dim=64, seq=4096, block=64, frames=4, frame_tokens=1024,
                   rho=(0.25, 0.25), kind="tiny", tensor_seed=1001, mask_seed=2001, plan_seed=3001),
    # Wan2.1-14B-shaped 480p, 81 frames -> 21 latent frames x 1560 tokens
    "wan480p": Config("wan480p", heads=40, head_dim=128, seq=32760, block=128, frames=21,
                      frame_tokens=1560, rho=(0.15, 0.15), w_s=(3, 3), f_band=(3, 3),
                      tensor_seed=1002, mask_seed=2002, plan_seed=3002),
    # Wan2.1-14B-shaped 720p, 81 frames -> 21 x 3600 tokens; even heads spatial, odd temporal
    "wan720p": Config("wan720p", heads=40, head_dim=128, seq=75600, block=128, frames=21,
                      frame_tokens=3600, rho=(0.10, 0.10), w_s=(12, 1), f_band=(1, 8),
                      tensor_seed=1003, mask_seed=2003, plan_seed=3003),
    # LTX-style mixed sparsity: per-head density 5-30 %, 10 % sink rows, 64x64 blocks
    "ltxmixed": Config("ltxmixed", heads=32, head_dim=128, seq=98304, block=64, frames=64,
                       frame_tokens=1536, rho=(0.05, 0.30), w_s=(3, 3), f_band=(3, 3),
                       sink_frac=0.10, tensor_seed=1004, mask_seed=2004, plan_seed=3004),
    # long-video 720p, 401 frames -> 101 x 3600 tokens
    "long720p": Config("long720p", heads=40, head_dim=128, seq=363600, block=128, frames=101,
                       frame_tokens=3600, rho=(0.04, 0.04), w_s=(2, 2), f_band=(4, 4),
                       tensor_seed=1005, mask_seed=2005, plan_seed=3005),
}
CONFIG_ORDER = ["tiny", "wan480p", "wan720p", "ltxmixed", "long720p"]


def scaled_config(cfg: Config, frames: int, heads: Optional[int] = None, name: Optional[str] = None) -> Config:
    """Same per-frame structure with fewer frames/heads (for oracle-sized parity cases)."""
    return dataclasses.replace(cfg, frames=frames, seq=frames * cfg.frame_tokens,
                               heads=cfg.heads if heads is None else heads,
                               name=name or f"{cfg.name}_f{frames}")


# --------------------------------------------------------------------------- masks

def head_density(cfg: Config, head: int) -> float:
    lo, hi = cfg.rho
    if lo == hi:
        return lo
    rng = np.random.default_rng([cfg.mask_seed, head, 7])
    return float(rng.uniform(lo, hi))


def _structured_priority(cfg: Config, head: int) -> np.ndarray:
    """float32 [N_B, N_B]: negative score for structured candidates (more negative = earlier),
    +inf elsewhere."""
    nb, b, lf = cfg.n_blocks, cfg.block, cfg.frame_tokens
    S = cfg.seq
    i = np.arange(nb)
    centre = np.minimum(i * b + b // 2, S - 1)
    frame = centre // lf
    off = centre % lf
    pri = np.full((nb, nb), np.inf, dtype=np.float32)
    w_s = cfg.w_s[head % 2]
    f_band = cfg.f_band[head % 2]
    if cfg.kind == "tiny":
        w_s, f_band = 2, cfg.frames - 1
    # temporal band (lowest structured priority first so that later writes override)
    for d in range(f_band, 0, -1):
        for sgn in (+1, -1):
            f2 = frame + sgn * d
            ok = (f2 >= 0) & (f2 < cfg.frames)
            tok = f2 * lf + off
            j = np.minimum(tok // b, nb - 1)
            pri[i[ok], j[ok]] = -1.0 + 0.5 * d / (f_band + 1) + (0.01 if sgn < 0 else 0.0)
    # spatial window inside the frame
    for d in range(w_s, 0, -1):
        for sgn in (+1, -1):
            j = i + sgn * d
            ok = (j >= 0) & (j < nb)
            jc = np.clip(j, 0, nb - 1)
            same = ok & (frame[jc] == frame)
            pri[i[same], jc[same]] = -2.0 + 0.5 * d / (w_s + 1) + (0.01 if sgn < 0 else 0.0)
    pri[i, i] = -3.0
    return pri


def make_mask(cfg: Config, head: int) -> np.ndarray:
    """Boolean block mask [M_B, N_B] of one head (M_B == N_B here)."""
    nb = cfg.n_blocks
    rng = np.random.default_rng([cfg.mask_seed, head])
    pri = _structured_priority(cfg, head)
    n_struct = np.isfinite(pri).sum(axis=1)
    if cfg.kind == "tiny":
        extra = 3 + rng.integers(0, 14, size=nb)
        n_row = np.minimum(n_struct + extra, nb)
        weights = np.ones((1, nb), dtype=np.float32)
        pool_of_row = np.zeros(nb, dtype=np.int64)
    else:
        rho = head_density(cfg, head)
        z = rng.standard_normal(nb)
        n_row = np.rint(rho * nb * np.exp(cfg.sigma * z - 0.5 * cfg.sigma ** 2)).astype(np.int64)
        n_row = np.clip(n_row, min(cfg.n_min, nb), nb)
        pool_size = min(nb, max(1, math.ceil(cfg.kappa * rho * nb)))
        weights = np.full((cfg.pools, nb), (1.0 - cfg.pool_q) / nb, dtype=np.float32)
        for g in range(cfg.pools):
            cols = rng.choice(nb, size=pool_size, replace=False)
            weights[g, cols] += cfg.pool_q / pool_size
        i = np.arange(nb)
        centre = np.minimum(i * cfg.block + cfg.block // 2, cfg.seq - 1)
        pool_of_row = (cfg.pools * (centre % cfg.frame_tokens)) // cfg.frame_tokens
        if cfg.sink_frac > 0.0:
            sink = rng.random(nb) < cfg.sink_frac
            n_row = np.where(sink, nb, n_row)
    # exponential race = weighted sampling without replacement; structured candidates win first
    e = rng.standard_exponential(size=(nb, nb), dtype=np.float32)
    score = e / weights[pool_of_row]
    score = np.where(np.isfinite(pri), pri, score)
    order = np.argsort(score, axis=1, kind="stable")
    take = np.arange(nb)[None, :] < n_row[:, None]
    mask = np.zeros((nb, nb), dtype=bool)
    np.put_along_axis(mask, order, take, axis=1)
    return mask


def random_mask(n_q: int, n_kv: int, density: float, seed: int) -> np.ndarray:
    """Unstructured mask: every row keeps round(density*n_kv) uniform columns (the
    'Random' row of Table 1)."""
    rng = np.random.default_rng(seed)
    k = max(1, int(round(density * n_kv)))
    score = rng.random((n_q, n_kv))
    order = np.argsort(score, axis=1)
    mask = np.zeros((n_q, n_kv), dtype=bool)
    np.put_along_axis(mask, order[:, :k], True, axis=1)
    return mask


def mask_to_bitmap(mask: np.ndarray) -> np.ndarray:
    """uint64 [M_B, ceil(N_B/64)]: bit (j & 63) of word (j >> 6) of row i is mask[i, j];
    padding bits are zero."""
    m, n = mask.shape
    words = (n + 63) // 64
    padded = np.zeros((m, words * 64), dtype=np.uint8)
    padded[:, :n] = mask
    by = np.packbits(padded, axis=1, bitorder="little")
    return np.ascontiguousarray(by).view("<u8").reshape(m, words)


def masks_to_csr(masks: Sequence[np.ndarray]) -> Tuple[np.ndarray, np.ndarray]:
    """Index-list form over the flattened (head, row) axis: row_ptr int32 [H*M_B + 1] and
    ascending column indices int32 [nnz]."""
    ptr = [0]
    idx: List[np.ndarray] = []
    total = 0
    for m in masks:
        rows, cols = np.nonzero(m)          # row-major => ascending columns inside each row
        counts = np.bincount(rows, minlength=m.shape[0])
        ptr.extend((total + np.cumsum(counts)).tolist())
        total += int(counts.sum())
        idx.append(cols.astype(np.int32))
    return np.asarray(ptr, dtype=np.int32), (np.concatenate(idx) if idx else np.zeros(0, np.int32))


# --------------------------------------------------------------------------- tensors

TENSOR_IDS = {"q": 0, "k": 1, "v": 2}


def make_head_tensor(cfg: Config, which: str, head: int, value_scale: float = 1.0):
    """bf16 torch tensor [S_pad, D] of one head of Q, K or V: i.i.d. N(0,1) rounded to bf16,
    rows >= S are zero.  Seeded per (config, tensor, head) so any head can be regenerated
    alone (the oracle only needs the sampled heads)."""
    import torch
    g = torch.Generator(device="cpu")
    g.manual_seed(cfg.tensor_seed * 1_000_003 + TENSOR_IDS[which] * 10_007 + head)
    x = torch.randn((cfg.seq, cfg.head_dim), generator=g, dtype=torch.float32)
    if value_scale != 1.0:
        x = x * value_scale
    out = torch.zeros((cfg.seq_pad, cfg.head_dim), dtype=torch.bfloat16)
    out[: cfg.seq] = x.to(torch.bfloat16)
    return out


def bf16_to_f64(t) -> np.ndarray:
    """Exact widening of a bf16 torch tensor to a float64 numpy array."""
    import torch
    return t.to(torch.float64).numpy()
