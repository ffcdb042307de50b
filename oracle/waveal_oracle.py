"""CPU oracle for WaveAlign-scheduled block-sparse attention.  TEST INFRASTRUCTURE ONLY.

This file is the slow, plain, fp64 statement of what the GPU library must compute.  It is
imported by the tests, by the smoke check and by the bench's cpu_baseline / reference
legs, and by nothing on the product path.  It shares no code with the CUDA sources and
imports nothing from the package.

Part A (exact definition): block-sparse softmax attention, Sections 2.1-2.3 of the paper:
each query block attends to the tokens of the K/V blocks its mask row selects.
Part B (a heuristic, followed step by step): the two-stage row reordering of Section 4 -
Algorithm 1 (matrix-free centred subspace iteration), Eq. 4 (polar angle), Algorithm 2
(angular sort, wave-sized buckets, descending block count inside each bucket) - and the
adaptive skip of Section 4.5.
Scores: the objective of Eq. 1 and the intra-wave K/V overlap it stands for.

Pins (tests/test_oracle_*.py): dense mask == textbook softmax attention and torch SDPA;
token-level brute force; closed forms; C twin (oracle_attn.c); Eq. 2 distance preservation;
Eq. 3 against a LAPACK SVD; implicit centred products against the explicit centred matrix;
subspace against numpy SVD on planted masks; Eq. 1 by brute-force pairwise distances;
Stage 2 against Python's sorted(); the Section 4.4 example's ordering relations; the start
block against splitmix64's published outputs; the sign rule on hand-made vectors; the
single-stage plan modes against the stage functions; the ring-cut variant by hand, as a
rotation of the Stage-1 order and by its invariance under rotation of the embedding.
Parity unpinned: the Stage-1 permutation at the working iteration count T (the paper prints
no worked permutation); the guard's numeric thresholds (the paper gives none).
"""
from __future__ import annotations

import math
from collections import OrderedDict
from typing import Dict, Optional, Sequence, Tuple

import numpy as np

# ----------------------------------------------------------------------------- Part A


def attention_block_row(Qb: np.ndarray, K: np.ndarray, V: np.ndarray, kv_blocks: Sequence[int],
                        block_kv: int, seq_kv: int, scale: float) -> Tuple[np.ndarray, np.ndarray]:
    """One query block (Section 2.3: one mask row = one task).

    Qb [rows, D], K/V [>=seq_kv, D], all float64.  The key set is the union of the selected
    K/V blocks' tokens below seq_kv (Section 2.2: only pairs with M_ij = 1 are executed).
    Plain two-pass softmax (Section 2.1): s = scale * q.k, p = exp(s - max s),
    O = sum p v / sum p, LSE = max s + log sum p.  A row that selects nothing gives O = 0,
    LSE = -inf.
    """
    rows, d = Qb.shape
    keys = [np.arange(j * block_kv, min((j + 1) * block_kv, seq_kv)) for j in kv_blocks]
    keys = np.concatenate(keys) if len(keys) else np.zeros(0, dtype=np.int64)
    if keys.size == 0:
        return np.zeros((rows, V.shape[1])), np.full(rows, -np.inf)
    s = scale * (Qb @ K[keys].T)
    m = s.max(axis=1)
    p = np.exp(s - m[:, None])
    l = p.sum(axis=1)
    o = (p @ V[keys]) / l[:, None]
    return o, m + np.log(l)


def block_sparse_attention(Q: np.ndarray, K: np.ndarray, V: np.ndarray, mask: np.ndarray,
                           block_q: int, block_kv: int, seq_q: int, seq_kv: int,
                           scale: Optional[float] = None) -> Tuple[np.ndarray, np.ndarray]:
    """All query blocks of one head.  Returns O [seq_q, D] and LSE [seq_q] (float64)."""
    d = Q.shape[1]
    scale = 1.0 / math.sqrt(d) if scale is None else scale
    out = np.zeros((seq_q, V.shape[1]))
    lse = np.zeros(seq_q)
    for i in range(mask.shape[0]):
        lo, hi = i * block_q, min((i + 1) * block_q, seq_q)
        if lo >= hi:
            break
        o, l = attention_block_row(Q[lo:hi], K, V, np.nonzero(mask[i])[0], block_kv, seq_kv, scale)
        out[lo:hi], lse[lo:hi] = o, l
    return out, lse


# ----------------------------------------------------------------------------- Part B

MODE_AUTO, MODE_FORCE_REORDER, MODE_FORCE_NATURAL, MODE_STAGE1_ONLY, MODE_STAGE2_ONLY = range(5)
FLAG_SKIPPED, FLAG_SHORT_SEQ, FLAG_TOO_SPARSE, FLAG_ALREADY_LOCAL = 1, 2, 4, 8


def row_nnz(mask: np.ndarray) -> np.ndarray:
    """n_i = sum_j M_ij (Section 2.2; Algorithm 2, Stage 2)."""
    return mask.astype(np.int64).sum(axis=1)


def col_count(mask: np.ndarray) -> np.ndarray:
    """c = M^T 1 (Algorithm 1, first step)."""
    return mask.astype(np.int64).sum(axis=0)


_M64 = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15


def _splitmix64(x: int) -> int:
    z = (x + _GOLDEN) & _M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _M64
    return z ^ (z >> 31)


def start_block(seed: int, head: int, m_b: int) -> np.ndarray:
    """The 'random' M_B x 2 start block of Algorithm 1 before orthonormalisation.  The paper
    names no distribution or seed; this reading is a counter-based formula so that any
    implementation can restate it: entry (i, k) = 2u - 1 with
    u = (splitmix64(seed ^ head*golden ^ (2i + k)) >> 11) * 2^-53."""
    x = np.empty((m_b, 2))
    hk = (head * _GOLDEN) & _M64
    for i in range(m_b):
        for k in range(2):
            u = (_splitmix64((seed & _M64) ^ hk ^ (2 * i + k)) >> 11) * (1.0 / 9007199254740992.0)
            x[i, k] = 2.0 * u - 1.0
    return x


def thin_qr2(z: np.ndarray) -> np.ndarray:
    """Q factor of the thin QR of an M_B x 2 block (Algorithm 1, 'X <- Q from Z = QR') by
    Gram-Schmidt with one re-orthogonalisation pass.  A column whose norm is not above
    1e-30*sqrt(M_B), or (second column) not above 1e-9 of its norm before projection, is
    numerically dependent and is returned as zeros (reading for rank-deficient centred
    masks such as the all-ones mask)."""
    m = z.shape[0]
    tiny = 1e-30 * math.sqrt(m)
    q = np.zeros_like(z)
    n1 = math.sqrt(float(z[:, 0] @ z[:, 0]))
    if n1 > tiny:
        q[:, 0] = z[:, 0] / n1
    v = z[:, 1].copy()
    n2_before = math.sqrt(float(v @ v))
    for _ in range(2):
        v = v - float(q[:, 0] @ v) * q[:, 0]
    n2 = math.sqrt(float(v @ v))
    if n2 > tiny and n2 > 1e-9 * n2_before:
        q[:, 1] = v / n2
    return q


def centred_mt_x(mask_f: np.ndarray, c: np.ndarray, x: np.ndarray) -> np.ndarray:
    """Y = M^T X - (1/m) c (1^T X)  (Algorithm 1; the centred transpose product without
    forming the centred matrix)."""
    m = mask_f.shape[0]
    return mask_f.T @ x - np.outer(c, x.sum(axis=0)) / m


def centred_m_y(mask_f: np.ndarray, c: np.ndarray, y: np.ndarray) -> np.ndarray:
    """Z = M Y - (1/m) 1 (c^T Y)  (Algorithm 1)."""
    m = mask_f.shape[0]
    return mask_f @ y - np.ones((m, 1)) * (c @ y)[None, :] / m


def sym2_rotation(a: float, b: float, d: float) -> Tuple[float, float]:
    """(cos t, sin t) of the eigenvector of [[a, b], [b, d]] for the larger eigenvalue:
    t = atan2(2b, a - d) / 2.  Equal eigenvalues (b = 0, a = d) give t = 0."""
    t = 0.5 * math.atan2(2.0 * b, a - d)
    return math.cos(t), math.sin(t)


def fix_sign(u: np.ndarray) -> np.ndarray:
    """Sign convention (the paper says the sort ignores sign flips, which holds only up to a
    reversal of the ring that moves bucket boundaries): make positive the first entry whose
    magnitude reaches half of the largest magnitude."""
    a = np.abs(u)
    mx = a.max() if a.size else 0.0
    if mx == 0.0:
        return u
    i = int(np.argmax(a >= 0.5 * mx))
    return -u if u[i] < 0 else u


def mfcsi(mask: np.ndarray, iters: int, x0: np.ndarray) -> np.ndarray:
    """Algorithm 1.  Returns U [M_B, 2]: approximate top-2 left singular vectors of the
    column-centred mask (Eq. 2), ordered by Ritz value, signs fixed by fix_sign."""
    mf = mask.astype(np.float64)
    c = mf.sum(axis=0)                      # c <- M^T 1
    x = thin_qr2(x0)                        # orthonormal start block
    for _ in range(iters):                  # subspace power iteration
        y = centred_mt_x(mf, c, x)
        z = centred_m_y(mf, c, y)
        x = thin_qr2(z)
    y = centred_mt_x(mf, c, x)              # order by singular value
    z = centred_m_y(mf, c, y)
    b = x.T @ z
    cs, sn = sym2_rotation(b[0, 0], 0.5 * (b[0, 1] + b[1, 0]), b[1, 1])
    r = np.array([[cs, -sn], [sn, cs]])
    x = x @ r
    u = np.stack([fix_sign(x[:, 0]), fix_sign(x[:, 1])], axis=1)
    return u + 0.0                          # -0.0 -> +0.0 so atan2 cannot land on -pi


def polar_angles(u: np.ndarray) -> np.ndarray:
    """a_i = atan2(u_2[i], u_1[i])  (Eq. 4)."""
    return np.arctan2(u[:, 1], u[:, 0])


def stage1_order(angles: np.ndarray) -> np.ndarray:
    """Rows sorted by ascending angle, ties by ascending row index (Algorithm 2, Stage 1)."""
    return np.argsort(angles, kind="stable").astype(np.int64)


def cut_ring_at_largest_gap(order1: np.ndarray, angles: np.ndarray) -> np.ndarray:
    """Variant of Stage 1 (not in the paper's Algorithm 2; Section 4.3.1 says the polar angle
    'unrolls the ring' of rows into a sequence but not where the ring is opened - Eq. 4's atan2
    opens it at -pi, wherever that falls).  Here the ring is opened where two neighbouring rows
    are farthest apart in angle: gaps of the sorted angles, the wrap-around gap
    angle[first] + 2 pi - angle[last] included; the first of equal largest gaps wins; the row
    behind the gap becomes the first of the sequence.  The result is a rotation of order1."""
    m = len(order1)
    if m < 2:
        return order1.copy()
    a = angles[order1]
    gaps = np.empty(m)
    gaps[:m - 1] = a[1:] - a[:-1]
    gaps[m - 1] = (a[0] + 2.0 * math.pi) - a[m - 1]
    k = int(np.argmax(gaps))               # first maximum
    return np.concatenate([order1[k + 1:], order1[:k + 1]])


def stage2_order(order1: np.ndarray, nnz: np.ndarray, wave: int) -> np.ndarray:
    """Algorithm 2, Stage 2: consecutive buckets of at most `wave` rows of order1; inside a
    bucket, descending block count, ties keeping their Stage-1 order; concatenate."""
    out = []
    for lo in range(0, len(order1), wave):
        bucket = order1[lo:lo + wave]
        keys = -nnz[bucket]
        out.append(bucket[np.argsort(keys, kind="stable")])
    return np.concatenate(out) if out else np.zeros(0, dtype=np.int64)


def wave_column_counts(mask: np.ndarray, order: np.ndarray, wave: int) -> np.ndarray:
    """c[l, j] = number of rows of wave l (consecutive chunks of `wave` of `order`) that
    touch column j."""
    mi = mask.astype(np.int64)[order]
    n_w = (len(order) + wave - 1) // wave
    return np.stack([mi[l * wave:(l + 1) * wave].sum(axis=0) for l in range(n_w)]) if n_w else \
        np.zeros((0, mask.shape[1]), dtype=np.int64)


def scores(mask: np.ndarray, order: np.ndarray, wave: int) -> Dict[str, int]:
    """Integer scores of an execution order.
    Ov: (row pair, shared column) incidences inside waves - the K/V-block overlap among rows
        of the same wave that Section 4.2 says is to be maximised.
    J:  the objective of Eq. 1 summed over ordered row pairs of each wave; for binary rows
        |a - b|^2 = n_a + n_b - 2<a, b>, which gives J = sum_l 2(|l| t_l - sum_j c_lj^2).
    U:  summed per-wave union sizes (distinct K/V blocks a wave touches)."""
    c = wave_column_counts(mask, order, wave)
    sizes = np.array([min(wave, len(order) - l * wave) for l in range(c.shape[0])], dtype=np.int64)
    t = c.sum(axis=1)
    ov = int((c * (c - 1) // 2).sum())
    j = int((2 * (sizes * t - (c * c).sum(axis=1))).sum())
    u = int((c > 0).sum())
    return {"Ov": ov, "J": j, "U": u}


def guard_stats(mask: np.ndarray, wave: int) -> Dict[str, int]:
    """Statistics the skip test uses: nnz, and the natural-order locality ratio
    lambda = ov_nat / pair_half with ov_nat = sum_l Ov_l(identity) and
    2*pair_half = sum_l (w_l - 1) t_l  (lambda = 1 iff all rows of every wave coincide)."""
    ident = np.arange(mask.shape[0])
    c = wave_column_counts(mask, ident, wave)
    sizes = np.array([min(wave, mask.shape[0] - l * wave) for l in range(c.shape[0])], dtype=np.int64)
    t = c.sum(axis=1)
    return {"nnz": int(mask.sum()), "ov_nat": int((c * (c - 1) // 2).sum()),
            "pair2": int(((sizes - 1) * t).sum())}


DEFAULT_GUARD = dict(kv_bytes_per_head=0, l2_bytes=0, l2_fit_num=9, l2_fit_den=16,
                     min_density_ppm=10000, min_nnz=0, local_num=1, local_den=2)


def guard_flags(mask: np.ndarray, wave: int, g: Dict[str, int]) -> int:
    """Adaptive skip (Section 4.5), decided before reordering, as integer comparisons:
    short sequence: kv_bytes * den <= l2_bytes * num (one head's K+V fit the cache budget;
    tested only when both byte counts are positive);
    too sparse: nnz < min_nnz or nnz * 1e6 < min_density_ppm * M_B * N_B;
    already local: 2 * ov_nat * local_den >= local_num * pair2 (and pair2 > 0).
    Returns the reason bits (FLAG_SHORT_SEQ | FLAG_TOO_SPARSE | FLAG_ALREADY_LOCAL)."""
    st = guard_stats(mask, wave)
    m_b, n_b = mask.shape
    flags = 0
    if g["kv_bytes_per_head"] > 0 and g["l2_bytes"] > 0 and \
            g["kv_bytes_per_head"] * g["l2_fit_den"] <= g["l2_bytes"] * g["l2_fit_num"]:
        flags |= FLAG_SHORT_SEQ
    if st["nnz"] < g["min_nnz"] or st["nnz"] * 1_000_000 < g["min_density_ppm"] * m_b * n_b:
        flags |= FLAG_TOO_SPARSE
    if st["pair2"] > 0 and 2 * st["ov_nat"] * g["local_den"] >= g["local_num"] * st["pair2"]:
        flags |= FLAG_ALREADY_LOCAL
    return flags


def plan_head(mask: np.ndarray, wave: int, iters: int, seed: int, head: int,
              mode: int = MODE_AUTO, guard: Optional[Dict[str, int]] = None,
              ring_cut: bool = False) -> Dict[str, np.ndarray]:
    """Algorithm 2 for one head, with the guard of Section 4.5 in front.
    Returns row_order (index list: position -> original row), order1 (Stage-1 order),
    row_nnz, col_count, u, angles and flags.  ring_cut=True opens the angular ring at its
    largest gap instead of at -pi (cut_ring_at_largest_gap; a variant, off by default)."""
    g = dict(DEFAULT_GUARD)
    if guard:
        g.update(guard)
    m_b = mask.shape[0]
    nnz = row_nnz(mask)
    flags = guard_flags(mask, wave, g)
    ident = np.arange(m_b, dtype=np.int64)
    skip = (mode == MODE_FORCE_NATURAL) or (mode == MODE_AUTO and flags != 0)
    res = {"row_nnz": nnz, "col_count": col_count(mask)}
    if skip:
        res.update(row_order=ident, order1=ident, flags=flags | FLAG_SKIPPED,
                   u=np.zeros((m_b, 2)), angles=np.zeros(m_b))
        return res
    if mode == MODE_STAGE2_ONLY:
        u = np.zeros((m_b, 2))
        ang = np.zeros(m_b)
        order1 = ident
    else:
        u = mfcsi(mask, iters, start_block(seed, head, m_b))
        ang = polar_angles(u)
        order1 = stage1_order(ang)
        if ring_cut:
            order1 = cut_ring_at_largest_gap(order1, ang)
    order = order1 if mode == MODE_STAGE1_ONLY else stage2_order(order1, nnz, wave)
    res.update(row_order=order, order1=order1, flags=flags, u=u, angles=ang)
    return res


def gather_blocks(x: np.ndarray, order: np.ndarray, block: int) -> np.ndarray:
    """Reorder operator of Section 5: block p of the result is block order[p] of x
    (x: [n_blocks*block, ...])."""
    n = len(order)
    return x.reshape(n, block, *x.shape[1:])[order].reshape(x.shape)


def scatter_blocks(x: np.ndarray, order: np.ndarray, block: int) -> np.ndarray:
    """Inverse operator of Section 5: block order[p] of the result is block p of x."""
    n = len(order)
    out = np.empty_like(x).reshape(n, block, *x.shape[1:])
    out[order] = x.reshape(n, block, *x.shape[1:])
    return out.reshape(x.shape)


# ----------------------------------------------------------------------------- wave model


def lru_wave_model(mask: np.ndarray, order: np.ndarray, workers: int, capacity: int) -> Dict[str, float]:
    """Streaming execution model of Section 2.3: `workers` SMs, each walks its row's K/V
    blocks in ascending order, one block per time step; a worker that finishes takes the
    next row of `order` at once (a wave is not a barrier).  Blocks pass through a fully
    associative LRU cache of `capacity` blocks.  Returns accesses, hits and hit rate.
    Explanatory tool only (not a parity target)."""
    lists = [np.nonzero(mask[r])[0] for r in order]
    nxt = 0
    cur = [None] * workers          # (list, position)
    cache: "OrderedDict[int, None]" = OrderedDict()
    hits = acc = 0
    active = 0
    for w in range(workers):
        if nxt < len(lists):
            cur[w] = [lists[nxt], 0]
            nxt += 1
            active += 1
    while active:
        for w in range(workers):
            st = cur[w]
            if st is None:
                continue
            while st is not None and st[1] >= len(st[0]):
                if nxt < len(lists):
                    st = cur[w] = [lists[nxt], 0]
                    nxt += 1
                else:
                    st = cur[w] = None
                    active -= 1
            if st is None:
                continue
            j = int(st[0][st[1]])
            st[1] += 1
            acc += 1
            if j in cache:
                hits += 1
                cache.move_to_end(j)
            else:
                cache[j] = None
                if len(cache) > capacity:
                    cache.popitem(last=False)
    return {"accesses": acc, "hits": hits, "hit_rate": hits / acc if acc else 0.0}
