"""Pins for the reordering part of the CPU oracle (no GPU)."""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import waveal_oracle as wo
from paper_2609_34814_b200 import inputs as I

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _mask(m, n, p, seed):
    mk = np.random.default_rng(seed).random((m, n)) < p
    mk[np.arange(min(m, n)), np.arange(min(m, n))] = True
    return mk


def test_counts_bruteforce():
    mk = _mask(13, 70, 0.3, 1)
    nnz = [sum(1 for j in range(70) if mk[i, j]) for i in range(13)]
    cc = [sum(1 for i in range(13) if mk[i, j]) for j in range(70)]
    assert wo.row_nnz(mk).tolist() == nnz and wo.col_count(mk).tolist() == cc
    assert sum(nnz) == sum(cc) == int(mk.sum())


def test_centering_preserves_row_distances_eq2():
    mk = _mask(20, 30, 0.3, 2).astype(float)
    mt = mk - mk.mean(axis=0, keepdims=True)          # (I - 11^T/M_B) M
    for i, j in itertools.combinations(range(20), 2):
        assert abs(np.linalg.norm(mt[i] - mt[j]) - np.linalg.norm(mk[i] - mk[j])) < 1e-12
    assert np.abs(mt.sum(axis=0)).max() < 1e-12       # 1^T M~ = 0


def test_distance_decomposition_eq3():
    mk = _mask(24, 40, 0.35, 3).astype(float)
    mt = mk - mk.mean(axis=0, keepdims=True)
    u, s, vt = np.linalg.svd(mt, full_matrices=False)
    for i, j in [(0, 5), (3, 17), (10, 23)]:
        lhs = np.sum((mt[i] - mt[j]) ** 2)
        rhs = np.sum(s ** 2 * (u[i] - u[j]) ** 2)
        assert abs(lhs - rhs) < 1e-10


def test_implicit_centred_products_equal_explicit():
    mk = _mask(17, 29, 0.3, 4)
    mf = mk.astype(float)
    mt = mf - mf.mean(axis=0, keepdims=True)
    c = mf.sum(axis=0)
    rng = np.random.default_rng(0)
    x = rng.standard_normal((17, 2))
    y = rng.standard_normal((29, 2))
    assert np.abs(wo.centred_mt_x(mf, c, x) - mt.T @ x).max() < 1e-12
    assert np.abs(wo.centred_m_y(mf, c, y) - mt @ y).max() < 1e-12


def test_thin_qr_orthonormal_and_span():
    z = np.random.default_rng(1).standard_normal((50, 2))
    q = wo.thin_qr2(z)
    assert np.abs(q.T @ q - np.eye(2)).max() < 1e-14
    qr, _ = np.linalg.qr(z)
    assert np.abs(q @ q.T - qr @ qr.T).max() < 1e-13   # same column space as LAPACK's QR
    # dependent second column and zero block
    q = wo.thin_qr2(np.stack([z[:, 0], 3 * z[:, 0]], axis=1))
    assert np.abs(q[:, 1]).max() == 0 and abs(np.linalg.norm(q[:, 0]) - 1) < 1e-14
    assert np.abs(wo.thin_qr2(np.zeros((9, 2)))).max() == 0


def test_sym2_rotation_against_eigh():
    rng = np.random.default_rng(2)
    for _ in range(50):
        a, b, d = rng.standard_normal(3)
        cs, sn = wo.sym2_rotation(a, b, d)
        w, v = np.linalg.eigh(np.array([[a, b], [b, d]]))
        assert abs(abs(cs * v[0, 1] + sn * v[1, 1]) - 1) < 1e-12   # parallel to the top eigenvector
    assert wo.sym2_rotation(2.0, 0.0, 1.0) == (1.0, 0.0)
    cs, sn = wo.sym2_rotation(1.0, 0.0, 2.0)
    assert abs(cs) < 1e-15 and abs(sn - 1) < 1e-15


def _planted(groups, rows_per, cols_per, seed):
    """k groups of identical rows with disjoint supports, shuffled."""
    k = groups
    mk = np.zeros((k * rows_per, k * cols_per), dtype=bool)
    for g in range(k):
        mk[g * rows_per:(g + 1) * rows_per, g * cols_per:(g + 1) * cols_per] = True
    perm = np.random.default_rng(seed).permutation(k * rows_per)
    return mk[perm], perm // rows_per


@pytest.mark.parametrize("k,sizes", [(3, (10, 8)), (4, (12, 5))])
def test_mfcsi_converges_to_svd_subspace_on_planted_masks(k, sizes):
    rows_per, cols_per = sizes
    # unequal group widths give a clear spectral gap: widen group g by g columns
    mk = np.zeros((k * rows_per, k * cols_per + k * (k - 1) // 2), dtype=bool)
    col = 0
    for g in range(k):
        wdt = cols_per + g
        mk[g * rows_per:(g + 1) * rows_per, col:col + wdt] = True
        col += wdt
    perm = np.random.default_rng(7).permutation(k * rows_per)
    mk = mk[perm]
    label = perm // rows_per
    u = wo.mfcsi(mk, 300, wo.start_block(5, 0, mk.shape[0]))
    mt = mk.astype(float) - mk.mean(axis=0, keepdims=True)
    us, s, _ = np.linalg.svd(mt, full_matrices=False)
    if k == 3:
        # centred rank is k-1 = 2: the top-2 subspace is the whole row-space image
        cosines = np.linalg.svd(u.T @ us[:, :2], compute_uv=False)
        assert cosines.min() > 1 - 1e-8
    else:
        assert s[1] - s[2] > 1e-3
        cosines = np.linalg.svd(u.T @ us[:, :2], compute_uv=False)
        assert cosines.min() > 1 - 1e-8
        # Ritz ordering: first column is the dominant singular vector
        assert abs(abs(u[:, 0] @ us[:, 0]) - 1) < 1e-7
    assert np.abs(u.T @ u - np.eye(2)).max() < 1e-12
    assert np.abs(u.sum(axis=0)).max() < 1e-10            # retained directions are orthogonal to 1
    # Stage 1 makes each group contiguous (identical rows share one angle)
    order1 = wo.stage1_order(wo.polar_angles(u))
    lab = label[order1]
    changes = int((lab[1:] != lab[:-1]).sum())
    assert changes == k - 1


def test_all_ones_and_identical_rows_degenerate_to_natural_order():
    mk = np.ones((12, 9), dtype=bool)
    res = wo.plan_head(mk, 4, 10, 1, 0, mode=wo.MODE_FORCE_REORDER)
    assert res["order1"].tolist() == list(range(12))
    assert res["row_order"].tolist() == list(range(12))
    assert np.isfinite(res["u"]).all()


def test_stage2_against_python_sorted():
    rng = np.random.default_rng(3)
    order1 = rng.permutation(37)
    nnz = rng.integers(1, 6, size=37)
    out = wo.stage2_order(order1, nnz, 8)
    exp = []
    for lo in range(0, 37, 8):
        b = list(order1[lo:lo + 8])
        exp += sorted(b, key=lambda r: -nnz[r])        # Python's sort is stable
    assert out.tolist() == exp
    assert sorted(out.tolist()) == list(range(37))


def _read_golden():
    vals = {}
    for line in open(os.path.join(GOLDEN, "stage2_example.txt")):
        if line.startswith("#") or not line.strip():
            continue
        k, *v = line.split()
        vals[k] = [int(x) for x in v]
    return vals


def test_section_4_4_example_relations():
    g = _read_golden()
    nnz = np.array(g["nnz"])
    W = g["sms"][0]
    ident = np.arange(g["rows"][0])
    out = wo.stage2_order(ident, nnz, W)
    assert out[0] == 4 and out[W - 1] == 6              # R2
    assert out[W] == 11 and out[W + 1] == 12            # R3
    # streaming model (Section 2.3): a freed SM takes the next row of the list at once
    def successor(order):
        """{row that finished: row its SM took next}, one K/V block per time step."""
        left = [int(nnz[order[w]]) for w in range(W)]
        running = [int(order[w]) for w in range(W)]
        nxt, succ = W, {}
        while nxt < 2 * W:
            for w in range(W):
                left[w] -= 1
                if left[w] == 0 and nxt < 2 * W:
                    succ[running[w]] = int(order[nxt])
                    running[w], left[w] = int(order[nxt]), int(nnz[order[nxt]])
                    nxt += 1
        return succ
    s_nat = successor(ident)
    assert s_nat[6] == 8 and s_nat[5] == 9              # R1
    s_sorted = successor(out)
    assert s_sorted[6] == 11 and s_sorted[5] == 12      # R3


def test_scores_bruteforce_eq1():
    mk = _mask(23, 31, 0.3, 8)
    order = np.random.default_rng(1).permutation(23)
    W = 5
    sc = wo.scores(mk, order, W)
    mf = mk.astype(float)
    J = Ov = U = 0
    for lo in range(0, 23, W):
        rows = order[lo:lo + W]
        for a in rows:
            for b in rows:
                J += np.sum((mf[a] - mf[b]) ** 2)       # Eq. 1 over ordered pairs
        for a, b in itertools.combinations(rows, 2):
            Ov += int((mk[a] & mk[b]).sum())
        U += int(mk[rows].any(axis=0).sum())
    assert sc == {"Ov": Ov, "J": int(round(J)), "U": U}
    # invariance under the order inside a wave (isolates Stage 1)
    o2 = order.copy()
    o2[:W] = o2[:W][::-1]
    assert wo.scores(mk, o2, W) == sc


def test_start_block_is_counter_based_and_in_range():
    a = wo.start_block(42, 3, 64)
    b = wo.start_block(42, 3, 128)
    assert np.array_equal(a, b[:64])                     # entry depends only on (seed, head, i, k)
    assert (np.abs(a) <= 1).all() and abs(a.mean()) < 0.2
    assert not np.array_equal(a, wo.start_block(42, 4, 64))
    # splitmix64 reference value: first output of the generator seeded with 0
    assert wo._splitmix64(0) == 0xE220A8397B1DCDAF


# the first three outputs of the published splitmix64 generator started from state 0 (the
# generator adds the golden-ratio constant to its state before every mix, so output n is the
# mix of n * golden)
SPLITMIX_SEED0 = (0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F)
GOLDEN64 = 0x9E3779B97F4A7C15


def _unit(z):
    """2u - 1 with u the top 53 bits of z as a fraction of 2^53, in exact integer arithmetic."""
    from fractions import Fraction
    return float(2 * Fraction(z >> 11, 1 << 53) - 1)


def test_start_block_known_answers_fix_the_index_mixing():
    o1, o2, o3 = SPLITMIX_SEED0
    assert wo._splitmix64(GOLDEN64) == o2 and wo._splitmix64((2 * GOLDEN64) & (2 ** 64 - 1)) == o3
    # seed 0, head 0: entry (0, 0) mixes counter 0
    x = wo.start_block(0, 0, 4)
    assert x[0, 0] == _unit(o1)
    # the head enters as head * golden: head 1 / head 2 at counter 0 are outputs two and three
    assert wo.start_block(0, 1, 4)[0, 0] == _unit(o2)
    assert wo.start_block(0, 2, 4)[0, 0] == _unit(o3)
    # the seed is xor-ed in: seed = golden cancels head 1, seed = golden at head 0 is output two
    assert wo.start_block(GOLDEN64, 1, 4)[0, 0] == _unit(o1)
    assert wo.start_block(GOLDEN64, 0, 4)[0, 0] == _unit(o2)
    # the counter of entry (i, k) is 2i + k: seed 5 cancels it at (2, 1) only, seed 6 at (3, 0) only
    x5 = wo.start_block(5, 0, 4)
    assert x5[2, 1] == _unit(o1) and (x5 == _unit(o1)).sum() == 1
    x6 = wo.start_block(6, 0, 4)
    assert x6[3, 0] == _unit(o1) and (x6 == _unit(o1)).sum() == 1
    x5h = wo.start_block(5, 1, 4)
    assert x5h[2, 1] == _unit(o2) and (x5h == _unit(o2)).sum() == 1
    # value map: o1 has its top bit set, o3 does not, so the signs differ
    assert 0.76 < _unit(o1) < 0.77 and _unit(o3) < -0.94


def test_fix_sign_is_flip_invariant_and_picks_the_first_large_entry():
    rng = np.random.default_rng(0)
    for _ in range(20):
        u = rng.standard_normal(17)
        a, b = wo.fix_sign(u), wo.fix_sign(-u)
        assert np.array_equal(a, b)
        assert np.array_equal(np.abs(a), np.abs(u))
        i = int(np.nonzero(np.abs(u) >= 0.5 * np.abs(u).max())[0][0])
        assert a[i] > 0
    # symmetric +- ties of the largest magnitude: the first qualifying entry decides, not the maximum
    u = np.array([0.1, -0.6, 1.0, -1.0, 0.6])
    assert wo.fix_sign(u).tolist() == [-0.1, 0.6, -1.0, 1.0, -0.6]
    assert wo.fix_sign(-u).tolist() == [-0.1, 0.6, -1.0, 1.0, -0.6]
    # an entry just below half of the maximum does not qualify
    u = np.array([-0.49, 1.0, -1.0])
    assert wo.fix_sign(u).tolist() == [-0.49, 1.0, -1.0]
    u = np.array([-0.5, 1.0, -1.0])
    assert wo.fix_sign(u).tolist() == [0.5, -1.0, 1.0]
    assert wo.fix_sign(np.zeros(4)).tolist() == [0, 0, 0, 0]


def test_plan_head_ablation_modes_are_the_single_stages():
    cfg = I.CONFIGS["wan480p"]
    mk = I.make_mask(cfg, 2)
    W = 37
    ident = np.arange(cfg.n_blocks)
    s1 = wo.plan_head(mk, W, 5, 9, 2, mode=wo.MODE_STAGE1_ONLY)
    both = wo.plan_head(mk, W, 5, 9, 2, mode=wo.MODE_FORCE_REORDER)
    s2 = wo.plan_head(mk, W, 5, 9, 2, mode=wo.MODE_STAGE2_ONLY)
    nat = wo.plan_head(mk, W, 5, 9, 2, mode=wo.MODE_FORCE_NATURAL)
    # Stage 1 alone: the angular order, untouched by the per-wave sort, and the same one S1+S2 starts from
    assert np.array_equal(s1["row_order"], s1["order1"])
    assert np.array_equal(s1["order1"], both["order1"])
    assert np.array_equal(s1["order1"], wo.stage1_order(wo.polar_angles(s1["u"])))
    assert not np.array_equal(s1["row_order"], ident)
    # Stage 2 alone: natural order cut into waves, each sorted by descending count (no embedding)
    assert np.array_equal(s2["order1"], ident)
    assert np.array_equal(s2["row_order"], wo.stage2_order(ident, wo.row_nnz(mk), W))
    exp = []
    for lo in range(0, cfg.n_blocks, W):
        exp += sorted(range(lo, min(lo + W, cfg.n_blocks)), key=lambda r: -int(mk[r].sum()))
    assert s2["row_order"].tolist() == exp
    assert np.abs(s2["u"]).max() == 0
    # S1+S2 = Stage 2 applied to Stage 1's order
    assert np.array_equal(both["row_order"], wo.stage2_order(s1["order1"], wo.row_nnz(mk), W))
    assert np.array_equal(nat["row_order"], ident) and nat["flags"] & wo.FLAG_SKIPPED


def test_plan_is_valid_permutation_and_bucket_invariants():
    cfg = I.CONFIGS["wan480p"]
    mk = I.make_mask(cfg, 1)
    W = 37
    res = wo.plan_head(mk, W, 10, cfg.plan_seed, 1, mode=wo.MODE_FORCE_REORDER)
    order, order1, nnz = res["row_order"], res["order1"], res["row_nnz"]
    assert sorted(order.tolist()) == list(range(cfg.n_blocks))
    for lo in range(0, len(order), W):
        assert sorted(order[lo:lo + W]) == sorted(order1[lo:lo + W])
        n = nnz[order[lo:lo + W]]
        assert (n[:-1] >= n[1:]).all()
    # the reordering raises intra-wave overlap on a video-shaped mask
    ident = np.arange(cfg.n_blocks)
    assert wo.scores(mk, order, W)["Ov"] > wo.scores(mk, ident, W)["Ov"]


def test_guard_cases():
    g = dict(wo.DEFAULT_GUARD)
    mk = _mask(64, 64, 0.3, 1)
    # short sequence: the head's K+V fit the cache budget
    f = wo.guard_flags(mk, 8, {**g, "kv_bytes_per_head": 10, "l2_bytes": 100})
    assert f & wo.FLAG_SHORT_SEQ
    f = wo.guard_flags(mk, 8, {**g, "kv_bytes_per_head": 56, "l2_bytes": 100})      # 56/100 <= 9/16
    assert f & wo.FLAG_SHORT_SEQ
    f = wo.guard_flags(mk, 8, {**g, "kv_bytes_per_head": 57, "l2_bytes": 100})
    assert not f & wo.FLAG_SHORT_SEQ
    # too sparse
    sparse = np.eye(200, dtype=bool)
    assert wo.guard_flags(sparse, 8, g) & wo.FLAG_TOO_SPARSE
    assert not wo.guard_flags(mk, 8, g) & wo.FLAG_TOO_SPARSE
    # already local: every wave's rows identical
    loc = np.zeros((32, 64), dtype=bool)
    for l in range(4):
        loc[l * 8:(l + 1) * 8, l * 10:l * 10 + 12] = True
    st = wo.guard_stats(loc, 8)
    assert 2 * st["ov_nat"] == st["pair2"]               # lambda == 1
    assert wo.guard_flags(loc, 8, g) & wo.FLAG_ALREADY_LOCAL
    assert not wo.guard_flags(_mask(64, 64, 0.1, 3), 8, g) & wo.FLAG_ALREADY_LOCAL
    # AUTO applies the skip, FORCE_REORDER does not
    res = wo.plan_head(loc, 8, 5, 1, 0, mode=wo.MODE_AUTO)
    assert res["flags"] & wo.FLAG_SKIPPED and res["row_order"].tolist() == list(range(32))
    res = wo.plan_head(loc, 8, 5, 1, 0, mode=wo.MODE_FORCE_REORDER)
    assert not res["flags"] & wo.FLAG_SKIPPED


def test_lru_model_orders_the_ablation_as_the_paper_does():
    # Section 6.5: Original < O+S1, O+S2 < O+S1+S2 in L2 hit ratio
    cfg = I.scaled_config(I.CONFIGS["long720p"], frames=24, heads=1)
    mk = I.make_mask(cfg, 0)
    W, cap = 32, 120
    rates = {}
    for name, mode in [("orig", wo.MODE_FORCE_NATURAL), ("s1", wo.MODE_STAGE1_ONLY),
                       ("s2", wo.MODE_STAGE2_ONLY), ("both", wo.MODE_FORCE_REORDER)]:
        order = wo.plan_head(mk, W, 10, 1, 0, mode=mode)["row_order"]
        rates[name] = wo.lru_wave_model(mk, order, W, cap)["hit_rate"]
    assert rates["both"] > rates["orig"]
    assert rates["both"] >= max(rates["s1"], rates["s2"]) - 0.02
    # trivial cache checks: capacity >= all blocks -> only compulsory misses
    full = wo.lru_wave_model(mk, np.arange(mk.shape[0]), W, mk.shape[1])
    assert full["accesses"] == int(mk.sum())
    assert full["accesses"] - full["hits"] == int(mk.any(axis=0).sum())


def test_gather_scatter_blocks_are_inverse_and_match_loops():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((6 * 4, 3))
    order = rng.permutation(6)
    g = wo.gather_blocks(x, order, 4)
    for p in range(6):
        assert np.array_equal(g[p * 4:(p + 1) * 4], x[order[p] * 4:(order[p] + 1) * 4])
    assert np.array_equal(wo.scatter_blocks(g, order, 4), x)


def test_ring_cut_by_hand_and_is_a_rotation():
    # sorted angles -3.0, -2.9, 0.1, 0.2, 3.0: gaps 0.1, 3.0, 0.1, 2.8 and 0.283 around the back
    ang = np.array([-3.0, -2.9, 0.1, 0.2, 3.0])
    o1 = wo.stage1_order(ang)
    assert o1.tolist() == [0, 1, 2, 3, 4]
    assert wo.cut_ring_at_largest_gap(o1, ang).tolist() == [2, 3, 4, 0, 1]
    # the wrap-around gap is the largest: nothing moves
    ang = np.array([0.5, -0.5, 0.0, 1.0])
    o1 = wo.stage1_order(ang)
    assert wo.cut_ring_at_largest_gap(o1, ang).tolist() == o1.tolist() == [1, 2, 0, 3]
    # equal largest gaps: the first one in sorted order
    ang = np.array([-2.0, -1.0, 0.0, 1.0])      # gaps 1, 1, 1 and 2 pi - 3 = 3.28 around the back
    assert wo.cut_ring_at_largest_gap(wo.stage1_order(ang), ang).tolist() == [0, 1, 2, 3]
    ang = np.array([-3.0, -1.0, 1.0, 3.0])      # gaps 2, 2, 2, 0.283: the first 2
    assert wo.cut_ring_at_largest_gap(wo.stage1_order(ang), ang).tolist() == [1, 2, 3, 0]
    # all angles equal (degenerate embedding): natural order stays
    z = np.zeros(7)
    assert wo.cut_ring_at_largest_gap(wo.stage1_order(z), z).tolist() == list(range(7))
    # random: a rotation of the Stage-1 order, and first/last are the two rows across the largest circular gap
    rng = np.random.default_rng(4)
    ang = rng.uniform(-math.pi, math.pi, 41)
    o1 = wo.stage1_order(ang)
    oc = wo.cut_ring_at_largest_gap(o1, ang)
    doubled = np.concatenate([o1, o1]).tolist()
    assert any(doubled[i:i + 41] == oc.tolist() for i in range(41))
    circ = lambda a, b: (ang[b] - ang[a]) % (2 * math.pi)        # going up from a to b around the ring
    best = max(circ(o1[i], o1[(i + 1) % 41]) for i in range(41))
    assert abs(circ(oc[-1], oc[0]) - best) < 1e-12


def test_ring_cut_is_invariant_under_rotation_of_the_embedding_and_keeps_groups_whole():
    rng = np.random.default_rng(9)
    ang = rng.uniform(-math.pi, math.pi, 60)
    base = wo.cut_ring_at_largest_gap(wo.stage1_order(ang), ang)
    wrap = lambda a: (a + math.pi) % (2 * math.pi) - math.pi
    for theta in (0.3, 1.7, 3.0, -2.2):
        rot = wrap(ang + theta)
        assert wo.cut_ring_at_largest_gap(wo.stage1_order(rot), rot).tolist() == base.tolist()
        # the plain -pi cut is not invariant: it starts wherever -pi happens to fall
    assert any(wo.stage1_order(wrap(ang + t)).tolist() != wo.stage1_order(ang).tolist() for t in (0.3, 1.7))
    # three tight groups, one of them straddling +-pi: the -pi cut splits it, the largest-gap cut does not
    lab = np.repeat([0, 1, 2], 8)
    centre = np.array([math.pi, -1.0, 1.0])
    a = wrap(centre[lab] + rng.uniform(-0.05, 0.05, 24))
    runs = lambda o: int((lab[o][1:] != lab[o][:-1]).sum())
    assert runs(wo.stage1_order(a)) == 3
    oc = wo.cut_ring_at_largest_gap(wo.stage1_order(a), a)
    assert runs(oc) == 2
    # with one wave per group the overlap score of identical-row groups can only gain
    mk = np.zeros((24, 30), dtype=bool)
    for g in range(3):
        mk[lab == g, g * 10:(g + 1) * 10] = True
    s_cut, s_pi = wo.scores(mk, oc, 8), wo.scores(mk, wo.stage1_order(a), 8)
    assert s_cut["Ov"] > s_pi["Ov"] and s_cut["U"] < s_pi["U"]


def test_plan_head_with_ring_cut_is_valid_and_not_worse_on_planted_masks():
    mk, label = _planted(4, 12, 6, 3)
    W = 12
    a = wo.plan_head(mk, W, 40, 5, 0, mode=wo.MODE_FORCE_REORDER)
    b = wo.plan_head(mk, W, 40, 5, 0, mode=wo.MODE_FORCE_REORDER, ring_cut=True)
    assert sorted(b["row_order"].tolist()) == list(range(48))
    assert np.array_equal(b["order1"], wo.cut_ring_at_largest_gap(a["order1"], a["angles"]))
    assert np.array_equal(b["row_order"], wo.stage2_order(b["order1"], wo.row_nnz(mk), W))
    sa, sb = wo.scores(mk, a["row_order"], W), wo.scores(mk, b["row_order"], W)
    assert sb["Ov"] >= sa["Ov"] and sb["U"] <= sa["U"]
    lab = label[b["order1"]]
    assert int((lab[1:] != lab[:-1]).sum()) == 3            # every group in one piece
