"""Pins for the attention part of the CPU oracle (no GPU)."""
import math

import numpy as np
import pytest
import torch

from oracle import waveal_oracle as wo
from oracle import c_twin
from paper_2609_34814_b200 import inputs as I


def _rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


def test_dense_mask_equals_textbook_softmax():
    # Section 2.2: dense attention computes every (Q_i, K_j) pair -> all-ones mask == softmax(QK^T)V
    S, D, b = 96, 16, 32
    Q, K, V = _rand((S, D), 1), _rand((S, D), 2), _rand((S, D), 3)
    mask = np.ones((3, 3), dtype=bool)
    o, lse = wo.block_sparse_attention(Q, K, V, mask, b, b, S, S)
    s = Q @ K.T / math.sqrt(D)
    w = np.exp(s - s.max(1, keepdims=True))
    ref = (w / w.sum(1, keepdims=True)) @ V
    assert np.abs(o - ref).max() < 1e-13
    ref_lse = np.log(np.exp(s).sum(1))
    assert np.abs(lse - ref_lse).max() < 1e-12
    sd = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(Q)[None], torch.from_numpy(K)[None], torch.from_numpy(V)[None])[0].numpy()
    assert np.abs(o - sd).max() < 1e-12


@pytest.mark.parametrize("seq", [160, 150])   # 150: ragged last block
def test_sparse_equals_token_level_bruteforce(seq):
    D, b = 8, 32
    nb = (seq + b - 1) // b
    rng = np.random.default_rng(5)
    mask = rng.random((nb, nb)) < 0.4
    mask[np.arange(nb), np.arange(nb)] = True
    Q, K, V = _rand((nb * b, D), 11), _rand((nb * b, D), 12), _rand((nb * b, D), 13)
    o, lse = wo.block_sparse_attention(Q, K, V, mask, b, b, seq, seq, scale=0.3)
    # a different formulation: token-level additive -inf mask on the dense score matrix
    tok = np.repeat(np.repeat(mask, b, axis=0), b, axis=1)[:seq, :seq]
    s = 0.3 * Q[:seq] @ K[:seq].T
    s = np.where(tok, s, -np.inf)
    w = np.exp(s - s.max(1, keepdims=True))
    ref = (w / w.sum(1, keepdims=True)) @ V[:seq]
    assert np.abs(o - ref).max() < 1e-13


def test_closed_forms():
    S, D, b = 128, 8, 32
    rng = np.random.default_rng(0)
    mask = rng.random((4, 4)) < 0.5
    mask[np.arange(4), np.arange(4)] = True
    Q, K = _rand((S, D), 1), _rand((S, D), 2)
    # constant V -> constant O
    V = np.tile(np.arange(D, dtype=float)[None], (S, 1))
    o, _ = wo.block_sparse_attention(Q, K, V, mask, b, b, S, S)
    assert np.abs(o - V[:1]).max() < 1e-12
    # Q = 0 -> uniform weights: O = mean of selected V rows, LSE = log(#keys); ragged tail counts real keys only
    V = _rand((S, D), 3)
    seq_kv = 120
    o, lse = wo.block_sparse_attention(np.zeros((S, D)), K, V, mask, b, b, S, seq_kv)
    for i in range(4):
        keys = np.concatenate([np.arange(j * b, min((j + 1) * b, seq_kv)) for j in np.nonzero(mask[i])[0]])
        assert np.abs(o[i * b] - V[keys].mean(0)).max() < 1e-13
        assert abs(lse[i * b] - math.log(len(keys))) < 1e-13
    # a row that selects nothing: O = 0, LSE = -inf
    o, lse = wo.attention_block_row(Q[:b], K, V, [], b, S, 1.0)
    assert (o == 0).all() and np.isneginf(lse).all()
    # a single selected block == dense attention restricted to that block
    o, _ = wo.attention_block_row(Q[:b], K, V, [2], b, S, 0.5)
    s = 0.5 * Q[:b] @ K[64:96].T
    w = np.exp(s - s.max(1, keepdims=True))
    assert np.abs(o - (w / w.sum(1, keepdims=True)) @ V[64:96]).max() < 1e-13


def test_row_order_invariance():
    # Section 4.1: query rows are independent, so any execution order gives the same outputs
    S, D, b = 128, 8, 16
    mask = np.random.default_rng(3).random((8, 8)) < 0.4
    Q, K, V = _rand((S, D), 1), _rand((S, D), 2), _rand((S, D), 3)
    ref, _ = wo.block_sparse_attention(Q, K, V, mask, b, b, S, S)
    perm = np.random.default_rng(4).permutation(8)
    out = np.zeros_like(ref)
    for i in perm:
        out[i * b:(i + 1) * b], _ = wo.attention_block_row(Q[i * b:(i + 1) * b], K, V, np.nonzero(mask[i])[0], b, S,
                                                          1 / math.sqrt(D))
    assert np.array_equal(out, ref)


def test_c_twin_matches_numpy_on_tiny_config():
    cfg = I.CONFIGS["tiny"]
    for head in range(cfg.heads):
        mask = I.make_mask(cfg, head)
        q, k, v = (I.make_head_tensor(cfg, w, head) for w in "qkv")
        Q, K, V = (I.bf16_to_f64(t) for t in (q, k, v))
        ref, ref_lse = wo.block_sparse_attention(Q, K, V, mask, cfg.block, cfg.block, cfg.seq, cfg.seq)
        bits = [t.view(torch.int16).numpy().view(np.uint16) for t in (q, k, v)]
        rows = list(range(cfg.n_blocks))
        out, lse = c_twin.attn_tasks(*bits, cfg.block, cfg.block, cfg.seq, cfg.seq, 1 / math.sqrt(cfg.head_dim),
                                     rows, [np.nonzero(mask[i])[0] for i in rows])
        assert np.abs(out.reshape(cfg.seq, -1) - ref).max() < 1e-12
        assert np.abs(lse.reshape(-1) - ref_lse).max() < 1e-12


def test_c_twin_ragged_and_empty():
    D, b, seq = 16, 32, 150
    rng = np.random.default_rng(9)
    nb = 5
    q, k, v = (torch.from_numpy(rng.standard_normal((nb * b, D))).to(torch.bfloat16) for _ in range(3))
    lists = [[0, 4], [], [4], [1, 2, 3]]
    rows = [0, 1, 4, 2]
    bits = [t.view(torch.int16).numpy().view(np.uint16) for t in (q, k, v)]
    out, lse = c_twin.attn_tasks(*bits, b, b, seq, seq, 0.25, rows, lists)
    Q, K, V = (I.bf16_to_f64(t) for t in (q, k, v))
    for t, (r, l) in enumerate(zip(rows, lists)):
        n = min(b, seq - r * b)
        o, ls = wo.attention_block_row(Q[r * b:r * b + n], K, V, l, b, seq, 0.25)
        assert np.abs(out[t, :n] - o).max() < 1e-12
        if l:
            assert np.abs(lse[t, :n] - ls).max() < 1e-12
        else:
            assert np.isneginf(lse[t, :n]).all()
        assert np.isnan(out[t, n:]).all()
