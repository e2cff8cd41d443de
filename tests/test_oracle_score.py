"""Pins for the CPU oracle's tolerance score (Eq. 1): the paper's worked number, hand cases,
closed forms, the row-sum invariant and a brute-force dense attention matrix."""
import math
import os

import numpy as np
import pytest

import oracle
from paper_2403_11805_b200 import synth
from conftest import read_golden


def desc(L, Hkv, Hq, d, T, CL, G=None):
    return oracle.make_desc(L, Hkv, Hq, d, T, CL, G or d)


def test_paper_worked_density_example(golden_dir):
    rows = read_golden(os.path.join(golden_dir, "density_worked_example.txt"))
    A = np.array(rows[:-1])
    col, want = int(rows[-1][0]), rows[-1][1]
    T = A.shape[0]
    scores = oracle.chunk_tolerance_from_probs(desc(1, 1, 1, 16, T, 1), A.reshape(1, 1, T, T), T)
    assert scores[col] == pytest.approx(want, abs=1e-15)


def test_three_by_three_hand_case():
    # A = [[1,0,0],[.5,.5,0],[.2,.3,.5]]: column 0 is seen by 3 rows, column 1 by 2, column 2 by 1:
    # tok = [(1+.5+.2)/3, (.5+.3)/2, .5/1] = [0.56667, 0.4, 0.5]
    A = np.array([[1, 0, 0], [.5, .5, 0], [.2, .3, .5]])
    s = oracle.chunk_tolerance_from_probs(desc(1, 1, 1, 16, 3, 1), A.reshape(1, 1, 3, 3), 3)
    assert s == pytest.approx([1.7 / 3, 0.4, 0.5], abs=1e-15)
    # one chunk of 3 tokens: the mean of the three
    s = oracle.chunk_tolerance_from_probs(desc(1, 1, 1, 16, 3, 3), A.reshape(1, 1, 3, 3), 3)
    assert s == pytest.approx([(1.7 / 3 + 0.4 + 0.5) / 3], abs=1e-15)
    # window of the last 2 rows: columns 0,1 are seen by 2 rows, column 2 by 1: [(.5+.2)/2, (.5+.3)/2, .5]
    s = oracle.chunk_tolerance_from_probs(desc(1, 1, 1, 16, 3, 1), A[1:].reshape(1, 1, 2, 3), 2)
    assert s == pytest.approx([0.35, 0.4, 0.5], abs=1e-15)


def test_masked_entries_are_ignored():
    A = np.array([[1, 9, 9], [.5, .5, 9], [.2, .3, .5]], dtype=float)   # garbage above the diagonal
    s = oracle.chunk_tolerance_from_probs(desc(1, 1, 1, 16, 3, 1), A.reshape(1, 1, 3, 3), 3)
    assert s == pytest.approx([1.7 / 3, 0.4, 0.5], abs=1e-15)


def test_layers_and_heads_are_averaged():
    rng = np.random.default_rng(0)
    L, H, W, T, CL = 3, 4, 5, 12, 4
    shape = synth.KVShape("t", L, H, H, 16, T, CL, 16, seed=3)
    P = synth.attention_probs(shape, W).numpy().astype(np.float64)
    full = oracle.chunk_tolerance_from_probs(desc(L, H, H, 16, T, CL), P, W)
    single = [oracle.chunk_tolerance_from_probs(desc(1, 1, 1, 16, T, CL), P[l, h][None, None], W)
              for l in range(L) for h in range(H)]
    assert full == pytest.approx(np.mean(single, axis=0), rel=1e-13)
    # tokens of a chunk are averaged: chunk_len 1 scores, grouped
    per_tok = oracle.chunk_tolerance_from_probs(desc(L, H, H, 16, T, 1), P, W)
    assert full == pytest.approx(per_tok.reshape(-1, CL).mean(1), rel=1e-13)


@pytest.mark.parametrize("T,W", [(9, 9), (40, 8), (33, 1), (16, 5)])
def test_row_sum_invariant(T, W):
    # every row sums to 1, so for one layer and head: sum over columns of n_vis(col) * tok(col) = number of rows
    shape = synth.KVShape("t", 1, 1, 1, 16, T, 1, 16, seed=T)
    P = synth.attention_probs(shape, W).numpy().astype(np.float64)
    tok = oracle.chunk_tolerance_from_probs(desc(1, 1, 1, 16, T, 1), P, W)
    n_vis = np.minimum(W, T - np.arange(T))
    assert float((n_vis * tok).sum()) == pytest.approx(W, rel=1e-6)   # inputs are fp32 probabilities


@pytest.mark.parametrize("T,W", [(8, 8), (24, 4)])
def test_zero_queries_give_harmonic_closed_form(T, W):
    # q = 0: every logit is 0, row r is uniform over its pos_r + 1 visible columns, so
    # tok(col) = (1/n_vis) * sum over rows r with pos_r >= col of 1/(pos_r + 1)
    shape = synth.KVShape("t", 2, 2, 4, 32, T, 4, 32, seed=1)
    kv = synth.kv_tensor(shape).numpy().view(np.uint16)
    q = np.zeros((2, 4, W, 32), dtype=np.uint16)
    got = oracle.chunk_tolerance(desc(2, 2, 4, 32, T, 4), kv, q, W)
    pos = T - W + np.arange(W)
    tok = np.array([sum(1.0 / (p + 1) for p in pos if p >= c) / min(W, T - c) for c in range(T)])
    assert got == pytest.approx(tok.reshape(-1, 4).mean(1), rel=1e-13)


def dense_attention(K, Q):
    """Brute force: the full causal T x T matrix softmax(mask(Q K^T / sqrt(d))) in float64."""
    T, d = K.shape
    logits = (Q @ K.T) / math.sqrt(d)
    A = np.zeros((T, T))
    for r in range(T):
        e = np.exp(logits[r, :r + 1] - logits[r, :r + 1].max())
        A[r, :r + 1] = e / e.sum()
    return A


@pytest.mark.parametrize("Hkv,Hq", [(2, 2), (2, 4), (1, 4)])
def test_brute_force_two_chunks(Hkv, Hq):
    # two chunks of 8 tokens; W = T reproduces the paper's full R x C matrix
    L, d, T, CL = 2, 32, 16, 8
    shape = synth.KVShape("t", L, Hkv, Hq, d, T, CL, d, seed=11)
    kv_t = synth.kv_tensor(shape)
    q_t = synth.q_window(shape, T)
    got = oracle.chunk_tolerance(desc(L, Hkv, Hq, d, T, CL), kv_t.numpy().view(np.uint16),
                                 q_t.numpy().view(np.uint16), T)
    K = kv_t.numpy().astype(np.float64)[:, 0]       # [L, Hkv, T, d]
    Q = q_t.numpy().astype(np.float64)              # [L, Hq, T, d]
    tok = np.zeros(T)
    for l in range(L):
        for hq in range(Hq):
            A = dense_attention(K[l, hq // (Hq // Hkv)], Q[l, hq])
            for c in range(T):
                tok[c] += A[c:, c].sum() / (T - c) / (L * Hq)
    assert got == pytest.approx(tok.reshape(2, CL).mean(1), rel=1e-12)
    # a window of the last W rows is the last W rows of the same matrix
    W = 5
    gotw = oracle.chunk_tolerance(desc(L, Hkv, Hq, d, T, CL), kv_t.numpy().view(np.uint16),
                                  np.ascontiguousarray(q_t.numpy()[:, :, T - W:]).view(np.uint16), W)
    tokw = np.zeros(T)
    for l in range(L):
        for hq in range(Hq):
            A = dense_attention(K[l, hq // (Hq // Hkv)], Q[l, hq])[T - W:]
            for c in range(T):
                rows = [r for r in range(W) if T - W + r >= c]
                tokw[c] += sum(A[r, c] for r in rows) / len(rows) / (L * Hq)
    assert gotw == pytest.approx(tokw.reshape(2, CL).mean(1), rel=1e-12)


def test_tail_tokens_are_not_a_chunk_but_stay_in_the_softmax():
    # T = 20, chunk_len 8: two chunks; tokens 16..19 are not scored, yet rows still attend to them
    L, H, d, T, CL, W = 1, 2, 32, 20, 8, 6
    shape = synth.KVShape("t", L, H, H, d, T, CL, d, seed=2)
    kv_t, q_t = synth.kv_tensor(shape), synth.q_window(shape, W)
    got = oracle.chunk_tolerance(desc(L, H, H, d, T, CL), kv_t.numpy().view(np.uint16), q_t.numpy().view(np.uint16), W)
    assert got.shape == (2,)
    per_tok = oracle.chunk_tolerance(desc(L, H, H, d, T, 1), kv_t.numpy().view(np.uint16),
                                     q_t.numpy().view(np.uint16), W)
    assert got == pytest.approx(per_tok[:16].reshape(2, 8).mean(1), rel=1e-13)


def test_attention_window_rows_are_probabilities():
    shape = synth.KVShape("t", 2, 2, 4, 32, 24, 8, 32, seed=4)
    P = oracle.attention_window(desc(2, 2, 4, 32, 24, 8), synth.kv_tensor(shape).numpy().view(np.uint16),
                                synth.q_window(shape, 8).numpy().view(np.uint16), 8)
    assert P.sum(-1) == pytest.approx(np.ones((2, 4, 8)), rel=1e-13)
    for r in range(8):
        assert not P[:, :, r, 24 - 8 + r + 1:].any()
        assert (P[:, :, r, :24 - 8 + r + 1] > 0).all()
