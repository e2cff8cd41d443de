"""Pins for the CPU oracle's host policies: rank -> bits (Eq. 2) and the LCTRU eviction order (Sec. 3.4)."""
import itertools

import numpy as np
import pytest

import oracle


def naive_rank(scores):
    """Rank by counting: chunk i is preceded by every chunk with a larger score, and by equal ones with a lower index."""
    n = len(scores)
    return [sum(1 for j in range(n) if scores[j] > scores[i] or (scores[j] == scores[i] and j < i)) for i in range(n)]


def test_assign_bits_exhaustive_small():
    frac = (1 / 3, 1 / 3, 1 / 3)
    for n in range(0, 7):
        for scores in itertools.product([0.1, 0.2, 0.3], repeat=n):   # many ties
            bits, order = oracle.assign_bits(scores, frac)
            rank = naive_rank(scores)
            n8 = int(np.floor(frac[0] * n + 0.5))
            n84 = int(np.floor((frac[0] + frac[1]) * n + 0.5))
            for i in range(n):
                assert order[rank[i]] == i
                assert bits[i] == (8 if rank[i] < n8 else 4 if rank[i] < n84 else 2)


def test_assign_bits_direction_low_density_gets_fewer_bits():
    # "compresses those with higher tolerance aggressively": the least informative third drops to 2 bits
    scores = [0.9, 0.1, 0.5, 0.8, 0.2, 0.4]
    bits, order = oracle.assign_bits(scores, (1 / 3, 1 / 3, 1 / 3))
    assert bits.tolist() == [8, 2, 4, 8, 2, 4]
    assert order.tolist() == [0, 3, 2, 5, 4, 1]


@pytest.mark.parametrize("n,frac,want", [
    (256, (1 / 3, 1 / 3, 1 / 3), (85, 86, 85)),
    (128, (1 / 3, 1 / 3, 1 / 3), (43, 42, 43)),
    (32, (1 / 3, 1 / 3, 1 / 3), (11, 10, 11)),
    (512, (0.1, 0.5, 0.4), (51, 256, 205)),
    (16, (1.0, 0.0, 0.0), (16, 0, 0)),
    (16, (0.0, 0.0, 1.0), (0, 0, 16)),
])
def test_assign_bits_counts(n, frac, want):
    rng = np.random.default_rng(n)
    bits, _ = oracle.assign_bits(rng.random(n), frac)
    assert tuple(int((bits == b).sum()) for b in (8, 4, 2)) == want


def test_global_ratio_of_the_paper_setting():
    # levels {8/8, 4/8, 2/8} with shares f8, f4, f2 = 2*f8 give the paper's 50% global ratio when
    # f8 + f4/2 + f2/4 = 1/2; the tertile split gives (1 + 1/2 + 1/4)/3 = 58.3% of the 8-bit size
    f = np.array([1 / 3, 1 / 3, 1 / 3])
    assert float((f * [1, .5, .25]).sum()) == pytest.approx(7 / 12)


def make_table(rows):
    t = np.zeros(len(rows), dtype=oracle.STATE_DTYPE)
    for i, (ctx, chunk, bits, resident, locked, last) in enumerate(rows):
        t[i] = (ctx, chunk, bits, resident, locked, 0, last)
    return t


def test_lctru_hand_case():
    # sub-queues concatenated 8 -> 4 -> 2 ("heavy chunks first"), each least-recently-used first;
    # swapped-out chunks and chunks of a locked (in-service) context never appear
    rows = [
        (0, 0, 2, 1, 0, 5),    # 0
        (0, 1, 8, 1, 0, 9),    # 1
        (1, 0, 8, 1, 0, 3),    # 2
        (1, 1, 4, 1, 0, 1),    # 3
        (2, 0, 8, 1, 1, 0),    # 4 locked
        (2, 1, 8, 0, 0, 0),    # 5 not resident
        (3, 0, 4, 1, 0, 1),    # 6 same bits and time as 3: context id breaks the tie
        (1, 2, 8, 1, 0, 3),    # 7 same as 2 but a later chunk
    ]
    assert oracle.lctru_order(make_table(rows)).tolist() == [2, 7, 1, 3, 6, 0]


def test_lctru_is_the_unique_sorted_permutation():
    rng = np.random.default_rng(7)
    for _ in range(50):
        n = int(rng.integers(1, 9))
        rows = [(int(rng.integers(0, 3)), i, int(rng.choice([8, 4, 2])), int(rng.random() < 0.8),
                 int(rng.random() < 0.2), int(rng.integers(0, 4))) for i in range(n)]
        order = oracle.lctru_order(make_table(rows)).tolist()
        eligible = [i for i, r in enumerate(rows) if r[3] and not r[4]]
        assert sorted(order) == eligible
        for a, b in zip(order, order[1:]):         # every adjacent pair respects the precedence
            ra, rb = rows[a], rows[b]
            assert (-ra[2], ra[5], ra[0], ra[1]) < (-rb[2], rb[5], rb[0], rb[1])
