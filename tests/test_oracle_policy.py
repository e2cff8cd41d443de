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


def test_assign_levels_other_level_sets():
    # atop a 4-bit base the further levels are 2 and 1 bits (Sec. 3.2): same ranks, other widths
    scores = [0.9, 0.1, 0.5, 0.8, 0.2, 0.4]
    bits, order = oracle.assign_levels(scores, (1 / 3, 1 / 3, 1 / 3), (4, 2, 1))
    assert bits.tolist() == [4, 1, 2, 4, 1, 2] and order.tolist() == [0, 3, 2, 5, 4, 1]
    rng = np.random.default_rng(11)
    s = rng.random(200)
    b842, o842 = oracle.assign_bits(s, (0.2, 0.5, 0.3))
    b421, o421 = oracle.assign_levels(s, (0.2, 0.5, 0.3), (4, 2, 1))
    assert np.array_equal(o842, o421) and np.array_equal(b842, 2 * b421)
    for bad in ((4, 4, 2), (2, 4, 8), (8, 3, 1)):
        with pytest.raises(RuntimeError):
            oracle.assign_levels(s, (0.2, 0.5, 0.3), bad)


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
        rows = [(int(rng.integers(0, 3)), i, int(rng.choice([8, 4, 2, 1])), int(rng.random() < 0.8),
                 int(rng.random() < 0.2), int(rng.integers(0, 4))) for i in range(n)]
        order = oracle.lctru_order(make_table(rows)).tolist()
        eligible = [i for i, r in enumerate(rows) if r[3] and not r[4]]
        assert sorted(order) == eligible
        for a, b in zip(order, order[1:]):         # every adjacent pair respects the precedence
            ra, rb = rows[a], rows[b]
            assert (-ra[2], ra[5], ra[0], ra[1]) < (-rb[2], rb[5], rb[0], rb[1])


# ----------------------------------------------------------------- Eq. 3: thresholds

def test_thresholds_uniform_density_means_uniform_bits():
    # every chunk equally dense: nothing is gained by moving bits around, the tie goes to n8 = 0 -> all 4-bit
    frac, counts = oracle.optimize_thresholds([0.25] * 12, 0.5)
    assert counts == [0, 12, 0] and frac.tolist() == [0.0, 1.0, 0.0]


def test_thresholds_one_dominant_chunk():
    # one chunk carries all the density: it alone keeps 8 bits, paid for by two chunks at 2 bits (f2 = 2 f8 at 50%)
    frac, counts = oracle.optimize_thresholds([0.001] * 5 + [0.9] + [0.001] * 6, 0.5)
    assert counts == [1, 9, 2]


def test_thresholds_closed_form_relation_and_achieved_ratio():
    rng = np.random.default_rng(4)
    for n in (3, 16, 32, 256, 511):
        for R in (0.5, 0.4, 0.7, 0.25, 1.0):
            s = rng.random(n) ** 3
            frac, (n8, n4, n2) = oracle.optimize_thresholds(s, R)
            assert n8 + n4 + n2 == n and min(n8, n4, n2) >= 0
            assert n2 == int(np.floor(2 * n8 + (2 - 4 * np.float64(np.float32(R))) * n + 0.5))
            assert abs((n8 + n4 / 2 + n2 / 4) / n - R) <= 1 / (8 * n) + 1e-7
            bits, _ = oracle.assign_bits(s, frac)          # the shares reproduce the counts
            assert [int((bits == b).sum()) for b in (8, 4, 2)] == [n8, n4, n2]


def test_thresholds_brute_force_over_all_level_assignments():
    # every assignment of levels to chunks (not only rank-ordered ones) whose counts obey the ratio rule
    rng = np.random.default_rng(9)
    for n in (4, 6, 7):
        for _ in range(6):
            s = (rng.random(n) ** 2).astype(np.float32)
            _, (n8, n4, n2) = oracle.optimize_thresholds(s, 0.5)
            order = np.argsort(-s, kind="stable")
            got = s[order[:n8]].sum(dtype=np.float64) + s[order[n8:n8 + n4]].sum(dtype=np.float64) / 2 \
                + s[order[n8 + n4:]].sum(dtype=np.float64) / 4
            best = -1.0
            for levels in itertools.product((1.0, 0.5, 0.25), repeat=n):
                c8, c2 = levels.count(1.0), levels.count(0.25)
                if c2 != 2 * c8:                      # f2 = 2 f8 at a 50% global ratio
                    continue
                best = max(best, float(np.dot(np.array(levels), s.astype(np.float64))))
            assert got == pytest.approx(best, rel=1e-12)


@pytest.mark.parametrize("levels", [(8, 4, 2), (4, 2, 1), (8, 2, 1), (8, 4, 1)])
def test_thresholds_for_other_level_sets(levels):
    b0, b1, b2 = levels
    r1, r2 = b1 / b0, b2 / b0
    rng = np.random.default_rng(b0 * 100 + b1 * 10 + b2)
    # counts obey the ratio rule and reproduce through the rank -> bits rule; the ratio is met to half a chunk step
    for n in (5, 32, 257):
        for R in (0.5, 0.3, 0.8, r2, 1.0):
            s = (rng.random(n) ** 3).astype(np.float32)
            try:
                frac, (c0, c1, c2) = oracle.optimize_thresholds_levels(s, R, levels)
            except RuntimeError:
                assert n == 5                               # only so few chunks can leave a ratio without any count triple
                continue
            assert c0 + c1 + c2 == n and min(c0, c1, c2) >= 0
            Rd = np.float64(np.float32(R))
            assert c2 == int(np.floor(((1 - r1) * c0 + (r1 - Rd) * n) / (r1 - r2) + 0.5))
            assert abs((c0 + r1 * c1 + r2 * c2) / n - R) <= (r1 - r2) / (2 * n) + 1e-7
            bits, _ = oracle.assign_levels(s, frac, levels)
            assert [int((bits == b).sum()) for b in levels] == [c0, c1, c2]
    # brute force over every assignment of levels to chunks whose counts obey the rule
    for n in (4, 6, 7):
        for R in (0.5, 0.4):
            s = (rng.random(n) ** 2).astype(np.float32)
            try:
                _, (c0, c1, c2) = oracle.optimize_thresholds_levels(s, R, levels)
            except RuntimeError:
                continue                                    # no count triple meets this ratio for so few chunks
            order = np.argsort(-s, kind="stable")
            sd = s.astype(np.float64)
            got = sd[order[:c0]].sum() + r1 * sd[order[c0:c0 + c1]].sum() + r2 * sd[order[c0 + c1:]].sum()
            Rd = np.float64(np.float32(R))
            best = -1.0
            for assign in itertools.product((0, 1, 2), repeat=n):
                k0, k2 = assign.count(0), assign.count(2)
                if k2 != int(np.floor(((1 - r1) * k0 + (r1 - Rd) * n) / (r1 - r2) + 0.5)):
                    continue
                w = np.array([(1.0, r1, r2)[a] for a in assign])
                best = max(best, float(np.dot(w, sd)))
            assert got == pytest.approx(best, rel=1e-12)


def test_thresholds_levels_842_is_the_original_rule():
    rng = np.random.default_rng(3)
    for n in (3, 16, 255):
        for R in (0.5, 0.4, 0.7, 0.25, 1.0):
            s = rng.random(n).astype(np.float32) ** 2
            a = oracle.optimize_thresholds(s, R)
            b = oracle.optimize_thresholds_levels(s, R, (8, 4, 2))
            assert a[1] == b[1] and np.array_equal(a[0], b[0])
