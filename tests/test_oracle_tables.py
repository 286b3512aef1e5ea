"""Pins for the oracle's sampling tables: the unigram^(3/4) alias table and the
sub-sampling thresholds."""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from oracle import Oracle

TWO32 = 1 << 32


def _tables(counts, t=0.0):
    o = Oracle(len(counts), 4, 1)
    o.build_tables(np.asarray(counts, dtype=np.uint64), t)
    return o, o.tables()


def exact_distribution(thr, alias):
    """Probability of each outcome of (uniform bucket, uniform 32-bit word < thr ? bucket : alias),
    as exact fractions.  An entry aliased to itself is accepted whatever the word."""
    V = len(thr)
    mass = [0] * V
    for j in range(V):
        a = int(alias[j])
        if a == j:
            mass[j] += TWO32
        else:
            mass[j] += int(thr[j])
            mass[a] += TWO32 - int(thr[j])
    return [Fraction(m, V * TWO32) for m in mass]


def test_three_word_table_by_hand():
    # counts (16, 1, 81) -> weights c^(3/4) = (8, 1, 27) -> p = (2/9, 1/36, 3/4); scaled by V:
    # q = (2/3, 1/12, 9/4).  Words 0 and 1 are below 1 and both borrow from word 2.
    _, (thr, alias, _) = _tables([16, 1, 81])
    assert list(alias) == [2, 2, 2]
    assert int(thr[0]) == (2 * TWO32) // 3
    assert int(thr[1]) == TWO32 // 12
    assert int(thr[2]) == TWO32 - 1
    p = exact_distribution(thr, alias)
    for got, want in zip(p, (Fraction(2, 9), Fraction(1, 36), Fraction(3, 4))):
        assert abs(got - want) <= Fraction(3, TWO32)


@pytest.mark.parametrize("V,seed", [(2, 0), (3, 1), (7, 2), (64, 3), (1000, 4), (10000, 5)])
def test_table_distribution_is_unigram_three_quarters(V, seed):
    rng = np.random.default_rng(seed)
    if V >= 1000:   # Zipfian histogram
        counts = np.maximum(1, np.rint(5e5 / np.arange(1, V + 1))).astype(np.uint64)
    else:
        counts = rng.integers(1, 10000, size=V).astype(np.uint64)
    _, (thr, alias, _) = _tables(counts)
    assert np.all(alias < V)
    p = exact_distribution(thr, alias)
    assert sum(p) == 1
    w = counts.astype(np.float64) ** 0.75        # brute force, library pow
    want = w / w.sum()
    err = max(abs(float(pi) - wi) for pi, wi in zip(p, want))
    assert err <= V * 2.0 ** -32 + 1e-15


def test_uniform_counts_give_trivial_table():
    _, (thr, alias, _) = _tables([5] * 16)
    p = exact_distribution(thr, alias)
    assert all(abs(pi - Fraction(1, 16)) <= Fraction(2, TWO32) for pi in p)


def test_zero_count_is_rejected():
    o = Oracle(3, 4, 1)
    with pytest.raises(ValueError):
        o.build_tables(np.array([1, 0, 2], dtype=np.uint64), 0.0)


def test_empirical_draw_frequencies():
    counts = np.array([16, 1, 81, 7, 300, 2, 2, 50], dtype=np.uint64)
    o, _ = _tables(counts)
    rng = np.random.default_rng(11)
    n = 200_000
    words = rng.integers(0, TWO32, size=(n, 3), dtype=np.uint64)
    hits = np.zeros(len(counts))
    for r0, r1, r2 in words:
        hits[o.alias_draw(int(r0), int(r1), int(r2))] += 1
    w = counts.astype(np.float64) ** 0.75
    p = w / w.sum()
    sigma = np.sqrt(n * p * (1 - p))
    assert np.all(np.abs(hits - n * p) < 4.5 * sigma)


def test_bucket_choice_uses_high_product():
    # bucket = floor(r64 * V / 2^64): the top of the range lands in the last bucket, the bottom in
    # the first.  With thr = 2^32-1 everywhere except via aliasing, use an always-accept word (r2 = 0).
    counts = np.array([1, 1, 1, 1, 1], dtype=np.uint64)
    o, _ = _tables(counts)
    assert o.alias_draw(0, 0, 0) == 0
    assert o.alias_draw(0xFFFFFFFF, 0xFFFFFFFF, 0) == 4
    assert o.alias_draw(0x33333333, 0x33333333, 0) == 0      # just below 1/5
    assert o.alias_draw(0x33333333, 0x33333334, 0) == 1      # just above 1/5


# ---- sub-sampling thresholds: keep probability sqrt(x) + x, x = t * total / count ----
def test_keep_threshold_special_values():
    # total = 1,000,000; t = 1e-3 -> t*total = 1000.
    #   count 4000 -> x = 1/4   -> p = 1/2 + 1/4 = 3/4 exactly
    #   count 16000 -> x = 1/16 -> p = 1/4 + 1/16 = 5/16 exactly
    #   count 1000 -> x = 1 -> p >= 1 -> always kept
    #   count 2617 -> x = 0.38211.. just above (3 - sqrt 5)/2 = 0.381966 -> p just above 1 -> always
    #   count 2619 -> x = 0.381825 -> p = 0.99975 < 1
    counts = np.array([4000, 16000, 1000, 2617, 2619], dtype=np.uint64)
    rest = 1_000_000 - int(counts.sum())
    counts = np.append(counts, np.uint64(rest))
    _, (_, _, keep) = _tables(counts, 1e-3)
    assert int(keep[0]) == 3 * TWO32 // 4
    assert int(keep[1]) == 5 * TWO32 // 16
    assert int(keep[2]) == TWO32 - 1
    assert int(keep[3]) == TWO32 - 1
    x = 1000 / 2619
    assert abs(int(keep[4]) / TWO32 - (np.sqrt(x) + x)) < 1e-9
    assert int(keep[4]) < TWO32 - 1


def test_keep_disabled_when_t_not_positive():
    _, (_, _, keep) = _tables([10, 1000, 5], 0.0)
    assert np.all(keep == TWO32 - 1)


def test_keep_probability_decreases_with_count():
    counts = np.sort(np.random.default_rng(3).integers(1, 10**6, size=500))[::-1].astype(np.uint64)
    _, (_, _, keep) = _tables(counts, 1e-4)
    assert np.all(np.diff(keep.astype(np.int64)) >= 0)     # rarer words: never a smaller chance
