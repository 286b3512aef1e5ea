"""Pins for the oracle's index sets: sub-sampling, dirty-context windows and negatives."""
import numpy as np

from oracle import Oracle

TWO32 = 1 << 32


def make(V=50, counts=None, t=0.0, seed=5, d=4):
    o = Oracle(V, d, seed)
    if counts is None:
        counts = np.full(V, 10, dtype=np.uint64)
    o.build_tables(np.asarray(counts, dtype=np.uint64), t)
    return o


def test_radius_one_pairs_are_the_neighbours():
    # W = 1 fixes b = 1 whatever the random word, so the pair list is known by hand.
    o = make()
    toks = [3, 4, 5, -1, 6, -1, -1, 7, 8, -1]
    c, x, n = o.sample_pairs(toks, window=1, negatives=2)
    assert list(zip(c, x)) == [(3, 4), (4, 3), (4, 5), (5, 4), (7, 8), (8, 7)]
    assert n.shape == (6, 2)
    st = o.stats()
    assert st["pairs"] == 6 and st["centres"] == 5 and st["kept"] == 6 and st["tokens"] == 10
    assert st["neg_draws"] == 12 + st["neg_redraws"]


def test_windows_stop_at_sentence_ends_and_chunk_edges():
    o = make()
    toks = [1, 2, -1, 3, 4]                      # no trailing sentinel: the chunk edge ends it
    c, x, _ = o.sample_pairs(toks, window=4, negatives=1)
    assert sorted(zip(c, x)) == [(1, 2), (2, 1), (3, 4), (4, 3)]


def test_out_of_vocabulary_tokens_are_skipped_not_sentence_breaks():
    o = make(V=10)
    toks = [1, 99, 2, -5, 3, -1]
    c, x, _ = o.sample_pairs(toks, window=1, negatives=1)
    assert list(zip(c, x)) == [(1, 2), (2, 1), (2, 3), (3, 2)]
    assert o.stats()["oov"] == 2


def test_dropped_words_do_not_count_towards_the_window():
    # word 0 is so frequent that its keep chance is ~1e-4: sentences "1 0 0 0 2" contract to "1 2".
    counts = np.array([10**12, 10, 10, 10], dtype=np.uint64)
    o = make(V=4, counts=counts, t=1e-8)
    keep = o.tables()[2]
    assert keep[0] < 0.001 * TWO32 and np.all(keep[1:] == TWO32 - 1)
    toks = ([1, 0, 0, 0, 2, -1]) * 200
    c, x, _ = o.sample_pairs(toks, window=1, negatives=1)
    pairs = list(zip(c, x))
    assert pairs.count((1, 2)) >= 195 and pairs.count((2, 1)) >= 195


def test_window_is_symmetric_and_radius_uniform():
    W = 5
    o = make(V=1000, counts=np.full(1000, 3, dtype=np.uint64))
    L = 2 * W + 1
    sent = list(range(100, 100 + L)) + [-1]          # distinct words: contexts identify positions
    toks = sent * 4000
    c, x, _ = o.sample_pairs(toks, window=W, negatives=1)
    mid = 100 + W                                      # the middle word sees its full window
    radii = []
    i = 0
    c = np.asarray(c); x = np.asarray(x)
    idx = np.flatnonzero(c == mid)
    # contexts of one centre are consecutive in the list and ascending
    splits = np.flatnonzero(np.diff(idx) != 1) + 1
    for grp in np.split(idx, splits):
        ctx = x[grp]
        b = len(ctx) // 2
        assert list(ctx) == [mid + o_ for o_ in range(-b, b + 1) if o_ != 0]
        radii.append(b)
    radii = np.asarray(radii)
    assert len(radii) == 4000 and radii.min() == 1 and radii.max() == W
    hist = np.bincount(radii, minlength=W + 1)[1:]
    exp = len(radii) / W
    assert np.all(np.abs(hist - exp) < 4.5 * np.sqrt(exp * (1 - 1 / W)))
    # first word of the sentence: only right-hand contexts, between 1 and W of them
    first = x[c == 100]
    assert np.all(first > 100) and np.all(first <= 100 + W)


def test_pair_count_identity():
    rng = np.random.default_rng(2)
    V = 300
    counts = np.maximum(1, (3000 / np.arange(1, V + 1)).astype(np.int64)).astype(np.uint64)
    o = make(V=V, counts=counts, t=1e-2)
    toks = rng.integers(0, V, size=5000).astype(np.int32)
    toks[rng.random(5000) < 0.05] = -1
    c, x, n = o.sample_pairs(toks, window=3, negatives=4)
    st = o.stats()
    assert st["pairs"] == len(c)
    assert st["kept"] < (toks >= 0).sum()              # sub-sampling did drop something
    assert 1 <= st["pairs"] / max(1, st["centres"]) <= 6
    assert st["neg_draws"] == 4 * len(c) + st["neg_redraws"]
    # every pair's reverse is a possible pair: the context word is itself a kept token, so
    # (context -> centre) appears whenever the context's own radius reaches back; at least the
    # neighbours (radius >= 1 always) are mutual
    pairs = set(zip(c.tolist(), x.tolist()))
    assert sum((b, a) in pairs for a, b in pairs) > 0.5 * len(pairs)


def test_kept_fraction_matches_threshold_table():
    V = 2000
    p = 1.0 / np.arange(1, V + 1)
    p /= p.sum()
    counts = np.maximum(1, np.rint(p * 1e6)).astype(np.uint64)
    o = make(V=V, counts=counts, t=1e-3)
    keep = o.tables()[2].astype(np.float64)
    pk = np.where(keep == TWO32 - 1, 1.0, keep / TWO32)
    rng = np.random.default_rng(8)
    n = 60000
    toks = rng.choice(V, size=n, p=p).astype(np.int32)
    o.sample_pairs(toks, window=1, negatives=1)
    kept = o.stats()["kept"]
    mean = pk[toks].sum()
    sd = np.sqrt((pk[toks] * (1 - pk[toks])).sum())
    assert abs(kept - mean) < 4.5 * sd
    assert 0.2 < kept / n < 0.9


def test_negatives_never_equal_the_context_and_follow_the_conditional_law():
    # V = 3, counts (16, 1, 81): p = (2/9, 1/36, 3/4).  Re-drawing until != w_O is rejection
    # sampling: P(i | w_O) = p_i (1 - p_o^16) / (1 - p_o), plus p_o^16 on (w_O + 1) mod V
    # (the fallback after 16 collisions).
    o = make(V=3, counts=np.array([16, 1, 81], dtype=np.uint64))
    p = np.array([2 / 9, 1 / 36, 3 / 4])
    toks = ([0, 1, 2, 1, 0, 2, -1]) * 3000
    c, x, n = o.sample_pairs(toks, window=2, negatives=8)
    assert np.all(n != x[:, None])
    assert n.min() >= 0 and n.max() <= 2
    for wo in range(3):
        sel = n[x == wo].ravel()
        m = len(sel)
        law = p * (1 - p[wo] ** 16) / (1 - p[wo])
        law[wo] = 0.0
        law[(wo + 1) % 3] += p[wo] ** 16
        hist = np.bincount(sel, minlength=3)
        sd = np.sqrt(m * law * (1 - law)) + 1e-9
        assert np.all(np.abs(hist - m * law) < 4.5 * sd), (wo, hist, m * law)
    assert o.stats()["neg_redraws"] > 0


def test_same_seed_and_step_regenerate_the_same_negatives():
    toks = np.random.default_rng(4).integers(0, 50, size=400).astype(np.int32)
    a = make(seed=77)
    b = make(seed=77)
    ra = a.sample_pairs(toks, 3, 5)
    rb = b.sample_pairs(toks, 3, 5)
    assert all(np.array_equal(p, q) for p, q in zip(ra, rb))
    ra2 = a.sample_pairs(toks, 3, 5)                    # sampling alone does not advance the step
    assert all(np.array_equal(p, q) for p, q in zip(ra, ra2))
    b.set_step(1)
    rb1 = b.sample_pairs(toks, 3, 5)
    assert len(rb1[0]) != len(ra[0]) or not np.array_equal(rb1[2], ra[2])
    c = make(seed=78)
    rc = c.sample_pairs(toks, 3, 5)
    assert len(rc[0]) != len(ra[0]) or not np.array_equal(rc[2], ra[2])
    # the high half of the step number matters too
    b.set_step(1 << 32)
    rb2 = b.sample_pairs(toks, 3, 5)
    assert len(rb2[0]) != len(ra[0]) or not np.array_equal(rb2[2], ra[2])


def test_empty_and_degenerate_chunks():
    o = make()
    for toks in ([], [-1, -1, -1], [7], [7, -1, 8, -1]):
        c, x, n = o.sample_pairs(np.asarray(toks, dtype=np.int32), 2, 3)
        assert len(c) == 0 and len(x) == 0 and n.shape[0] == 0


# ---- interleaved minibatch formation (Section 5.1, last paragraph) ----
def test_interleaved_phases_partition_the_pairs_of_the_chunk():
    # same step number, phases 0..stride-1: every input word of the chunk is used exactly once, with
    # the same contexts and the same negatives as in the whole-chunk call
    rng = np.random.default_rng(8)
    V = 300
    counts = rng.integers(1, 2000, size=V).astype(np.uint64)
    o = make(V=V, counts=counts, t=5e-3, seed=12)
    toks = []
    for _ in range(40):
        toks += list(rng.integers(0, V, size=rng.integers(1, 30))) + [-1]
    whole = o.sample_pairs(toks, window=4, negatives=3)
    whole_rows = np.concatenate([whole[0][:, None], whole[1][:, None], whole[2]], axis=1)
    for stride in (1, 2, 7, 64):
        parts = []
        for phase in range(stride):
            o.set_interleave(phase, stride)
            c, x, n = o.sample_pairs(toks, window=4, negatives=3)
            parts.append(np.concatenate([c[:, None], x[:, None], n], axis=1))
        got = np.concatenate(parts, axis=0)
        assert len(got) == len(whole_rows)
        assert np.array_equal(got[np.lexsort(got.T[::-1])], whole_rows[np.lexsort(whole_rows.T[::-1])])
    o.set_interleave(0, 1)


def test_interleaved_input_words_are_a_stride_apart():
    # distinct words, nothing dropped: a centre word identifies its position in the chunk
    V = 500
    o = make(V=V, counts=np.full(V, 5, dtype=np.uint64), t=0.0)
    toks = np.arange(V, dtype=np.int32)                      # one long sentence
    for stride, phase in ((5, 0), (5, 3), (50, 49)):
        o.set_interleave(phase, stride)
        c, x, _ = o.sample_pairs(toks, window=3, negatives=1)
        assert len(c) > 0 and np.all(c % stride == phase)
        assert np.all(np.abs(x - c) <= 3) and np.all(x != c)   # contexts still come from the whole sentence
    o.set_interleave(0, 1)
    for bad in ((1, 1), (5, 5), (0, 0)):
        try:
            o.set_interleave(*bad)
            raise AssertionError("accepted phase >= stride")
        except ValueError:
            pass
