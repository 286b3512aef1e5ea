"""Pins for the oracle's continuous-bag-of-words variant (footnote to Section 5): it is checked
against the skip-gram step it reduces to, against finite differences of its objective, against the
closed form of a first step, and its index sets against hand enumeration."""
import numpy as np
import pytest

from oracle import Oracle


def tables(o):
    ids = np.arange(o.vocab)
    return o.read_rows(0, ids).astype(np.float64), o.read_rows(1, ids).astype(np.float64)


def seeded(V, d, seed=0, scale=0.3):
    rng = np.random.default_rng(seed)
    o = Oracle(V, d, 1)
    o.write_rows(0, np.arange(V), rng.normal(scale=scale, size=(V, d)).astype(np.float32))
    o.write_rows(1, np.arange(V), rng.normal(scale=scale, size=(V, d)).astype(np.float32))
    return o


@pytest.mark.parametrize("mode", [0, 1])
def test_one_context_word_is_a_skipgram_pair(mode):
    # with a single context word k the mean is u(k) itself: the example (centre c, context {k}) is the
    # skip-gram pair with input word k and output word c, which the skip-gram pins cover
    V, d = 12, 6
    centre, ctx, negs = [3, 7, 3], [5, 1, 9], [[2, 8], [4, 4], [11, 0]]
    a, b = seeded(V, d, 4), seeded(V, d, 4)
    a.cbow_step_examples(centre, negs, [0, 1, 2, 3], ctx, 0.07, mode)
    b.step_pairs(ctx, centre, negs, 0.07, mode)
    for x, y in zip(tables(a), tables(b)):
        assert np.array_equal(x, y)
    assert a.cbow_loss_examples(centre, negs, [0, 1, 2, 3], ctx) == pytest.approx(b.loss_pairs(ctx, centre, negs), abs=1e-12)


def test_snapshot_step_is_a_gradient_step_on_the_objective():
    # central finite differences of the loss in fp64 against (x' - x) / lr of a snapshot step
    V, d, lr = 7, 5, 1e-3
    centre = [0, 2, 5, 2]
    negs = [[1, 3, 6], [4, 0, 0], [2, 2, 1], [6, 3, 5]]
    ctx_off = [0, 3, 4, 8, 10]
    ctx = [1, 2, 3, 6, 0, 1, 3, 4, 5, 5]            # repeated context words and repeated rows on purpose
    o = seeded(V, d, 7)
    U0, V0 = tables(o)

    def loss_at(U, Vv):
        t = Oracle(V, d, 1)
        t.write_rows(0, np.arange(V), U.astype(np.float32)); t.write_rows(1, np.arange(V), Vv.astype(np.float32))
        return t.cbow_loss_examples(centre, negs, ctx_off, ctx)

    def loss64(U, Vv):                              # the objective itself, in numpy fp64
        tot = 0.0
        for e, c in enumerate(centre):
            h = U[ctx[ctx_off[e]:ctx_off[e + 1]]].mean(axis=0)
            tot -= np.log(1 / (1 + np.exp(-h @ Vv[c])))
            for t_ in negs[e]:
                tot -= np.log(1 / (1 + np.exp(h @ Vv[t_])))
        return tot

    assert loss_at(U0, V0) == pytest.approx(loss64(U0, V0), rel=1e-12)
    o.cbow_step_examples(centre, negs, ctx_off, ctx, lr, 0)
    U1, V1 = tables(o)
    eps = 1e-6
    for T0, T1, which in ((U0, U1, 0), (V0, V1, 1)):
        grad = np.zeros_like(T0)
        for r in range(V):
            for j in range(d):
                P, M = T0.copy(), T0.copy()
                P[r, j] += eps; M[r, j] -= eps
                lp = loss64(P, V0) if which == 0 else loss64(U0, P)
                lm = loss64(M, V0) if which == 0 else loss64(U0, M)
                grad[r, j] = (lp - lm) / (2 * eps)
        step = (T1 - T0) / lr
        assert np.allclose(step, -grad, rtol=0, atol=2e-4 * np.abs(grad).max())   # fp32 storage of x' limits this
        assert np.abs(step + grad).max() <= 2e-4 * np.abs(grad).max()


def test_first_step_from_zero_output_vectors():
    # V = 0: every dot is 0, sigma = 1/2, so U does not move and v(t) = lr (label - 1/2) * sum of the means
    V, d, lr = 9, 4, 0.1
    o = Oracle(V, d, 3)                              # U from the initialiser, V = 0
    U0, _ = tables(o)
    centre, negs, ctx_off, ctx = [1, 4], [[2, 4], [1, 8]], [0, 2, 5], [0, 3, 5, 6, 7]
    h0, h1 = U0[[0, 3]].mean(axis=0), U0[[5, 6, 7]].mean(axis=0)
    sig = lambda z: 1 / (1 + np.exp(-z))
    # mode 0: both examples see V = 0
    t = Oracle(V, d, 3)
    t.cbow_step_examples(centre, negs, ctx_off, ctx, lr, 0)
    U1, V1 = tables(t)
    assert np.array_equal(U1, U0)
    want = np.zeros((V, d))
    want[1] += 0.5 * lr * h0; want[2] -= 0.5 * lr * h0; want[4] -= 0.5 * lr * h0
    want[4] += 0.5 * lr * h1; want[8] -= 0.5 * lr * h1; want[1] -= 0.5 * lr * h1
    assert np.allclose(V1, want, rtol=0, atol=1e-9)
    # mode 1: example 2 sees v(4) and v(1) as example 1 left them; its context words then move
    t = Oracle(V, d, 3)
    t.cbow_step_examples(centre, negs, ctx_off, ctx, lr, 1)
    U1, V1 = tables(t)
    v1, v2, v4 = 0.5 * lr * h0, -0.5 * lr * h0, -0.5 * lr * h0
    g4, g1, g8 = lr * (1 - sig(h1 @ v4)), -lr * sig(h1 @ v1), -0.5 * lr
    e = g4 * v4 + g1 * v1
    assert np.allclose(V1[2], v2, rtol=0, atol=1e-9) and np.allclose(V1[8], g8 * h1, rtol=0, atol=1e-9)
    assert np.allclose(V1[4], v4 + g4 * h1, rtol=0, atol=1e-9) and np.allclose(V1[1], v1 + g1 * h1, rtol=0, atol=1e-9)
    assert np.array_equal(U1[[0, 1, 2, 3, 4, 8]], U0[[0, 1, 2, 3, 4, 8]])
    assert np.allclose(U1[[5, 6, 7]], U0[[5, 6, 7]] + e / 3, rtol=0, atol=1e-8)
    assert np.abs(e).max() > 1e-7


def test_example_lists_by_hand():
    o = Oracle(50, 4, 5)
    o.build_tables(np.full(50, 10, dtype=np.uint64), 0.0)
    toks = [3, 4, 5, -1, 6, -1, -1, 7, 8, -1]
    centre, negs, off, ctx = o.cbow_examples(toks, window=1, negatives=3)
    assert list(centre) == [3, 4, 5, 7, 8]                        # 6 has no context
    assert [list(ctx[off[e]:off[e + 1]]) for e in range(5)] == [[4], [3, 5], [4], [8], [7]]
    assert negs.shape == (5, 3) and np.all(negs != centre[:, None])
    st = o.stats()
    assert st["centres"] == 5 and st["pairs"] == 6 and st["kept"] == 6
    assert st["neg_draws"] == 15 + st["neg_redraws"]
    # the contexts are those of the skip-gram pairs with the same centre
    c2, x2, _ = o.sample_pairs(toks, window=1, negatives=3)
    assert list(x2) == list(ctx) and list(c2) == [3, 4, 4, 5, 7, 8]


def test_negatives_avoid_the_centre_word_and_follow_the_table():
    V = 4
    counts = np.array([1, 16, 81, 256], dtype=np.uint64)           # weights 1, 8, 27, 64
    o = Oracle(V, 4, 9)
    o.build_tables(counts, 0.0)
    toks = np.array(([3, 0, -1]) * 4000, dtype=np.int32)
    centre, negs, _, _ = o.cbow_examples(toks, window=1, negatives=4)
    assert np.all(negs != centre[:, None])
    # given centre 3, a negative is 0, 1 or 2 with chances 1 : 8 : 27 (re-draws only remove word 3)
    got = np.bincount(negs[centre == 3].ravel(), minlength=V)[:3]
    n = got.sum()
    p = np.array([1, 8, 27]) / 36.0
    assert np.all(np.abs(got - n * p) <= 4 * np.sqrt(n * p * (1 - p)))
    assert o.stats()["neg_redraws"] > 1000


def test_interleaving_partitions_the_examples():
    rng = np.random.default_rng(2)
    o = Oracle(100, 4, 5)
    o.build_tables(rng.integers(1, 500, 100).astype(np.uint64), 1e-2)
    toks = []
    for _ in range(30):
        toks += list(rng.integers(0, 100, size=rng.integers(1, 20))) + [-1]
    whole = o.cbow_examples(toks, 3, 2)
    E = 0
    for phase in range(5):
        o.set_interleave(phase, 5)
        E += len(o.cbow_examples(toks, 3, 2)[0])
    assert E == len(whole[0])
