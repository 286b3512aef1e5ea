"""Pins for the oracle's cosine retrieval (Section 2, Section 7.2)."""
import numpy as np
import pytest

from oracle import Oracle


def model(rows, which=0):
    rows = np.asarray(rows, dtype=np.float32)
    o = Oracle(len(rows), rows.shape[1], 1)
    o.write_rows(which, np.arange(len(rows)), rows)
    return o


def test_known_angles():
    # row 0 = e1; the others at 0, 45, 60, 90, 120, 180 degrees from it, with assorted lengths
    r = np.zeros((7, 4), dtype=np.float32)
    r[0, 0] = 2.0
    for k, deg in enumerate((0, 45, 60, 90, 120, 180), start=1):
        a = np.deg2rad(deg)
        r[k, :2] = (k + 0.5) * np.array([np.cos(a), np.sin(a)])
    o = model(r)
    ids, cs = o.topk_cosine(0, [0], 0, 7, 6, -2.0)
    assert list(ids[0]) == [1, 2, 3, 4, 5, 6]                       # the query itself is left out
    assert cs[0] == pytest.approx([1.0, np.sqrt(0.5), 0.5, 0.0, -0.5, -1.0], abs=1e-7)
    ids, cs = o.topk_cosine(0, [0], 0, 7, 6, 0.65)                  # threshold of Section 7.2
    assert list(ids[0]) == [1, 2, -1, -1, -1, -1] and cs[0][2:].tolist() == [0.0] * 4
    ids, _ = o.topk_cosine(0, [0], 0, 7, 1, -2.0)
    assert list(ids[0]) == [1]
    ids, _ = o.topk_cosine(0, [0], 3, 6, 3, -2.0)                   # candidate range
    assert list(ids[0]) == [3, 4, 5]


def test_against_a_full_sort_and_scale_invariance():
    rng = np.random.default_rng(0)
    V, d, K = 400, 20, 9
    X = rng.normal(size=(V, d)).astype(np.float32)
    o = model(X, which=1)
    q = rng.integers(0, V, 25)
    ids, cs = o.topk_cosine(1, q, 50, 350, K, -2.0)
    Xd = X.astype(np.float64)
    C = (Xd[q] @ Xd[50:350].T) / (np.linalg.norm(Xd[q], axis=1)[:, None] * np.linalg.norm(Xd[50:350], axis=1)[None, :])
    for i, qi in enumerate(q):
        c = C[i].copy()
        if 50 <= qi < 350:
            c[qi - 50] = -np.inf
        order = np.argsort(-c, kind="stable")[:K]
        assert list(ids[i]) == list(order + 50)
        assert cs[i] == pytest.approx(c[order], abs=1e-12)
    # cosine does not depend on the length of the rows
    scale = rng.uniform(0.1, 10.0, size=(V, 1)).astype(np.float32)
    ids2, cs2 = model(X * scale, which=1).topk_cosine(1, q, 50, 350, K, -2.0)
    assert np.array_equal(ids, ids2) and np.allclose(cs, cs2, atol=1e-6)


def test_zero_rows_bad_queries_and_ties():
    r = np.array([[1, 0], [0, 0], [2, 0], [3, 0], [0, 1]], dtype=np.float32)
    o = model(r)
    ids, cs = o.topk_cosine(0, [0, 1, -1, 9], 0, 5, 3, -2.0)
    assert list(ids[0]) == [2, 3, 1] and cs[0].tolist() == [1.0, 1.0, 0.0]   # ties by id; zero row scores 0
    assert list(ids[1]) == [0, 2, 3] and cs[1].tolist() == [0.0, 0.0, 0.0]   # zero query: every cosine is 0
    assert list(ids[2]) == [-1, -1, -1] and list(ids[3]) == [-1, -1, -1]     # out-of-range query ids
    with pytest.raises(ValueError):
        o.topk_cosine(0, [0], 3, 6, 3, 0.0)
