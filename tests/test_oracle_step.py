"""Pins for the oracle's arithmetic: coefficients, deferred updates, sequential updates,
partial dots, loss and initialisation."""
import numpy as np
import pytest

from oracle import Oracle


def sig(x):
    return 1.0 / (1.0 + np.exp(-x))


def set_tables(o, U, V):
    o.write_rows(0, np.arange(len(U)), np.asarray(U, dtype=np.float32))
    o.write_rows(1, np.arange(len(V)), np.asarray(V, dtype=np.float32))


def get_tables(o):
    ids = np.arange(o.vocab)
    return o.read_rows(0, ids).astype(np.float64), o.read_rows(1, ids).astype(np.float64)


UB = [(0.5, -0.25), (0.25, 0.25), (-0.5, 0.5)]
VB = [(1, 0), (1, 2), (2, 0)]


def fl(rows):
    return np.array([float(x) for x in rows], dtype=np.float64)


def test_hand_example_A(golden):
    g = golden("hand_examples.txt")
    o = Oracle(3, 2, 0)
    set_tables(o, UB, VB)
    assert o.partial_dots([[0, 1], [0, 2]], 0, 2) == pytest.approx(fl(g["A_F"][0]), abs=1e-15)
    assert o.loss_pairs([0], [1], [[2]]) == pytest.approx(fl(g["A_loss"][0])[0], abs=2e-12)
    for mode in (0, 1):
        o = Oracle(3, 2, 0)
        set_tables(o, UB, VB)
        o.step_pairs([0], [1], [[2]], 0.1, mode)
        U, V = get_tables(o)
        assert U[0] == pytest.approx(fl(g["A_u0"][0]), abs=5e-8)
        assert V[1] == pytest.approx(fl(g["A_v1"][0]), abs=2e-7)
        assert V[2] == pytest.approx(fl(g["A_v2"][0]), abs=2e-7)
        assert np.array_equal(U[1:], np.array(UB, dtype=np.float64)[1:])
        assert np.array_equal(V[0], np.array(VB[0], dtype=np.float64))


def test_hand_example_B_deferred_and_sequential(golden):
    g = golden("hand_examples.txt")
    o = Oracle(3, 2, 0)
    set_tables(o, UB, VB)
    F = o.partial_dots([[0, 1], [0, 2], [1, 0], [1, 2]], 0, 2)
    assert F == pytest.approx(fl(g["B_F"][0]), abs=1e-15)
    G = np.array([0.1 * (1 - sig(F[0])), -0.1 * sig(F[1]), 0.1 * (1 - sig(F[2])), -0.1 * sig(F[3])])
    assert G == pytest.approx(fl(g["B_G"][0]), abs=1e-11)
    o.step_pairs([0, 1], [1, 0], [[2], [2]], 0.1, 0)
    U, V = get_tables(o)
    assert U.ravel() == pytest.approx(fl(g["B_snap_U"][0]), abs=1e-7)
    assert V.ravel() == pytest.approx(fl(g["B_snap_V"][0]), abs=2e-7)
    o = Oracle(3, 2, 0)
    set_tables(o, UB, VB)
    o.step_pairs([0, 1], [1, 0], [[2], [2]], 0.1, 1)
    U2, V2 = get_tables(o)
    assert U2[1] == pytest.approx(fl(g["B_seq_U1"][0]), abs=1e-7)
    assert V2[2] == pytest.approx(fl(g["B_seq_V2"][0]), abs=2e-7)
    assert U2[0] == pytest.approx(U[0], abs=1e-7) and V2[1] == pytest.approx(V[1], abs=1e-7)
    # the second pair saw the first pair's write to v2, so the two modes differ there
    assert abs(V2[2][0] - V[2][0]) > 1e-5


def random_problem(seed, V=6, d=5, P=9, N=3, grid=2.0 ** -12):
    rng = np.random.default_rng(seed)
    U = np.round(rng.uniform(-1, 1, (V, d)) / grid) * grid          # exactly representable in fp32
    Vv = np.round(rng.uniform(-1, 1, (V, d)) / grid) * grid
    c = rng.integers(0, V, P)
    x = rng.integers(0, V, P)
    n = rng.integers(0, V, (P, N))
    return U, Vv, c, x, n


def numpy_deferred_step(U, Vv, c, x, n, lr):
    """Eq. (4)/(5) evaluated with array operations (not the oracle's loops)."""
    P, N = n.shape
    tgt = np.concatenate([x[:, None], n], axis=1)                       # [P, 1+N]
    lab = np.zeros((P, 1 + N)); lab[:, 0] = 1.0
    F = np.einsum("pd,pkd->pk", U[c], Vv[tgt])
    G = lr * (lab - sig(F))
    dU = np.zeros_like(U); dV = np.zeros_like(Vv)
    np.add.at(dU, c, np.einsum("pk,pkd->pd", G, Vv[tgt]))
    np.add.at(dV, tgt.ravel(), (G[:, :, None] * U[c][:, None, :]).reshape(-1, U.shape[1]))
    return U + dU, Vv + dV


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_deferred_step_matches_eq4_eq5_in_numpy(seed):
    U, Vv, c, x, n = random_problem(seed)
    o = Oracle(len(U), U.shape[1], 0)
    set_tables(o, U, Vv)
    o.step_pairs(c, x, n, 0.05, 0)
    gotU, gotV = get_tables(o)
    wantU, wantV = numpy_deferred_step(U, Vv, c, x, n, 0.05)
    assert gotU == pytest.approx(wantU, abs=1.2e-7)
    assert gotV == pytest.approx(wantV, abs=1.2e-7)


def test_update_is_lr_times_finite_difference_gradient_of_eq3():
    # Lambda = -loss_pairs.  Central differences with a step that fp32 storage holds exactly.
    U, Vv, c, x, n = random_problem(7, V=4, d=3, P=6, N=2)
    V_, d = U.shape
    lr, h = 2.0 ** -4, 2.0 ** -10
    o = Oracle(V_, d, 0)

    def lam(Ua, Va):
        set_tables(o, Ua, Va)
        return -o.loss_pairs(c, x, n)

    gU = np.zeros_like(U); gV = np.zeros_like(Vv)
    for T, gT, isu in ((U, gU, True), (Vv, gV, False)):
        for i in range(V_):
            for j in range(d):
                Tp = T.copy(); Tm = T.copy()
                Tp[i, j] += h; Tm[i, j] -= h
                hi = lam(Tp, Vv) if isu else lam(U, Tp)
                lo = lam(Tm, Vv) if isu else lam(U, Tm)
                gT[i, j] = (hi - lo) / (2 * h)
    set_tables(o, U, Vv)
    o.step_pairs(c, x, n, lr, 0)
    newU, newV = get_tables(o)
    scale = max(np.abs(gU).max(), np.abs(gV).max())
    assert np.abs((newU - U) / lr - gU).max() < 3e-5 * scale + 2e-6
    assert np.abs((newV - Vv) / lr - gV).max() < 3e-5 * scale + 2e-6
    assert scale > 0.1       # the test is not vacuous


def test_deferred_step_is_order_invariant():
    U, Vv, c, x, n = random_problem(3, V=5, d=4, P=40, N=4)
    res = []
    for perm_seed in (None, 1, 2):
        o = Oracle(len(U), U.shape[1], 0)
        set_tables(o, U, Vv)
        idx = np.arange(len(c)) if perm_seed is None else np.random.default_rng(perm_seed).permutation(len(c))
        o.step_pairs(c[idx], x[idx], n[idx], 0.05, 0)
        res.append(get_tables(o))
    for r in res[1:]:
        assert np.abs(r[0] - res[0][0]).max() <= 1.2e-7 and np.abs(r[1] - res[0][1]).max() <= 1.2e-7


def test_sequential_mode_sees_earlier_writes():
    # two identical pairs: the second one must be computed from the tables the first one left.
    U, Vv, _, _, _ = random_problem(5, V=3, d=4)
    c, x, n = np.array([0, 0]), np.array([1, 1]), np.array([[2], [2]])
    o = Oracle(3, 4, 0)
    set_tables(o, U, Vv)
    o.step_pairs(c, x, n, 0.1, 1)
    got = get_tables(o)
    Uc, Vc = U.copy(), Vv.copy()
    for _ in range(2):
        Uf, Vf = Uc.astype(np.float32).astype(np.float64), Vc.astype(np.float32).astype(np.float64)
        e = np.zeros(4)
        for t, lab in ((1, 1.0), (2, 0.0)):
            g = 0.1 * (lab - sig(Uf[0] @ Vf[t]))
            e += g * Vf[t]
            Vf[t] = (Vf[t] + g * Uf[0]).astype(np.float32)
        Uf[0] = (Uf[0] + e).astype(np.float32)
        Uc, Vc = Uf, Vf
    assert got[0] == pytest.approx(Uc, abs=1e-7) and got[1] == pytest.approx(Vc, abs=1e-7)


def test_first_step_from_initial_tables_closed_form():
    # V = 0 at the start: every dot is 0, sigma = 1/2, so U does not move and
    # V[w] = lr/2 (sum of u(c) over positive pairs with context w - sum over negative draws of w).
    V_, d, lr = 200, 12, 0.025
    o = Oracle(V_, d, 99)
    counts = np.maximum(1, (2000 / np.arange(1, V_ + 1)).astype(np.int64)).astype(np.uint64)
    o.build_tables(counts, 1e-2)
    rng = np.random.default_rng(1)
    toks = rng.integers(0, V_, 3000).astype(np.int32)
    toks[::40] = -1
    U0, V0 = get_tables(o)
    assert np.all(V0 == 0)
    c, x, n = o.sample_pairs(toks, 4, 3)
    o.step(toks, 4, 3, lr, 0)
    assert o.get_step() == 1
    U1, V1 = get_tables(o)
    assert np.array_equal(U1, U0)
    want = np.zeros_like(V0)
    np.add.at(want, x, 0.5 * lr * U0[c])
    for k in range(n.shape[1]):
        np.add.at(want, n[:, k], -0.5 * lr * U0[c])
    assert V1 == pytest.approx(want, rel=2e-7, abs=1e-10)
    assert np.abs(V1).max() > 0


def test_slice_partial_dots_sum_to_the_full_dot():
    V_, d = 40, 300
    rng = np.random.default_rng(0)
    o = Oracle(V_, d, 3)
    Vt = rng.normal(size=(V_, d)).astype(np.float32)
    o.write_rows(1, np.arange(V_), Vt)
    Ut = o.read_rows(0, np.arange(V_))
    pairs = rng.integers(0, V_, (64, 2)).astype(np.int32)
    full = np.einsum("pd,pd->p", Ut[pairs[:, 0]].astype(np.float64), Vt[pairs[:, 1]].astype(np.float64))
    assert o.partial_dots(pairs, 0, d) == pytest.approx(full, rel=1e-13, abs=1e-15)
    for S in (1, 2, 10, 15, 75, d):
        edges = np.linspace(0, d, S + 1).astype(int)
        tot = sum(o.partial_dots(pairs, int(a), int(b)) for a, b in zip(edges[:-1], edges[1:]))
        assert tot == pytest.approx(full, rel=1e-12, abs=1e-14)
    # the paper's example: d = 300 over 10 shards, shard s holds columns 30 s .. 30 s + 29
    s3 = o.partial_dots(pairs, 90, 120)
    want = np.einsum("pd,pd->p", Ut[pairs[:, 0], 90:120].astype(np.float64), Vt[pairs[:, 1], 90:120].astype(np.float64))
    assert s3 == pytest.approx(want, rel=1e-13, abs=1e-15)
    with pytest.raises(ValueError):
        o.partial_dots(pairs, 10, 10)
    with pytest.raises(ValueError):
        o.partial_dots(pairs, 0, d + 1)


def test_loss_of_zero_output_table():
    # all dots 0 -> every term is log 2 -> (1 + N) log 2 per positive pair
    o = Oracle(100, 8, 1)
    o.build_tables(np.full(100, 4, dtype=np.uint64), 0.0)
    toks = np.random.default_rng(0).integers(0, 100, 500).astype(np.int32)
    s, P = o.loss(toks, 3, 6, step_id=17)
    assert P > 0 and s / P == pytest.approx(7 * np.log(2.0), rel=1e-14)
    assert o.get_step() == 0


def test_initial_rows():
    d = 100
    o = Oracle(5000, d, 42)
    U = o.read_rows(0, np.arange(5000)).astype(np.float64)
    assert U.min() >= -0.5 / d and U.max() < 0.5 / d
    n = U.size
    assert abs(U.mean()) < 4.5 * (1 / d) / np.sqrt(12 * n)
    assert U.var() == pytest.approx((1 / d) ** 2 / 12, rel=0.02)
    # values sit on the 2^-24 grid of the uniform variate: (u d + 1/2) 2^24 is an integer up to
    # the rounding of the fp32 division
    grid = (U * d + 0.5) * 2 ** 24
    assert np.abs(grid - np.rint(grid)).max() < 0.51
    assert len(np.unique(U[:, 0])) > 4900
    assert np.array_equal(o.init_row(17), o.read_rows(0, [17])[0])
    assert not np.array_equal(Oracle(5000, d, 43).init_row(17), o.init_row(17))


def test_sparse_store_equals_dense_store():
    V_, d = 500, 8
    counts = np.maximum(1, (5000 / np.arange(1, V_ + 1)).astype(np.int64)).astype(np.uint64)
    toks = np.random.default_rng(3).integers(0, V_, 2000).astype(np.int32)
    toks[::25] = -1
    outs = []
    for sparse in (False, True):
        o = Oracle(V_, d, 5, sparse=sparse)
        o.build_tables(counts, 1e-3)
        o.step(toks, 3, 4, 0.05, 0)
        o.step(toks, 3, 4, 0.05, 1)
        outs.append(get_tables(o))
        if sparse:
            assert o.rows_resident(0) <= V_
    assert np.array_equal(outs[0][0], outs[1][0]) and np.array_equal(outs[0][1], outs[1][1])
