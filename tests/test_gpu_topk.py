"""Cosine retrieval on the GPU against the CPU checker's brute force in fp64.

Cosines must agree to 2e-6 (fp32 dot products of unit-scaled rows).  Where two candidates' exact
cosines differ by less than that, either order is right, so ids are compared position by position
only where the checker's neighbouring cosines are further apart, and otherwise through the value:
the checker's cosine of the row the GPU returned must match the checker's cosine at that rank."""
import numpy as np
import pytest

from oracle import Oracle
from paper_1606_08495_b200 import binding

pytestmark = pytest.mark.gpu

TOL = 2e-6
KERNELS = [0, 1, 2, 3]    # fp32 on the CUDA cores; tensor cores with the TF32 head/tail split; tensor-core screen + exact fp32; the screen on pairs of SMs


def tolerance(kernel, d):
    """fp32 CUDA cores: rounding of a d-term fp32 dot product of unit-scaled rows, 2e-6.  Tensor cores:
    the head/tail split leaves ~2^-21 per product, but the accumulator in tensor memory is updated
    3 * d/8 times (three MMAs per 8 columns) with rounding toward zero, each time up to 2^-24 of the
    running sum (|cos| <= 1): a bias of up to 3 (d/8) 2^-24 on top."""
    if kernel in (0, 2, 3):                            # the screens rank and return fp32 dot products
        return TOL
    return TOL + 3 * ((d + 7) // 8) * 2.0 ** -24


def pair(V, d, seed, which=0, scale=1.0, row_stride=None, rows=None, kernel=0):
    rng = np.random.default_rng(seed)
    X = rng.normal(scale=scale, size=(V, d)).astype(np.float32) if rows is None else np.asarray(rows, dtype=np.float32)
    gpu = binding.W2V(V, d, 1, row_stride=row_stride)
    cpu = Oracle(V, d, 1)
    ids = np.arange(V)
    gpu.write_rows(which, ids, X); cpu.write_rows(which, ids, X)
    binding.w2v_set_retrieval_kernel(gpu.h, kernel)
    return gpu, cpu, X


def compare(gi, gc, wi, wc, X, queries, lo, hi, K, tau, TOL=TOL):
    """GPU lists (gi, gc) against the checker's (wi, wc) for the same queries; X holds the table rows."""
    assert gi.shape == wi.shape

    def exact(q, a):                                       # fp64 cosine of rows q and a
        x, y = X[q].astype(np.float64), X[a].astype(np.float64)
        nx, ny = np.linalg.norm(x), np.linalg.norm(y)
        return float(x @ y / (nx * ny)) if nx > 0 and ny > 0 else 0.0

    for r, q in enumerate(np.asarray(queries)):
        n_want = int((wi[r] >= 0).sum())
        n_got = int((gi[r] >= 0).sum())
        # the number kept can differ only through candidates within TOL of tau
        if n_got != n_want:
            k = min(n_got, n_want)
            edge = wc[r][k] if n_want > n_got else None
            assert n_want < K or n_got < K
            assert edge is None or abs(edge - tau) <= TOL, (r, n_got, n_want)
        for s in range(min(n_got, n_want)):
            assert abs(gc[r, s] - wc[r, s]) <= TOL, (r, s, gc[r, s], wc[r, s])
            if gi[r, s] != wi[r, s]:
                a = gi[r, s]
                assert abs(exact(q, a) - wc[r, s]) <= TOL and lo <= a < hi and a != q, (r, s)
        assert np.all(gi[r, n_got:] == -1) and not gc[r, n_got:].any()
        assert len(set(gi[r, :n_got].tolist())) == n_got


def check(gpu, cpu, X, which, queries, lo, hi, K, tau, TOL=TOL):
    gi, gc = gpu.topk_cosine(which, queries, lo, hi, K, tau)
    wi, wc = cpu.topk_cosine(which, queries, lo, hi, K, tau)
    compare(gi, gc, wi, wc, X, queries, lo, hi, K, tau, TOL)
    return gi, gc


@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("V,d,K,m", [(3000, 300, 30, 200), (1000, 100, 5, 70), (5000, 64, 64, 10), (700, 4, 1, 700),
                                     (900, 1024, 30, 40), (129, 132, 7, 129)])
def test_topk_matches_brute_force(V, d, K, m, kernel):
    gpu, cpu, X = pair(V, d, seed=V + d, kernel=kernel)
    rng = np.random.default_rng(1)
    q = rng.integers(0, V, m)
    check(gpu, cpu, X, 0, q, 0, V, K, -2.0, tolerance(kernel, d))
    check(gpu, cpu, X, 0, q, V // 5, V - 7, K, 0.0, tolerance(kernel, d))
    gpu.close()


@pytest.mark.parametrize("kernel", KERNELS)
def test_topk_threshold_of_the_paper_on_clustered_vectors(kernel):
    # rows = cluster centre + noise, so that some neighbours are above tau = 0.65 and most are not
    rng = np.random.default_rng(3)
    V, d, C = 20_000, 300, 400
    centres = rng.normal(size=(C, d))
    X = (centres[rng.integers(0, C, V)] + 0.55 * rng.normal(size=(V, d))).astype(np.float32)
    gpu, cpu, X = pair(V, d, 0, which=1, rows=X, row_stride=320, kernel=kernel)
    q = rng.integers(0, V, 300)
    gi, gc = check(gpu, cpu, X, 1, q, 5000, 20_000, 30, 0.65, tolerance(kernel, d))
    kept = (gi >= 0).sum(axis=1)
    assert kept.max() == 30 and kept.min() < 30 and (gc[gi >= 0] > 0.65).all()
    gpu.close()


@pytest.mark.parametrize("kernel", KERNELS)
def test_topk_many_queries_few_candidates_and_edge_cases(kernel):
    gpu, cpu, X = pair(5000, 32, seed=9, scale=3.0, kernel=kernel)
    q = np.arange(5000)                                   # more query blocks than SMs: no candidate split
    check(gpu, cpu, X, 0, q, 100, 150, 8, -2.0, tolerance(kernel, 32))
    gi, gc = gpu.topk_cosine(0, [5, -1, 5000, 7], 0, 5000, 4, -2.0)
    assert (gi[1] == -1).all() and (gi[2] == -1).all() and (gi[0] >= 0).all() and (gi[3] >= 0).all()
    gi, gc = gpu.topk_cosine(0, [5], 10, 10, 4, -2.0)     # empty candidate range
    assert (gi == -1).all() and not gc.any()
    gi, gc = gpu.topk_cosine(0, [5], 5, 6, 4, -2.0)       # the only candidate is the query itself
    assert (gi == -1).all()
    for args in ((2, [1], 0, 10, 4, 0.0), (0, [1], 0, 10, 0, 0.0), (0, [1], 0, 10, 65, 0.0), (0, [1], 5, 4, 4, 0.0),
                 (0, [1], 0, 5001, 4, 0.0)):
        with pytest.raises(binding.W2VError) as e:
            gpu.topk_cosine(*args)
        assert e.value.code == binding.W2V_ERR_ARG
    gpu.close()


@pytest.mark.parametrize("kernel", KERNELS)
def test_topk_zero_rows_and_exact_ties(kernel):
    rows = np.zeros((200, 8), dtype=np.float32)
    rows[:, 0] = 1.0                                      # every row the same direction: all cosines 1
    rows[50] = 0.0                                        # a zero row: cosine 0 with everything
    rows[100:, 0] = np.arange(100, 200)                   # other lengths, same direction
    gpu, cpu, X = pair(200, 8, 0, rows=rows, kernel=kernel)
    gi, gc = gpu.topk_cosine(0, [0, 50, 150], 0, 200, 6, -2.0)
    wi, wc = cpu.topk_cosine(0, [0, 50, 150], 0, 200, 6, -2.0)
    assert np.array_equal(gi, wi)                         # ties go to the smaller row number
    assert np.allclose(gc, wc, atol=tolerance(kernel, 8))
    gpu.close()


@pytest.mark.parametrize("kernel", KERNELS)
def test_topk_candidate_range_longer_than_one_chunk(kernel):
    # the screening kernel takes the candidates in chunks of 2^22 rows, each with its own partial lists
    V, d = (1 << 22) + 70_001, 8
    gpu, cpu, X = pair(V, d, seed=11, kernel=kernel)
    q = np.array([0, 5, (1 << 22) - 1, 1 << 22, V - 1, 123_456])
    check(gpu, cpu, X, 0, q, 0, V, 20, -2.0, tolerance(kernel, d))
    check(gpu, cpu, X, 0, q, 3, V - 5, 7, 0.9, tolerance(kernel, d))
    gpu.close()


@pytest.mark.parametrize("kernel", KERNELS)
def test_topk_rows_that_are_all_alike(kernel):
    # every candidate is (almost) the same direction as every query: nothing can be dismissed early, every
    # pair gets an exact cosine, and the order is decided in the last bits
    rng = np.random.default_rng(17)
    V, d = 4000, 64
    v = rng.normal(size=d)
    rows = (rng.uniform(0.5, 2.0, size=(V, 1)) * v + 1e-4 * rng.normal(size=(V, d))).astype(np.float32)
    gpu, cpu, X = pair(V, d, 0, rows=rows, kernel=kernel)
    q = rng.integers(0, V, 96)
    check(gpu, cpu, X, 0, q, 0, V, 10, -2.0, tolerance(kernel, d))
    check(gpu, cpu, X, 0, q, 100, 3000, 30, 0.999, tolerance(kernel, d))
    gpu.close()


def test_a_wait_that_runs_out_is_reported_once_and_nothing_faults():
    # the retrieval kernels' bounded wait on a barrier nobody arrives at: the block gives up after the
    # limit, w2v_sync reports it once, and the same handle goes on to answer a query correctly
    import time
    gpu, cpu, X = pair(500, 32, seed=4, kernel=2)
    t0 = time.time()
    binding.w2v_selftest_bounded_wait(gpu.h, 250)
    with pytest.raises(binding.W2VError) as e:
        gpu.sync()
    waited = time.time() - t0
    assert e.value.code == binding.W2V_ERR_CUDA and "gave up waiting" in str(e.value)
    assert 0.2 <= waited < 3.0, waited
    gpu.sync()                                            # reported once
    check(gpu, cpu, X, 0, np.arange(40), 0, 500, 5, -2.0, tolerance(2, 32))
    with pytest.raises(binding.W2VError) as e:
        binding.w2v_selftest_bounded_wait(gpu.h, 0)
    assert e.value.code == binding.W2V_ERR_ARG
    gpu.close()
