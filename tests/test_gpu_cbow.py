"""The continuous-bag-of-words step on the GPU against the CPU checker: index sets bit-exact,
snapshot-mode vectors to 1e-5 per row, Hogwild-mode training to 1 % of held-out loss."""
import numpy as np
import pytest

from oracle import Oracle
from paper_1606_08495_b200 import binding, corpus
from paper_1606_08495_b200.train import train
from gpu_common import make_pair, row_rel_err

pytestmark = pytest.mark.gpu

SNAPSHOT_TOL = 1e-5
TINY = corpus.CONFIGS["tiny"]


def assert_same_examples(gpu, cpu, toks, W, N):
    c0, n0, off0, ctx0 = cpu.cbow_examples(toks, W, N)
    so = cpu.stats()
    c1, n1, st = gpu.sample_cbow(toks, W, N)
    assert np.array_equal(c0, c1) and np.array_equal(n0, n1)
    for k in ("tokens", "kept", "centres", "pairs", "neg_draws", "neg_redraws", "oov"):
        assert st[k] == so[k], (k, st[k], so[k])
    # the contexts are those of the pair list, grouped by centre
    x = gpu.sample_pairs(toks, W, N, allow=(binding.W2V_ERR_TOKEN_RANGE,))[1]
    assert np.array_equal(x, ctx0)
    return c0, n0, off0, ctx0


@pytest.mark.parametrize("cfg,W,N", [(TINY, 5, 5), (corpus.CONFIGS["small"], 5, 5),
                                     (corpus.scaled(TINY, minibatch=3000, sentence_len=400), 127, 3),
                                     (corpus.scaled(TINY, minibatch=3000), 2, 64), (TINY, 1, 1)])
def test_cbow_examples_bit_exact(cfg, W, N):
    gpu, cpu, cp = make_pair(cfg)
    for i in range(2):
        gpu.set_step(i); cpu.set_step(i)
        c, n, off, ctx = assert_same_examples(gpu, cpu, cp.chunk(i), W, N)
        assert len(c) > 500
    gpu.close()


def test_cbow_examples_three_words_and_edge_chunks():
    gpu, cpu, _ = make_pair(dict(vocab=3, d=4), counts=[16, 1, 81], t=0.0)
    toks = np.array(([0, 1, 2, 1, 0, 2, 2, 2, -1]) * 300, dtype=np.int32)
    assert_same_examples(gpu, cpu, toks, 2, 8)
    assert cpu.stats()["neg_redraws"] > 500
    for t in ([], [-1], [2], [2, -1, 1, -1], [0, 1], [0, 5, 1, -3, 2, -1]):
        c0, n0, _, _ = cpu.cbow_examples(np.asarray(t, dtype=np.int32), 2, 3)
        c1, n1, st = gpu.sample_cbow(np.asarray(t, dtype=np.int32), 2, 3, allow=(binding.W2V_ERR_TOKEN_RANGE,))
        assert np.array_equal(c0, c1) and np.array_equal(n0, n1)
    gpu.close()


def check_cbow_snapshot(cfg, steps, words=None, row_stride=None):
    gpu, cpu, cp = make_pair(cfg, row_stride=row_stride)
    W, N, lr = cfg["window"], cfg["negatives"], cfg["lr"]
    for i in range(steps):
        toks = cp.chunk(i, words)
        c, n, off, ctx = cpu.cbow_examples(toks, W, N)
        st = gpu.cbow_step(toks, W, N, lr, binding.MODE_SNAPSHOT)
        so = cpu.cbow_step(toks, W, N, lr, 0)
        for k in ("kept", "centres", "pairs", "neg_draws", "neg_redraws"):
            assert st[k] == so[k], k
        ru, rv = np.unique(ctx), np.unique(np.concatenate([c, n.ravel()]))
        eu = row_rel_err(gpu.read_rows(0, ru), cpu.read_rows(0, ru))
        ev = row_rel_err(gpu.read_rows(1, rv), cpu.read_rows(1, rv))
        assert eu <= SNAPSHOT_TOL and ev <= SNAPSHOT_TOL, (i, eu, ev)
    assert gpu.get_step() == steps == cpu.get_step()
    ids = np.arange(cfg["vocab"])
    assert row_rel_err(gpu.read_rows(0, ids), cpu.read_rows(0, ids)) <= SNAPSHOT_TOL
    assert row_rel_err(gpu.read_rows(1, ids), cpu.read_rows(1, ids)) <= SNAPSHOT_TOL
    gpu.close()


def test_cbow_snapshot_steps_tiny():
    check_cbow_snapshot(TINY, steps=6)


def test_cbow_snapshot_steps_small_and_medium_shapes():
    check_cbow_snapshot(corpus.CONFIGS["small"], steps=2, words=20_000)
    check_cbow_snapshot(corpus.scaled(corpus.CONFIGS["medium"], vocab=200_000, corpus_tokens=40_000_000,
                                      minibatch=32_768), steps=2, words=8_000, row_stride=320)


@pytest.mark.parametrize("N", [1, 13, 33, 64])
def test_cbow_snapshot_other_negative_counts(N):
    cfg = corpus.scaled(TINY, vocab=3000, d=100, negatives=N, minibatch=600, corpus_tokens=60_000)
    check_cbow_snapshot(cfg, steps=2)


@pytest.mark.parametrize("d", [4, 64, 132, 512, 1024])
def test_cbow_snapshot_other_dimensions(d):
    check_cbow_snapshot(corpus.scaled(TINY, vocab=3000, d=d, minibatch=1500, corpus_tokens=100_000), steps=2)


def test_cbow_hogwild_single_example_equals_checker():
    gpu, cpu, _ = make_pair(dict(vocab=50, d=100), counts=np.full(50, 7), t=0.0)
    rng = np.random.default_rng(2)
    Vt = rng.normal(scale=0.2, size=(50, 100)).astype(np.float32)
    for m in (gpu, cpu):
        m.write_rows(1, np.arange(50), Vt)
    # examples (8 | 9) and (9 | 8) run in two warps at once and may share output rows through their
    # negatives; the second then sees the first's additions or not
    toks = np.array([7, -1, 8, 9, -1], dtype=np.int32)
    gpu.cbow_step(toks, 1, 5, 0.05, binding.MODE_HOGWILD)
    cpu.cbow_step(toks, 1, 5, 0.05, 1)
    ids = np.arange(50)
    assert row_rel_err(gpu.read_rows(0, ids), cpu.read_rows(0, ids)) <= 2e-3
    assert row_rel_err(gpu.read_rows(1, ids), cpu.read_rows(1, ids)) <= 2e-3
    # a chunk with exactly one example has no concurrency at all: the sequential result
    Ut = cpu.read_rows(0, ids)
    for m in (gpu, cpu):
        m.write_rows(0, ids, Ut); m.write_rows(1, ids, Vt)
    one = np.array([20, 21, 22, -1], dtype=np.int32)
    for m in (gpu, cpu):
        m.set_step(5); m.set_interleave(1, 3)                # only token 1 (word 21) is an input position
    gpu.cbow_step(one, 1, 5, 0.05, binding.MODE_HOGWILD)
    cpu.cbow_step(one, 1, 5, 0.05, 1)
    assert cpu.stats()["centres"] == 1 and cpu.stats()["pairs"] == 2
    assert row_rel_err(gpu.read_rows(0, ids), cpu.read_rows(0, ids)) <= 1e-5
    assert row_rel_err(gpu.read_rows(1, ids), cpu.read_rows(1, ids)) <= 1e-5
    gpu.close()


def heldout_cbow_loss(vectors_from, cfg, cp, held, seed):
    ev = Oracle(cfg["vocab"], cfg["d"], seed)
    ev.build_tables(cp.counts, cfg["subsample_t"])
    ids = np.arange(cfg["vocab"])
    ev.write_rows(0, ids, vectors_from.read_rows(0, ids)); ev.write_rows(1, ids, vectors_from.read_rows(1, ids))
    tot, E = 0.0, 0
    for j in held:
        s, e = ev.cbow_loss(cp.chunk(j), cfg["window"], cfg["negatives"], step_id=10**9 + j)
        tot += s; E += e
    return tot / E


def test_cbow_hogwild_training_loss_within_one_percent():
    # Three passes over the tiny corpus.  The checker's mode 1 is the sequential limit (every example
    # sees all earlier ones); its mode 0 is the other limit (every example of a chunk sees the
    # chunk's start).  Thousands of warps at once put the GPU between the two.
    cfg, seed, epochs, lr0 = TINY, 31, 3, 0.05
    gpu, cpu, cp = make_pair(cfg, seed=seed)
    W, N = cfg["window"], cfg["negatives"]
    chunks = [cp.chunk(i) for i in range(120)]
    held = [10_000, 10_001]
    base = heldout_cbow_loss(cpu, cfg, cp, held, seed)

    def run(step):
        train(lambda t, lr, num, ph, st: step(t, lr, num), chunks, epochs=epochs, lr0=lr0)

    def cpu_mode(model, mode):
        def step(t, lr, num):
            model.set_step(num)
            model.cbow_step(t, W, N, lr, mode)
        return step

    run(cpu_mode(cpu, 1))
    want = heldout_cbow_loss(cpu, cfg, cp, held, seed)
    stale = Oracle(cfg["vocab"], cfg["d"], seed)
    stale.build_tables(cp.counts, cfg["subsample_t"])
    run(cpu_mode(stale, 0))
    upper = heldout_cbow_loss(stale, cfg, cp, held, seed)
    assert want < 0.9 * base
    losses = []
    for rep in range(3):
        g = binding.W2V(cfg["vocab"], cfg["d"], seed)
        g.build_alias(cp.counts, cfg["subsample_t"])

        def gstep(t, lr, num, g=g):
            g.set_step(num)
            g.cbow_step(t, W, N, lr, binding.MODE_HOGWILD, want_stats=False)
        run(gstep)
        losses.append(heldout_cbow_loss(g, cfg, cp, held, seed))
        g.close()
    print("cbow held-out loss: sequential %.5f, chunk-stale %.5f, gpu %s (untrained %.5f)" % (want, upper, losses, base))
    for got in losses:
        assert abs(got - want) / want <= 0.01, (got, want)
        assert want * 0.99 <= got <= upper * 1.01
    gpu.close()


def test_cbow_refused_on_a_shard_and_bad_arguments():
    m = binding.W2V(100, 16, 1, columns=(0, 8))
    m.build_alias(np.full(100, 3, dtype=np.uint64), 0.0)
    toks = np.array([1, 2, 3, -1], dtype=np.int32)
    with pytest.raises(binding.W2VError) as e:
        m.cbow_step(toks, 2, 2, 0.1, 0)
    assert e.value.code == binding.W2V_ERR_STATE
    m.close()
    g = binding.W2V(100, 16, 1)
    with pytest.raises(binding.W2VError) as e:
        g.cbow_step(toks, 2, 2, 0.1, 0)                    # no tables yet
    assert e.value.code == binding.W2V_ERR_STATE
    g.build_alias(np.full(100, 3, dtype=np.uint64), 0.0)
    for W, N, mode in ((0, 2, 0), (2, 65, 1), (2, 2, 2)):
        with pytest.raises(binding.W2VError) as e:
            g.cbow_step(toks, W, N, 0.1, mode)
        assert e.value.code == binding.W2V_ERR_ARG
    g.close()
