"""Parity of the CUDA library (through its C ABI) with the CPU checker, on the same seeded inputs.

Integer results (tables, kept tokens, windows, negatives, counters) must be identical.
Snapshot-mode vectors must agree to 1e-5 relative to each row's largest element.
Hogwild-mode training must reach a held-out loss within 1 % of the sequential checker's.
"""
import numpy as np
import pytest
import torch

from oracle import Oracle
from paper_1606_08495_b200 import binding, corpus
from gpu_common import assert_same_pairs, elem_rel_err, make_pair, row_rel_err, touched_rows

pytestmark = pytest.mark.gpu

SNAPSHOT_TOL = 1e-5       # max over touched rows of ||gpu - cpu||_inf / ||cpu||_inf
HOGWILD_LOSS_TOL = 0.01   # relative difference of held-out loss per positive pair

TINY = corpus.CONFIGS["tiny"]
SMALL = corpus.CONFIGS["small"]
MEDIUM_CUT = corpus.scaled(corpus.CONFIGS["medium"], vocab=200_000, corpus_tokens=40_000_000, minibatch=32_768)


# ---------------------------------------------------------------- initialisation and tables
@pytest.mark.parametrize("vocab,d", [(1000, 100), (333, 4), (70, 300), (64, 1024), (5000, 200), (20000, 256)])
def test_initial_tables_bit_exact(vocab, d):
    gpu = binding.W2V(vocab, d, seed=0xDEADBEEF12345)
    cpu = Oracle(vocab, d, seed=0xDEADBEEF12345)
    ids = np.arange(vocab)
    assert np.array_equal(gpu.read_rows(0, ids).view(np.uint32), cpu.read_rows(0, ids).view(np.uint32))
    assert not gpu.read_rows(1, ids).any()
    gpu.close()


@pytest.mark.parametrize("name", ["tiny", "small"])
def test_sampling_tables_integer_equal(name):
    cfg = corpus.CONFIGS[name]
    gpu, cpu, _ = make_pair(cfg)
    for a, b in zip(gpu.tables(), cpu.tables()):
        assert np.array_equal(a, b)
    gpu.close()


def test_sampling_tables_random_histograms():
    rng = np.random.default_rng(5)
    for V in (2, 3, 17, 1000, 50_000):
        counts = rng.integers(1, 10**7, size=V).astype(np.uint64)
        cfg = dict(vocab=V, d=8)
        gpu, cpu, _ = make_pair(cfg, counts=counts, t=3e-5)
        for a, b in zip(gpu.tables(), cpu.tables()):
            assert np.array_equal(a, b)
        gpu.close()


# ---------------------------------------------------------------- sampled indices
@pytest.mark.parametrize("cfg,chunks", [(TINY, 3), (SMALL, 2), (MEDIUM_CUT, 1)])
def test_sampled_indices_bit_exact(cfg, chunks):
    gpu, cpu, cp = make_pair(cfg)
    for i in range(chunks):
        toks = cp.chunk(i)
        gpu.set_step(i); cpu.set_step(i)
        c, x, n = assert_same_pairs(gpu, cpu, toks, cfg["window"], cfg["negatives"])
        assert len(c) > 1000
    gpu.close()


def test_sampled_indices_sponsored_shape():
    cfg = corpus.scaled(corpus.CONFIGS["sponsored"], vocab=300_000, corpus_tokens=50_000_000, minibatch=50_000)
    gpu, cpu, cp = make_pair(cfg)
    assert_same_pairs(gpu, cpu, cp.chunk(0), cfg["window"], cfg["negatives"])
    gpu.close()


def test_sampled_indices_three_word_vocabulary_with_collisions():
    cfg = dict(vocab=3, d=4)
    gpu, cpu, _ = make_pair(cfg, counts=[16, 1, 81], t=0.0)
    toks = np.array(([0, 1, 2, 1, 0, 2, 2, 2, -1]) * 500, dtype=np.int32)
    c, x, n = assert_same_pairs(gpu, cpu, toks, 2, 8)
    assert cpu.stats()["neg_redraws"] > 1000
    gpu.close()


@pytest.mark.parametrize("W,N", [(1, 1), (127, 3), (2, 64), (10, 33)])
def test_sampled_indices_extreme_window_and_negatives(W, N):
    cfg = corpus.scaled(TINY, minibatch=3000, sentence_len=400)
    gpu, cpu, cp = make_pair(cfg)
    assert_same_pairs(gpu, cpu, cp.chunk(0), W, N)
    gpu.close()


def test_sampled_indices_edge_chunks():
    cfg = corpus.scaled(TINY, minibatch=500)
    gpu, cpu, _ = make_pair(cfg, t=0.0)
    V = cfg["vocab"]
    cases = [
        [], [-1], [-1, -1, -1], [5], [5, -1], [5, 6], [5, -1, 6, -1],
        [1, 2, 3, V, 4, -7, 5, -1, 2 ** 31 - 1, 6, 7],          # out-of-vocabulary ids
        list(range(10, 2059)),                                    # one tile + 1 token, no sentinel
        ([3, 4, -1] * 683) + [9],                                 # ragged tail across a tile edge
    ]
    for toks in cases:
        toks = np.asarray(toks, dtype=np.int32)
        assert_same_pairs(gpu, cpu, toks, 3, 4)
    gpu.close()


def test_sampling_depends_on_seed_and_step_only():
    gpu, cpu, cp = make_pair(TINY)
    toks = cp.chunk(0)
    a = gpu.sample_pairs(toks, 5, 5)[:3]
    gpu.set_tuning(rows_in_flight=1, blocks_per_sm=1)
    b = gpu.sample_pairs(toks, 5, 5)[:3]
    assert all(np.array_equal(p, q) for p, q in zip(a, b))
    assert gpu.get_step() == 0
    gpu.set_step(1 << 32); cpu.set_step(1 << 32)          # high half of the step number
    assert_same_pairs(gpu, cpu, toks, 5, 5)
    gpu.close()


def test_pair_capacity_is_reported():
    gpu, cpu, cp = make_pair(TINY)
    toks = cp.chunk(0)
    c0, x0, n0 = cpu.sample_pairs(toks, 5, 5)
    c, x, n, st, rc, P = gpu.sample_pairs(toks, 5, 5, cap=100, allow=(binding.W2V_ERR_CAPACITY,))
    assert rc == binding.W2V_ERR_CAPACITY and P == len(c0) and len(c) == 100
    assert np.array_equal(c, c0[:100]) and np.array_equal(n, n0[:100])
    gpu.close()


# ---------------------------------------------------------------- partial dot products
def test_partial_dots_and_slice_sum_identity():
    V, d = 4000, 300
    gpu = binding.W2V(V, d, seed=3)
    cpu = Oracle(V, d, seed=3)
    rng = np.random.default_rng(0)
    Vt = rng.normal(scale=0.3, size=(V, d)).astype(np.float32)
    gpu.write_rows(1, np.arange(V), Vt); cpu.write_rows(1, np.arange(V), Vt)
    pairs = rng.integers(0, V, size=(5000, 2)).astype(np.int32)
    Ut = cpu.read_rows(0, np.arange(V)).astype(np.float64)
    absdot = np.einsum("pd,pd->p", np.abs(Ut[pairs[:, 0]]), np.abs(Vt[pairs[:, 1]].astype(np.float64)))
    bound = 4 * d * 2.0 ** -24 * absdot + 1e-30
    full = cpu.partial_dots(pairs, 0, d)
    assert np.all(np.abs(gpu.partial_dots(pairs, 0, d) - full) <= bound)
    for lo, hi in [(0, 1), (1, 2), (3, 9), (5, 6), (90, 120), (7, 300), (0, 299), (297, 300), (4, 8)]:
        want = cpu.partial_dots(pairs, lo, hi)
        assert np.all(np.abs(gpu.partial_dots(pairs, lo, hi) - want) <= bound), (lo, hi)
    for S in (2, 10, 15, 75, d):
        edges = np.linspace(0, d, S + 1).astype(int)
        tot = sum(gpu.partial_dots(pairs, int(a), int(b)).astype(np.float64) for a, b in zip(edges[:-1], edges[1:]))
        assert np.all(np.abs(tot - full) <= 2 * bound), S
    gpu.close()


def test_partial_dots_rejects_bad_slices_and_flags_bad_rows():
    gpu = binding.W2V(50, 8, seed=1)
    for lo, hi in [(0, 0), (5, 4), (0, 9)]:
        with pytest.raises(binding.W2VError) as e:
            gpu.partial_dots([[0, 1]], lo, hi)
        assert e.value.code == binding.W2V_ERR_ARG
    out = gpu.partial_dots([[0, 1], [50, 1], [0, -1]], 0, 8)
    assert np.isfinite(out[0]) and np.isnan(out[1]) and np.isnan(out[2])
    gpu.close()


def test_read_write_rows_roundtrip():
    V, d = 1000, 100
    gpu = binding.W2V(V, d, seed=2)
    rng = np.random.default_rng(1)
    ids = rng.permutation(V)[:300]
    rows = rng.normal(size=(300, d)).astype(np.float32)
    gpu.write_rows(0, ids, rows)
    assert np.array_equal(gpu.read_rows(0, ids), rows)
    back = gpu.read_rows(0, np.array([ids[0], -3, V, ids[1]]))
    assert np.array_equal(back[0], rows[0]) and np.array_equal(back[3], rows[1])
    assert not back[1].any() and not back[2].any()          # bad ids leave the output untouched
    gpu.close()


# ---------------------------------------------------------------- snapshot mode
def check_snapshot_steps(cfg, steps, words=None, seed=11, row_stride=None, tuning=None):
    gpu, cpu, cp = make_pair(cfg, seed=seed, row_stride=row_stride)
    if tuning is not None:
        gpu.set_tuning(*tuning)
    W, N, lr = cfg["window"], cfg["negatives"], cfg["lr"]
    worst = 0.0
    for i in range(steps):
        toks = cp.chunk(i, words)
        c, x, n = cpu.sample_pairs(toks, W, N)
        st = gpu.sgns_step(toks, W, N, lr, binding.MODE_SNAPSHOT)
        so = cpu.step(toks, W, N, lr, 0)
        for k in ("kept", "centres", "pairs", "neg_draws", "neg_redraws"):
            assert st[k] == so[k], k
        ru, rv = touched_rows(c, x, n)
        eu = row_rel_err(gpu.read_rows(0, ru), cpu.read_rows(0, ru))
        ev = row_rel_err(gpu.read_rows(1, rv), cpu.read_rows(1, rv))
        worst = max(worst, eu, ev)
        assert eu <= SNAPSHOT_TOL and ev <= SNAPSHOT_TOL, (i, eu, ev)
    assert gpu.get_step() == steps == cpu.get_step()
    # rows nobody touched in the last step are still identical to the checker's
    rng = np.random.default_rng(0)
    ids = rng.integers(0, cfg["vocab"], 2000)
    assert row_rel_err(gpu.read_rows(0, ids), cpu.read_rows(0, ids)) <= SNAPSHOT_TOL
    assert row_rel_err(gpu.read_rows(1, ids), cpu.read_rows(1, ids)) <= SNAPSHOT_TOL
    gpu.close()
    return worst


def test_snapshot_steps_tiny():
    check_snapshot_steps(TINY, steps=6)


def test_snapshot_steps_small():
    check_snapshot_steps(SMALL, steps=2, words=20_000)


def test_snapshot_steps_medium_shape():
    check_snapshot_steps(MEDIUM_CUT, steps=2, words=8_000)


@pytest.mark.parametrize("d", [4, 64, 128, 132, 512, 1024])
def test_snapshot_other_dimensions(d):
    cfg = corpus.scaled(TINY, vocab=3000, d=d, minibatch=1500, corpus_tokens=100_000)
    check_snapshot_steps(cfg, steps=2)


@pytest.mark.parametrize("N,W", [(1, 3), (13, 2), (33, 2), (64, 1)])
def test_snapshot_other_negative_counts(N, W):
    # more targets per pair than one batch of row touches (12), than one register of draws per lane (32)
    cfg = corpus.scaled(TINY, vocab=3000, d=100, negatives=N, window=W, minibatch=400, corpus_tokens=60_000)
    check_snapshot_steps(cfg, steps=2)


@pytest.mark.parametrize("d,N,W,tuned", [(300, 10, 5, False), (300, 10, 5, True), (260, 1, 3, False), (384, 13, 2, False),
                                         (300, 64, 1, False), (320, 5, 127, False)])
def test_snapshot_rows_of_the_papers_width(d, N, W, tuned):
    # rows of 260..384 columns take pass 1 through the shared-memory ring (bulk copies, groups of four
    # rows that also run across the boundary between two centres); a requested register shape
    # (tuned) takes the other kernel: both must give the checker's step
    cfg = corpus.scaled(TINY, vocab=3000, d=d, negatives=N, window=W, minibatch=1200, corpus_tokens=80_000)
    check_snapshot_steps(cfg, steps=2, tuning=(4, 0) if tuned else None)


@pytest.mark.parametrize("d,row_stride", [(300, 320), (300, 304), (100, 128), (8, 16), (132, 2048)])
def test_snapshot_padded_rows(d, row_stride):
    # rows on 64-byte boundaries: same vectors, same step, only the addresses differ
    cfg = corpus.scaled(TINY, vocab=3000, d=d, minibatch=1500, corpus_tokens=100_000)
    check_snapshot_steps(cfg, steps=2, row_stride=row_stride)


def test_padded_rows_init_dots_and_padding_untouched():
    V, d, ld = 2000, 300, 304
    gpu = binding.W2V(V, d, seed=5, row_stride=ld)
    cpu = Oracle(V, d, seed=5)
    assert binding.w2v_get_row_stride(gpu.h) == ld
    ids = np.arange(V)
    assert np.array_equal(gpu.read_rows(0, ids).view(np.uint32), cpu.read_rows(0, ids).view(np.uint32))
    rng = np.random.default_rng(3)
    Vt = rng.normal(scale=0.3, size=(V, d)).astype(np.float32)
    gpu.write_rows(1, ids, Vt); cpu.write_rows(1, ids, Vt)
    pairs = rng.integers(0, V, size=(3000, 2)).astype(np.int32)
    for lo, hi in [(0, d), (3, 9), (297, 300), (90, 120)]:
        want = cpu.partial_dots(pairs, lo, hi)
        assert np.allclose(gpu.partial_dots(pairs, lo, hi), want, rtol=0, atol=1e-6)
    counts = np.full(V, 50, dtype=np.uint64)
    gpu.build_alias(counts, 0.0)
    toks = np.append(rng.integers(0, V, size=4000).astype(np.int32), -1)
    gpu.sgns_step(toks, 5, 5, 0.025, binding.MODE_HOGWILD)
    gpu.sgns_step(toks, 5, 5, 0.025, binding.MODE_SNAPSHOT)
    pad_u = gpu.U.view(V, ld)[:, d:]
    pad_v = gpu.V.view(V, ld)[:, d:]
    assert not pad_u.any().item() and not pad_v.any().item()
    gpu.close()


def test_create_strided_rejects_bad_strides():
    for d, ld in [(300, 296), (300, 302), (8, 2052)]:
        with pytest.raises(binding.W2VError) as e:
            binding.W2V(10, d, seed=1, row_stride=ld)
        assert e.value.code == binding.W2V_ERR_ARG


def test_snapshot_result_does_not_depend_on_launch_shape():
    cfg = corpus.scaled(TINY, vocab=3000, minibatch=2000, corpus_tokens=100_000)
    outs = []
    for rif, bps in ((0, 0), (1, 1), (3, 2)):
        gpu, cpu, cp = make_pair(cfg)
        gpu.set_tuning(rif, bps)
        toks = cp.chunk(0)
        gpu.sgns_step(toks, 5, 5, 0.025, binding.MODE_SNAPSHOT)
        gpu.sgns_step(cp.chunk(1), 5, 5, 0.025, binding.MODE_SNAPSHOT)
        ids = np.arange(cfg["vocab"])
        outs.append((gpu.read_rows(0, ids), gpu.read_rows(1, ids)))
        gpu.close()
    for u, v in outs[1:]:
        assert row_rel_err(u, outs[0][0]) <= 2e-6 and row_rel_err(v, outs[0][1]) <= 2e-6


def test_snapshot_hand_example_through_the_step(golden):
    # Example B of the hand-worked fixtures, driven through the real step: a 3-word vocabulary
    # in which "0 1" is the whole chunk, so the pairs are (0 -> 1) and (1 -> 0); the negatives are
    # whatever the sampler draws, and the checker gets the same ones.
    gpu, cpu, _ = make_pair(dict(vocab=3, d=4), counts=[5, 5, 5], t=0.0)
    U = np.array([(0.5, -0.25, 0, 0), (0.25, 0.25, 0, 0), (-0.5, 0.5, 0, 0)], dtype=np.float32)
    Vv = np.array([(1, 0, 0, 0), (1, 2, 0, 0), (2, 0, 0, 0)], dtype=np.float32)
    for m in (gpu, cpu):
        m.write_rows(0, np.arange(3), U); m.write_rows(1, np.arange(3), Vv)
    toks = np.array([0, 1, -1], dtype=np.int32)
    gpu.sgns_step(toks, 1, 1, 0.1, binding.MODE_SNAPSHOT)
    cpu.step(toks, 1, 1, 0.1, 0)
    ids = np.arange(3)
    assert row_rel_err(gpu.read_rows(0, ids), cpu.read_rows(0, ids)) <= 1e-6
    assert row_rel_err(gpu.read_rows(1, ids), cpu.read_rows(1, ids)) <= 1e-6
    gpu.close()


# ---------------------------------------------------------------- hogwild mode
def test_hogwild_single_pair_equals_checker():
    # with one pair in the chunk there is no concurrency: the result is the sequential one
    gpu, cpu, _ = make_pair(dict(vocab=50, d=100), counts=np.full(50, 7), t=0.0)
    rng = np.random.default_rng(2)
    Vt = rng.normal(scale=0.2, size=(50, 100)).astype(np.float32)
    for m in (gpu, cpu):
        m.write_rows(1, np.arange(50), Vt)
    toks = np.array([4, -1, 9, -1], dtype=np.int32)       # no pair at all
    st = gpu.sgns_step(toks, 2, 5, 0.05, binding.MODE_HOGWILD)
    assert st["pairs"] == 0
    cpu.step(toks, 2, 5, 0.05, 1)
    # exactly one pair: of the sentence (7, 8) only the token at an even index is an input word
    toks = np.array([7, 8, -1], dtype=np.int32)
    for m in (gpu, cpu):
        m.set_interleave(0, 2)
    st = gpu.sgns_step(toks, 1, 5, 0.05, binding.MODE_HOGWILD)
    cpu.step(toks, 1, 5, 0.05, 1)
    assert st["pairs"] == 1 and st["centres"] == 1
    ids = np.arange(50)
    assert row_rel_err(gpu.read_rows(0, ids), cpu.read_rows(0, ids)) <= 1e-5
    assert row_rel_err(gpu.read_rows(1, ids), cpu.read_rows(1, ids)) <= 1e-5
    gpu.close()


def run_training(model, cp, cfg, steps, mode, words=None):
    W, N = cfg["window"], cfg["negatives"]
    for i in range(steps):
        lr = cfg["lr"] * max(1.0 - i / (steps + 1.0), 1e-4)
        if isinstance(model, Oracle):
            model.step(cp.chunk(i, words), W, N, lr, mode)
        else:
            model.sgns_step(cp.chunk(i, words), W, N, lr, mode, want_stats=False)


def heldout_loss(vectors_from, cfg, cp, held_chunks, seed):
    """Loss of Eq. (1) per positive pair, evaluated by the checker in fp64 on the given vectors."""
    ev = Oracle(cfg["vocab"], cfg["d"], seed)
    ev.build_tables(cp.counts, cfg["subsample_t"])
    ids = np.arange(cfg["vocab"])
    ev.write_rows(0, ids, vectors_from.read_rows(0, ids))
    ev.write_rows(1, ids, vectors_from.read_rows(1, ids))
    tot, P = 0.0, 0
    for j in held_chunks:
        s, p = ev.loss(cp.chunk(j), cfg["window"], cfg["negatives"], step_id=10**9 + j)
        tot += s; P += p
    return tot / P


@pytest.mark.parametrize("cfg,steps,words", [(TINY, 120, None), (corpus.scaled(SMALL, d=64), 12, 65_536)])
def test_hogwild_training_loss_within_one_percent(cfg, steps, words):
    seed = 21
    gpu, cpu, cp = make_pair(cfg, seed=seed)
    base = heldout_loss(cpu, cfg, cp, [10_000, 10_001], seed)
    run_training(cpu, cp, cfg, steps, 1, words)
    want = heldout_loss(cpu, cfg, cp, [10_000, 10_001], seed)
    assert want < 0.9 * base                                   # training did something
    losses = []
    for rep in range(3):
        g = binding.W2V(cfg["vocab"], cfg["d"], seed)
        g.build_alias(cp.counts, cfg["subsample_t"])
        run_training(g, cp, cfg, steps, binding.MODE_HOGWILD, words)
        losses.append(heldout_loss(g, cfg, cp, [10_000, 10_001], seed))
        g.close()
    print("hogwild held-out loss: checker %.5f gpu %s (untrained %.5f)" % (want, losses, base))
    for got in losses:
        assert abs(got - want) / want <= HOGWILD_LOSS_TOL, (got, want)
    gpu.close()


# ---------------------------------------------------------------- error paths
def test_error_codes():
    gpu = binding.W2V(100, 8, seed=1)
    toks = torch.zeros(10, dtype=torch.int32, device="cuda")
    with pytest.raises(binding.W2VError) as e:
        gpu.sgns_step(toks, 5, 5, 0.1, 1)
    assert e.value.code == binding.W2V_ERR_STATE
    with pytest.raises(binding.W2VError) as e:
        gpu.build_alias(np.array([1] * 99 + [0], dtype=np.uint64), 1e-3)
    assert e.value.code == binding.W2V_ERR_ARG
    gpu.build_alias(np.full(100, 3, dtype=np.uint64), 0.0)
    for W, N, mode in ((0, 5, 1), (128, 5, 1), (5, 0, 1), (5, 65, 1), (5, 5, 2)):
        with pytest.raises(binding.W2VError) as e:
            gpu.sgns_step(toks, W, N, 0.1, mode)
        assert e.value.code == binding.W2V_ERR_ARG
    bad = torch.tensor([1, 2, 100, 3, -1], dtype=torch.int32, device="cuda")
    with pytest.raises(binding.W2VError) as e:
        gpu.sgns_step(bad, 2, 2, 0.1, 0)
    assert e.value.code == binding.W2V_ERR_TOKEN_RANGE
    st = gpu.sgns_step(bad, 2, 2, 0.1, 1, allow=(binding.W2V_ERR_TOKEN_RANGE,))
    assert st["oov"] == 1 and st["kept"] == 3 and st["status"] & 1
    assert gpu.get_step() == 2                                  # the steps still completed
    gpu.close()


def test_host_token_entry_point_matches_device_entry_point():
    cfg = corpus.scaled(TINY, vocab=3000, minibatch=2000, corpus_tokens=100_000)
    outs = []
    for host in (False, True):
        gpu, cpu, cp = make_pair(cfg)
        toks = cp.chunk(0)
        if host:
            pinned = torch.from_numpy(toks).pin_memory()
            st = gpu.sgns_step_host(pinned, 5, 5, 0.025, binding.MODE_SNAPSHOT)
        else:
            st = gpu.sgns_step(toks, 5, 5, 0.025, binding.MODE_SNAPSHOT)
        ids = np.arange(cfg["vocab"])
        outs.append((st, gpu.read_rows(0, ids), gpu.read_rows(1, ids)))
        gpu.close()
    assert outs[0][0] == outs[1][0]
    assert row_rel_err(outs[1][1], outs[0][1]) <= 2e-6 and row_rel_err(outs[1][2], outs[0][2]) <= 2e-6


def test_resume_from_saved_rows_and_step_number():
    # vectors + step number are the whole training state: a model rebuilt from them continues exactly
    cfg = corpus.scaled(TINY, vocab=3000, minibatch=2000, corpus_tokens=100_000)
    gpu, cpu, cp = make_pair(cfg)
    W, N, lr = cfg["window"], cfg["negatives"], cfg["lr"]
    ids = np.arange(cfg["vocab"])
    for i in range(2):
        gpu.sgns_step(cp.chunk(i), W, N, lr, binding.MODE_SNAPSHOT)
    saved_u, saved_v, saved_step = gpu.read_rows(0, ids), gpu.read_rows(1, ids), gpu.get_step()
    for i in range(2, 4):
        gpu.sgns_step(cp.chunk(i), W, N, lr, binding.MODE_SNAPSHOT)
    again = binding.W2V(cfg["vocab"], cfg["d"], 11, row_stride=binding.aligned_row_stride(cfg["d"]))
    again.build_alias(cp.counts, cfg["subsample_t"])
    again.write_rows(0, ids, saved_u); again.write_rows(1, ids, saved_v); again.set_step(saved_step)
    for i in range(2, 4):
        again.sgns_step(cp.chunk(i), W, N, lr, binding.MODE_SNAPSHOT)
    assert again.get_step() == gpu.get_step() == 4
    assert row_rel_err(again.read_rows(0, ids), gpu.read_rows(0, ids)) <= 2e-6     # atomics' order only
    assert row_rel_err(again.read_rows(1, ids), gpu.read_rows(1, ids)) <= 2e-6
    gpu.close(); again.close()


def test_sampled_indices_random_chunk_structures():
    # seeded random chunks: sentence lengths from 0 up, runs of sentinels, out-of-vocabulary ids, every
    # window and negative count, with and without sub-sampling, several step numbers and interleavings
    rng = np.random.default_rng(77)
    V = 400
    counts = rng.integers(1, 10**5, size=V).astype(np.uint64)
    for case in range(40):
        t = [0.0, 1e-3, 1e-2][case % 3]
        gpu, cpu, _ = make_pair(dict(vocab=V, d=8), counts=counts, t=t, seed=1000 + case)
        toks = []
        for _ in range(int(rng.integers(0, 60))):
            n = int(rng.integers(0, 70))
            sent = rng.integers(0, V, size=n)
            if n and rng.random() < 0.3:
                sent[rng.integers(0, n)] = V + int(rng.integers(0, 5))         # out of vocabulary
            if n and rng.random() < 0.1:
                sent[rng.integers(0, n)] = -int(rng.integers(2, 9))
            toks += list(sent) + [-1] * int(rng.integers(0 if n else 1, 3))
        toks = np.asarray(toks, dtype=np.int32)
        W, N = int(rng.integers(1, 20)), int(rng.integers(1, 40))
        step = int(rng.integers(0, 2**40))
        stride = int(rng.integers(1, 6)); phase = int(rng.integers(0, stride))
        for m in (gpu, cpu):
            m.set_step(step); m.set_interleave(phase, stride)
        assert_same_pairs(gpu, cpu, toks, W, N)
        c0, n0, _, ctx0 = cpu.cbow_examples(toks, W, N)
        c1, n1, _ = gpu.sample_cbow(toks, W, N, allow=(binding.W2V_ERR_TOKEN_RANGE,)) if len(toks) else (c0, n0, None)
        assert np.array_equal(c0, c1) and np.array_equal(n0, n1)
        gpu.close()


def test_memory_probe_leaves_the_table_as_it_was():
    # the probe's additions add zero: V keeps its bits; every access pattern runs and reports a time
    cfg = corpus.scaled(corpus.CONFIGS["tiny"], vocab=5000, d=100)
    gpu, cpu, cp = make_pair(cfg, row_stride=128)
    ids = np.arange(cfg["vocab"])
    rng = np.random.default_rng(2)
    Vv = rng.normal(scale=0.1, size=(cfg["vocab"], cfg["d"])).astype(np.float32)
    gpu.write_rows(1, ids, Vv)
    for access in range(5):
        for span in (cfg["vocab"], 17):
            ms, done = binding.w2v_probe_rows(gpu.h, access, span, 100_000)
            assert ms > 0 and done >= 100_000
    assert np.array_equal(gpu.read_rows(1, ids), Vv)
    # the ring of bulk copies only reads the table too
    for stage, stages, producers in ((4096, 4, 1), (16384, 3, 2), (1024, 64, 4)):
        ms, done = binding.w2v_probe_bulk_ring(gpu.h, stage, stages, producers, 1 << 20)
        assert ms > 0 and done == (1 << 20) // stage * stage
    # and so does the producer / ring / MMA pipeline (two streams of 5 tiles fit this table; the tensor
    # pipe alone needs 19 x 128 cycles per tile, so no configuration can be faster than that)
    for kps, stages, span in ((3, 3, 0), (3, 3, 1), (2, 4, 1), (1, 9, 0), (4, 2, 1)):
        cyc, waited = binding.w2v_probe_mma_ring(gpu.h, kps, stages, 5, span)
        assert cyc >= 19 * 128 * 0.9 and 0 <= waited <= cyc
    gpu.sync()
    assert np.array_equal(gpu.read_rows(1, ids), Vv)
    for args in ((3, 1, 5, 0), (5, 2, 5, 0), (0, 3, 5, 0), (3, 3, 0, 0), (3, 3, 100, 0)):       # one stage, ring too large, ..., table too small
        with pytest.raises(binding.W2VError) as e:
            binding.w2v_probe_mma_ring(gpu.h, *args)
        assert e.value.code == binding.W2V_ERR_ARG
    for args in ((24, 4, 1, 1 << 20), (4096, 0, 1, 1 << 20), (65536, 4, 1, 1 << 20), (4096, 4, 5, 1 << 20), (4096, 4, 1, 100)):
        with pytest.raises(binding.W2VError) as e:
            binding.w2v_probe_bulk_ring(gpu.h, *args)
        assert e.value.code == binding.W2V_ERR_ARG
    for args in ((5, 10, 10), (0, 0, 10), (0, cfg["vocab"] + 1, 10), (0, 10, 0)):
        with pytest.raises(binding.W2VError) as e:
            binding.w2v_probe_rows(gpu.h, *args)
        assert e.value.code == binding.W2V_ERR_ARG
    gpu.close()
