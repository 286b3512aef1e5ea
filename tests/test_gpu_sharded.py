"""The column-sharded step (Section 5.1, Algorithms 1-3) against the CPU checker's snapshot step.

S shards of one model live on one GPU and run one after another; every shard's kernel adds its
partial dot products into every shard's array, as it would into its peers' memory.  Side by side,
the shards' columns must equal the checker's whole vectors to the snapshot tolerance.
"""
import numpy as np
import pytest
import torch

from oracle import Oracle
from paper_1606_08495_b200 import binding, corpus
from paper_1606_08495_b200.sharded import LocalShards, shard_columns
from gpu_common import row_rel_err, touched_rows

pytestmark = pytest.mark.gpu

SNAPSHOT_TOL = 1e-5
TINY = corpus.CONFIGS["tiny"]


def make_sharded(cfg, shards, seed=11, aligned=False, exchange="p2p"):
    cp = corpus.Corpus(cfg)
    gpu = LocalShards(cfg["vocab"], cfg["d"], seed, shards, aligned_rows=aligned, exchange=exchange)
    cpu = Oracle(cfg["vocab"], cfg["d"], seed)
    gpu.build_alias(cp.counts, cfg["subsample_t"])
    cpu.build_tables(cp.counts, cfg["subsample_t"])
    return gpu, cpu, cp


@pytest.mark.parametrize("d,shards", [(100, 1), (100, 2), (100, 5), (300, 8), (64, 16), (8, 2)])
def test_shards_hold_the_columns_of_the_whole_initial_model(d, shards):
    V = 500
    gpu = LocalShards(V, d, 5, shards)
    cpu = Oracle(V, d, 5)
    ids = np.arange(V)
    assert np.array_equal(gpu.read_rows(0, ids).view(np.uint32), cpu.read_rows(0, ids).view(np.uint32))
    assert not gpu.read_rows(1, ids).any()
    gpu.close()


@pytest.mark.parametrize("exchange", ["p2p", "allreduce"])
@pytest.mark.parametrize("d,shards,aligned", [(100, 1, False), (100, 2, False), (100, 3, True), (300, 8, False),
                                              (300, 10, True), (64, 16, False)])
def test_sharded_step_equals_snapshot_step(d, shards, aligned, exchange):
    cfg = corpus.scaled(TINY, vocab=3000, d=d, minibatch=2000, corpus_tokens=100_000)
    gpu, cpu, cp = make_sharded(cfg, shards, aligned=aligned, exchange=exchange)
    W, N, lr = cfg["window"], cfg["negatives"], cfg["lr"]
    for i in range(3):
        toks = cp.chunk(i)
        c, x, n = cpu.sample_pairs(toks, W, N)
        st = gpu.step(toks, W, N, lr)
        so = cpu.step(toks, W, N, lr, 0)
        for k in ("kept", "centres", "pairs"):
            assert st[k] == so[k], k
        ru, rv = touched_rows(c, x, n)
        eu = row_rel_err(gpu.read_rows(0, ru), cpu.read_rows(0, ru))
        ev = row_rel_err(gpu.read_rows(1, rv), cpu.read_rows(1, rv))
        assert eu <= SNAPSHOT_TOL and ev <= SNAPSHOT_TOL, (i, eu, ev)
    ids = np.arange(cfg["vocab"])
    assert row_rel_err(gpu.read_rows(0, ids), cpu.read_rows(0, ids)) <= SNAPSHOT_TOL
    assert row_rel_err(gpu.read_rows(1, ids), cpu.read_rows(1, ids)) <= SNAPSHOT_TOL
    gpu.close()


def test_sharded_step_small_shape_many_negatives():
    cfg = corpus.scaled(corpus.CONFIGS["small"], vocab=20_000, corpus_tokens=2_000_000, minibatch=8_000)
    gpu, cpu, cp = make_sharded(cfg, 5)
    toks = cp.chunk(0)
    for W, N in ((5, 5), (2, 40)):
        c, x, n = cpu.sample_pairs(toks, W, N)
        gpu.step(toks, W, N, 0.025)
        cpu.step(toks, W, N, 0.025, 0)
        ru, rv = touched_rows(c, x, n)
        assert row_rel_err(gpu.read_rows(0, ru), cpu.read_rows(0, ru)) <= SNAPSHOT_TOL
        assert row_rel_err(gpu.read_rows(1, rv), cpu.read_rows(1, rv)) <= SNAPSHOT_TOL
    gpu.close()


def test_summed_partials_are_the_full_dot_products():
    # Algorithm 3, "(F+, F-) <- sum over shards": after all shards' w2v_shard_dots every array holds
    # u(centre).v(target) over all d columns, in the order of the pair list
    cfg = corpus.scaled(TINY, vocab=2000, d=100, minibatch=1500, corpus_tokens=100_000)
    gpu, cpu, cp = make_sharded(cfg, 4)
    rng = np.random.default_rng(2)
    ids = np.arange(cfg["vocab"])
    Vt = rng.normal(scale=0.3, size=(cfg["vocab"], cfg["d"])).astype(np.float32)
    gpu.write_rows(1, ids, Vt); cpu.write_rows(1, ids, Vt)
    toks = cp.chunk(0)
    W, N = 5, 5
    c, x, n = cpu.sample_pairs(toks, W, N)
    t = gpu.models[0]._dev_tokens(toks)
    cap = len(c) * (N + 1)
    F = [torch.zeros(cap, dtype=torch.float32, device="cuda") for _ in gpu.models]
    for m in gpu.models:
        binding.w2v_shard_dots(m.h, t, t.numel(), W, N, F, cap)
    torch.cuda.synchronize()
    pairs = np.stack([np.repeat(c, N + 1), np.concatenate([x[:, None], n], axis=1).ravel()], axis=1)
    want = cpu.partial_dots(pairs, 0, cfg["d"])
    Ut = cpu.read_rows(0, ids).astype(np.float64)
    bound = 4 * cfg["d"] * 2.0 ** -24 * np.einsum("pd,pd->p", np.abs(Ut[pairs[:, 0]]), np.abs(Vt[pairs[:, 1]].astype(np.float64)))
    for f in F:
        assert np.all(np.abs(f.cpu().numpy().astype(np.float64) - want) <= bound + 1e-30)
    gpu.close()


def test_shard_call_order_and_capacity_errors():
    cfg = corpus.scaled(TINY, vocab=500, d=16, minibatch=400, corpus_tokens=50_000)
    gpu, cpu, cp = make_sharded(cfg, 2)
    m = gpu.models[0]
    t = m._dev_tokens(cp.chunk(0))
    F = torch.zeros(1 << 20, dtype=torch.float32, device="cuda")
    with pytest.raises(binding.W2VError) as e:
        binding.w2v_shard_adjust(m.h, F, 0.1)                      # no dots before it
    assert e.value.code == binding.W2V_ERR_STATE
    with pytest.raises(binding.W2VError) as e:
        binding.w2v_sgns_step(m.h, t, t.numel(), 5, 5, 0.1, 0)     # a shard has no step of its own
    assert e.value.code == binding.W2V_ERR_STATE
    with pytest.raises(binding.W2VError) as e:
        binding.w2v_shard_dots(m.h, t, t.numel(), 5, 5, [F], 10)   # too small for the chunk
    assert e.value.code == binding.W2V_ERR_CAPACITY
    assert not F.any().item()
    binding.w2v_shard_dots(m.h, t, t.numel(), 5, 5, [F], F.numel())
    m.set_step(3)                                                  # cancels the pending step
    with pytest.raises(binding.W2VError) as e:
        binding.w2v_shard_adjust(m.h, F, 0.1)
    assert e.value.code == binding.W2V_ERR_STATE
    for lo, hi in [(0, 6), (2, 8), (8, 8), (0, 20)]:
        with pytest.raises(binding.W2VError):
            binding.W2V(10, 16, 1, columns=(lo, hi))
    gpu.close()


def test_sharded_step_with_interleaved_minibatches():
    cfg = corpus.scaled(TINY, vocab=2000, d=100, minibatch=1500, corpus_tokens=100_000)
    gpu, cpu, cp = make_sharded(cfg, 4)
    W, N, lr, stride = cfg["window"], cfg["negatives"], 0.05, 5
    toks = cp.chunk(0)
    for phase in range(stride):
        cpu.set_step(0); cpu.set_interleave(phase, stride)
        for m in gpu.models:
            m.set_step(0); m.set_interleave(phase, stride)
        st = gpu.step(toks, W, N, lr)
        so = cpu.step(toks, W, N, lr, 0)
        assert st["pairs"] == so["pairs"] and st["centres"] == so["centres"]
    ids = np.arange(cfg["vocab"])
    assert row_rel_err(gpu.read_rows(0, ids), cpu.read_rows(0, ids)) <= SNAPSHOT_TOL
    assert row_rel_err(gpu.read_rows(1, ids), cpu.read_rows(1, ids)) <= SNAPSHOT_TOL
    gpu.close()
