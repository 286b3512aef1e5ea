"""Interleaved minibatch formation and the multi-epoch loop (Section 5.1) on the GPU against the
CPU checker: same index sets per phase, same snapshot updates, same training result."""
import numpy as np
import pytest

from oracle import Oracle
from paper_1606_08495_b200 import binding, corpus
from paper_1606_08495_b200.train import gpu_step, train
from gpu_common import assert_same_pairs, make_pair, row_rel_err

pytestmark = pytest.mark.gpu

CFG = corpus.scaled(corpus.CONFIGS["tiny"], vocab=2000, corpus_tokens=100_000, minibatch=2000, d=100)


@pytest.mark.parametrize("stride", [2, 7, 50, 4096])
def test_interleaved_index_sets_bit_exact(stride):
    gpu, cpu, cp = make_pair(CFG)
    toks = cp.chunk(0)
    total = 0
    for phase in sorted({0, 1, stride // 2, stride - 1}):
        gpu.set_interleave(phase, stride); cpu.set_interleave(phase, stride)
        c, x, n = assert_same_pairs(gpu, cpu, toks, CFG["window"], CFG["negatives"])
        total += len(c)
    assert total > 0
    with pytest.raises(binding.W2VError) as e:
        gpu.set_interleave(stride, stride)
    assert e.value.code == binding.W2V_ERR_ARG
    gpu.close()


def test_interleaved_snapshot_steps_equal_the_checker():
    gpu, cpu, cp = make_pair(CFG)
    W, N, lr, stride = CFG["window"], CFG["negatives"], 0.05, 10       # ~100 input words per step
    ids = np.arange(CFG["vocab"])
    for block in range(2):
        toks = cp.chunk(block)
        pairs = 0
        for phase in range(stride):
            for m in (gpu, cpu):
                m.set_step(block); m.set_interleave(phase, stride)
            st = gpu.sgns_step(toks, W, N, lr, binding.MODE_SNAPSHOT)
            so = cpu.step(toks, W, N, lr, 0)
            assert st["pairs"] == so["pairs"] and st["centres"] == so["centres"]
            pairs += st["pairs"]
        # together the phases used every input word of the chunk once
        for m in (gpu, cpu):
            m.set_step(block); m.set_interleave(0, 1)
        assert pairs == len(cpu.sample_pairs(toks, W, N)[0])
        assert row_rel_err(gpu.read_rows(0, ids), cpu.read_rows(0, ids)) <= 1e-5
        assert row_rel_err(gpu.read_rows(1, ids), cpu.read_rows(1, ids)) <= 1e-5
    gpu.close()


def test_two_epochs_of_interleaved_training_match_the_checker():
    seed = 23
    gpu, cpu, cp = make_pair(CFG, seed=seed)
    W, N = CFG["window"], CFG["negatives"]
    chunks = [cp.chunk(i) for i in range(8)]

    def cpu_step(tokens, lr, number, phase, stride):
        cpu.set_step(number); cpu.set_interleave(phase, stride)
        cpu.step(tokens, W, N, lr, 0)

    calls = train(gpu_step(gpu, W, N, binding.MODE_SNAPSHOT), chunks, epochs=2, lr0=0.05, stride=10)
    assert calls == train(cpu_step, chunks, epochs=2, lr0=0.05, stride=10) == 160
    ids = np.arange(CFG["vocab"])
    # 160 deterministic steps: the fp32 rounding differences of each step carry over, no more
    assert row_rel_err(gpu.read_rows(0, ids), cpu.read_rows(0, ids)) <= 2e-4
    assert row_rel_err(gpu.read_rows(1, ids), cpu.read_rows(1, ids)) <= 2e-4
    cpu.set_interleave(0, 1)
    held = cp.chunk(900)
    s_cpu, p_cpu = cpu.loss(held, W, N, step_id=10**9)
    ev = Oracle(CFG["vocab"], CFG["d"], seed)
    ev.build_tables(cp.counts, CFG["subsample_t"])
    ev.write_rows(0, ids, gpu.read_rows(0, ids)); ev.write_rows(1, ids, gpu.read_rows(1, ids))
    s_gpu, p_gpu = ev.loss(held, W, N, step_id=10**9)
    assert p_cpu == p_gpu and abs(s_gpu - s_cpu) / s_cpu <= 1e-4
    fresh = Oracle(CFG["vocab"], CFG["d"], seed)
    fresh.build_tables(cp.counts, CFG["subsample_t"])
    s0, _ = fresh.loss(held, W, N, step_id=10**9)
    assert s_cpu < 0.95 * s0                                        # training did something
    gpu.close()
