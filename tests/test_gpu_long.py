"""Hogwild-mode training at the lengths the acceptance criterion names: one pass over the small
corpus (17 M tokens) and a 20 M-token prefix of the medium corpus, held-out loss of the GPU result
against the sequential CPU checker's, three GPU repeats.  The checker needs several minutes per run
on one core, so these are skipped unless W2V_LONG_TESTS=1."""
import os

import numpy as np
import pytest

from oracle import Oracle
from paper_1606_08495_b200 import binding, corpus
from paper_1606_08495_b200.train import train

pytestmark = [pytest.mark.gpu,
              pytest.mark.skipif(os.environ.get("W2V_LONG_TESTS") != "1", reason="set W2V_LONG_TESTS=1 (minutes of CPU time)")]


def heldout(vectors_from, cfg, cp, held, seed):
    ev = Oracle(cfg["vocab"], cfg["d"], seed)
    ev.build_tables(cp.counts, cfg["subsample_t"])
    tot, P = 0.0, 0
    ids = np.arange(cfg["vocab"])
    for lo in range(0, cfg["vocab"], 100_000):
        part = ids[lo:lo + 100_000]
        ev.write_rows(0, part, vectors_from.read_rows(0, part))
        ev.write_rows(1, part, vectors_from.read_rows(1, part))
    for j in held:
        s, p = ev.loss(cp.chunk(j), cfg["window"], cfg["negatives"], step_id=10**9 + j)
        tot += s; P += p
    ev.close()
    return tot / P


@pytest.mark.parametrize("name,tokens", [("small", 17_000_000), ("medium", 20_000_000)])
def test_hogwild_loss_after_a_long_run(name, tokens):
    cfg, seed = corpus.CONFIGS[name], 41
    cp = corpus.Corpus(cfg)
    W, N = cfg["window"], cfg["negatives"]
    n_chunks = tokens // cfg["minibatch"]
    chunks = [cp.chunk(i) for i in range(n_chunks)]
    held = [1_000_000, 1_000_001]
    cpu = Oracle(cfg["vocab"], cfg["d"], seed)
    cpu.build_tables(cp.counts, cfg["subsample_t"])

    def cpu_step(t, lr, num, ph, st):
        cpu.set_step(num)
        cpu.step(t, W, N, lr, 1)

    train(cpu_step, chunks, epochs=1, lr0=cfg["lr"])
    want = heldout(cpu, cfg, cp, held, seed)
    losses = []
    for rep in range(3):
        g = binding.W2V(cfg["vocab"], cfg["d"], seed, row_stride=binding.aligned_row_stride(cfg["d"]))
        g.build_alias(cp.counts, cfg["subsample_t"])

        def gstep(t, lr, num, ph, st, g=g):
            g.set_step(num)
            g.sgns_step(t, W, N, lr, binding.MODE_HOGWILD, want_stats=False)
        train(gstep, chunks, epochs=1, lr0=cfg["lr"])
        losses.append(heldout(g, cfg, cp, held, seed))
        g.close()
    print("LONG %s: %d chunks, held-out loss checker %.5f gpu %s" % (name, n_chunks, want, losses))
    for got in losses:
        assert abs(got - want) / want <= 0.01, (got, want)
