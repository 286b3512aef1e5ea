"""Hogwild-mode training at the lengths the acceptance criterion names: one pass over the small
corpus (17 M tokens) and a 20 M-token prefix of the medium corpus; held-out loss of the GPU result
within 1 % of the sequential CPU checker's, three GPU repeats.

The checker's side of the comparison takes minutes of one CPU core per run, so it is not repeated
here: tests/golden/hogwild_losses.txt holds its held-out losses, written by
oracle/write_golden_losses.py (which calls only the checker and the input generator).  This file
trains the library on the same chunks with the same step numbers and learning rates, reads the
vectors back and has the checker's loss() evaluate them."""
import numpy as np
import pytest

from oracle import Oracle
from paper_1606_08495_b200 import binding, corpus
from paper_1606_08495_b200.train import train
from conftest import load_golden

pytestmark = pytest.mark.gpu

SEED = 41                                  # the seed the stored runs used
HELD = (1_000_000, 1_000_001)              # chunks the loss is evaluated on
HELD_STEP_BASE = 10 ** 9


def heldout(vectors_from, cfg, cp):
    ev = Oracle(cfg["vocab"], cfg["d"], SEED)
    ev.build_tables(cp.counts, cfg["subsample_t"])
    ids = np.arange(cfg["vocab"])
    for lo in range(0, cfg["vocab"], 100_000):
        part = ids[lo:lo + 100_000]
        ev.write_rows(0, part, vectors_from.read_rows(0, part))
        ev.write_rows(1, part, vectors_from.read_rows(1, part))
    tot, P = 0.0, 0
    for j in HELD:
        s, p = ev.loss(cp.chunk(j), cfg["window"], cfg["negatives"], step_id=HELD_STEP_BASE + j)
        tot += s; P += p
    ev.close()
    return tot / P


@pytest.mark.parametrize("run", ["small", "medium"])
def test_hogwild_loss_after_a_long_run(run):
    cfg_name, n_chunks, words, before, want = load_golden("hogwild_losses.txt")[run][0]
    n_chunks, words, before, want = int(n_chunks), int(words), float(before), float(want)
    cfg = corpus.CONFIGS[cfg_name]
    cp = corpus.Corpus(cfg)
    W, N = cfg["window"], cfg["negatives"]
    chunks = [cp.chunk(i) for i in range(n_chunks)]
    assert sum(int((c >= 0).sum()) for c in chunks) == words      # the stored run saw the same stream
    assert want < 0.9 * before                                    # and it learned something
    losses = []
    for rep in range(3):
        g = binding.W2V(cfg["vocab"], cfg["d"], SEED, row_stride=binding.aligned_row_stride(cfg["d"]))
        g.build_alias(cp.counts, cfg["subsample_t"])
        if rep == 0:
            # untrained vectors give the stored starting loss: the evaluation protocol is the same
            assert abs(heldout(g, cfg, cp) - before) <= 1e-6 * before

        def gstep(t, lr, num, ph, st, g=g):
            g.set_step(num)
            g.sgns_step(t, W, N, lr, binding.MODE_HOGWILD, want_stats=False)
        train(gstep, chunks, epochs=1, lr0=cfg["lr"])
        losses.append(heldout(g, cfg, cp))
        g.close()
    print("LONG %s: %d chunks, held-out loss checker %.5f gpu %s" % (run, n_chunks, want, losses))
    for got in losses:
        assert abs(got - want) / want <= 0.01, (got, want)
