"""Writes tests/golden/hogwild_losses.txt: the held-out loss per positive pair (Eq. (1)) that the
sequential CPU oracle reaches after training, for the runs whose length the Hogwild acceptance
criterion names (one pass over the small corpus; a 20 M-token prefix of the medium corpus).

TEST INFRASTRUCTURE.  It calls only the oracle and the seeded input generator; nothing of the CUDA
library runs here, so every stored value is the oracle's own.  The GPU tests train the library on
the same chunks with the same learning rates and compare their loss with the stored one.

    python oracle/write_golden_losses.py            # all runs, one process per run (minutes of CPU)
    python oracle/write_golden_losses.py small      # one run, printed only

Training protocol (harness level, restated here so that this file needs nothing but the oracle):
chunk i of the corpus is step number i; the learning rate of a step is
lr0 * max(1 - words_done / (words_total + 1), 1e-4), evaluated before the step; Hogwild mode of the
oracle = one target after another (Section 5.1: lock-free operation, sequential limit); the loss
is evaluated on chunks 1,000,000 and 1,000,001 of the same corpus with step numbers 10^9 + chunk.
"""
from __future__ import annotations

import multiprocessing as mp
import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from oracle import Oracle  # noqa: E402
from paper_1606_08495_b200 import corpus  # noqa: E402  (inputs only)

OUT = os.path.join(ROOT, "tests", "golden", "hogwild_losses.txt")
SEED = 41
HELD = (1_000_000, 1_000_001)
HELD_STEP_BASE = 10 ** 9
# name -> (configuration, tokens of the corpus to train on)
RUNS = {
    "small": ("small", 17_000_000),
    "medium": ("medium", 20_000_000),
}


def heldout_loss(model: Oracle, cfg: dict, cp: corpus.Corpus) -> float:
    tot, pairs = 0.0, 0
    for j in HELD:
        s, p = model.loss(cp.chunk(j), cfg["window"], cfg["negatives"], step_id=HELD_STEP_BASE + j)
        tot += s
        pairs += p
    return tot / pairs


def run(name: str):
    cfg_name, tokens = RUNS[name]
    cfg = corpus.CONFIGS[cfg_name]
    cp = corpus.Corpus(cfg)
    n_chunks = tokens // cfg["minibatch"]
    model = Oracle(cfg["vocab"], cfg["d"], SEED)
    model.build_tables(cp.counts, cfg["subsample_t"])
    before = heldout_loss(model, cfg, cp)
    sizes = []
    chunks = []
    for i in range(n_chunks):
        c = cp.chunk(i)
        chunks.append(c)
        sizes.append(int((c >= 0).sum()))
    total = sum(sizes)
    done = 0
    t0 = time.time()
    for i, c in enumerate(chunks):
        lr = cfg["lr"] * max(1.0 - done / (total + 1.0), 1e-4)
        model.set_step(i)
        model.step(c, cfg["window"], cfg["negatives"], lr, 1)
        done += sizes[i]
    after = heldout_loss(model, cfg, cp)
    model.close()
    return name, cfg_name, n_chunks, total, before, after, time.time() - t0


def main(argv):
    names = argv[1:] or list(RUNS)
    with mp.Pool(len(names)) as pool:
        results = pool.map(run, names)
    lines = [
        "# Held-out loss per positive pair (Eq. (1)) of the sequential CPU oracle after training.",
        "# Written by: python oracle/write_golden_losses.py   (calls only oracle/ and the input generator)",
        "# Protocol: seed %d; chunk i = step number i; lr0 max(1 - words_done/(words_total+1), 1e-4) per step;" % SEED,
        "# Hogwild mode of the oracle (one target after another); loss on chunks %s with step numbers 10^9 + chunk." % (HELD,),
        "# <run>: <configuration> <chunks> <word tokens trained on> <loss before training> <loss after>",
    ]
    for name, cfg_name, n_chunks, total, before, after, secs in results:
        print("%s: %d chunks, %d words, loss %.9f -> %.9f (%.0f s)" % (name, n_chunks, total, before, after, secs))
        lines.append("%s: %s %d %d %.9f %.9f" % (name, cfg_name, n_chunks, total, before, after))
    if len(argv) == 1:
        with open(OUT, "w") as f:
            f.write("\n".join(lines) + "\n")
        print("wrote", OUT)


if __name__ == "__main__":
    main(sys.argv)
