"""The training loop around the step (Section 5.1: several passes over the data, with the learning
rate lowered from pass to pass in the way the word2vec program lowers it; optional
interleaved minibatch formation).

Harness level only: it decides which chunk, which step number, which learning rate and which
interleaving phase each call gets, and hands them to a `step` callable; none of the method's
arithmetic is here, so the same loop can drive the CUDA library and any other implementation of
the step.
"""
from __future__ import annotations

from typing import Callable, Iterable, Sequence

MIN_LR_FRACTION = 1e-4


def learning_rate(lr0: float, words_done: int, words_total: int, schedule: str = "linear",
                  epoch: int = 0, epochs: int = 1) -> float:
    """"linear": lr0 * max(1 - words_done / (words_total + 1), 1e-4), evaluated once per step (the
    open-source word2vec program's decay, to which the paper refers); "epoch": the same line
    evaluated at the start of each pass over the data and held during it (Section 5.1 speaks of a
    reduction per pass)."""
    if schedule == "linear":
        frac = 1.0 - words_done / (words_total + 1.0)
    elif schedule == "epoch":
        frac = 1.0 - epoch / float(epochs)
    else:
        raise ValueError("schedule must be 'linear' or 'epoch'")
    return lr0 * max(frac, MIN_LR_FRACTION)


def train(step: Callable[..., object], chunks: Sequence, epochs: int, lr0: float, stride: int = 1,
          schedule: str = "linear", on_step: Callable[[dict], None] | None = None) -> int:
    """Runs `epochs` passes over `chunks` (token arrays).

    step(tokens, lr, step_number, phase, stride) performs one minibatch step.  With stride > 1 each
    chunk is visited `stride` times in a row with the same step number and phases 0..stride-1
    (interleaved minibatches); the step number is the running chunk count, so a resumed run that
    passes the same numbers redraws the same samples.  Returns the number of step calls made.
    """
    if stride < 1 or epochs < 1:
        raise ValueError("epochs and stride must be at least 1")
    sizes = [int((c >= 0).sum()) if hasattr(c, "sum") else sum(1 for t in c if t >= 0) for c in chunks]
    total = epochs * sum(sizes)
    done = calls = number = 0
    for epoch in range(epochs):
        for chunk, words in zip(chunks, sizes):
            lr = learning_rate(lr0, done, total, schedule, epoch, epochs)
            for phase in range(stride):
                step(chunk, lr, number, phase, stride)
                calls += 1
                if on_step is not None:
                    on_step(dict(epoch=epoch, step_number=number, phase=phase, lr=lr, words_done=done))
            done += words
            number += 1
    return calls


def gpu_step(model, window: int, negatives: int, mode: int):
    """The `step` callable for a binding.W2V model."""
    def run(tokens, lr, number, phase, stride):
        model.set_step(number)
        model.set_interleave(phase, stride)
        model.sgns_step(tokens, window, negatives, lr, mode, want_stats=False)
    return run
