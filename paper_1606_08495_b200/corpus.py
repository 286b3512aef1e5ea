"""Seeded synthetic corpora shaped like the paper's workloads.

This module only makes INPUTS (vocabulary histograms and token streams).  It
holds none of the method's arithmetic, so that both the CUDA library's tests and
the CPU checker can be fed exactly the same arrays.  The paper's own corpora
(a public news-text benchmark corpus and proprietary search sessions, Section 7)
are not available; Zipfian rank-frequency streams with the same vocabulary
sizes, sentence lengths and hyper-parameters stand in for them.

Token stream convention: int32 word ids in [0, vocab), ids ordered by
decreasing frequency (Section 5.1, the ordering O); -1 ends a sentence.
"""
from __future__ import annotations

import numpy as np

BASE_SEED = 160608495

# name -> workload description (sizes follow the five benchmark configurations)
CONFIGS = {
    "tiny": dict(index=0, vocab=10_000, zipf_s=1.0, corpus_tokens=500_000, sentence_len=50,
                 d=100, window=5, negatives=5, subsample_t=1e-4, lr=0.025, minibatch=4_096),
    "small": dict(index=1, vocab=71_000, zipf_s=1.05, corpus_tokens=17_000_000, sentence_len=1_000,
                  d=200, window=5, negatives=5, subsample_t=1e-4, lr=0.025, minibatch=65_536),
    "medium": dict(index=2, vocab=1_000_000, zipf_s=1.0, corpus_tokens=200_000_000, sentence_len=100,
                   d=300, window=10, negatives=5, subsample_t=1e-5, lr=0.025, minibatch=262_144),
    "sponsored": dict(index=3, vocab=20_000_000, zipf_s=0.8, classes=(0.60, 0.25, 0.15),
                      corpus_tokens=500_000_000, sentence_len=(5, 40),
                      d=300, window=5, negatives=5, subsample_t=1e-5, lr=0.025, minibatch=1_000_000),
    "large": dict(index=4, vocab=60_000_000, zipf_s=0.9, corpus_tokens=1_000_000_000, sentence_len=30,
                  d=300, window=5, negatives=10, subsample_t=1e-5, lr=0.025, minibatch=1_000_000),
}


def scaled(cfg: dict, **over) -> dict:
    """A copy of a configuration with some fields replaced (reduced test sizes)."""
    out = dict(cfg)
    out.update(over)
    return out


def word_probabilities(cfg: dict) -> np.ndarray:
    """Rank-frequency probabilities, fp64, sorted in decreasing order (id = rank)."""
    V = int(cfg["vocab"])
    s = float(cfg["zipf_s"])
    classes = cfg.get("classes")
    if not classes:
        p = np.arange(1, V + 1, dtype=np.float64) ** (-s)
        return p / p.sum()
    # several id classes (queries / links / ads), each Zipfian inside; the chance
    # of a class equals its share of the vocabulary; ids re-ranked by probability
    parts = []
    left = V
    for k, share in enumerate(classes):
        nk = left if k == len(classes) - 1 else int(round(V * share))
        left -= nk
        pk = np.arange(1, nk + 1, dtype=np.float64) ** (-s)
        parts.append(pk / pk.sum() * (nk / V))
    p = np.concatenate(parts)
    p = np.sort(p)[::-1].copy()
    return p / p.sum()


def word_counts(cfg: dict, p: np.ndarray | None = None) -> np.ndarray:
    """The vocabulary histogram handed to the table builders: max(1, round(T p_r))."""
    if p is None:
        p = word_probabilities(cfg)
    c = np.rint(p * float(cfg["corpus_tokens"]))
    return np.maximum(c, 1.0).astype(np.uint64)


class Corpus:
    """Draws reproducible chunks of the token stream of one configuration."""

    def __init__(self, cfg: dict, seed: int = BASE_SEED):
        self.cfg = dict(cfg)
        self.seed = int(seed) + 1000 * int(cfg.get("index", 0))
        self.p = word_probabilities(cfg)
        self.counts = word_counts(cfg, self.p)
        self.cdf = np.cumsum(self.p)
        self.cdf[-1] = 1.0

    def _words(self, rng: np.random.Generator, n: int) -> np.ndarray:
        u = rng.random(n)
        ids = np.searchsorted(self.cdf, u, side="right")
        return np.minimum(ids, len(self.cdf) - 1).astype(np.int32)

    def chunk(self, index: int, words: int | None = None) -> np.ndarray:
        """Chunk number `index`: whole sentences holding at most `words` word
        tokens (default: the configuration's minibatch), each followed by -1."""
        cfg = self.cfg
        words = int(words if words is not None else cfg["minibatch"])
        rng = np.random.Generator(np.random.PCG64([self.seed, int(index)]))
        sl = cfg["sentence_len"]
        if isinstance(sl, (tuple, list)):
            lo, hi = int(sl[0]), int(sl[1])
            lens = rng.integers(lo, hi + 1, size=max(1, words // lo + 1))
            keep = np.cumsum(lens) <= words
            keep[0] = True
            lens = lens[keep]
        else:
            lens = np.full(max(1, words // int(sl)), int(sl), dtype=np.int64)
        total = int(lens.sum())
        toks = self._words(rng, total)
        out = np.full(total + len(lens), -1, dtype=np.int32)
        ends = np.cumsum(lens) + np.arange(len(lens))          # positions of the -1 entries
        mask = np.ones(len(out), dtype=bool)
        mask[ends] = False
        out[mask] = toks
        return out


def clustered_rows(n: int, d: int, seed: int, cluster_size: int = 50, noise: float = 0.55,
                   loose: float = 0.2) -> np.ndarray:
    """Stand-in for trained vectors as the retrieval stage sees them (Section 7.2): fp32 rows
    [n, d] that have neighbours.  A row is a cluster centre plus `noise` times a standard normal
    vector (cosine between two rows of a cluster about 1 / (1 + noise^2), 0.77 for 0.55, above the
    paper's threshold of 0.65; rows of different clusters are nearly orthogonal); clusters have
    `cluster_size` rows on average; a share `loose` of the rows is plain noise and has no neighbour.
    Inputs only: written into a table by the caller."""
    rng = np.random.default_rng([int(seed), 7])
    n_clusters = max(1, n // cluster_size)
    centres = rng.standard_normal((n_clusters, d), dtype=np.float32)
    out = np.empty((n, d), dtype=np.float32)
    for a in range(0, n, 1 << 18):
        b = min(n, a + (1 << 18))
        which = rng.integers(0, n_clusters, b - a)
        is_loose = rng.random(b - a) < loose
        rows = noise * rng.standard_normal((b - a, d), dtype=np.float32)
        rows += np.where(is_loose[:, None], np.float32(0), centres[which])
        rows[is_loose] *= np.float32(1.0 / noise)
        out[a:b] = rows
    return out
