"""Helpers shared by the GPU parity tests: a GPU model and a CPU checker fed the same inputs."""
import numpy as np

from oracle import Oracle
from paper_1606_08495_b200 import binding, corpus


def make_pair(cfg, seed=11, sparse=False, counts=None, t=None, row_stride=None):
    cp = corpus.Corpus(cfg) if counts is None else None
    counts = cp.counts if counts is None else np.asarray(counts, dtype=np.uint64)
    t = cfg["subsample_t"] if t is None else t
    gpu = binding.W2V(cfg["vocab"], cfg["d"], seed, row_stride=row_stride)
    cpu = Oracle(cfg["vocab"], cfg["d"], seed, sparse=sparse)
    gpu.build_alias(counts, t)
    cpu.build_tables(counts, t)
    return gpu, cpu, cp


def row_rel_err(a, b):
    """max over rows of ||a - b||_inf / ||b||_inf (rows of zeros compared absolutely)."""
    a = a.astype(np.float64); b = b.astype(np.float64)
    den = np.abs(b).max(axis=1)
    err = np.abs(a - b).max(axis=1)
    return float((err / np.where(den > 0, den, 1.0)).max()) if len(a) else 0.0


def elem_rel_err(a, b):
    """elementwise error with floor max(|b|, 1e-3 ||row||_inf)."""
    a = a.astype(np.float64); b = b.astype(np.float64)
    floor = 1e-3 * np.abs(b).max(axis=1, keepdims=True)
    den = np.maximum(np.abs(b), floor)
    return float((np.abs(a - b) / np.where(den > 0, den, 1.0)).max()) if len(a) else 0.0


def touched_rows(c, x, n):
    return np.unique(c), np.unique(np.concatenate([x, n.ravel()]))


def assert_same_pairs(gpu, cpu, toks, W, N):
    c0, x0, n0 = cpu.sample_pairs(toks, W, N)
    c1, x1, n1, st, rc, P = gpu.sample_pairs(toks, W, N, allow=(binding.W2V_ERR_TOKEN_RANGE,))
    assert P == len(c0), (P, len(c0))
    assert np.array_equal(c0, c1)
    assert np.array_equal(x0, x1)
    assert np.array_equal(n0, n1)
    so = cpu.stats()
    for k in ("tokens", "kept", "centres", "pairs", "neg_draws", "neg_redraws", "oov"):
        assert st[k] == so[k], (k, st[k], so[k])
    return c0, x0, n0
