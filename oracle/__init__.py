"""CPU oracle for the SGNS minibatch step -- TEST INFRASTRUCTURE, not the product.

A ctypes wrapper over ``w2v_oracle.c`` (plain C, fp64 arithmetic on fp32
storage).  Only the tests, the smoke check and the benchmark's CPU-baseline /
reference arm may import this package; nothing under the CUDA package does,
and this package imports nothing from it.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "w2v_oracle.c")
_LIB = os.path.join(_HERE, "libw2v_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-ffp-contract=off", "-fno-fast-math",
               "-Wall", "-Wextra", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    build()
    L = C.CDLL(_LIB)
    u32, u64, i32p = C.c_uint32, C.c_uint64, C.POINTER(C.c_int32)
    vp = C.c_void_p
    L.orc_philox.argtypes = [u32] * 6 + [vp]
    L.orc_create.restype = vp
    L.orc_create.argtypes = [u64, u32, u64, C.c_int]
    L.orc_destroy.argtypes = [vp]
    L.orc_set_step.argtypes = [vp, u64]
    L.orc_set_interleave.argtypes = [vp, u32, u32]
    L.orc_get_step.restype = u64
    L.orc_get_step.argtypes = [vp]
    L.orc_init_row.argtypes = [vp, u64, vp]
    L.orc_read_rows.argtypes = [vp, u32, vp, u64, vp]
    L.orc_write_rows.argtypes = [vp, u32, vp, u64, vp]
    L.orc_build_tables.argtypes = [vp, vp, C.c_double]
    L.orc_get_tables.argtypes = [vp, vp, vp, vp]
    L.orc_alias_draw.restype = u32
    L.orc_alias_draw.argtypes = [vp, u32, u32, u32]
    L.orc_get_stats.argtypes = [vp, vp]
    L.orc_sample_pairs.argtypes = [vp, vp, u64, u32, u32, vp, vp, vp, u64, vp]
    L.orc_step.argtypes = [vp, vp, u64, u32, u32, C.c_double, u32]
    L.orc_step_pairs.argtypes = [vp, vp, vp, vp, u64, u32, C.c_double, u32]
    L.orc_partial_dots.argtypes = [vp, vp, u64, u32, u32, vp]
    L.orc_loss.argtypes = [vp, vp, u64, u32, u32, u64, vp, vp]
    L.orc_loss_pairs.restype = C.c_double
    L.orc_loss_pairs.argtypes = [vp, vp, vp, vp, u64, u32]
    L.orc_cbow_examples.argtypes = [vp, vp, u64, u32, u32, vp, vp, vp, vp, u64, u64, vp, vp]
    L.orc_cbow_step.argtypes = [vp, vp, u64, u32, u32, C.c_double, u32]
    L.orc_cbow_step_examples.argtypes = [vp, vp, vp, vp, vp, u64, u32, C.c_double, u32]
    L.orc_cbow_loss.argtypes = [vp, vp, u64, u32, u32, u64, vp, vp]
    L.orc_cbow_loss_examples.restype = C.c_double
    L.orc_cbow_loss_examples.argtypes = [vp, vp, vp, vp, vp, u64, u32]
    L.orc_topk_cosine.argtypes = [vp, u32, vp, u64, u64, u64, u32, C.c_double, vp, vp]
    L.orc_rows_resident.restype = u64
    L.orc_rows_resident.argtypes = [vp, u32]
    _lib = L
    return L


def philox(k0, k1, c0, c1, c2, c3):
    out = np.zeros(4, dtype=np.uint32)
    _load().orc_philox(k0, k1, c0, c1, c2, c3, out.ctypes.data)
    return out


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


STAT_NAMES = ("tokens", "kept", "centres", "pairs", "neg_draws", "neg_redraws", "oov")


class Oracle:
    """One pair of fp32 tables (U input, V output) plus the sampling tables."""

    def __init__(self, vocab: int, d: int, seed: int, sparse: bool = False):
        self.L = _load()
        self.vocab, self.d, self.seed = int(vocab), int(d), int(seed)
        self.h = self.L.orc_create(self.vocab, self.d, self.seed, 1 if sparse else 0)
        if not self.h:
            raise ValueError("orc_create rejected its arguments")

    def close(self):
        if self.h:
            self.L.orc_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- state -----------------------------------------------------------
    def set_step(self, s):
        self.L.orc_set_step(self.h, int(s))

    def get_step(self):
        return int(self.L.orc_get_step(self.h))

    def set_interleave(self, phase, stride):
        if self.L.orc_set_interleave(self.h, int(phase), int(stride)) != 0:
            raise ValueError("need stride >= 1 and phase < stride")

    def init_row(self, row):
        out = np.empty(self.d, dtype=np.float32)
        self.L.orc_init_row(self.h, int(row), out.ctypes.data)
        return out

    def read_rows(self, which, ids):
        ids = np.ascontiguousarray(ids, dtype=np.int64)
        out = np.empty((len(ids), self.d), dtype=np.float32)
        self.L.orc_read_rows(self.h, int(which), ids.ctypes.data, len(ids), out.ctypes.data)
        return out

    def write_rows(self, which, ids, rows):
        ids = np.ascontiguousarray(ids, dtype=np.int64)
        rows = np.ascontiguousarray(rows, dtype=np.float32).reshape(len(ids), self.d)
        self.L.orc_write_rows(self.h, int(which), ids.ctypes.data, len(ids), rows.ctypes.data)

    # -- tables ----------------------------------------------------------
    def build_tables(self, counts, subsample_t):
        counts = np.ascontiguousarray(counts, dtype=np.uint64)
        assert len(counts) == self.vocab
        rc = self.L.orc_build_tables(self.h, counts.ctypes.data, float(subsample_t))
        if rc != 0:
            raise ValueError("counts must all be >= 1")

    def tables(self):
        thr = np.empty(self.vocab, dtype=np.uint32)
        alias = np.empty(self.vocab, dtype=np.uint32)
        keep = np.empty(self.vocab, dtype=np.uint32)
        assert self.L.orc_get_tables(self.h, thr.ctypes.data, alias.ctypes.data, keep.ctypes.data) == 0
        return thr, alias, keep

    def alias_draw(self, r0, r1, r2):
        return int(self.L.orc_alias_draw(self.h, r0, r1, r2))

    def stats(self):
        out = np.zeros(7, dtype=np.uint64)
        self.L.orc_get_stats(self.h, out.ctypes.data)
        return dict(zip(STAT_NAMES, (int(x) for x in out)))

    # -- sampling ----------------------------------------------------------
    def sample_pairs(self, tokens, window, negatives, cap=None):
        tokens = _i32(tokens)
        n = len(tokens)
        if cap is None:
            cap = max(1, n * 2 * window)
        centre = np.empty(cap, dtype=np.int32)
        context = np.empty(cap, dtype=np.int32)
        negs = np.empty((cap, negatives), dtype=np.int32)
        P = C.c_uint64(0)
        rc = self.L.orc_sample_pairs(self.h, tokens.ctypes.data, n, window, negatives,
                                     centre.ctypes.data, context.ctypes.data, negs.ctypes.data,
                                     cap, C.byref(P))
        if rc != 0:
            raise ValueError("orc_sample_pairs rejected its arguments")
        P = min(int(P.value), cap)
        return centre[:P].copy(), context[:P].copy(), negs[:P].copy()

    # -- the step ------------------------------------------------------------
    def step(self, tokens, window, negatives, lr, mode):
        tokens = _i32(tokens)
        rc = self.L.orc_step(self.h, tokens.ctypes.data, len(tokens), window, negatives, float(lr), mode)
        if rc != 0:
            raise ValueError("orc_step rejected its arguments")
        return self.stats()

    def step_pairs(self, centre, context, negs, lr, mode):
        centre, context = _i32(centre), _i32(context)
        negs = _i32(negs).reshape(len(centre), -1)
        rc = self.L.orc_step_pairs(self.h, centre.ctypes.data, context.ctypes.data, negs.ctypes.data,
                                   len(centre), negs.shape[1], float(lr), mode)
        assert rc == 0

    def partial_dots(self, pairs, col_lo, col_hi):
        pairs = _i32(pairs).reshape(-1, 2)
        out = np.empty(len(pairs), dtype=np.float64)
        rc = self.L.orc_partial_dots(self.h, pairs.ctypes.data, len(pairs), col_lo, col_hi, out.ctypes.data)
        if rc != 0:
            raise ValueError("bad column range")
        return out

    def loss(self, tokens, window, negatives, step_id):
        """(sum of -log-likelihood terms of Eq. (1) over the chunk, number of positive pairs)."""
        tokens = _i32(tokens)
        s = C.c_double(0.0)
        P = C.c_uint64(0)
        rc = self.L.orc_loss(self.h, tokens.ctypes.data, len(tokens), window, negatives, int(step_id),
                             C.byref(s), C.byref(P))
        assert rc == 0
        return s.value, int(P.value)

    def loss_pairs(self, centre, context, negs):
        centre, context = _i32(centre), _i32(context)
        negs = _i32(negs).reshape(len(centre), -1)
        return float(self.L.orc_loss_pairs(self.h, centre.ctypes.data, context.ctypes.data,
                                           negs.ctypes.data, len(centre), negs.shape[1]))

    # -- continuous bag of words -------------------------------------------
    def cbow_examples(self, tokens, window, negatives):
        """(centre[E], negs[E, N], ctx_off[E + 1], ctx[sum |C|]) of the chunk's examples."""
        tokens = _i32(tokens)
        n = len(tokens)
        cap_ex, cap_ctx = max(1, n), max(1, n * 2 * window)
        centre = np.empty(cap_ex, dtype=np.int32)
        negs = np.empty((cap_ex, negatives), dtype=np.int32)
        ctx_off = np.zeros(cap_ex + 1, dtype=np.uint64)
        ctx = np.empty(cap_ctx, dtype=np.int32)
        E, M = C.c_uint64(0), C.c_uint64(0)
        rc = self.L.orc_cbow_examples(self.h, tokens.ctypes.data, n, window, negatives, centre.ctypes.data,
                                      negs.ctypes.data, ctx_off.ctypes.data, ctx.ctypes.data, cap_ex, cap_ctx,
                                      C.byref(E), C.byref(M))
        if rc != 0:
            raise ValueError("orc_cbow_examples rejected its arguments")
        E, M = int(E.value), int(M.value)
        return centre[:E].copy(), negs[:E].copy(), ctx_off[:E + 1].copy(), ctx[:M].copy()

    def cbow_step(self, tokens, window, negatives, lr, mode):
        tokens = _i32(tokens)
        rc = self.L.orc_cbow_step(self.h, tokens.ctypes.data, len(tokens), window, negatives, float(lr), mode)
        if rc != 0:
            raise ValueError("orc_cbow_step rejected its arguments")
        return self.stats()

    @staticmethod
    def _examples(centre, negs, ctx_off, ctx):
        centre = _i32(centre)
        negs = _i32(negs).reshape(len(centre), -1)
        ctx_off = np.ascontiguousarray(ctx_off, dtype=np.uint64)
        ctx = _i32(ctx)
        assert len(ctx_off) == len(centre) + 1 and int(ctx_off[-1]) == len(ctx)
        return centre, negs, ctx_off, ctx

    def cbow_step_examples(self, centre, negs, ctx_off, ctx, lr, mode):
        centre, negs, ctx_off, ctx = self._examples(centre, negs, ctx_off, ctx)
        rc = self.L.orc_cbow_step_examples(self.h, centre.ctypes.data, negs.ctypes.data, ctx_off.ctypes.data,
                                           ctx.ctypes.data, len(centre), negs.shape[1], float(lr), mode)
        assert rc == 0

    def cbow_loss(self, tokens, window, negatives, step_id):
        """(sum of -log-likelihood terms over the chunk's examples, number of examples)."""
        tokens = _i32(tokens)
        s, E = C.c_double(0.0), C.c_uint64(0)
        rc = self.L.orc_cbow_loss(self.h, tokens.ctypes.data, len(tokens), window, negatives, int(step_id),
                                  C.byref(s), C.byref(E))
        assert rc == 0
        return s.value, int(E.value)

    def cbow_loss_examples(self, centre, negs, ctx_off, ctx):
        centre, negs, ctx_off, ctx = self._examples(centre, negs, ctx_off, ctx)
        return float(self.L.orc_cbow_loss_examples(self.h, centre.ctypes.data, negs.ctypes.data,
                                                   ctx_off.ctypes.data, ctx.ctypes.data, len(centre),
                                                   negs.shape[1]))

    def topk_cosine(self, which, queries, cand_lo, cand_hi, K, tau):
        """(ids[m, K] padded with -1, cosines[m, K]) of the K nearest candidate rows above tau."""
        q = np.ascontiguousarray(queries, dtype=np.int64)
        ids = np.empty((len(q), K), dtype=np.int64)
        cs = np.empty((len(q), K), dtype=np.float64)
        rc = self.L.orc_topk_cosine(self.h, int(which), q.ctypes.data, len(q), int(cand_lo), int(cand_hi), int(K),
                                    float(tau), ids.ctypes.data, cs.ctypes.data)
        if rc != 0:
            raise ValueError("orc_topk_cosine rejected its arguments")
        return ids, cs

    def rows_resident(self, which):
        return int(self.L.orc_rows_resident(self.h, which))
