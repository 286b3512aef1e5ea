"""ctypes binding of libw2v.so: one Python function per C entry point, same names,
argument marshalling only.  Torch provides device memory and streams; every step of
the method runs in the library's kernels.  There is no fallback: if the library is
missing or cannot be built, loading raises.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

from . import build as _build

W2V_OK = 0
W2V_ERR_ARG, W2V_ERR_STATE, W2V_ERR_NOMEM, W2V_ERR_CUDA = -1, -2, -3, -4
W2V_ERR_TOKEN_RANGE, W2V_ERR_CAPACITY = -5, -6
MODE_SNAPSHOT, MODE_HOGWILD = 0, 1
TABLE_U, TABLE_V = 0, 1
MAX_SHARDS = 16                  # most column shards (and epoch words per barrier array)

EXPORTS = (
    "w2v_create", "w2v_create_strided", "w2v_create_shard", "w2v_shard_dots", "w2v_shard_adjust",
    "w2v_get_row_stride", "w2v_set_interleave", "w2v_cbow_step", "w2v_cbow_step_host", "w2v_sample_cbow",
    "w2v_topk_cosine", "w2v_set_retrieval_kernel", "w2v_destroy", "w2v_build_alias", "w2v_get_tables", "w2v_sgns_step",
    "w2v_sgns_step_host", "w2v_sample_pairs", "w2v_partial_dots", "w2v_read_rows", "w2v_write_rows",
    "w2v_set_step", "w2v_get_step", "w2v_get_table_ptrs", "w2v_sync", "w2v_profile_enable",
    "w2v_profile_read", "w2v_get_launch_count", "w2v_set_tuning", "w2v_last_error",
    "w2v_sample_pairs_noalloc", "w2v_peer_barrier", "w2v_probe_rows",
    "w2v_selftest_bounded_wait", "w2v_probe_bulk_ring", "w2v_probe_mma_ring",
)


class StepStats(C.Structure):
    _fields_ = [("tokens", C.c_uint64), ("kept", C.c_uint64), ("centres", C.c_uint64),
                ("pairs", C.c_uint64), ("neg_draws", C.c_uint64), ("neg_redraws", C.c_uint64),
                ("oov", C.c_uint64), ("status", C.c_uint32), ("reserved", C.c_uint32)]

    def as_dict(self):
        return {k: int(getattr(self, k)) for k, _ in self._fields_ if k != "reserved"}


class W2VError(RuntimeError):
    def __init__(self, code, text):
        super().__init__(f"libw2v error {code}: {text}")
        self.code = code


_lib = None


def library_path() -> str:
    return _build.LIB


def load():
    """Load libw2v.so (building it first if the sources are newer and nvcc is here)."""
    global _lib
    if _lib is not None:
        return _lib
    try:
        _build.build()
    except Exception as exc:                     # no nvcc on this machine: use the shipped binary
        if not os.path.exists(_build.LIB):
            raise RuntimeError(f"libw2v.so is missing and could not be built: {exc}") from exc
    L = C.CDLL(_build.LIB)
    vp, u32, u64, i32 = C.c_void_p, C.c_uint32, C.c_uint64, C.c_int32
    sig = {
        "w2v_create": [u64, u32, u64, vp, vp, vp, C.POINTER(vp)],
        "w2v_create_strided": [u64, u32, u32, u64, vp, vp, vp, C.POINTER(vp)],
        "w2v_get_row_stride": [vp, C.POINTER(u32)],
        "w2v_create_shard": [u64, u32, u32, u32, u32, u64, vp, vp, vp, C.POINTER(vp)],
        "w2v_shard_dots": [vp, vp, u64, u32, u32, C.POINTER(vp), u32, u64, C.POINTER(StepStats)],
        "w2v_shard_adjust": [vp, vp, C.c_float],
        "w2v_peer_barrier": [vp, C.POINTER(vp), u32, u32, u32, u32],
        "w2v_probe_rows": [vp, u32, u64, u64, C.POINTER(C.c_double), C.POINTER(u64)],
        "w2v_selftest_bounded_wait": [vp, u32],
        "w2v_probe_bulk_ring": [vp, u32, u32, u32, u64, C.POINTER(C.c_double), C.POINTER(u64)],
        "w2v_probe_mma_ring": [vp, u32, u32, u32, u32, C.POINTER(C.c_double), C.POINTER(C.c_double)],
        "w2v_destroy": [vp],
        "w2v_build_alias": [vp, vp, C.c_double],
        "w2v_get_tables": [vp, vp, vp, vp],
        "w2v_sgns_step": [vp, vp, u64, u32, u32, C.c_float, u32, C.POINTER(StepStats)],
        "w2v_sgns_step_host": [vp, vp, u64, u32, u32, C.c_float, u32, C.POINTER(StepStats)],
        "w2v_cbow_step": [vp, vp, u64, u32, u32, C.c_float, u32, C.POINTER(StepStats)],
        "w2v_cbow_step_host": [vp, vp, u64, u32, u32, C.c_float, u32, C.POINTER(StepStats)],
        "w2v_sample_cbow": [vp, vp, u64, u32, u32, vp, vp, u64, C.POINTER(u64), C.POINTER(StepStats)],
        "w2v_sample_pairs": [vp, vp, u64, u32, u32, vp, vp, vp, u64, C.POINTER(u64), C.POINTER(StepStats)],
        "w2v_sample_pairs_noalloc": [vp, vp, u64, u32, u32, vp, vp, vp, u64, C.POINTER(u64), C.POINTER(StepStats)],
        "w2v_partial_dots": [vp, vp, u64, u32, u32, vp],
        "w2v_read_rows": [vp, u32, vp, u64, vp],
        "w2v_write_rows": [vp, u32, vp, u64, vp],
        "w2v_topk_cosine": [vp, u32, vp, u64, u64, u64, u32, C.c_float, vp, vp],
        "w2v_set_retrieval_kernel": [vp, u32],
        "w2v_set_step": [vp, u64],
        "w2v_set_interleave": [vp, u32, u32],
        "w2v_get_step": [vp, C.POINTER(u64)],
        "w2v_get_table_ptrs": [vp, C.POINTER(vp), C.POINTER(vp)],
        "w2v_sync": [vp],
        "w2v_profile_enable": [vp, i32],
        "w2v_profile_read": [vp, C.POINTER(C.c_double), C.POINTER(u64)],
        "w2v_get_launch_count": [vp, C.POINTER(u64)],
        "w2v_set_tuning": [vp, u32, u32],
        "w2v_last_error": [vp],
    }
    for name, argtypes in sig.items():
        fn = getattr(L, name)
        fn.argtypes = argtypes
        fn.restype = C.c_char_p if name == "w2v_last_error" else i32
    _lib = L
    return L


def _check(h, rc, allow=()):
    if rc != W2V_OK and rc not in allow:
        text = load().w2v_last_error(h)
        raise W2VError(rc, text.decode() if text else "?")
    return rc


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, torch.Tensor):
        assert t.is_contiguous()
        return t.data_ptr()
    if isinstance(t, np.ndarray):
        assert t.flags["C_CONTIGUOUS"]
        return t.ctypes.data
    return int(t)


# ---- one function per C entry point ---------------------------------------------------
def w2v_create(vocab, d, seed, U, V, stream):
    h = C.c_void_p()
    rc = load().w2v_create(int(vocab), int(d), int(seed), _ptr(U), _ptr(V), stream, C.byref(h))
    if rc != W2V_OK:
        raise W2VError(rc, "w2v_create rejected its arguments or could not allocate")
    return h


def w2v_create_strided(vocab, d, row_stride, seed, U, V, stream):
    h = C.c_void_p()
    rc = load().w2v_create_strided(int(vocab), int(d), int(row_stride), int(seed), _ptr(U), _ptr(V), stream,
                                   C.byref(h))
    if rc != W2V_OK:
        raise W2VError(rc, "w2v_create_strided rejected its arguments or could not allocate")
    return h


def w2v_create_shard(vocab, d_full, col_lo, col_hi, row_stride, seed, U, V, stream):
    h = C.c_void_p()
    rc = load().w2v_create_shard(int(vocab), int(d_full), int(col_lo), int(col_hi), int(row_stride), int(seed),
                                 _ptr(U), _ptr(V), stream, C.byref(h))
    if rc != W2V_OK:
        raise W2VError(rc, "w2v_create_shard rejected its arguments or could not allocate")
    return h


def w2v_shard_dots(h, tokens, n, window, negatives, F_peers, cap, stats=None, allow=()):
    """F_peers: device pointers (ints or tensors), one array of `cap` floats per shard."""
    ptrs = (C.c_void_p * len(F_peers))(*[_ptr(f) for f in F_peers])
    ref = C.byref(stats) if stats is not None else None
    return _check(h, load().w2v_shard_dots(h, _ptr(tokens), int(n), window, negatives, ptrs, len(F_peers),
                                           int(cap), ref), allow)


def w2v_shard_adjust(h, F, lr):
    return _check(h, load().w2v_shard_adjust(h, _ptr(F), float(lr)))


def w2v_peer_barrier(h, flags_peers, rank, epoch, timeout_ms):
    """flags_peers: device pointers (ints or tensors), one array of len(flags_peers) uint32 per shard."""
    ptrs = (C.c_void_p * len(flags_peers))(*[_ptr(f) for f in flags_peers])
    return _check(h, load().w2v_peer_barrier(h, ptrs, len(flags_peers), int(rank), int(epoch), int(timeout_ms)))


PROBE_GATHER, PROBE_GATHER_RED, PROBE_GATHER_ALIAS, PROBE_GATHER_RED_ALIAS, PROBE_TOUCH_RED = range(5)


def w2v_probe_rows(h, access, span_rows, rows):
    """(milliseconds, rows touched) of one probe launch."""
    ms, done = C.c_double(0.0), C.c_uint64(0)
    _check(h, load().w2v_probe_rows(h, int(access), int(span_rows), int(rows), C.byref(ms), C.byref(done)))
    return ms.value, int(done.value)


def w2v_probe_bulk_ring(h, stage_bytes, stages, producers, bytes_per_sm):
    """(milliseconds, bytes copied per SM) of one launch of the bulk-copy ring probe."""
    ms, done = C.c_double(0.0), C.c_uint64(0)
    _check(h, load().w2v_probe_bulk_ring(h, int(stage_bytes), int(stages), int(producers), int(bytes_per_sm),
                                         C.byref(ms), C.byref(done)))
    return ms.value, int(done.value)


def w2v_probe_mma_ring(h, kblocks_per_stage, stages, tiles, span_tiles):
    """(SM cycles per tile, cycles of them spent waiting for data) of the producer / ring / MMA probe."""
    cyc, waited = C.c_double(0.0), C.c_double(0.0)
    _check(h, load().w2v_probe_mma_ring(h, int(kblocks_per_stage), int(stages), int(tiles), int(bool(span_tiles)),
                                        C.byref(cyc), C.byref(waited)))
    return cyc.value, waited.value


def w2v_selftest_bounded_wait(h, timeout_ms):
    return _check(h, load().w2v_selftest_bounded_wait(h, int(timeout_ms)))


def w2v_get_row_stride(h):
    s = C.c_uint32(0)
    _check(h, load().w2v_get_row_stride(h, C.byref(s)))
    return int(s.value)


def w2v_destroy(h):
    return load().w2v_destroy(h)


def w2v_build_alias(h, counts, subsample_t):
    counts = np.ascontiguousarray(counts, dtype=np.uint64)
    return _check(h, load().w2v_build_alias(h, counts.ctypes.data, float(subsample_t)))


def w2v_get_tables(h, vocab):
    thr = np.empty(vocab, dtype=np.uint32)
    alias = np.empty(vocab, dtype=np.uint32)
    keep = np.empty(vocab, dtype=np.uint32)
    _check(h, load().w2v_get_tables(h, thr.ctypes.data, alias.ctypes.data, keep.ctypes.data))
    return thr, alias, keep


def w2v_sgns_step(h, tokens, n, window, negatives, lr, mode, stats=None, allow=()):
    ref = C.byref(stats) if stats is not None else None
    return _check(h, load().w2v_sgns_step(h, _ptr(tokens), int(n), window, negatives, float(lr), mode, ref), allow)


def w2v_sgns_step_host(h, tokens_host, n, window, negatives, lr, mode, stats=None, allow=()):
    ref = C.byref(stats) if stats is not None else None
    return _check(h, load().w2v_sgns_step_host(h, _ptr(tokens_host), int(n), window, negatives, float(lr), mode, ref), allow)


def w2v_cbow_step(h, tokens, n, window, negatives, lr, mode, stats=None, allow=()):
    ref = C.byref(stats) if stats is not None else None
    return _check(h, load().w2v_cbow_step(h, _ptr(tokens), int(n), window, negatives, float(lr), mode, ref), allow)


def w2v_cbow_step_host(h, tokens_host, n, window, negatives, lr, mode, stats=None, allow=()):
    ref = C.byref(stats) if stats is not None else None
    return _check(h, load().w2v_cbow_step_host(h, _ptr(tokens_host), int(n), window, negatives, float(lr), mode, ref), allow)


def w2v_sample_cbow(h, tokens, n, window, negatives, centre, negs, cap, stats=None, allow=()):
    nex = C.c_uint64(0)
    ref = C.byref(stats) if stats is not None else None
    rc = _check(h, load().w2v_sample_cbow(h, _ptr(tokens), int(n), window, negatives, _ptr(centre), _ptr(negs),
                                          int(cap), C.byref(nex), ref), allow)
    return rc, int(nex.value)


def w2v_sample_pairs(h, tokens, n, window, negatives, centre, context, negs, cap, stats=None, allow=()):
    npairs = C.c_uint64(0)
    ref = C.byref(stats) if stats is not None else None
    rc = _check(h, load().w2v_sample_pairs(h, _ptr(tokens), int(n), window, negatives, _ptr(centre), _ptr(context),
                                           _ptr(negs), int(cap), C.byref(npairs), ref), allow)
    return rc, int(npairs.value)


def w2v_sample_pairs_noalloc(h, tokens, n, window, negatives, centre, context, negs, cap, stats=None, allow=()):
    """w2v_sample_pairs on the library's fixed scratch: no device allocation, at most 65536 tokens."""
    npairs = C.c_uint64(0)
    ref = C.byref(stats) if stats is not None else None
    rc = _check(h, load().w2v_sample_pairs_noalloc(h, _ptr(tokens), int(n), window, negatives, _ptr(centre),
                                                   _ptr(context), _ptr(negs), int(cap), C.byref(npairs), ref), allow)
    return rc, int(npairs.value)


def w2v_partial_dots(h, pairs, m, col_lo, col_hi, out):
    return _check(h, load().w2v_partial_dots(h, _ptr(pairs), int(m), col_lo, col_hi, _ptr(out)))


def w2v_read_rows(h, which, ids, m, out):
    return _check(h, load().w2v_read_rows(h, which, _ptr(ids), int(m), _ptr(out)))


def w2v_write_rows(h, which, ids, m, rows):
    return _check(h, load().w2v_write_rows(h, which, _ptr(ids), int(m), _ptr(rows)))


def w2v_topk_cosine(h, which, queries, m, cand_lo, cand_hi, K, tau, out_ids, out_cos):
    return _check(h, load().w2v_topk_cosine(h, int(which), _ptr(queries), int(m), int(cand_lo), int(cand_hi), int(K),
                                            float(tau), _ptr(out_ids), _ptr(out_cos)))


def w2v_set_retrieval_kernel(h, kind):
    return _check(h, load().w2v_set_retrieval_kernel(h, int(kind)))


def w2v_set_step(h, step_id):
    return _check(h, load().w2v_set_step(h, int(step_id)))


def w2v_set_interleave(h, phase, stride):
    return _check(h, load().w2v_set_interleave(h, int(phase), int(stride)))


def w2v_get_step(h):
    s = C.c_uint64(0)
    _check(h, load().w2v_get_step(h, C.byref(s)))
    return int(s.value)


def w2v_sync(h):
    return _check(h, load().w2v_sync(h))


def w2v_profile_enable(h, on):
    return _check(h, load().w2v_profile_enable(h, 1 if on else 0))


def w2v_profile_read(h):
    ms, k = C.c_double(0.0), C.c_uint64(0)
    _check(h, load().w2v_profile_read(h, C.byref(ms), C.byref(k)))
    return ms.value, int(k.value)


def w2v_get_launch_count(h):
    k = C.c_uint64(0)
    _check(h, load().w2v_get_launch_count(h, C.byref(k)))
    return int(k.value)


def w2v_set_tuning(h, rows_in_flight, blocks_per_sm):
    return _check(h, load().w2v_set_tuning(h, int(rows_in_flight), int(blocks_per_sm)))


def aligned_row_stride(d):
    """Smallest row stride (in floats) >= d that puts every row on a 128-byte boundary, the
    granularity at which the GPU's L2 cache fetches and writes back: a gathered row then moves
    no bytes of its neighbours."""
    return (int(d) + 31) // 32 * 32


# ---- convenience wrapper: owns the torch tensors the handle points at ----------------------
class W2V:
    """Tables U and V as torch tensors on one GPU plus the library handle."""

    def __init__(self, vocab, d, seed, device="cuda:0", row_stride=None, columns=None):
        """columns=(col_lo, col_hi) makes this model one column shard of vectors with d columns;
        its own d is then the slice width."""
        load()
        if not torch.cuda.is_available():
            raise RuntimeError("libw2v needs a CUDA device; there is no CPU path")
        self.device = torch.device(device)
        self.vocab, self.seed = int(vocab), int(seed)
        self.d_full = int(d)
        self.col_lo, self.col_hi = (0, self.d_full) if columns is None else (int(columns[0]), int(columns[1]))
        self.d = self.col_hi - self.col_lo
        self.row_stride = self.d if row_stride is None else int(row_stride)
        with torch.cuda.device(self.device):
            self.U = torch.empty(self.vocab * self.row_stride, dtype=torch.float32, device=self.device)
            self.V = torch.empty(self.vocab * self.row_stride, dtype=torch.float32, device=self.device)
            self.stream = torch.cuda.current_stream(self.device)
            self.h = w2v_create_shard(self.vocab, self.d_full, self.col_lo, self.col_hi, self.row_stride,
                                      self.seed, self.U, self.V, self.stream.cuda_stream)

    def close(self):
        if getattr(self, "h", None):
            w2v_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def build_alias(self, counts, subsample_t):
        assert len(counts) == self.vocab
        w2v_build_alias(self.h, counts, subsample_t)

    def tables(self):
        return w2v_get_tables(self.h, self.vocab)

    def _dev_tokens(self, tokens):
        if isinstance(tokens, torch.Tensor):
            return tokens.to(device=self.device, dtype=torch.int32).contiguous()
        return torch.from_numpy(np.ascontiguousarray(tokens, dtype=np.int32)).to(self.device)

    def sgns_step(self, tokens, window, negatives, lr, mode, want_stats=True, allow=()):
        t = self._dev_tokens(tokens)
        st = StepStats() if want_stats else None
        w2v_sgns_step(self.h, t, t.numel(), window, negatives, lr, mode, st, allow)
        return st.as_dict() if want_stats else None

    def sgns_step_host(self, tokens_host, window, negatives, lr, mode, want_stats=True, allow=()):
        n = tokens_host.numel() if isinstance(tokens_host, torch.Tensor) else len(tokens_host)
        st = StepStats() if want_stats else None
        w2v_sgns_step_host(self.h, tokens_host, n, window, negatives, lr, mode, st, allow)
        return st.as_dict() if want_stats else None

    def cbow_step(self, tokens, window, negatives, lr, mode, want_stats=True, allow=()):
        t = self._dev_tokens(tokens)
        st = StepStats() if want_stats else None
        w2v_cbow_step(self.h, t, t.numel(), window, negatives, lr, mode, st, allow)
        return st.as_dict() if want_stats else None

    def sample_cbow(self, tokens, window, negatives, cap=None, allow=()):
        """(centre[E], negs[E, N], counters) of the examples the next cbow_step would use."""
        t = self._dev_tokens(tokens)
        n = t.numel()
        if cap is None:
            cap = max(1, n)
        centre = torch.empty(cap, dtype=torch.int32, device=self.device)
        negs = torch.empty(cap * negatives, dtype=torch.int32, device=self.device)
        st = StepStats()
        rc, E = w2v_sample_cbow(self.h, t, n, window, negatives, centre, negs, cap, st, allow)
        m = min(E, cap)
        return centre[:m].cpu().numpy(), negs[: m * negatives].view(m, negatives).cpu().numpy(), st.as_dict()

    def sample_pairs(self, tokens, window, negatives, cap=None, allow=()):
        t = self._dev_tokens(tokens)
        n = t.numel()
        if cap is None:
            cap = max(1, n * 2 * window)
        centre = torch.empty(cap, dtype=torch.int32, device=self.device)
        context = torch.empty(cap, dtype=torch.int32, device=self.device)
        negs = torch.empty(cap * negatives, dtype=torch.int32, device=self.device)
        st = StepStats()
        rc, P = w2v_sample_pairs(self.h, t, n, window, negatives, centre, context, negs, cap, st, allow)
        m = min(P, cap)
        return (centre[:m].cpu().numpy(), context[:m].cpu().numpy(),
                negs[: m * negatives].view(m, negatives).cpu().numpy(), st.as_dict(), rc, P)

    def partial_dots(self, pairs, col_lo, col_hi):
        p = torch.as_tensor(np.ascontiguousarray(pairs, dtype=np.int32)).reshape(-1, 2).to(self.device)
        out = torch.empty(p.shape[0], dtype=torch.float32, device=self.device)
        w2v_partial_dots(self.h, p, p.shape[0], col_lo, col_hi, out)
        return out.cpu().numpy()

    def read_rows(self, which, ids):
        i = torch.as_tensor(np.ascontiguousarray(ids, dtype=np.int64)).to(self.device)
        out = torch.zeros(i.numel() * self.d, dtype=torch.float32, device=self.device)
        w2v_read_rows(self.h, which, i, i.numel(), out)
        return out.view(i.numel(), self.d).cpu().numpy()

    def write_rows(self, which, ids, rows):
        i = torch.as_tensor(np.ascontiguousarray(ids, dtype=np.int64)).to(self.device)
        r = torch.as_tensor(np.ascontiguousarray(rows, dtype=np.float32)).reshape(-1).to(self.device)
        assert r.numel() == i.numel() * self.d
        w2v_write_rows(self.h, which, i, i.numel(), r)
        w2v_sync(self.h)

    def topk_cosine(self, which, queries, cand_lo, cand_hi, K, tau):
        """(ids[m, K] padded with -1, cosines[m, K]) of the K nearest candidate rows above tau."""
        q = torch.as_tensor(np.ascontiguousarray(queries, dtype=np.int64)).to(self.device)
        ids = torch.empty(q.numel() * K, dtype=torch.int64, device=self.device)
        cs = torch.empty(q.numel() * K, dtype=torch.float32, device=self.device)
        w2v_topk_cosine(self.h, which, q, q.numel(), cand_lo, cand_hi, K, tau, ids, cs)
        w2v_sync(self.h)
        return ids.view(-1, K).cpu().numpy(), cs.view(-1, K).cpu().numpy()

    def set_step(self, s):
        w2v_set_step(self.h, s)

    def get_step(self):
        return w2v_get_step(self.h)

    def set_interleave(self, phase, stride):
        w2v_set_interleave(self.h, phase, stride)

    def sync(self):
        w2v_sync(self.h)

    def set_tuning(self, rows_in_flight=0, blocks_per_sm=0):
        w2v_set_tuning(self.h, rows_in_flight, blocks_per_sm)

    def launch_count(self):
        return w2v_get_launch_count(self.h)
