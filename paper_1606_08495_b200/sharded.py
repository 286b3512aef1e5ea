"""The paper's column partition over several GPUs (Section 5.1, Eq. (6)-(7)).

Shard s holds columns [a_s, a_{s+1}) of every input and output vector.  One minibatch is:
every shard computes the partial dot products of its slice for index sets that all shards
regenerate from the same seed (Algorithm 1), the partials are summed over the shards
(Algorithm 3), and every shard applies the coefficients to its own columns (Algorithm 2).
Per minibatch a shard sends 4 bytes per target instead of 4 d bytes per vector.

Only argument marshalling and the exchange plumbing live here; all arithmetic runs in the
library's kernels (w2v_shard_dots, w2v_shard_adjust).

LocalShards       all shards in one process on one GPU: each shard's kernel adds its partials
                  into the F arrays of all shards through the peer-pointer list, one launch
                  after the other on one stream.  Used to check the decomposition on one GPU.
DistributedShard  one shard per rank of a torch.distributed group (one process per GPU).
                  exchange="allreduce": partials into a local array, then one NCCL all-reduce.
                  exchange="p2p": the arrays live in symmetric memory and the dots kernel adds
                  into every peer's array directly over NVLink; one time-limited device barrier
                  (w2v_peer_barrier) per step.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding


def shard_columns(d: int, shards: int):
    """Column ranges [(lo, hi)] of `shards` slices of a d-column vector: contiguous, covering
    [0, d), boundaries on multiples of 4 (one 16-byte load), widths as even as possible (the
    slowest shard sets the pace, so no slice is more than 4 columns wider than another)."""
    d, shards = int(d), int(shards)
    if d % 4 or d < 4:
        raise ValueError("d must be a positive multiple of 4")
    quads = d // 4
    if not 1 <= shards <= quads:
        raise ValueError(f"between 1 and {quads} shards fit {d} columns")
    base, extra = divmod(quads, shards)
    out, lo = [], 0
    for s in range(shards):
        w = 4 * (base + (1 if s < extra else 0))
        out.append((lo, lo + w))
        lo += w
    return out


def conventional_bytes_per_input_word(w: float, n: float, d: int) -> float:
    """Eq. (2): bytes a conventional parameter server moves, in each direction, per minibatch input
    word: the input and output vectors of the word plus the output vectors of its w * n negatives,
    d single-precision numbers each."""
    return (2.0 + w * n) * d * 4.0


def exchange_bytes_per_input_word(w: float, n: float, shards: int) -> float:
    """Eq. (7): bytes of partial dot products (or, in the other direction, of coefficients) per
    minibatch input word summed over the shards: one 4-byte number per target and shard, whatever d."""
    return w * (n + 1.0) * shards * 4.0


def exchange_bytes_per_step(pairs: int, negatives: int) -> int:
    """What ONE shard sends (and receives) in a step of this library: 4 bytes per target, the
    per-shard term of Eq. (6) with b * w = the step's positive pairs."""
    return 4 * int(pairs) * (1 + int(negatives))


def _targets_capacity(n_tokens: int, window: int, negatives: int) -> int:
    return max(1, int(n_tokens) * 2 * int(window) * (1 + int(negatives)))


class LocalShards:
    """S column shards of one model on one GPU (the ranks of the multi-GPU run, one after another)."""

    def __init__(self, vocab, d, seed, shards, device="cuda:0", aligned_rows=False, exchange="p2p"):
        """exchange="p2p": every shard's kernel adds into every shard's array (peer pointers);
        "allreduce": every shard stores its partials in its own array and the arrays are summed
        afterwards, as an all-reduce would (here: a torch sum on the one GPU)."""
        if exchange not in ("p2p", "allreduce"):
            raise ValueError("exchange must be 'p2p' or 'allreduce'")
        self.exchange = exchange
        self.vocab, self.d, self.seed = int(vocab), int(d), int(seed)
        self.columns = shard_columns(d, shards)
        self.device = torch.device(device)
        self.models = []
        for lo, hi in self.columns:
            stride = binding.aligned_row_stride(hi - lo) if aligned_rows else hi - lo
            self.models.append(binding.W2V(vocab, d, seed, device=device, row_stride=stride, columns=(lo, hi)))
        self.F = []          # one array of summed dot products per shard, as on separate GPUs
        self.cap = 0

    def close(self):
        for m in self.models:
            m.close()
        self.models = []

    def build_alias(self, counts, subsample_t):
        for m in self.models:
            m.build_alias(counts, subsample_t)

    def set_step(self, s):
        for m in self.models:
            m.set_step(s)

    def _ensure(self, cap):
        if cap > self.cap:
            self.F = [torch.empty(cap, dtype=torch.float32, device=self.device) for _ in self.models]
            self.cap = cap

    def step(self, tokens, window, negatives, lr):
        """One minibatch on all shards; returns the counters of the step."""
        t = self.models[0]._dev_tokens(tokens)
        n = t.numel()
        self._ensure(_targets_capacity(n, window, negatives))
        st = binding.StepStats()
        if self.exchange == "p2p":
            for f in self.F:
                f.zero_()
            for m in self.models:                               # every shard adds into every shard's array
                binding.w2v_shard_dots(m.h, t, n, window, negatives, self.F, self.cap, st)
            for m, f in zip(self.models, self.F):               # stream order stands in for the barrier
                binding.w2v_shard_adjust(m.h, f, lr)
        else:
            for m, f in zip(self.models, self.F):               # partials into the shard's own array
                binding.w2v_shard_dots(m.h, t, n, window, negatives, [f], self.cap, st)
            targets = st.pairs * (1 + negatives)
            total = self.F[0][:targets]
            for f in self.F[1:]:                                # the all-reduce, on one GPU
                total += f[:targets]
            for m in self.models:
                binding.w2v_shard_adjust(m.h, total, lr)
        return st.as_dict()

    def read_rows(self, which, ids):
        """Whole vectors: the shards' slices side by side."""
        return np.concatenate([m.read_rows(which, ids) for m in self.models], axis=1)

    def write_rows(self, which, ids, rows):
        rows = np.ascontiguousarray(rows, dtype=np.float32).reshape(len(ids), self.d)
        for m, (lo, hi) in zip(self.models, self.columns):
            m.write_rows(which, ids, rows[:, lo:hi])

    def sync(self):
        for m in self.models:
            m.sync()

    def launch_count(self):
        return sum(m.launch_count() for m in self.models)


class DistributedShard:
    """This rank's column shard of a model spread over a torch.distributed group, one rank per GPU.

    Every rank must be given the same vocab, d, seed, histogram, token chunks and step numbers;
    nothing but the dot products crosses between GPUs.
    """

    def __init__(self, vocab, d, seed, device, group=None, exchange="allreduce", aligned_rows=True,
                 max_tokens=1 << 20, window=5, negatives=5, barrier_timeout_ms=5000):
        """barrier_timeout_ms (exchange="p2p"): how long a rank's barrier kernel waits for the other
        ranks before it gives up; the next sync() of that rank then raises, and no GPU hangs on a
        rank that failed."""
        import torch.distributed as dist

        if exchange not in ("allreduce", "p2p"):
            raise ValueError("exchange must be 'allreduce' or 'p2p'")
        self.dist, self.group, self.exchange = dist, group, exchange
        self.rank = dist.get_rank(group)
        self.world = dist.get_world_size(group)
        self.columns = shard_columns(d, self.world)
        lo, hi = self.columns[self.rank]
        stride = binding.aligned_row_stride(hi - lo) if aligned_rows else hi - lo
        self.device = torch.device(device)
        self.model = binding.W2V(vocab, d, seed, device=device, row_stride=stride, columns=(lo, hi))
        self.cap = _targets_capacity(max_tokens, window, negatives)
        self.steps = 0
        if exchange == "allreduce":
            self.F = torch.zeros(self.cap, dtype=torch.float32, device=self.device)
            self.peer_ptrs = None
        else:
            # two arrays per rank in symmetric memory: step k uses array k % 2, so that one device
            # barrier per step orders both "all partials added" and "array of step k-2 zeroed"
            import torch.distributed._symmetric_memory as symm_mem

            # and, behind them, one epoch word per rank for the library's time-limited barrier
            self.barrier_timeout_ms = int(barrier_timeout_ms)
            self.buf = symm_mem.empty(2 * self.cap + binding.MAX_SHARDS, dtype=torch.float32, device=self.device)
            self.buf.zero_()
            self.symm = symm_mem.rendezvous(self.buf, group if group is not None else dist.group.WORLD)
            self.peer_ptrs = [int(p) for p in self.symm.buffer_ptrs]
            self.flag_ptrs = [p + 4 * 2 * self.cap for p in self.peer_ptrs]
            torch.cuda.synchronize(self.device)
            dist.barrier(group)

    def close(self):
        self.model.close()

    def build_alias(self, counts, subsample_t):
        self.model.build_alias(counts, subsample_t)

    def step(self, tokens, window, negatives, lr):
        m = self.model
        t = m._dev_tokens(tokens)
        n = t.numel()
        if _targets_capacity(n, window, negatives) > self.cap:
            raise ValueError("chunk larger than the capacity this shard was created with")
        st = binding.StepStats()
        if self.exchange == "allreduce":
            binding.w2v_shard_dots(m.h, t, n, window, negatives, [self.F], self.cap, st)    # one array: stored
            targets = st.pairs * (1 + negatives)
            if targets:
                self.dist.all_reduce(self.F[:targets], op=self.dist.ReduceOp.SUM, group=self.group)
            binding.w2v_shard_adjust(m.h, self.F, lr)
        else:
            half = (self.steps & 1) * self.cap
            peers = [p + 4 * half for p in self.peer_ptrs]
            binding.w2v_shard_dots(m.h, t, n, window, negatives, peers, self.cap, st)
            # every rank's additions have landed once every rank has announced this step
            binding.w2v_peer_barrier(m.h, self.flag_ptrs, self.rank, self.steps + 1, self.barrier_timeout_ms)
            mine = self.buf[half: half + self.cap]
            binding.w2v_shard_adjust(m.h, mine, lr)
            mine.zero_()                                          # ready for step k + 2
        self.steps += 1
        return st.as_dict()

    def set_step(self, s):
        self.model.set_step(s)

    def set_interleave(self, phase, stride):
        self.model.set_interleave(phase, stride)

    def sync(self):
        """Waits for this rank's stream; raises if one of its barriers gave up waiting for a peer."""
        self.model.sync()

    def read_rows(self, which, ids):
        """This rank's columns of the rows."""
        return self.model.read_rows(which, ids)
