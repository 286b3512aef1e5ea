"""The time-limited barrier of the peer-to-peer exchange (w2v_peer_barrier), on one GPU.

Kernels of different ranks must never wait for one another on one GPU, so the other rank is played
by the host: its epoch word is either written before the launch (it "arrived first") or never
written (it failed before its launch).  In the second case the wait has to run out, the kernel has
to return, w2v_sync has to report it once, and the device has to stay usable: nothing traps."""
import time

import numpy as np
import pytest
import torch

from paper_1606_08495_b200 import binding

pytestmark = pytest.mark.gpu


@pytest.fixture()
def shard():
    m = binding.W2V(64, 8, seed=1, columns=(0, 4))
    yield m
    m.close()


def _flags(n):
    return [torch.zeros(binding.MAX_SHARDS, dtype=torch.int32, device="cuda") for _ in range(n)]


def test_single_shard_passes_at_once(shard):
    f = _flags(1)
    for epoch in (1, 2, 3):
        binding.w2v_peer_barrier(shard.h, f, 0, epoch, 1000)
        shard.sync()
        assert int(f[0][0]) == epoch


def test_peer_that_arrived_first_lets_the_barrier_pass(shard):
    f = _flags(2)
    f[0][1] = 5                      # rank 1 announced epoch 5 in rank 0's array already
    torch.cuda.synchronize()
    t0 = time.time()
    binding.w2v_peer_barrier(shard.h, f, 0, 5, 2000)
    shard.sync()                     # no error
    assert time.time() - t0 < 1.0
    assert f[0].tolist()[:2] == [5, 5] and f[1].tolist()[:2] == [5, 0]     # announced to itself and to rank 1
    f[0][1] = 9                      # a peer that is already steps ahead does not hold anyone up either
    torch.cuda.synchronize()
    binding.w2v_peer_barrier(shard.h, f, 0, 6, 2000)
    shard.sync()


def test_peer_that_never_arrives_times_out_without_a_fault(shard):
    f = _flags(2)
    t0 = time.time()
    binding.w2v_peer_barrier(shard.h, f, 0, 1, 300)
    with pytest.raises(binding.W2VError) as exc:
        shard.sync()
    waited = time.time() - t0
    assert exc.value.code == binding.W2V_ERR_CUDA and "barrier" in str(exc.value)
    assert 0.25 <= waited < 5.0, waited
    assert f[1].tolist()[0] == 1     # this rank did announce itself
    shard.sync()                     # reported once; the flag is cleared and the stream goes on
    ids = np.arange(4)
    assert shard.read_rows(0, ids).shape == (4, 4)
    x = torch.arange(10, device="cuda").sum().item()
    assert x == 45


def test_bad_arguments_are_refused(shard):
    f = _flags(2)
    for args in [(f, 2, 1, 100), (f, 0, 1, 0), (f, 0, 1, 700000), ([], 0, 1, 100)]:
        with pytest.raises(binding.W2VError) as exc:
            binding.w2v_peer_barrier(shard.h, *args)
        assert exc.value.code == binding.W2V_ERR_ARG
