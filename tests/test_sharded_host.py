"""Host side of the multi-GPU paths, on CPU with two gloo ranks.

The kernels need a GPU; what runs here is the plan around them: which columns a rank owns, that
the all-reduce of the ranks' partial dot products (computed by the CPU checker on each rank's own
slice) gives the full dot products of Algorithm 3, and the benchmark's reduction over ranks.
"""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_1606_08495_b200.sharded import (conventional_bytes_per_input_word, exchange_bytes_per_input_word,
                                           exchange_bytes_per_step, shard_columns)


@pytest.mark.parametrize("d,shards", [(300, 1), (300, 2), (300, 8), (300, 10), (300, 75), (8, 2), (1024, 16)])
def test_shard_columns_partition(d, shards):
    cols = shard_columns(d, shards)
    assert len(cols) == shards and cols[0][0] == 0 and cols[-1][1] == d
    widths = []
    for (lo, hi), nxt in zip(cols, cols[1:] + [(d, d)]):
        assert lo % 4 == 0 and hi % 4 == 0 and lo < hi and hi == nxt[0]
        widths.append(hi - lo)
    assert max(widths) - min(widths) <= 4


def test_shard_columns_rejects_impossible_splits():
    for d, s in [(300, 0), (300, 76), (10, 2), (0, 1)]:
        with pytest.raises(ValueError):
            shard_columns(d, s)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from oracle import Oracle
        import bench

        V, d = 400, 100
        cpu = Oracle(V, d, seed=9)
        rng = np.random.default_rng(1)                        # same inputs on every rank
        Vt = rng.normal(scale=0.3, size=(V, d)).astype(np.float32)
        cpu.write_rows(1, np.arange(V), Vt)
        pairs = rng.integers(0, V, size=(2000, 2)).astype(np.int32)
        lo, hi = shard_columns(d, world)[rank]
        part = torch.from_numpy(cpu.partial_dots(pairs, lo, hi))
        dist.all_reduce(part, op=dist.ReduceOp.SUM)
        full = cpu.partial_dots(pairs, 0, d)
        ok_dots = bool(np.allclose(part.numpy(), full, rtol=0, atol=1e-12))
        # the benchmark's reduction: slowest rank's time, work summed over ranks
        ms, e2e_ms, pairs_sum, e2e_sum, launches = bench.reduce_over_ranks(
            10.0 + rank, 20.0 - rank, 1000.0 * (rank + 1), 500.0, 7, world, torch.device("cpu"))
        ok_red = (ms, e2e_ms, pairs_sum, e2e_sum, launches) == (10.0 + world - 1, 20.0, 1000.0 * world * (world + 1) / 2,
                                                              500.0 * world, 7 * world)
        with open(os.path.join(out_dir, f"rank{rank}.txt"), "w") as f:
            f.write(f"{int(ok_dots)} {int(ok_red)}\n")
    finally:
        dist.destroy_process_group()


def test_two_ranks_sum_their_slices_and_reduce_the_timing(tmp_path):
    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    for r in range(world):
        assert open(tmp_path / f"rank{r}.txt").read().split() == ["1", "1"]


def test_network_bytes_of_the_paper():
    # Section 4 works Eq. (2) for w = 10, n = 10, d = 500: about 200,000 bytes per word and direction, and
    # from it, for 10 passes over 5e10 words in a week, at least 1300 Gbit/s
    r = conventional_bytes_per_input_word(10, 10, 500)
    assert r == 204_000 and abs(r - 200_000) / 200_000 < 0.03
    gbits = 10 * 5e10 * 2e5 * 8 / (7 * 24 * 60 * 60 * 1e9)
    assert 1300 <= gbits < 1330
    # Section 5.2: the shards' partial dot products take S in the place of d, so the ratio is about S / d
    for S, d in [(10, 300), (15, 300), (20, 1000), (25, 1000)]:
        ratio = exchange_bytes_per_input_word(10, 10, S) / conventional_bytes_per_input_word(10, 10, d)
        assert abs(ratio / (S / d) - 1) < 0.1
        assert 1 / 100 - 1e-9 <= S / d <= 1 / 15
    # Section 6.2: at 1.6e6 input words/s with about 20 targets per word on 15 shards the scheme needs a few
    # Gbit/s of dot products each way where a conventional server would need ~300 Gbit/s for d = 300
    words = 1.6e6
    conventional = words * 21 * 300 * 4 * 8 / 1e9            # 21 vectors of 300 floats per input word
    assert 300 <= conventional <= 340
    ours = words * 20 * 15 * 4 * 8 / 1e9
    assert ours < 20
    # this library's exchange: one float per target per shard and direction
    assert exchange_bytes_per_step(4_541_742, 10) == 4 * 4_541_742 * 11 == 199_836_648
    b, w, n, S = 1000, 6, 5, 8
    assert exchange_bytes_per_step(b * w, n) * S == b * exchange_bytes_per_input_word(w, n, S)
