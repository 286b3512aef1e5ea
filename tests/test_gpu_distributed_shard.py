"""DistributedShard through real torch.distributed groups on the one GPU there is.

One rank (NCCL): a world of one rank holds all columns, so the step must equal the checker's
snapshot step, and the exchange code (the NCCL all-reduce, or the symmetric-memory arrays with the
library's barrier) is executed for real.

Two ranks (gloo, both processes on the same GPU, exchange="allreduce"): each rank holds half of the
columns, the partial dot products are summed by a real all-reduce between the processes, and the
halves put side by side must equal the checker's snapshot step.  No kernel of one rank waits for
the other here (the collective runs on the host), so the two processes may share the GPU.  The
peer-to-peer exchange with two or more ranks needs a GPU per rank and is not run."""
import os
import socket
import subprocess
import sys
import textwrap

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = textwrap.dedent("""
    import os, sys
    import numpy as np
    import torch
    import torch.distributed as dist
    sys.path.insert(0, os.environ["W2V_ROOT"]); sys.path.insert(0, os.path.join(os.environ["W2V_ROOT"], "tests"))
    from oracle import Oracle
    from paper_1606_08495_b200 import corpus
    from paper_1606_08495_b200.sharded import DistributedShard
    from gpu_common import row_rel_err

    exchange = sys.argv[1]
    torch.cuda.set_device(0)
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", 0))
    cfg = corpus.scaled(corpus.CONFIGS["tiny"], vocab=3000, d=100, minibatch=2000, corpus_tokens=100_000)
    cp = corpus.Corpus(cfg)
    try:
        shard = DistributedShard(cfg["vocab"], cfg["d"], 11, "cuda:0", exchange=exchange, max_tokens=4096,
                                 window=cfg["window"], negatives=cfg["negatives"])
    except Exception as exc:                       # symmetric memory may be unavailable for a single rank
        print("UNAVAILABLE", type(exc).__name__, exc)
        dist.destroy_process_group()
        sys.exit(0)
    cpu = Oracle(cfg["vocab"], cfg["d"], 11)
    shard.build_alias(cp.counts, cfg["subsample_t"]); cpu.build_tables(cp.counts, cfg["subsample_t"])
    for i in range(3):
        st = shard.step(cp.chunk(i), cfg["window"], cfg["negatives"], cfg["lr"])
        so = cpu.step(cp.chunk(i), cfg["window"], cfg["negatives"], cfg["lr"], 0)
        assert st["pairs"] == so["pairs"]
    ids = np.arange(cfg["vocab"])
    eu = row_rel_err(shard.read_rows(0, ids), cpu.read_rows(0, ids))
    ev = row_rel_err(shard.read_rows(1, ids), cpu.read_rows(1, ids))
    torch.cuda.synchronize()
    shard.close()
    dist.destroy_process_group()
    assert eu <= 1e-5 and ev <= 1e-5, (eu, ev)
    print("OK", eu, ev)
""")


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


@pytest.mark.parametrize("exchange", ["allreduce", "p2p"])
def test_single_rank_group_runs_the_exchange_code(exchange, tmp_path):
    script = tmp_path / "child.py"
    script.write_text(CHILD)
    env = dict(os.environ, W2V_ROOT=ROOT, MASTER_ADDR="127.0.0.1", MASTER_PORT=str(_free_port()),
               NCCL_NVLS_ENABLE="0")
    out = subprocess.run([sys.executable, str(script), exchange], env=env, capture_output=True, text=True, timeout=600)
    print(out.stdout[-2000:], out.stderr[-2000:])
    assert out.returncode == 0, out.stderr[-3000:]
    if "UNAVAILABLE" in out.stdout:
        pytest.skip("symmetric memory not available for a one-rank group: " + out.stdout.strip()[:300])
    assert "OK" in out.stdout


TWO_RANKS = textwrap.dedent("""
    import os, sys
    import numpy as np
    import torch
    import torch.distributed as dist
    sys.path.insert(0, os.environ["W2V_ROOT"]); sys.path.insert(0, os.path.join(os.environ["W2V_ROOT"], "tests"))
    from oracle import Oracle
    from paper_1606_08495_b200 import corpus
    from paper_1606_08495_b200.sharded import DistributedShard, shard_columns
    from gpu_common import row_rel_err

    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    torch.cuda.set_device(0)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = corpus.scaled(corpus.CONFIGS["tiny"], vocab=3000, d=100, minibatch=2000, corpus_tokens=100_000)
    cp = corpus.Corpus(cfg)
    W, N, lr = cfg["window"], cfg["negatives"], cfg["lr"]
    shard = DistributedShard(cfg["vocab"], cfg["d"], 11, "cuda:0", exchange="allreduce", max_tokens=4096,
                             window=W, negatives=N)
    assert shard.columns == shard_columns(cfg["d"], world) and shard.world == world
    lo, hi = shard.columns[rank]
    assert shard.model.d == hi - lo
    shard.build_alias(cp.counts, cfg["subsample_t"])
    cpu = Oracle(cfg["vocab"], cfg["d"], 11)
    cpu.build_tables(cp.counts, cfg["subsample_t"])
    for i in range(3):
        st = shard.step(cp.chunk(i), W, N, lr)
        so = cpu.step(cp.chunk(i), W, N, lr, 0)
        assert st["pairs"] == so["pairs"]
    # one chunk as two interleaved minibatches with the same step number
    for phase in range(2):
        shard.set_step(3); shard.set_interleave(phase, 2)
        cpu.set_step(3); cpu.set_interleave(phase, 2)
        st = shard.step(cp.chunk(3), W, N, lr)
        so = cpu.step(cp.chunk(3), W, N, lr, 0)
        assert st["pairs"] == so["pairs"] and st["centres"] == so["centres"]
    shard.sync()
    ids = np.arange(cfg["vocab"])
    parts = [None] * world
    dist.all_gather_object(parts, (shard.read_rows(0, ids), shard.read_rows(1, ids)))
    shard.close()
    dist.destroy_process_group()
    if rank == 0:
        U = np.concatenate([p[0] for p in parts], axis=1)
        V = np.concatenate([p[1] for p in parts], axis=1)
        assert U.shape == (cfg["vocab"], cfg["d"])
        eu, ev = row_rel_err(U, cpu.read_rows(0, ids)), row_rel_err(V, cpu.read_rows(1, ids))
        assert eu <= 1e-5 and ev <= 1e-5, (eu, ev)
        # each half alone is NOT the answer: the halves really came from different ranks
        assert np.abs(parts[0][1]).max() > 0 and np.abs(parts[1][1]).max() > 0
        print("OK", eu, ev)
""")


def test_two_ranks_hold_half_of_the_columns_each(tmp_path):
    script = tmp_path / "child2.py"
    script.write_text(TWO_RANKS)
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, W2V_ROOT=ROOT, MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                   WORLD_SIZE="2")
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        try:
            outs.append(p.communicate(timeout=600))
        except subprocess.TimeoutExpired:
            for q in procs:
                q.kill()
            raise
    for rank, (p, (so, se)) in enumerate(zip(procs, outs)):
        print(rank, so[-2000:], se[-2000:])
        assert p.returncode == 0, se[-3000:]
    assert "OK" in outs[0][0]
