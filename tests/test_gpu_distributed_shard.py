"""DistributedShard through a real torch.distributed group on the one GPU there is: a world of one
rank holds all columns, so the step must equal the checker's snapshot step, and the exchange code
(the NCCL all-reduce, or the symmetric-memory arrays with the device barrier) is executed for real.
More than one rank needs more than one GPU and is not run here."""
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
