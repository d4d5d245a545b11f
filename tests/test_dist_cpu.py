"""World-size-2 CPU (gloo) run of the rank plumbing the benchmark uses at N > 1: rendezvous
from the environment, batch sharding without overlap or gap, max- and sum-over-ranks."""
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys
sys.path.insert(0, %r)
from paper_2006_11735_b200 import dist as D
rank, local_rank, size = D.world()
assert D.init("gloo")
first, count = D.shard(257, rank, size)
total = D.sum_over_ranks(count)
slow = D.max_over_ranks(10.0 + rank)
firsts = D.sum_over_ranks(first)
D.barrier()
print("RANK %%d first %%d count %%d total %%d max %%.1f firsts %%d" %% (rank, first, count, int(total), slow, int(firsts)))
D.finish()
"""


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def test_two_gloo_ranks_shard_and_reduce():
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), CUDA_VISIBLE_DEVICES="")
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER % ROOT], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=180)
        assert p.returncode == 0, err
        outs.append(out.strip().splitlines()[-1])
    got = sorted(outs)
    assert got[0] == "RANK 0 first 0 count 129 total 257 max 11.0 firsts 129"
    assert got[1] == "RANK 1 first 129 count 128 total 257 max 11.0 firsts 129"


def test_shard_covers_every_unit_once():
    from paper_2006_11735_b200 import dist as D
    for n in (0, 1, 7, 256, 1000):
        for size in (1, 2, 3, 8):
            spans = [D.shard(n, r, size) for r in range(size)]
            assert spans[0][0] == 0 and sum(c for _, c in spans) == n
            for (f0, c0), (f1, _) in zip(spans[:-1], spans[1:]):
                assert f0 + c0 == f1
