"""Row sharding of one large picture (host logic): the partition covers every row once with the
halo clipped at the picture's border, the halo follows from the network's paddings, strips run
through the ORACLE reproduce the unsplit oracle result bit for bit, and two gloo ranks gather
their owned rows into the whole picture."""
import os
import socket
import subprocess
import sys

import numpy as np
import pytest

from oracle import networks as ON
from paper_2006_11735_b200 import rowshard as RS
from workloads import networks as N

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_halo_is_the_sum_of_the_widest_paddings():
    assert RS.halo_rows(N.vrcnn(n=1, h=32, w=32)) == 6          # 2 (5x5) + 2 (5x5 | 3x3) + 1 (3x3 | 1x1) + 1 (3x3)
    assert RS.halo_rows(N.vdsr(n=1, h=32, w=32)) == 20          # twenty 3x3 layers
    assert RS.halo_rows(N.vdsr(n=1, h=32, w=32, depth=5)) == 5
    with pytest.raises(ValueError):
        RS.halo_rows(N.resnet(1, (1,), h=32, w=32, widths=(16,), classes=8))      # strided layers do not shard by rows


@pytest.mark.parametrize("h,parts,halo", [(1600, 2, 6), (1600, 3, 6), (1080, 8, 20), (17, 4, 20), (5, 8, 2), (64, 1, 6)])
def test_partition_covers_every_row_once_and_clips_the_halo(h, parts, halo):
    strips = RS.partition(h, parts, halo)
    assert len(strips) == parts and strips[0].own0 == 0 and strips[-1].own1 == h
    for a, b in zip(strips[:-1], strips[1:]):
        assert a.own1 == b.own0                                   # contiguous, no gap, no overlap
    sizes = [s.own1 - s.own0 for s in strips]
    assert max(sizes) - min(sizes) <= 1 and sum(sizes) == h
    for s in strips:
        assert s.in0 == max(0, s.own0 - halo) and s.in1 == min(h, s.own1 + halo)
        assert 0 <= s.in0 <= s.own0 <= s.own1 <= s.in1 <= h
        k = s.keep
        assert k.stop - k.start == s.own1 - s.own0 and s.in0 + k.start == s.own0


@pytest.mark.parametrize("parts", [2, 3, 5])
def test_strips_through_the_oracle_equal_the_unsplit_oracle(parts):
    net = N.vrcnn(n=1, h=56, w=40)
    params = ON.calibrate(net)
    x = ON.net_input(net)
    whole = ON.forward(net, params, x)[net.output]
    halo = RS.halo_rows(net)

    def forward(strip):
        small = N.vrcnn(n=1, h=strip.shape[1], w=strip.shape[2])
        return ON.forward(small, params, strip)[small.output]

    got = RS.stitch([RS.run_strip(x, s, forward) for s in RS.partition(56, parts, halo)])
    assert np.array_equal(got, whole)
    # one row less of halo is not enough: some owned row next to a cut changes
    short = RS.stitch([RS.run_strip(x, s, forward) for s in RS.partition(56, parts, halo - 1)])
    assert not np.array_equal(short, whole)


WORKER = r"""
import os, sys
sys.path.insert(0, %r)
import numpy as np
from oracle import networks as ON
from paper_2006_11735_b200 import dist as D, rowshard as RS
from workloads import networks as N
rank, _, size = D.world()
assert D.init("gloo")
net = N.vdsr(n=1, h=40, w=24, depth=4)
params = ON.calibrate(net)
x = ON.net_input(net)
strips = RS.partition(40, size, RS.halo_rows(net))
def forward(strip):
    small = N.vdsr(n=1, h=strip.shape[1], w=strip.shape[2], depth=4)
    return ON.forward(small, params, strip)[small.output]
owned = RS.run_strip(x, strips[rank], forward)
whole = RS.gather_rows(owned, strips, rank)
if rank == 0:
    want = ON.forward(net, params, x)[net.output]
    print("RANK 0 stitched %%s equal %%s" %% (whole.shape, np.array_equal(whole, want)))
else:
    print("RANK %%d owned %%d rows, gathered %%s" %% (rank, owned.shape[1], whole))
D.finish()
"""


def test_two_gloo_ranks_compute_their_strips_and_gather_the_picture():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), CUDA_VISIBLE_DEVICES="")
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER % ROOT], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=300)
        assert p.returncode == 0, err
        outs.append(out.strip().splitlines()[-1])
    got = sorted(outs)
    assert got[0] == "RANK 0 stitched (1, 40, 24, 1) equal True"
    assert got[1] == "RANK 1 owned 20 rows, gathered None"
