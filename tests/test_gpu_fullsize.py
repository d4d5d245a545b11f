"""GPU parity at the full sizes of the benchmark configurations, in the launch configuration
``bench.py`` times (same plans, same batch, kernel family chosen by the plan).

Images are independent units through every layer, so the oracle's forward of ONE image is the
exact expectation for that image's slice of every tensor of the full-batch GPU run: the first
and the last image of each batch are checked, every layer, bit for bit.  Parameters are the
cached ones of ``workloads/params`` (written by the oracle's calibration)."""
import numpy as np
import pytest
import torch

from oracle import networks as ON
from paper_2006_11735_b200 import binding as B
from paper_2006_11735_b200.network import Network, load_params, net_input
from workloads import networks as N

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["vdsr", "vrcnn", "resnet50", "resnet152"])
def test_full_size_configuration_matches_oracle_on_sampled_images(name):
    net = N.by_name(name)
    params = load_params(name)
    g = Network(net, params)
    x = net_input(net)
    out = g.forward(torch.from_numpy(x).cuda())
    B.iconv_check(torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    for img in (0, net.n - 1):
        want = ON.forward(net, params, x[img:img + 1])
        for op in net.ops:
            if op.name in g.fused:        # a fused projection's int32 tensor is never written
                continue
            got = g.tensors[op.dst][img:img + 1].cpu().numpy()
            assert np.array_equal(got, want[op.dst]), "%s image %d layer %s: %d mismatches" % (
                name, img, op.name, (got != want[op.dst]).sum())
        assert np.array_equal(out[img:img + 1].cpu().numpy(), want[net.output])
        zeros = (want[net.output] == 0).mean()
        assert zeros < 0.95
    g.close()
    del g
    torch.cuda.empty_cache()
