"""GPU parity at the full sizes of the benchmark configurations, in the launch configuration
``bench.py`` times (same plans, same batch, kernel family chosen by the plan).

Images are independent units through every layer, so the oracle's forward of ONE image is the
exact expectation for that image's slice of every tensor of the full-batch GPU run.  Persistent
CTAs walk the 128-pixel tiles round-robin, so the images are picked from the tile schedule: the
first and the last of the batch, the middle one, and two that sit where the last, partial wave
of tiles begins in the deep stages (e.g. ResNet-50 at batch 256, stage 4: 196 tiles on 148 SMs,
the partial wave starts inside image 193; ResNet-152 at batch 128, stage 3: inside image 120).
Every layer of each is checked bit for bit.  Parameters are the
cached ones of ``workloads/params`` (written by the oracle's calibration)."""
import numpy as np
import pytest
import torch

from oracle import networks as ON
from paper_2006_11735_b200 import binding as B
from paper_2006_11735_b200.network import Network, load_params, net_input
from workloads import networks as N

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["vdsr", "vrcnn", "resnet18", "resnet50", "resnet152"])
def test_full_size_configuration_matches_oracle_on_sampled_images(name):
    net = N.by_name(name)
    params = load_params(name)
    g = Network(net, params)
    x = net_input(net)
    out = g.forward(torch.from_numpy(x).cuda())
    B.iconv_check(torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    for img in sorted({0, net.n // 2, (3 * net.n) // 4 + 1, (15 * net.n) // 16, net.n - 1}):
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


def test_single_2560x1600_picture_matches_oracle_on_crops():
    """The VRCNN-shaped network on one 2560 x 1600 picture (the size of Table 6's timing).  The
    oracle runs crops of the picture; away from a crop's artificial edges by the network's
    receptive-field radius (2 + 2 + 1 + 1 = 6 pixels) every layer of the crop equals the same
    region of the full picture, and a crop that touches the picture's border shares its padding."""
    net = N.by_name("vrcnn_hd")
    params = load_params("vrcnn_hd")
    g = Network(net, params)
    assert len(g.merged) == 2
    x = net_input(net)
    H, W = x.shape[1], x.shape[2]
    assert (H, W) == (1600, 2560)
    out = g.forward(torch.from_numpy(x).cuda())
    B.iconv_check(torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    ch, cw, r = 160, 192, 6
    # (top, left) of the crop and the slice of the crop that is exact
    crops = [(0, 0, slice(0, ch - r), slice(0, cw - r)),                           # top-left corner: real padding on two sides
             (H - ch, W - cw, slice(r, ch), slice(r, cw)),                         # bottom-right corner
             (0, 1111, slice(0, ch - r), slice(r, cw - r)),                        # top edge
             (733, 1283, slice(r, ch - r), slice(r, cw - r))]                      # interior, odd offsets
    small = N.vrcnn(n=1, h=ch, w=cw)
    for top, left, ys, xs in crops:
        want = ON.forward(small, params, np.ascontiguousarray(x[:, top:top + ch, left:left + cw, :]))
        for op in net.ops:
            got = g.tensors[op.dst][:, top:top + ch, left:left + cw, :].cpu().numpy()
            a, b = got[:, ys, xs, :], want[op.dst][:, ys, xs, :]
            assert np.array_equal(a, b), "crop (%d, %d) layer %s: %d mismatches" % (top, left, op.name, (a != b).sum())
        assert np.unique(want[net.output]).size > 16
    assert out.shape == (1, H, W, 1)
    g.close()
    del g
    torch.cuda.empty_cache()


def test_single_1920x1080_picture_through_the_vdsr_stack_matches_oracle_on_crops():
    """The VDSR-shaped network on one picture-sized input (Table 4 times VDSR on whole pictures).
    Receptive-field radius: twenty 3x3 layers = 20 pixels."""
    net = N.by_name("vdsr_hd")
    params = load_params("vdsr_hd")
    g = Network(net, params)
    x = net_input(net)
    H, W = x.shape[1], x.shape[2]
    assert (H, W) == (1080, 1920)
    out = g.forward(torch.from_numpy(x).cuda())
    B.iconv_check(torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    ch, cw, r = 112, 128, 20
    crops = [(0, 0, slice(0, ch - r), slice(0, cw - r)),
             (H - ch, W - cw, slice(r, ch), slice(r, cw)),
             (517, 0, slice(r, ch - r), slice(0, cw - r)),                         # left edge
             (301, 1001, slice(r, ch - r), slice(r, cw - r))]
    small = N.vdsr(n=1, h=ch, w=cw)
    for top, left, ys, xs in crops:
        want = ON.forward(small, params, np.ascontiguousarray(x[:, top:top + ch, left:left + cw, :]))
        for op in (net.ops[0], net.ops[9], net.ops[-1]):
            got = g.tensors[op.dst][:, top:top + ch, left:left + cw, :].cpu().numpy()
            a, b = got[:, ys, xs, :], want[op.dst][:, ys, xs, :]
            assert np.array_equal(a, b), "crop (%d, %d) layer %s: %d mismatches" % (top, left, op.name, (a != b).sum())
        assert np.unique(want[net.output]).size > 16
    assert out.shape == (1, H, W, 1)
    g.close()
    del g
    torch.cuda.empty_cache()


@pytest.mark.parametrize("name,parts", [("vrcnn_hd", 2), ("vrcnn_hd", 3), ("vdsr_hd", 2), ("vdsr_hd", 3)])
def test_row_sharded_picture_equals_the_unsplit_one(name, parts):
    """The strips of a 2- and a 3-way row split, each run through the CUDA library as the rank that
    owns it would (here one after another on one GPU), stitched: bit-identical to the unsplit GPU
    forward, which the tests above tie to the oracle."""
    from paper_2006_11735_b200 import rowshard as RS
    net = N.by_name(name)
    params = load_params(name)
    x = net_input(net)
    g = Network(net, params)
    whole = g.forward(torch.from_numpy(x).cuda()).cpu().numpy()
    B.iconv_check(torch.cuda.current_stream().cuda_stream)
    g.close()
    del g
    torch.cuda.empty_cache()
    halo = RS.halo_rows(net)
    assert halo == (6 if name == "vrcnn_hd" else 20)

    def forward(strip):
        sn = N.by_name(name, h=strip.shape[1], w=strip.shape[2])
        gs = Network(sn, params)
        out = gs.forward(torch.from_numpy(strip).cuda()).cpu().numpy()
        B.iconv_check(torch.cuda.current_stream().cuda_stream)
        gs.close()
        return out

    strips = RS.partition(x.shape[1], parts, halo)
    got = RS.stitch([RS.run_strip(x, s, forward) for s in strips])
    assert got.shape == whole.shape
    bad = np.argwhere(got != whole)
    assert bad.shape[0] == 0, "%d mismatches, first at %s" % (bad.shape[0], bad[:1])
    assert sum(s.rows for s in strips) == x.shape[1] + 2 * halo * (parts - 1)      # the redundant halo rows
    torch.cuda.empty_cache()
