"""Network shapes of the five benchmark configurations, as plain data.

A network is a list of operations over named NHWC tensors.  Nothing here computes
anything: the CPU oracle and the CUDA path each interpret the list with their own layer
implementations.  The shapes follow the networks the paper evaluates (Section 4: ResNet
with bottleneck blocks, VDSR's 20 3x3 layers, VRCNN's four layers with two
concatenations) with random-initialised weights.
"""
from dataclasses import dataclass, field
from typing import Dict, List, Optional


@dataclass
class Tensor:
    name: str
    h: int
    w: int
    c: int
    dtype: str          # "u8" | "i32"


@dataclass
class Conv:
    name: str
    layer: int          # index used to seed the layer's weights and bias
    src: str
    dst: str
    c_in: int
    c_out: int
    k: int
    stride: int = 1
    pad: int = 0
    in_dtype: str = "u8"        # "u8" | "u8_raw128" (raw image, 128 subtracted on load)
    in_c_offset: int = 0
    out_c_offset: int = 0
    # "act": BReLU + requantisation to 8 bits; "raw": int32 Y (projection skip, logits);
    # "regression": last layer of VDSR / VRCNN (no BReLU, output ratio reset to the input's)
    role: str = "act"
    skip: Optional[str] = None
    skip_dtype: Optional[str] = None   # "u8" | "i32" | "u8_raw128"
    concat: Optional[str] = None       # name of the concatenation this branch belongs to


@dataclass
class MaxPool:
    name: str
    src: str
    dst: str
    k: int = 3
    stride: int = 2
    pad: int = 1


@dataclass
class AvgPool:
    name: str
    src: str
    dst: str


@dataclass
class Net:
    name: str
    seed: int
    n: int
    input: str
    output: str
    tensors: Dict[str, Tensor] = field(default_factory=dict)
    ops: List[object] = field(default_factory=list)
    max_int: int = 255
    input_ratio: float = 256.0   # raw pixel / 256 after the -128 re-normalisation
    input_kind: str = "smooth"   # "smooth": generators.image_batch; "uniform": generators.uniform_u8
    fixed_h_rf: Optional[float] = None   # a BReLU bound given in float units instead of calibrated

    def add_tensor(self, name, h, w, c, dtype="u8"):
        self.tensors[name] = Tensor(name, h, w, c, dtype)
        return name

    def convs(self):
        return [op for op in self.ops if isinstance(op, Conv)]


def _out(sz, k, s, p):
    return (sz + 2 * p - k) // s + 1


def single_conv(n=1, h=32, w=32, c_in=64, c_out=64, k=3, stride=1, pad=1, seed=1) -> Net:
    """Configuration 1: one 3x3 layer on uniform uint8 activations."""
    net = Net("single_conv", seed, n, "x", "v", input_ratio=255.0 / 6.0, input_kind="uniform",
              fixed_h_rf=6.0)
    net.add_tensor("x", h, w, c_in)
    net.add_tensor("v", _out(h, k, stride, pad), _out(w, k, stride, pad), c_out)
    net.ops.append(Conv("conv", 0, "x", "v", c_in, c_out, k, stride, pad))
    return net


def vdsr(n=16, h=256, w=256, depth=20, width=64, seed=2) -> Net:
    """Configuration 2: VDSR-shaped, depth 3x3 layers, global residual with the input."""
    net = Net("vdsr", seed, n, "x0", "out")
    net.add_tensor("x0", h, w, 1)
    prev, c_prev = "x0", 1
    for i in range(depth - 1):
        t = net.add_tensor("v%d" % (i + 1), h, w, width)
        net.ops.append(Conv("conv%d" % (i + 1), i, prev, t, c_prev, width, 3, 1, 1,
                            in_dtype="u8_raw128" if i == 0 else "u8"))
        prev, c_prev = t, width
    net.add_tensor("out", h, w, 1)
    net.ops.append(Conv("conv%d" % depth, depth - 1, prev, "out", c_prev, 1, 3, 1, 1,
                        role="regression", skip="x0", skip_dtype="u8_raw128"))
    return net


def vrcnn(n=16, h=512, w=512, seed=3) -> Net:
    """Configuration 3: VRCNN-shaped, two concatenation layers, global residual."""
    net = Net("vrcnn", seed, n, "x0", "out")
    net.add_tensor("x0", h, w, 1)
    net.add_tensor("v1", h, w, 64)
    net.add_tensor("v2", h, w, 48)
    net.add_tensor("v3", h, w, 48)
    net.add_tensor("out", h, w, 1)
    net.ops.append(Conv("conv1", 0, "x0", "v1", 1, 64, 5, 1, 2, in_dtype="u8_raw128"))
    net.ops.append(Conv("conv2a", 1, "v1", "v2", 64, 16, 5, 1, 2, out_c_offset=0, concat="cat2"))
    net.ops.append(Conv("conv2b", 2, "v1", "v2", 64, 32, 3, 1, 1, out_c_offset=16, concat="cat2"))
    net.ops.append(Conv("conv3a", 3, "v2", "v3", 48, 16, 3, 1, 1, out_c_offset=0, concat="cat3"))
    net.ops.append(Conv("conv3b", 4, "v2", "v3", 48, 32, 1, 1, 0, out_c_offset=16, concat="cat3"))
    net.ops.append(Conv("conv4", 5, "v3", "out", 48, 1, 3, 1, 1, role="regression",
                        skip="x0", skip_dtype="u8_raw128"))
    return net


def resnet(n, blocks, h=224, w=224, widths=(64, 128, 256, 512), classes=1000, seed=4,
           name="resnet") -> Net:
    """Bottleneck ResNet: 7x7/2 stem, 3x3/2 max-pool, stages of 1x1 -> 3x3 -> 1x1(+skip)
    with the stride on the 3x3, a projection skip in the first block of each stage, global
    average pool and a fully connected layer emitting int32 logits."""
    net = Net(name, seed, n, "x0", "logits")
    net.add_tensor("x0", h, w, 3)
    layer = 0
    hh, ww = _out(h, 7, 2, 3), _out(w, 7, 2, 3)
    net.add_tensor("stem", hh, ww, widths[0])
    net.ops.append(Conv("stem", layer, "x0", "stem", 3, widths[0], 7, 2, 3, in_dtype="u8_raw128"))
    layer += 1
    hh, ww = _out(hh, 3, 2, 1), _out(ww, 3, 2, 1)
    net.add_tensor("pool", hh, ww, widths[0])
    net.ops.append(MaxPool("maxpool", "stem", "pool"))
    prev, c_prev = "pool", widths[0]
    for si, (nb, width) in enumerate(zip(blocks, widths)):
        for b in range(nb):
            s = 2 if (b == 0 and si > 0) else 1
            c_out = width * 4
            tag = "s%db%d" % (si + 1, b)
            h2, w2 = _out(hh, 3, s, 1), _out(ww, 3, s, 1)
            ta = net.add_tensor(tag + "_a", hh, ww, width)
            net.ops.append(Conv(tag + "_1x1a", layer, prev, ta, c_prev, width, 1))
            layer += 1
            tb = net.add_tensor(tag + "_b", h2, w2, width)
            net.ops.append(Conv(tag + "_3x3", layer, ta, tb, width, width, 3, s, 1))
            layer += 1
            if b == 0:
                tp = net.add_tensor(tag + "_p", h2, w2, c_out, "i32")
                net.ops.append(Conv(tag + "_proj", layer, prev, tp, c_prev, c_out, 1, s, 0, role="raw"))
                layer += 1
                skip, skip_dtype = tp, "i32"
            else:
                skip, skip_dtype = prev, "u8"
            tc = net.add_tensor(tag + "_c", h2, w2, c_out)
            net.ops.append(Conv(tag + "_1x1b", layer, tb, tc, width, c_out, 1,
                                skip=skip, skip_dtype=skip_dtype))
            layer += 1
            prev, c_prev, hh, ww = tc, c_out, h2, w2
    net.add_tensor("avg", 1, 1, c_prev)
    net.ops.append(AvgPool("avgpool", prev, "avg"))
    net.add_tensor("logits", 1, 1, classes, "i32")
    net.ops.append(Conv("fc", layer, "avg", "logits", c_prev, classes, 1, role="raw"))
    return net


def resnet_basic(n, blocks, h=224, w=224, widths=(64, 128, 256, 512), classes=1000, seed=6,
                 name="resnet_basic") -> Net:
    """Basic-block ResNet (the paper's Figure 3): 7x7/2 stem, 3x3/2 max-pool, stages of blocks
    of two 3x3 convolutions, the second one closing the block with the skip: the block input
    itself (type 1) or, where the block strides or widens, its 1x1 projection (type 2)."""
    net = Net(name, seed, n, "x0", "logits")
    net.add_tensor("x0", h, w, 3)
    layer = 0
    hh, ww = _out(h, 7, 2, 3), _out(w, 7, 2, 3)
    net.add_tensor("stem", hh, ww, widths[0])
    net.ops.append(Conv("stem", layer, "x0", "stem", 3, widths[0], 7, 2, 3, in_dtype="u8_raw128"))
    layer += 1
    hh, ww = _out(hh, 3, 2, 1), _out(ww, 3, 2, 1)
    net.add_tensor("pool", hh, ww, widths[0])
    net.ops.append(MaxPool("maxpool", "stem", "pool"))
    prev, c_prev = "pool", widths[0]
    for si, (nb, width) in enumerate(zip(blocks, widths)):
        for b in range(nb):
            s = 2 if (b == 0 and si > 0) else 1
            tag = "s%db%d" % (si + 1, b)
            h2, w2 = _out(hh, 3, s, 1), _out(ww, 3, s, 1)
            ta = net.add_tensor(tag + "_a", h2, w2, width)
            net.ops.append(Conv(tag + "_3x3a", layer, prev, ta, c_prev, width, 3, s, 1))
            layer += 1
            if s != 1 or c_prev != width:
                tp = net.add_tensor(tag + "_p", h2, w2, width, "i32")
                net.ops.append(Conv(tag + "_proj", layer, prev, tp, c_prev, width, 1, s, 0, role="raw"))
                layer += 1
                skip, skip_dtype = tp, "i32"
            else:
                skip, skip_dtype = prev, "u8"
            tc = net.add_tensor(tag + "_c", h2, w2, width)
            net.ops.append(Conv(tag + "_3x3b", layer, ta, tc, width, width, 3, 1, 1,
                                skip=skip, skip_dtype=skip_dtype))
            layer += 1
            prev, c_prev, hh, ww = tc, width, h2, w2
    net.add_tensor("avg", 1, 1, c_prev)
    net.ops.append(AvgPool("avgpool", prev, "avg"))
    net.add_tensor("logits", 1, 1, classes, "i32")
    net.ops.append(Conv("fc", layer, "avg", "logits", c_prev, classes, 1, role="raw"))
    return net


def resnet18(n=256, h=224, w=224, seed=6) -> Net:
    """The paper's second classification network (Tables 1 and 2), basic blocks (2, 2, 2, 2)."""
    return resnet_basic(n, (2, 2, 2, 2), h, w, seed=seed, name="resnet18")


def resnet50(n=256, h=224, w=224, seed=4) -> Net:
    """Configuration 4."""
    return resnet(n, (3, 4, 6, 3), h, w, seed=seed, name="resnet50")


def resnet152(n=128, h=224, w=224, seed=5) -> Net:
    """Configuration 5."""
    return resnet(n, (3, 8, 36, 3), h, w, seed=seed, name="resnet152")


def vrcnn_hd(n=1, h=1600, w=2560, seed=3) -> Net:
    """The VRCNN-shaped network on one 2560 x 1600 picture (the size the paper times its
    in-loop filter on, Table 6): the layers, weights and parameters of configuration 3."""
    return vrcnn(n=n, h=h, w=w, seed=seed)


def vdsr_hd(n=1, h=1080, w=1920, seed=2) -> Net:
    """The VDSR-shaped network on one picture-sized input (the paper times VDSR on whole Set-5
    pictures, Table 4; 1920 x 1080 stands in for them): the layers, weights and parameters of
    configuration 2."""
    return vdsr(n=n, h=h, w=w, seed=seed)


def by_name(name: str, **kw) -> Net:
    return {"single_conv": single_conv, "vdsr": vdsr, "vrcnn": vrcnn, "vrcnn_hd": vrcnn_hd, "vdsr_hd": vdsr_hd,
            "resnet18": resnet18, "resnet50": resnet50, "resnet152": resnet152}[name](**kw)
