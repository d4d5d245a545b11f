"""Sequences the C-ABI calls of a whole network (``workloads.networks.Net``).

PyTorch supplies device memory and the stream; every layer runs in the CUDA library.
Per-layer integer parameters (quantisation step, mul, shift, h_i, skip rescale) arrive as
a dict, e.g. read from ``workloads/params/*.json``; weights are re-created from the
network's seed with the library's own Eq. 1 (``iq_quantize_weights``).
"""
import json
import os

import numpy as np
import torch

from workloads import generators as gen
from workloads.networks import AvgPool, Conv, MaxPool, Net

from . import binding as B

_TORCH = {"u8": torch.uint8, "i32": torch.int32}
PARAMS_DIR = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "workloads", "params")


def load_params(name: str) -> dict:
    """Cached per-layer parameters of a full-size configuration (``float.hex`` strings for
    doubles so that the quantisation steps round-trip exactly)."""
    with open(os.path.join(PARAMS_DIR, name + ".json")) as f:
        raw = json.load(f)
    for p in raw["layers"].values():
        if "delta" in p:
            p["delta"] = float.fromhex(p["delta"])
    return raw["layers"]


def net_input(net: Net, first: int = 0, count=None) -> np.ndarray:
    t = net.tensors[net.input]
    count = net.n - first if count is None else count
    if net.input_kind == "uniform":
        return np.ascontiguousarray(gen.uniform_u8(net.seed, (net.n, t.h, t.w, t.c))[first:first + count])
    return gen.image_batch(net.seed, count, t.h, t.w, t.c, first=first)


class Network:
    """Plans every layer once; ``forward`` enqueues the whole network on the current stream."""

    def __init__(self, net: Net, params: dict, n=None, device="cuda:0", kernel=B.KERNEL_AUTO):
        self.net, self.n, self.device = net, net.n if n is None else n, torch.device(device)
        self.plans, self.steps, self.tensors = {}, [], {}
        torch.cuda.set_device(self.device)
        for name, t in net.tensors.items():
            self.tensors[name] = torch.zeros((self.n, t.h, t.w, t.c), dtype=_TORCH[t.dtype], device=self.device)
        for op in net.ops:
            src, dst = net.tensors[op.src], net.tensors[op.dst]
            if isinstance(op, MaxPool):
                self.steps.append(("max", op, None))
            elif isinstance(op, AvgPool):
                self.steps.append(("avg", op, params[op.name]))
            else:
                p = params[op.name]
                w_f = gen.weights_f(net.seed, op.layer, op.c_out, op.k, op.k, op.c_in)
                kw = dict(n=self.n, h=src.h, w=src.w, c_in=op.c_in, c_out=op.c_out, kh=op.k, kw=op.k,
                          stride=op.stride, pad=op.pad, in_dtype=B.DTYPE_CODE[op.in_dtype], in_c_total=src.c,
                          in_c_offset=op.in_c_offset, out_c_total=dst.c, out_c_offset=op.out_c_offset,
                          weights=B.iq_quantize_weights(w_f, p["delta"]),
                          bias=gen.bias_i32(net.seed, op.layer, op.c_out), kernel=kernel)
                if op.skip:
                    kw.update(skip_dtype=B.DTYPE_CODE[op.skip_dtype], skip_c_total=net.tensors[op.skip].c,
                              skip_mul=p["skip_mul"], skip_shift=p["skip_shift"])
                if op.role == "raw":
                    kw.update(out_dtype=B.I32, brelu=0)
                else:
                    kw.update(out_dtype=B.U8, brelu=p["brelu"], mul=p["mul"], shift=p["shift"], h_i=p["h_i"],
                              out_lo=p["out_lo"], out_hi=p["out_hi"], out_zero=p["out_zero"])
                self.plans[op.name] = B.iconv_plan(**kw)
                self.steps.append(("conv", op, None))

    def kernels(self) -> dict:
        return {k: B.KERNEL_NAME[B.iconv_plan_kernel(p)] for k, p in self.plans.items()}

    def conv_macs(self) -> dict:
        """True multiply-accumulates per forward of every convolution (M * N * K)."""
        out = {}
        for op in self.net.convs():
            dst = self.net.tensors[op.dst]
            out[op.name] = self.n * dst.h * dst.w * op.c_out * op.c_in * op.k * op.k
        return out

    def forward(self, x: torch.Tensor = None, marks: list = None) -> torch.Tensor:
        """x: uint8 device tensor [n][h][w][c] (or None to reuse the resident input).
        marks: if a list, receives (op name, event recorded after that op's launch); the
        first entry (None, event) marks the start."""
        ts = torch.cuda.current_stream(self.device)
        stream = ts.cuda_stream
        T = self.tensors
        if x is not None:
            T[self.net.input] = x
        if marks is not None:
            ev = torch.cuda.Event(enable_timing=True)
            ev.record(ts)
            marks.append((None, ev))
        for kind, op, p in self.steps:
            src = self.net.tensors[op.src]
            if kind == "conv":
                B.iconv_forward(self.plans[op.name], T[op.src].data_ptr(),
                                T[op.skip].data_ptr() if op.skip else None, T[op.dst].data_ptr(), stream)
            elif kind == "max":
                B.ipool_max(T[op.src].data_ptr(), T[op.dst].data_ptr(), self.n, src.h, src.w, src.c,
                            op.k, op.stride, op.pad, stream)
            else:
                B.ipool_avg_requant(T[op.src].data_ptr(), T[op.dst].data_ptr(), self.n, src.h, src.w, src.c,
                                    p["mul"], p["shift"], self.net.max_int, stream)
            if marks is not None:
                ev = torch.cuda.Event(enable_timing=True)
                ev.record(ts)
                marks.append((op.name, ev))
        return T[self.net.output]

    def close(self):
        for p in self.plans.values():
            B.iconv_plan_destroy(p)
        self.plans = {}

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
