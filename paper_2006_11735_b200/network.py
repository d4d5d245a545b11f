"""Sequences the C-ABI calls of a whole network (``workloads.networks.Net``).

PyTorch supplies device memory and the stream; every layer runs in the CUDA library.
Per-layer integer parameters (quantisation step, mul, shift, h_i, skip rescale) arrive as
a dict, e.g. read from ``workloads/params/*.json``; weights are re-created from the
network's seed with the library's own Eq. 1 (``iq_quantize_weights``).
"""
import numpy as np
import torch

from workloads import generators as gen
from workloads.networks import AvgPool, Conv, MaxPool, Net
from workloads.params import load_params  # noqa: F401  (re-exported: callers read cached parameters through here too)

from . import binding as B

_TORCH = {"u8": torch.uint8, "i32": torch.int32}

def net_input(net: Net, first: int = 0, count=None) -> np.ndarray:
    t = net.tensors[net.input]
    count = net.n - first if count is None else count
    if net.input_kind == "uniform":
        return np.ascontiguousarray(gen.uniform_u8(net.seed, (net.n, t.h, t.w, t.c))[first:first + count])
    return gen.image_batch(net.seed, count, t.h, t.w, t.c, first=first)


class Network:
    """Plans every layer once; ``forward`` enqueues the whole network on the current stream."""

    def __init__(self, net: Net, params: dict, n=None, device="cuda:0", kernel=B.KERNEL_AUTO, fuse_projection=True,
                 merge_branches=True, fuse_chain=True):
        """fuse_projection: run a projection skip (a "raw" convolution whose int32 output only feeds
        the next layer's skip) inside that layer's kernel; its int32 tensor is then never written.
        merge_branches: plan two convolutions that read the same tensor and write neighbouring
        channel ranges of the same concatenation (a variable-filter-size block) as one layer: the
        smaller filter sits zero-padded in the middle of the larger one, every channel keeps its
        own bias, h_i, mul and shift.  The sums only gain zero terms, so the bytes are the same.
        fuse_chain: run a block-closing 1x1 layer with an 8-bit identity skip and the 1x1 layer that
        reads its output as ONE kernel where the library takes the pair (``iconv_plan_chain``): the
        wide tensor is still written (later layers read it as their skip) but not read back by the
        next layer, and one launch goes."""
        self.net, self.n, self.device = net, net.n if n is None else n, torch.device(device)
        self.plans, self.steps, self.tensors = {}, [], {}
        self.chains = {}         # name of a closing layer -> chain handle; self.chained: second op name -> closing layer
        self.chained = {}
        self.fused = {}          # name of a fused projection op -> name of the layer that absorbed it
        self.merged = {}         # name of a branch convolution -> name of the sibling whose plan runs both
        self._pending = {}
        torch.cuda.set_device(self.device)
        convs = {op.name: op for op in net.convs()}
        fusable = {}             # skip tensor name -> projection op
        if fuse_projection and kernel in (B.KERNEL_AUTO, B.KERNEL_UMMA):
            for op in net.convs():
                if op.role == "raw" and op.dst != net.output:
                    users = [o for o in net.ops if getattr(o, "src", None) == op.dst or getattr(o, "skip", None) == op.dst]
                    if len(users) == 1 and getattr(users[0], "skip", None) == op.dst and getattr(users[0], "src", None) != op.dst:
                        fusable[op.dst] = op
        for name, t in net.tensors.items():
            self.tensors[name] = torch.zeros((self.n, t.h, t.w, t.c), dtype=_TORCH[t.dtype], device=self.device)
        partner = {}             # first op of a merged pair -> second
        if merge_branches and kernel in (B.KERNEL_AUTO, B.KERNEL_UMMA):
            for a, b in zip(net.ops, net.ops[1:]):
                if a.name not in self.merged and self._mergeable(a, b, params):
                    partner[a.name] = b
                    self.merged[b.name] = a.name
        for op in net.ops:
            src, dst = net.tensors[op.src], net.tensors[op.dst]
            if op.name in self.merged or op.name in self.chained:
                continue
            if op.name in partner:
                self.plans[op.name] = self._plan_merged(op, partner[op.name], params, kernel)
                self.steps.append(("conv", op, None))
                continue
            if isinstance(op, MaxPool):
                self.steps.append(("max", op, None))
            elif isinstance(op, AvgPool):
                self.steps.append(("avg", op, params[op.name]))
            else:
                if op.dst in fusable and self._try_fuse(op, fusable, params, kernel):
                    continue
                p = params[op.name]
                w_f = gen.weights_f(net.seed, op.layer, op.c_out, op.k, op.k, op.c_in)
                kw = dict(n=self.n, h=src.h, w=src.w, c_in=op.c_in, c_out=op.c_out, kh=op.k, kw=op.k,
                          stride=op.stride, pad=op.pad, in_dtype=B.DTYPE_CODE[op.in_dtype], in_c_total=src.c,
                          in_c_offset=op.in_c_offset, out_c_total=dst.c, out_c_offset=op.out_c_offset,
                          weights=B.iq_quantize_weights(w_f, p["delta"]),
                          bias=gen.bias_i32(net.seed, op.layer, op.c_out), kernel=kernel)
                fused = self._pending.pop(op.skip, None) if op.skip else None
                if fused is not None:
                    kw.update(skip_dtype=fused["skip_dtype"], skip_mul=p["skip_mul"], skip_shift=p["skip_shift"],
                              proj=fused["proj"])
                elif op.skip:
                    kw.update(skip_dtype=B.DTYPE_CODE[op.skip_dtype], skip_c_total=net.tensors[op.skip].c,
                              skip_mul=p["skip_mul"], skip_shift=p["skip_shift"])
                if op.role == "raw":
                    kw.update(out_dtype=B.I32, brelu=0)
                else:
                    kw.update(out_dtype=B.U8, brelu=p["brelu"], mul=p["mul"], shift=p["shift"], h_i=p["h_i"],
                              out_lo=p["out_lo"], out_hi=p["out_hi"], out_zero=p["out_zero"])
                if fused is not None:
                    try:
                        self.plans[op.name] = B.iconv_plan(**kw)
                    except B.IconvError as e:
                        if e.status != B.ERR_UNSUPPORTED:
                            raise
                        raise RuntimeError("fused projection refused for %s: %s (build the network with "
                                           "fuse_projection=False)" % (op.name, e))
                    self.fused[fused["op"].name] = op.name
                    self.tensors.pop(fused["op"].dst, None)        # the projection's int32 output is never written
                    self.steps.append(("conv", op, fused["op"].src))
                    continue
                nxt = self._chain_partner(op, kernel) if fuse_chain else None
                if nxt is not None:
                    try:
                        self.chains[op.name] = B.iconv_plan_chain(kw, self._conv_kwargs(nxt, params, kernel))
                        self.chained[nxt.name] = op.name
                        self.steps.append(("chain", op, nxt))
                        continue
                    except B.IconvError as e:
                        if e.status != B.ERR_UNSUPPORTED:
                            raise
                self.plans[op.name] = B.iconv_plan(**kw)
                self.steps.append(("conv", op, None))
        self._alloc_workspace()

    def _chain_partner(self, op, kernel):
        """The layer to run in the same kernel as the closing layer `op`, or None: the next
        operation, a plain 1x1 layer (no skip, 8-bit output) that reads op's whole output."""
        if kernel not in (B.KERNEL_AUTO, B.KERNEL_UMMA) or op.k != 1 or not op.skip or op.skip_dtype != "u8" or op.role != "act":
            return None
        ops = self.net.ops
        i = ops.index(op)
        if i + 1 >= len(ops):
            return None
        nxt = ops[i + 1]
        if not isinstance(nxt, Conv) or nxt.src != op.dst or nxt.k != 1 or nxt.stride != 1 or nxt.skip or nxt.role != "act":
            return None
        if nxt.c_in != op.c_out or nxt.in_c_offset != op.out_c_offset:
            return None
        return nxt

    def _conv_kwargs(self, op, params, kernel) -> dict:
        """iconv_plan's keyword arguments of a plain layer (8-bit output, no skip)."""
        net = self.net
        src, dst = net.tensors[op.src], net.tensors[op.dst]
        p = params[op.name]
        w_f = gen.weights_f(net.seed, op.layer, op.c_out, op.k, op.k, op.c_in)
        return dict(n=self.n, h=src.h, w=src.w, c_in=op.c_in, c_out=op.c_out, kh=op.k, kw=op.k, stride=op.stride, pad=op.pad,
                    in_dtype=B.DTYPE_CODE[op.in_dtype], in_c_total=src.c, in_c_offset=op.in_c_offset, out_c_total=dst.c,
                    out_c_offset=op.out_c_offset, weights=B.iq_quantize_weights(w_f, p["delta"]),
                    bias=gen.bias_i32(net.seed, op.layer, op.c_out), kernel=kernel, out_dtype=B.U8, brelu=p["brelu"],
                    mul=p["mul"], shift=p["shift"], h_i=p["h_i"], out_lo=p["out_lo"], out_hi=p["out_hi"], out_zero=p["out_zero"])

    def _alloc_workspace(self):
        """One buffer of the largest workspace any plan asks for: the layers run one after another
        on one stream, so they can share it."""
        size = max([B.iconv_workspace_bytes(p) for p in self.plans.values()] + [0])
        self.workspace = torch.empty((size,), dtype=torch.uint8, device=self.device) if size else None
        self._ws_ptr = self.workspace.data_ptr() if size else None

    def _mergeable(self, a, b, params) -> bool:
        if not (isinstance(a, Conv) and isinstance(b, Conv)):
            return False
        if a.role == "raw" or b.role == "raw" or a.skip or b.skip or a.dst == self.net.output:
            return False
        same = (a.src == b.src and a.dst == b.dst and a.c_in == b.c_in and a.in_c_offset == b.in_c_offset and
                a.in_dtype == b.in_dtype and a.stride == b.stride and b.out_c_offset == a.out_c_offset + a.c_out)
        if not same or (a.k - b.k) % 2 or a.pad - b.pad != (a.k - b.k) // 2:
            return False
        pa, pb = params[a.name], params[b.name]
        return all(pa[k] == pb[k] for k in ("brelu", "out_lo", "out_hi", "out_zero")) and pa["brelu"] == 1 and \
            len(pa["mul"]) == 1 and len(pb["mul"]) == 1

    def _plan_merged(self, a, b, params, kernel):
        """One plan for the sibling branches a and b (see merge_branches)."""
        net = self.net
        src, dst = net.tensors[a.src], net.tensors[a.dst]
        k = max(a.k, b.k)
        W = np.zeros((a.c_out + b.c_out, k, k, a.c_in), dtype=np.int8)
        row = 0
        for op in (a, b):
            w_f = gen.weights_f(net.seed, op.layer, op.c_out, op.k, op.k, op.c_in)
            o = (k - op.k) // 2
            W[row:row + op.c_out, o:o + op.k, o:o + op.k, :] = B.iq_quantize_weights(w_f, params[op.name]["delta"])
            row += op.c_out
        per = lambda key: np.concatenate([np.repeat(np.asarray(params[op.name][key], dtype=np.int32), op.c_out) for op in (a, b)])
        pa = params[a.name]
        big = a if a.k >= b.k else b
        return B.iconv_plan(n=self.n, h=src.h, w=src.w, c_in=a.c_in, c_out=a.c_out + b.c_out, kh=k, kw=k, stride=a.stride,
                            pad=big.pad, in_dtype=B.DTYPE_CODE[a.in_dtype], in_c_total=src.c, in_c_offset=a.in_c_offset,
                            out_c_total=dst.c, out_c_offset=a.out_c_offset, weights=W,
                            bias=np.concatenate([gen.bias_i32(net.seed, op.layer, op.c_out) for op in (a, b)]),
                            kernel=kernel, out_dtype=B.U8, brelu=1, mul=per("mul"), shift=per("shift"), h_i=per("h_i"),
                            out_lo=pa["out_lo"], out_hi=pa["out_hi"], out_zero=pa["out_zero"])

    def _try_fuse(self, op, fusable, params, kernel) -> bool:
        """Remember a projection op so that its consumer plans it as a fused skip."""
        src = self.net.tensors[op.src]
        if op.in_dtype != "u8" or op.c_in % 16 or src.c % 16 or op.in_c_offset % 16:
            return False
        p = params[op.name]
        w_f = gen.weights_f(self.net.seed, op.layer, op.c_out, op.k, op.k, op.c_in)
        self._pending[op.dst] = dict(op=op, skip_dtype=B.U8, proj=dict(
            weights=B.iq_quantize_weights(w_f, p["delta"]), bias=gen.bias_i32(self.net.seed, op.layer, op.c_out),
            h=src.h, w=src.w, c_total=src.c, c_offset=op.in_c_offset, stride=op.stride, pad=op.pad))
        return True

    def kernels(self) -> dict:
        out = {k: B.KERNEL_NAME[B.iconv_plan_kernel(p)] for k, p in self.plans.items()}
        out.update({k: "umma" for k in self.chains})
        return out

    def describe(self) -> dict:
        out = {k: B.iconv_plan_describe(p) for k, p in self.plans.items()}
        out.update({k: "umma chain: this layer and %s in one kernel" % [b for b, a in self.chained.items() if a == k][0] for k in self.chains})
        return out

    def conv_macs(self) -> dict:
        """True multiply-accumulates per forward of every convolution (M * N * K)."""
        out = {}
        for op in self.net.convs():
            dst = self.net.tensors[op.dst]
            name = self.fused.get(op.name, op.name)          # a fused projection counts with the layer that runs it
            name = self.merged.get(name, name)               # and so does a merged sibling branch
            name = self.chained.get(name, name)              # and the second layer of a two-layer kernel
            out[name] = out.get(name, 0) + self.n * dst.h * dst.w * op.c_out * op.c_in * op.k * op.k
        return out

    def algorithmic_bytes(self) -> dict:
        """Bytes every executed step must move at least once when the network runs layer at a time:
        its input slice, its output slice, its skip operand and its weights (a fused projection
        adds its own input and weights to the layer that runs it and writes nothing)."""
        esz = {"u8": 1, "i32": 4}
        out = {}
        for op in self.net.ops:
            src, dst = self.net.tensors[op.src], self.net.tensors[op.dst]
            if isinstance(op, (MaxPool, AvgPool)):
                out[op.name] = self.n * (src.h * src.w * src.c + dst.h * dst.w * dst.c)
                continue
            b = self.n * src.h * src.w * op.c_in + op.c_out * op.c_in * op.k * op.k + 4 * op.c_out
            if op.name in self.chained:                      # its input never comes back from memory
                name = self.chained[op.name]
                b += self.n * dst.h * dst.w * op.c_out * esz[dst.dtype] - self.n * src.h * src.w * op.c_in
            elif op.name in self.fused:
                name = self.fused[op.name]
            elif op.name in self.merged:                     # shares its sibling's input read
                name = self.merged[op.name]
                b += self.n * dst.h * dst.w * op.c_out * esz[dst.dtype] - self.n * src.h * src.w * op.c_in
            else:
                name = op.name
                b += self.n * dst.h * dst.w * op.c_out * esz[dst.dtype]
                if op.skip and op.skip in self.tensors:
                    sk = self.net.tensors[op.skip]
                    b += self.n * sk.h * sk.w * op.c_out * esz[sk.dtype]
            out[name] = out.get(name, 0) + b
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
            if kind == "chain":
                B.iconv_forward_chain(self.chains[op.name], T[op.src].data_ptr(), T[op.skip].data_ptr(), T[op.dst].data_ptr(),
                                      T[p.dst].data_ptr(), stream)
            elif kind == "conv":
                skip_name = p if p is not None else op.skip       # a fused projection reads its own input
                B.iconv_forward(self.plans[op.name], T[op.src].data_ptr(),
                                T[skip_name].data_ptr() if skip_name else None, T[op.dst].data_ptr(), self._ws_ptr, stream)
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
        for c in self.chains.values():
            B.iconv_chain_destroy(c)
        self.plans, self.chains = {}, {}

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
