"""TEST INFRASTRUCTURE -- whole-network runs and parameter calibration on the CPU oracle.

``calibrate`` walks a network (``workloads.networks.Net``) in order on ONE image and
fixes every layer's integer parameters the way the paper does offline:

  * weights by Eq. 1-2 from the seeded float kernels,
  * ratios accumulated along the path (Eq. 3),
  * the BReLU bound h_rf by the 3-sigma rule of Section 3.2.2 (the smallest of the
    largest 0.15 % of the layer's Y on that image), then mul / shift / h_i by Eq. 7-13,
  * residual additions by the ratio synchronisation of Section 4.1 (skip rescaled by
    multiply / shift, quantisation step of the convolution adjusted to match exactly),
  * concatenations by Algorithm 2,
  * the regression output rescaled so that the overall ratio returns to the input's
    (Section 3.1, "reset to 1 by rescaling the output").

``forward`` then runs any batch through the oracle layers with those parameters.
"""
import numpy as np

from workloads import generators as gen
from workloads.networks import AvgPool, Conv, MaxPool, Net

from . import layers as L
from . import planner as P

_NP = {"u8": np.uint8, "i32": np.int32}


def net_input(net: Net, first: int = 0, count=None) -> np.ndarray:
    """The network's seeded raw input, images [first, first + count)."""
    t = net.tensors[net.input]
    count = net.n - first if count is None else count
    if net.input_kind == "uniform":
        full = gen.uniform_u8(net.seed, (net.n, t.h, t.w, t.c))
        return np.ascontiguousarray(full[first:first + count])
    return gen.image_batch(net.seed, count, t.h, t.w, t.c, first=first)


def layer_weights(net: Net, op: Conv, delta: float):
    """int8 kernel and int32 bias of one layer from the seeded float draw and its step."""
    W_f = gen.weights_f(net.seed, op.layer, op.c_out, op.k, op.k, op.c_in)
    return P.quantize_weights(W_f, delta), gen.bias_i32(net.seed, op.layer, op.c_out)


def _run_conv(net, op, p, W, b, tensors, raw_Y=False):
    """Run one Conv op on the oracle.  raw_Y: return the int32 Y (with skip) instead."""
    X = tensors[op.src]
    skip = tensors[op.skip] if op.skip else None
    kw = dict(stride=op.stride, pad=op.pad, in_dtype=L.DTYPE_CODE[op.in_dtype],
              in_c_offset=op.in_c_offset, c_in=op.c_in,
              skip=skip, skip_dtype=L.DTYPE_CODE[op.skip_dtype] if op.skip else -1,
              skip_mul=p.get("skip_mul", 1), skip_shift=p.get("skip_shift", 0))
    if raw_Y or op.role == "raw":
        out, ovf = L.conv(X, W, b, [1], [0], [0], out_dtype=L.I32, brelu=False, **kw)
        if not raw_Y:
            tensors[op.dst] = out
    else:
        dst = tensors[op.dst]
        out, ovf = L.conv(X, W, b, p["mul"], p["shift"], p["h_i"], out_dtype=L.U8, out=dst,
                          out_c_offset=op.out_c_offset, brelu=p["brelu"], out_lo=p["out_lo"],
                          out_hi=p["out_hi"], out_zero=p["out_zero"], **kw)
    if ovf:
        raise OverflowError("layer %s: Y does not fit int32" % op.name)
    return out


def _alloc(net, tensors, name, n):
    if name not in tensors:
        t = net.tensors[name]
        tensors[name] = np.zeros((n, t.h, t.w, t.c), dtype=_NP[t.dtype])


def _three_sigma_bound(Y) -> int:
    """Section 3.2.2: the minimal value among the largest 0.15 % of the feature map."""
    flat = np.sort(Y.reshape(-1))
    k = max(1, int(np.ceil(flat.size * 0.0015)))
    return max(1, int(flat[flat.size - k]))


def calibrate(net: Net, image: int = 0, shift_min: int = 16) -> dict:
    """Per-layer integer parameters from one image.  Returns {op name: parameter dict}."""
    tensors = {net.input: net_input(net, image, 1)}
    ratio = {net.input: net.input_ratio}
    params = {}
    ops = list(net.ops)
    i = 0
    while i < len(ops):
        op = ops[i]
        if isinstance(op, MaxPool):
            tensors[op.dst] = L.maxpool(tensors[op.src], op.k, op.stride, op.pad)
            ratio[op.dst] = ratio[op.src]
            params[op.name] = {}
            i += 1
            continue
        if isinstance(op, AvgPool):
            t = net.tensors[op.src]
            m, s = P.avgpool_mul_shift(t.h * t.w)
            tensors[op.dst] = L.avgpool_requant(tensors[op.src], m, s, net.max_int)
            ratio[op.dst] = ratio[op.src] * m / float(1 << s) * (t.h * t.w)
            params[op.name] = dict(mul=int(m), shift=int(s))
            i += 1
            continue
        group = [op]
        if op.concat:
            while i + len(group) < len(ops) and getattr(ops[i + len(group)], "concat", None) == op.concat:
                group.append(ops[i + len(group)])
        done = []
        for g in group:
            _alloc(net, tensors, g.dst, 1)
            W_f = gen.weights_f(net.seed, g.layer, g.c_out, g.k, g.k, g.c_in)
            b = gen.bias_i32(net.seed, g.layer, g.c_out)
            delta = P.weight_delta(W_f)                                    # Eq. 2
            ratio_X = ratio[g.src]
            ratio_Y = ratio_X / delta                                      # Eq. 3 accumulated
            p = dict(delta=delta, ratio_X=ratio_X, brelu=int(g.role == "act"),
                     out_zero=0, out_lo=0, out_hi=net.max_int)
            if g.skip:
                sy = P.skip_sync(ratio_Y, ratio[g.skip])
                p.update(skip_mul=sy["skip_mul"], skip_shift=sy["skip_shift"])
                delta = delta * sy["delta_scale"]
                ratio_Y = sy["ratio_Y_new"]
                p["delta"] = delta
            p["ratio_Y"] = ratio_Y
            W = P.quantize_weights(W_f, delta)                             # Eq. 1
            if g.role == "raw":
                _run_conv(net, g, p, W, b, tensors)
                ratio[g.dst] = ratio_Y
            elif g.role == "regression":
                m, s = P.mul_shift(net.input_ratio / ratio_Y, shift_min)
                p.update(mul=[m], shift=[s], h_i=[0], out_zero=128, out_lo=0, out_hi=255,
                         ratio_V=ratio_Y * m / float(1 << s))
                _run_conv(net, g, p, W, b, tensors)
                ratio[g.dst] = p["ratio_V"]
            else:
                if net.fixed_h_rf is not None:
                    q = P.brelu_params(net.fixed_h_rf, ratio_Y, net.max_int, shift_min)
                else:
                    Y = _run_conv(net, g, p, W, b, tensors, raw_Y=True)
                    q = P.brelu_params_from_h_ri(_three_sigma_bound(Y), ratio_Y, net.max_int, shift_min)
                p.update(mul=[q["mul"]], shift=[q["shift"]], h_i=[q["h_i"]], h_ri=q["h_ri"],
                         ratio_V=q["ratio_V"], h_f=q["h_f"])
            params[g.name] = p
            done.append((g, W_f, b))
        if op.concat:
            sync = P.concat_sync([params[g.name]["ratio_Y"] for g in group],
                                 [params[g.name]["ratio_V"] for g in group], shift_min)   # Algorithm 2
            for k, (g, W_f, b) in enumerate(done):
                p = params[g.name]
                p["delta"] = p["delta"] * sync["delta_scale"][k]
                p["ratio_Y"] = sync["ratio_Y_new"][k]
                p["mul"], p["shift"] = [sync["mul"][k]], [sync["shift"][k]]
                p["h_i"] = [int(P.round_half_up(P.Fraction(net.max_int * (1 << sync["shift"][k]), sync["mul"][k])))]
                p["ratio_V"] = sync["ratio_V_min"]
        for g, W_f, b in done:
            p = params[g.name]
            if g.role == "act":
                _run_conv(net, g, p, P.quantize_weights(W_f, p["delta"]), b, tensors)
                ratio[g.dst] = p["ratio_V"]
        i += len(group)
    return params


def forward(net: Net, params: dict, x: np.ndarray, weights: dict = None) -> dict:
    """Run a batch through the network on the oracle.  Returns every named tensor."""
    n = x.shape[0]
    tensors = {net.input: np.ascontiguousarray(x)}
    for op in net.ops:
        if isinstance(op, MaxPool):
            tensors[op.dst] = L.maxpool(tensors[op.src], op.k, op.stride, op.pad)
        elif isinstance(op, AvgPool):
            p = params[op.name]
            tensors[op.dst] = L.avgpool_requant(tensors[op.src], p["mul"], p["shift"], net.max_int)
        else:
            p = params[op.name]
            W, b = weights[op.name] if weights else layer_weights(net, op, p["delta"])
            _alloc(net, tensors, op.dst, n)
            _run_conv(net, op, p, W, b, tensors)
    return tensors
