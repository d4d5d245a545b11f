"""ctypes binding of ``libiconv_b200.so``: the same names as ``include/iconv.h``, argument
marshalling only.  Tensors are passed as raw device addresses (``torch.Tensor.data_ptr()``)
and streams as raw ``cudaStream_t`` handles."""
import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libiconv_b200.so")

OK, ERR_ARG, ERR_SHAPE, ERR_ALIGN, ERR_OVERFLOW, ERR_UNSUPPORTED, ERR_CUDA, ERR_TIMEOUT = 0, -1, -2, -3, -4, -5, -6, -7
U8, S8, I32, U8_RAW128 = 0, 1, 2, 3
KERNEL_AUTO, KERNEL_DIRECT, KERNEL_UMMA, KERNEL_THIN, KERNEL_STEM, KERNEL_UMMA_IM2COL = 0, 1, 2, 3, 4, 5
DTYPE_CODE = {"u8": U8, "s8": S8, "i32": I32, "u8_raw128": U8_RAW128}
KERNEL_NAME = {KERNEL_DIRECT: "direct", KERNEL_UMMA: "umma", KERNEL_THIN: "thin", KERNEL_STEM: "stem"}

EXPORTS = ("iconv_plan", "iconv_plan_destroy", "iconv_plan_kernel", "iconv_plan_describe", "iconv_workspace_bytes", "iconv_forward",
           "iconv_check", "iconv_selftest_wait_timeout", "iconv_device_initialised", "iconv_plan_chain", "iconv_chain_destroy",
           "iconv_forward_chain",
           "iadd_requant", "ipool_max", "ipool_avg_requant", "iq_weight_delta", "iq_quantize_weights",
           "iq_mul_shift", "iq_brelu_params", "iq_skip_sync", "iq_sigma_bound", "iq_bn_fold", "iconcat_plan",
           "iconv_stem_forward_static", "iconv_last_error")


class IconvError(RuntimeError):
    def __init__(self, status, text):
        super().__init__("iconv status %d: %s" % (status, text))
        self.status = status


class iconv_desc(C.Structure):
    _fields_ = [(k, C.c_int32) for k in (
        "n", "h", "w", "c_in", "c_out", "kh", "kw", "stride", "pad",
        "in_dtype", "in_c_total", "in_c_offset", "out_dtype", "out_c_total", "out_c_offset",
        "brelu", "per_channel", "out_lo", "out_hi", "out_zero",
        "skip_dtype", "skip_c_total", "skip_c_offset", "skip_mul", "skip_shift", "kernel",
        "proj_h", "proj_w", "proj_c_in", "proj_c_total", "proj_c_offset", "proj_k", "proj_stride", "proj_pad")] + [
        ("weights", C.c_void_p), ("bias", C.c_void_p), ("mul", C.c_void_p), ("shift", C.c_void_p),
        ("h_i", C.c_void_p), ("proj_weights", C.c_void_p), ("proj_bias", C.c_void_p)]


class iadd_desc(C.Structure):
    _fields_ = [("n_elems", C.c_int64)] + [(k, C.c_int32) for k in (
        "a_dtype", "b_dtype", "out_dtype", "a_zero", "b_zero", "mul_a", "sh_a", "mul_b", "sh_b",
        "brelu", "h_i", "mul", "shift", "out_zero", "out_lo", "out_hi")]


class istem_desc(C.Structure):
    _fields_ = [(k, C.c_int32) for k in (
        "n", "h", "w", "c_out", "in_dtype", "out_c_total", "out_c_offset", "mul", "shift", "h_i",
        "out_lo", "out_hi", "out_zero")]


STEM_STATIC_BYTES = 32 * 1024 * 1024


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError("%s is missing: build it with `python -m paper_2006_11735_b200.build` "
                          "(there is no fallback path)" % LIB_PATH)
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64, dbl = C.c_void_p, C.c_int32, C.c_int64, C.c_double
    P = C.POINTER
    lib.iconv_plan.argtypes = [P(iconv_desc), P(vp)]
    lib.iconv_plan_destroy.argtypes = [vp]
    lib.iconv_plan_kernel.argtypes = [vp]
    lib.iconv_plan_describe.argtypes = [vp, C.c_char_p, C.c_size_t]
    lib.iconv_workspace_bytes.argtypes = [vp]
    lib.iconv_forward.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.iconv_plan_chain.argtypes = [P(iconv_desc), P(iconv_desc), P(vp)]
    lib.iconv_chain_destroy.argtypes = [vp]
    lib.iconv_forward_chain.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.iconv_selftest_wait_timeout.argtypes = [i32, i64, vp]
    lib.iconv_device_initialised.argtypes = [i32]
    lib.iconv_check.argtypes = [vp]
    lib.iadd_requant.argtypes = [P(iadd_desc), vp, vp, vp, vp]
    lib.ipool_max.argtypes = [vp, vp, i32, i32, i32, i32, i32, i32, i32, vp]
    lib.ipool_avg_requant.argtypes = [vp, vp, i32, i32, i32, i32, i32, i32, i32, vp]
    lib.iq_weight_delta.argtypes = [vp, i64, P(dbl)]
    lib.iq_quantize_weights.argtypes = [vp, i64, dbl, vp]
    lib.iq_mul_shift.argtypes = [dbl, i32, P(i32), P(i32)]
    lib.iq_brelu_params.argtypes = [dbl, dbl, i32, i32, P(i32), P(i32), P(i32), P(i32), P(dbl), P(dbl)]
    lib.iq_skip_sync.argtypes = [dbl, dbl, i32, P(i32), P(i32), P(dbl), P(dbl)]
    lib.iq_sigma_bound.argtypes = [C.c_void_p, C.c_int64, dbl, P(i32), C.c_void_p]
    lib.iq_bn_fold.argtypes = [vp, vp, vp, vp, vp, vp, dbl, i32, i64, vp, vp, vp]
    lib.iconcat_plan.argtypes = [i32, vp, vp, i32, vp, vp, vp, vp, P(dbl)]
    lib.iconv_stem_forward_static.argtypes = [P(istem_desc), vp, vp, vp, vp, vp]
    lib.iconv_last_error.restype = C.c_char_p
    for name in EXPORTS:
        if name not in ("iconv_last_error", "iconv_workspace_bytes"):
            getattr(lib, name).restype = C.c_int
    lib.iconv_workspace_bytes.restype = C.c_size_t
    return lib


lib = _load()


def iconv_last_error() -> str:
    return lib.iconv_last_error().decode()


def _check(rc):
    if rc != OK:
        raise IconvError(rc, iconv_last_error())


def _i32(a):
    return np.ascontiguousarray(np.atleast_1d(np.asarray(a)), dtype=np.int32)


def _make_desc(*, n, h, w, c_in, c_out, kh, kw, stride=1, pad=0, in_dtype=U8, in_c_total=None, in_c_offset=0,
               out_dtype=U8, out_c_total=None, out_c_offset=0, brelu=1, out_lo=0, out_hi=255, out_zero=0,
               skip_dtype=-1, skip_c_total=0, skip_c_offset=0, skip_mul=1, skip_shift=0, kernel=KERNEL_AUTO,
               weights, bias, mul=None, shift=None, h_i=None, proj=None):
    """The C descriptor of one layer and the host arrays it points to (which must outlive the call
    that reads it)."""
    weights = np.ascontiguousarray(weights, dtype=np.int8)
    assert weights.shape == (c_out, kh, kw, c_in), weights.shape
    bias = _i32(bias)
    d = iconv_desc(n=n, h=h, w=w, c_in=c_in, c_out=c_out, kh=kh, kw=kw, stride=stride, pad=pad,
                   in_dtype=in_dtype, in_c_total=c_in if in_c_total is None else in_c_total, in_c_offset=in_c_offset,
                   out_dtype=out_dtype, out_c_total=c_out if out_c_total is None else out_c_total,
                   out_c_offset=out_c_offset, brelu=int(brelu), per_channel=0,
                   out_lo=out_lo, out_hi=out_hi, out_zero=out_zero, skip_dtype=skip_dtype,
                   skip_c_total=skip_c_total, skip_c_offset=skip_c_offset, skip_mul=int(skip_mul),
                   skip_shift=int(skip_shift), kernel=kernel)
    keep = [weights, bias]
    d.weights, d.bias = weights.ctypes.data, bias.ctypes.data
    if mul is not None:
        mul, shift, h_i = _i32(mul), _i32(shift), _i32(h_i)
        assert mul.shape == shift.shape == h_i.shape and mul.shape[0] in (1, c_out)
        d.per_channel = int(mul.shape[0] == c_out and c_out > 1)
        d.mul, d.shift, d.h_i = mul.ctypes.data, shift.ctypes.data, h_i.ctypes.data
        keep += [mul, shift, h_i]
    if proj is not None:
        pw = np.ascontiguousarray(proj["weights"], dtype=np.int8)
        pb = _i32(proj["bias"])
        assert pw.shape[0] == c_out and pw.shape[1] == pw.shape[2] and pb.shape[0] == c_out
        d.proj_h, d.proj_w, d.proj_c_in, d.proj_k = proj["h"], proj["w"], pw.shape[3], pw.shape[1]
        d.proj_c_total = proj.get("c_total", pw.shape[3])
        d.proj_c_offset = proj.get("c_offset", 0)
        d.proj_stride, d.proj_pad = proj.get("stride", 1), proj.get("pad", 0)
        d.proj_weights, d.proj_bias = pw.ctypes.data, pb.ctypes.data
        keep += [pw, pb]
    return d, keep


def iconv_plan(**kw):
    """Plan one layer; returns an opaque handle (int).  Arrays are host numpy arrays.
    proj: optional fused projection skip, a dict with ``weights`` [c_out][k][k][c_in], ``bias``,
    ``h``, ``w``, ``c_total``, ``c_offset``, ``stride``, ``pad`` of the projection's input; the
    forward's skip tensor is then that input and ``skip_dtype`` its storage type."""
    d, keep = _make_desc(**kw)
    plan = C.c_void_p()
    _check(lib.iconv_plan(C.byref(d), C.byref(plan)))
    del keep
    return plan.value


def iconv_plan_chain(first: dict, second: dict):
    """Plan two consecutive 1x1 layers as one kernel (``iconv_plan``'s keyword arguments for each);
    raises IconvError(ERR_UNSUPPORTED) when the pair does not qualify."""
    d1, k1 = _make_desc(**first)
    d2, k2 = _make_desc(**second)
    chain = C.c_void_p()
    _check(lib.iconv_plan_chain(C.byref(d1), C.byref(d2), C.byref(chain)))
    del k1, k2
    return chain.value


def iconv_chain_destroy(chain):
    _check(lib.iconv_chain_destroy(chain))


def iconv_forward_chain(chain, x_ptr, skip_ptr, out_ptr, out2_ptr, stream=0):
    _check(lib.iconv_forward_chain(chain, x_ptr, skip_ptr, out_ptr, out2_ptr, stream))


def iconv_plan_destroy(plan):
    _check(lib.iconv_plan_destroy(plan))


def iconv_plan_kernel(plan) -> int:
    rc = lib.iconv_plan_kernel(plan)
    if rc < 0:
        _check(rc)
    return rc


def iconv_plan_describe(plan) -> str:
    buf = C.create_string_buffer(256)
    _check(lib.iconv_plan_describe(plan, buf, 256))
    return buf.value.decode()


def iconv_workspace_bytes(plan) -> int:
    return int(lib.iconv_workspace_bytes(plan))


def iconv_forward(plan, x_ptr, skip_ptr, out_ptr, workspace_ptr=None, stream=0):
    _check(lib.iconv_forward(plan, x_ptr, skip_ptr, out_ptr, workspace_ptr, stream))


def iconv_selftest_wait_timeout(which: int, limit_cycles: int, stream=0):
    _check(lib.iconv_selftest_wait_timeout(which, limit_cycles, stream))


def iconv_device_initialised(device: int) -> int:
    return int(lib.iconv_device_initialised(device))


def iconv_check(stream=0):
    _check(lib.iconv_check(stream))


def iadd_requant(a_ptr, b_ptr, out_ptr, stream=0, **kw):
    _check(lib.iadd_requant(C.byref(iadd_desc(**kw)), a_ptr, b_ptr, out_ptr, stream))


def ipool_max(x_ptr, out_ptr, n, h, w, c, k=3, stride=2, pad=1, stream=0):
    _check(lib.ipool_max(x_ptr, out_ptr, n, h, w, c, k, stride, pad, stream))


def ipool_avg_requant(x_ptr, out_ptr, n, h, w, c, mul, shift, max_int=255, stream=0):
    _check(lib.ipool_avg_requant(x_ptr, out_ptr, n, h, w, c, mul, shift, max_int, stream))


def iq_weight_delta(w_f) -> float:
    w_f = np.ascontiguousarray(w_f, dtype=np.float32)
    out = C.c_double()
    _check(lib.iq_weight_delta(w_f.ctypes.data, w_f.size, C.byref(out)))
    return out.value


def iq_quantize_weights(w_f, delta: float):
    w_f = np.ascontiguousarray(w_f, dtype=np.float32)
    out = np.empty(w_f.shape, dtype=np.int8)
    _check(lib.iq_quantize_weights(w_f.ctypes.data, w_f.size, float(delta), out.ctypes.data))
    return out


def iq_mul_shift(r: float, shift_min: int = 16):
    m, s = C.c_int32(), C.c_int32()
    _check(lib.iq_mul_shift(float(r), shift_min, C.byref(m), C.byref(s)))
    return m.value, s.value


def iq_brelu_params(h_rf: float, ratio_y: float, max_int: int = 255, shift_min: int = 16):
    h_ri, m, s, h_i = C.c_int32(), C.c_int32(), C.c_int32(), C.c_int32()
    h_f, rv = C.c_double(), C.c_double()
    _check(lib.iq_brelu_params(float(h_rf), float(ratio_y), max_int, shift_min, C.byref(h_ri), C.byref(m),
                               C.byref(s), C.byref(h_i), C.byref(h_f), C.byref(rv)))
    return dict(h_ri=h_ri.value, mul=m.value, shift=s.value, h_i=h_i.value, h_f=h_f.value, ratio_V=rv.value)


def iq_skip_sync(ratio_y: float, ratio_s: float, shift_min: int = 8):
    m, s, ry, ds = C.c_int32(), C.c_int32(), C.c_double(), C.c_double()
    _check(lib.iq_skip_sync(float(ratio_y), float(ratio_s), shift_min, C.byref(m), C.byref(s), C.byref(ry),
                            C.byref(ds)))
    return dict(skip_mul=m.value, skip_shift=s.value, ratio_Y_new=ry.value, delta_scale=ds.value)


def iq_bn_fold(w_f, b_f, gamma, beta, mean, var, eps: float):
    """Batch normalisation merged into the convolution before it; returns (W', b', delta per channel)."""
    w_f = np.ascontiguousarray(w_f, dtype=np.float32)
    c_out = w_f.shape[0]
    k = w_f.size // c_out
    f32 = lambda a: None if a is None else np.ascontiguousarray(a, dtype=np.float32)
    b_f, gamma, beta, mean, var = f32(b_f), f32(gamma), f32(beta), f32(mean), f32(var)
    w_out = np.empty(w_f.shape, dtype=np.float64)
    b_out, delta = np.empty(c_out, dtype=np.float64), np.empty(c_out, dtype=np.float64)
    _check(lib.iq_bn_fold(w_f.ctypes.data, None if b_f is None else b_f.ctypes.data, gamma.ctypes.data, beta.ctypes.data,
                          mean.ctypes.data, var.ctypes.data, float(eps), c_out, k, w_out.ctypes.data, b_out.ctypes.data,
                          delta.ctypes.data))
    return w_out, b_out, delta


def iq_sigma_bound(y_ptr, count: int, fraction: float = 0.0015, stream=0) -> int:
    """The n-sigma bound (Section 3.2.2) of ``count`` int32 values at the device pointer ``y_ptr``."""
    b = C.c_int32()
    _check(lib.iq_sigma_bound(y_ptr, int(count), float(fraction), C.byref(b), stream))
    return b.value


def iconcat_plan(ratio_y, ratio_v, shift_min: int = 16):
    ry = np.ascontiguousarray(ratio_y, dtype=np.float64)
    rv = np.ascontiguousarray(ratio_v, dtype=np.float64)
    n = ry.shape[0]
    mul, shift = np.zeros(n, np.int32), np.zeros(n, np.int32)
    scale, ry_new = np.zeros(n, np.float64), np.zeros(n, np.float64)
    rmin = C.c_double()
    _check(lib.iconcat_plan(n, ry.ctypes.data, rv.ctypes.data, shift_min, mul.ctypes.data, shift.ctypes.data,
                            scale.ctypes.data, ry_new.ctypes.data, C.byref(rmin)))
    return dict(ratio_V_min=rmin.value, mul=mul.tolist(), shift=shift.tolist(), delta_scale=scale.tolist(),
                ratio_Y_new=ry_new.tolist())


def iconv_stem_forward_static(x_ptr, weights_ptr, bias_ptr, out_ptr, stream=0, *, n, h, w, c_out, in_dtype=U8_RAW128,
                              out_c_total=None, out_c_offset=0, mul, shift, h_i, out_lo=0, out_hi=255, out_zero=0):
    """The 7x7/2 first layer without any allocation: weights and bias are DEVICE addresses,
    the scratch is the library's static device array (see ``include/iconv.h``)."""
    d = istem_desc(n=n, h=h, w=w, c_out=c_out, in_dtype=in_dtype,
                   out_c_total=c_out if out_c_total is None else out_c_total, out_c_offset=out_c_offset,
                   mul=int(mul), shift=int(shift), h_i=int(h_i), out_lo=out_lo, out_hi=out_hi, out_zero=out_zero)
    _check(lib.iconv_stem_forward_static(C.byref(d), x_ptr, weights_ptr, bias_ptr, out_ptr, stream))
