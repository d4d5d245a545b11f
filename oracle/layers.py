"""TEST INFRASTRUCTURE -- numpy front end of the C oracle (``iconv_oracle.c``).

Argument checking and pointer marshalling only; the arithmetic is in the C file, which
follows the paper's layer statement (Section 3.1, Eq. 4, Eq. 5) step by step in int64.
"""
import ctypes as C

import numpy as np

from . import build as _build

U8, S8, I32, U8_RAW128 = 0, 1, 2, 3
DTYPE_CODE = {"u8": U8, "s8": S8, "i32": I32, "u8_raw128": U8_RAW128}
_NP_OF = {U8: np.uint8, S8: np.int8, I32: np.int32, U8_RAW128: np.uint8}

_lib = None


class _ConvDesc(C.Structure):
    _fields_ = [(k, C.c_int64) for k in (
        "n", "h", "w", "c_in", "c_out", "kh", "kw", "stride", "pad",
        "in_dtype", "in_c_total", "in_c_offset",
        "out_dtype", "out_c_total", "out_c_offset",
        "brelu", "per_channel", "out_lo", "out_hi", "out_zero",
        "skip_dtype", "skip_c_total", "skip_c_offset", "skip_mul", "skip_shift",
        "check_partial")]


class _AddDesc(C.Structure):
    _fields_ = [(k, C.c_int64) for k in (
        "n_elems", "a_dtype", "b_dtype", "out_dtype", "a_zero", "b_zero",
        "mul_a", "sh_a", "mul_b", "sh_b",
        "brelu", "h_i", "mul", "shift", "out_zero", "out_lo", "out_hi")]


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build.build())
        _lib.orc_round_shift.restype = C.c_int64
        _lib.orc_round_shift.argtypes = [C.c_int64, C.c_int64]
        _lib.orc_conv.restype = C.c_int
        _lib.orc_add_requant.restype = C.c_int
        _lib.orc_maxpool.restype = C.c_int
        _lib.orc_avgpool_requant.restype = C.c_int
    return _lib


def round_shift(v: int, s: int) -> int:
    """[v / 2^s], ties toward +infinity (the bracket of Eq. 4)."""
    return int(lib().orc_round_shift(int(v), int(s)))


def _ptr(a):
    return a.ctypes.data_as(C.c_void_p)


def _as(a, code):
    a = np.ascontiguousarray(a)
    if a.dtype != _NP_OF[code]:
        raise TypeError("array dtype %s does not match storage code %d" % (a.dtype, code))
    return a


def out_hw(h, w, k_h, k_w, stride, pad):
    return (h + 2 * pad - k_h) // stride + 1, (w + 2 * pad - k_w) // stride + 1


def conv(X, W, b, mul, shift, h_i, *, stride=1, pad=0, in_dtype=U8, in_c_offset=0, c_in=None,
         out_dtype=U8, out=None, out_c_offset=0, brelu=True, out_lo=0, out_hi=255, out_zero=0,
         skip=None, skip_dtype=-1, skip_c_offset=0, skip_mul=1, skip_shift=0,
         check_partial=False):
    """One integer convolution layer (Figure 1's integer branch).

    X is NHWC storage (its last axis may be wider than ``c_in``; the layer then reads the
    slice starting at ``in_c_offset``).  W is [c_out][kh][kw][c_in] int8.  ``out`` may be a
    wider NHWC tensor that the layer writes at ``out_c_offset`` (concatenation).  Returns
    (out, overflow_flag).
    """
    X = _as(X, in_dtype)
    W = _as(W, S8)
    n, h, w, in_c_total = X.shape
    c_out, kh, kw, wc_in = W.shape
    c_in = wc_in if c_in is None else c_in
    assert c_in == wc_in and in_c_offset + c_in <= in_c_total
    ho, wo = out_hw(h, w, kh, kw, stride, pad)
    b = _as(np.asarray(b, dtype=np.int32), I32)
    assert b.shape == (c_out,)
    mul = np.atleast_1d(np.asarray(mul, dtype=np.int32))
    shift = np.atleast_1d(np.asarray(shift, dtype=np.int32))
    h_i = np.atleast_1d(np.asarray(h_i, dtype=np.int32))
    assert mul.shape == shift.shape == h_i.shape and mul.shape[0] in (1, c_out)
    per_channel = int(mul.shape[0] == c_out and c_out > 1)
    if out is None:
        out = np.zeros((n, ho, wo, c_out), dtype=_NP_OF[out_dtype])
    assert out.flags["C_CONTIGUOUS"] and out.dtype == _NP_OF[out_dtype]
    assert out.shape[:3] == (n, ho, wo) and out_c_offset + c_out <= out.shape[3]
    d = _ConvDesc(n=n, h=h, w=w, c_in=c_in, c_out=c_out, kh=kh, kw=kw, stride=stride, pad=pad,
                  in_dtype=in_dtype, in_c_total=in_c_total, in_c_offset=in_c_offset,
                  out_dtype=out_dtype, out_c_total=out.shape[3], out_c_offset=out_c_offset,
                  brelu=int(bool(brelu)), per_channel=per_channel,
                  out_lo=out_lo, out_hi=out_hi, out_zero=out_zero,
                  skip_dtype=-1, skip_c_total=0, skip_c_offset=0, skip_mul=1, skip_shift=0,
                  check_partial=int(bool(check_partial)))
    sp = None
    if skip is not None:
        skip = _as(skip, skip_dtype)
        assert skip.shape[:3] == (n, ho, wo) and skip_c_offset + c_out <= skip.shape[3]
        d.skip_dtype, d.skip_c_total, d.skip_c_offset = skip_dtype, skip.shape[3], skip_c_offset
        d.skip_mul, d.skip_shift = int(skip_mul), int(skip_shift)
        sp = _ptr(skip)
    rc = lib().orc_conv(C.byref(d), _ptr(X), _ptr(W), _ptr(b), _ptr(mul), _ptr(shift), _ptr(h_i),
                        sp, _ptr(out))
    if rc == 2:
        raise ValueError("bad convolution descriptor")
    return out, bool(rc)


def add_requant(A, B, *, a_dtype=U8, b_dtype=U8, out_dtype=U8, a_zero=0, b_zero=0,
                mul_a=1, sh_a=0, mul_b=1, sh_b=0, brelu=True, h_i=0, mul=1, shift=0,
                out_zero=0, out_lo=0, out_hi=255):
    """Stand-alone feature-map addition with ratio synchronisation (Section 4.1)."""
    A = _as(A, a_dtype)
    B = _as(B, b_dtype)
    assert A.shape == B.shape
    out = np.zeros(A.shape, dtype=_NP_OF[out_dtype])
    d = _AddDesc(n_elems=A.size, a_dtype=a_dtype, b_dtype=b_dtype, out_dtype=out_dtype,
                 a_zero=a_zero, b_zero=b_zero, mul_a=mul_a, sh_a=sh_a, mul_b=mul_b, sh_b=sh_b,
                 brelu=int(bool(brelu)), h_i=h_i, mul=mul, shift=shift,
                 out_zero=out_zero, out_lo=out_lo, out_hi=out_hi)
    rc = lib().orc_add_requant(C.byref(d), _ptr(A), _ptr(B), _ptr(out))
    return out, bool(rc)


def maxpool(X, k=3, stride=2, pad=1):
    X = _as(X, U8)
    n, h, w, c = X.shape
    ho, wo = out_hw(h, w, k, k, stride, pad)
    out = np.zeros((n, ho, wo, c), dtype=np.uint8)
    rc = lib().orc_maxpool(_ptr(X), C.c_int64(n), C.c_int64(h), C.c_int64(w), C.c_int64(c),
                           C.c_int64(k), C.c_int64(stride), C.c_int64(pad), _ptr(out))
    assert rc == 0
    return out


def avgpool_requant(X, mul, shift, max_int=255):
    X = _as(X, U8)
    n, h, w, c = X.shape
    out = np.zeros((n, 1, 1, c), dtype=np.uint8)
    rc = lib().orc_avgpool_requant(_ptr(X), C.c_int64(n), C.c_int64(h), C.c_int64(w), C.c_int64(c),
                                   C.c_int64(mul), C.c_int64(shift), C.c_int64(max_int), _ptr(out))
    assert rc == 0
    return out
